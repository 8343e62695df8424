// Fused RoPE(q), RoPE(k) + append(k, v) for one chunk.
//
// Section 2 of the paper: the new tokens' position identifiers continue from the chunk's
// absolute start, so the rotations line up with the original sequence; Figure "KV-Fold": the
// chunk's K/V are appended to the cache and earlier rows are left as they are.
//
// Numerics (the cache bits are a contract): theta = pos * inv_freq[j] in fp64, cos/sin in fp64,
// each rounded once to fp32; then per output two fp32 operations,
//     lo' = fma(x_lo, c, -(x_hi * s))      hi' = fma(x_hi, c, x_lo * s)
// with the cross product rounded first, and one round-to-nearest-even to the cache dtype.
// Values are copied verbatim.  All global accesses are 16-byte vectors.
#include "kvfold_internal.h"

namespace kvf {
namespace {

constexpr int kTok = 1;        // tokens per CTA: with 512 threads every thread has one 16-byte item of a bf16
constexpr int kThreads = 512;  // Llama-shaped token (320 rotated segments + 128 value segments), all loads in flight at once

template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ void load(const float *p, float (&x)[4]) {
        float4 v = *reinterpret_cast<const float4 *>(p);
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    }
    static __device__ __forceinline__ void store(float *p, const float (&x)[4]) {
        *reinterpret_cast<float4 *>(p) = make_float4(x[0], x[1], x[2], x[3]);
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ void load(const __nv_bfloat16 *p, float (&x)[8]) {
        uint4 v = *reinterpret_cast<const uint4 *>(p);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    static __device__ __forceinline__ void store(__nv_bfloat16 *p, const float (&x)[8]) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t lo = __bfloat16_as_ushort(__float2bfloat16_rn(x[2 * i]));
            uint32_t hi = __bfloat16_as_ushort(__float2bfloat16_rn(x[2 * i + 1]));
            w[i] = lo | (hi << 16);
        }
        *reinterpret_cast<uint4 *>(p) = make_uint4(w[0], w[1], w[2], w[3]);
    }
};

__device__ __forceinline__ void rotate(float a, float b, float c, float s, float &ra, float &rb) {
    float cross_a = __fmul_rn(b, s);
    float cross_b = __fmul_rn(a, s);
    ra = __fmaf_rn(a, c, -cross_a);
    rb = __fmaf_rn(b, c, cross_b);
}

template <typename T, bool INTERLEAVED>
__global__ void __launch_bounds__(kThreads) rope_append_kernel(const RopeAppendArgs a) {
    constexpr int VEC = Vec16<T>::N;
    __shared__ float2 cs[kTok][kMaxHalfDim];   // (cos, sin) per (token, pair)

    const int d = a.d, half = d / 2;
    const int n_tok_blocks = (a.n + kTok - 1) / kTok;      // (a.n: the longest chunk of the launch)
    const int b = blockIdx.y;      // cache of a batch (0 when there is one cache)
    const RowMap rows{a.page_tables ? a.page_tables[b] : a.page_table, a.capacity, a.page_elems, a.d};
    // (the per-cache arrays of a ragged batch were written by an earlier kernel of the stream: under
    // a dependent launch they are visible only after the wait)
    if (a.prefixes || a.pos0s) pdl_wait();
    const int64_t prefix = a.prefixes ? a.prefixes[b] : a.prefix;
    const int64_t pos0 = a.pos0s ? a.pos0s[b] : a.pos0;
    const int n = a.ns ? (int)a.ns[b] : a.n;               // tokens this cache folds

    pdl_launch_dependents();
    if ((int)blockIdx.x >= n_tok_blocks) {
        pdl_wait();   // the attention of the step before may still be reading these rows' tile
        // Clear value rows between the new end of the cache and the next key-tile boundary,
        // so that a zero probability never multiplies stale non-finite bits.
        const int vec_per_row = d / VEC;
        const int zero_rows = n == 0 ? 0 : a.prefixes ? (int)((kKvTile - (prefix + n) % kKvTile) % kKvTile) : a.zero_rows;
        const int64_t total = (int64_t)zero_rows * a.Hkv * vec_per_row;
        const int64_t start = ((int64_t)blockIdx.x - n_tok_blocks) * kThreads + threadIdx.x;
        const int64_t stride = (int64_t)(gridDim.x - n_tok_blocks) * kThreads;
        T *vp = reinterpret_cast<T *>(a.v_plane);
        for (int64_t i = start; i < total; i += stride) {
            int c = (int)(i % vec_per_row);
            int64_t t = i / vec_per_row;
            int g = (int)(t % a.Hkv);
            int64_t row = prefix + n + t / a.Hkv;
            *reinterpret_cast<uint4 *>(vp + rows.offset(g, row) + c * VEC) =
                make_uint4(0, 0, 0, 0);
        }
        return;
    }

    const int tok0 = blockIdx.x * kTok;
    const int ntok = min(kTok, n - tok0);
    if (ntok <= 0) return;                                  // a shorter member of a batch

    for (int idx = threadIdx.x; idx < ntok * half; idx += kThreads) {
        int t = idx / half, j = idx % half;
        double theta = (double)(pos0 + tok0 + t) * a.table.inv_freq[j];
        double sn, cn;
        sincos(theta, &sn, &cn);
        cs[t][j] = make_float2((float)cn, (float)sn);
    }
    __syncthreads();
    pdl_wait();   // the table above needs nothing from earlier kernels; the writes below do

    const int64_t qoff = (int64_t)b * a.n * a.H * d, koff = (int64_t)b * a.n * a.Hkv * d;
    const T *q = reinterpret_cast<const T *>(a.q) + qoff;
    const T *k = reinterpret_cast<const T *>(a.k_new) + koff;
    const T *v = reinterpret_cast<const T *>(a.v_new) + koff;
    T *qr = reinterpret_cast<T *>(a.q_rot) + qoff;
    T *kp = reinterpret_cast<T *>(a.k_plane);
    T *vp = reinterpret_cast<T *>(a.v_plane);
    const int heads = a.H + (a.k_new ? a.Hkv : 0);     // (queries only when no keys are given: kvf_attend)

    // One loop over the rotated segments of q and k and, behind them, the value segments (verbatim
    // 16-byte copies): a thread's items are independent, so their loads go out back to back.
    const int rot_chunks = INTERLEAVED ? d / VEC : half / VEC;       // vectors per row (interleaved) or per half row
    const int rot_items = ntok * heads * rot_chunks;
    const int v_chunks = d / VEC;
    const int items = rot_items + (a.v_new ? ntok * a.Hkv * v_chunks : 0);
    float amax = 0.f;               // largest magnitude written (tracked only under a range limit, fp32 caches)
    const bool ranged = sizeof(T) == 4 && a.range_limit > 0.f;
    for (int idx = threadIdx.x; idx < items; idx += kThreads) {
        if (idx >= rot_items) {
            const int i = idx - rot_items;
            const int c = i % v_chunks;
            const int g = (i / v_chunks) % a.Hkv;
            const int t = i / (v_chunks * a.Hkv);
            const uint4 val = *reinterpret_cast<const uint4 *>(v + ((int64_t)(tok0 + t) * a.Hkv + g) * d + c * VEC);
            *reinterpret_cast<uint4 *>(vp + rows.offset(g, prefix + tok0 + t) + c * VEC) = val;
            if (ranged)
                amax = fmaxf(fmaxf(amax, fmaxf(fabsf(__uint_as_float(val.x)), fabsf(__uint_as_float(val.y)))),
                             fmaxf(fabsf(__uint_as_float(val.z)), fabsf(__uint_as_float(val.w))));
            continue;
        }
        const int c = idx % rot_chunks;
        const int hh = (idx / rot_chunks) % heads;
        const int t = idx / (rot_chunks * heads);
        const T *src;
        T *dst;
        if (hh < a.H) {
            src = q + ((int64_t)(tok0 + t) * a.H + hh) * d;
            dst = qr + ((int64_t)(tok0 + t) * a.H + hh) * d;
        } else {
            const int g = hh - a.H;
            src = k + ((int64_t)(tok0 + t) * a.Hkv + g) * d;
            dst = kp + rows.offset(g, prefix + tok0 + t);
        }
        if (!INTERLEAVED) {
            float lo[VEC], hi[VEC], rlo[VEC], rhi[VEC];
            Vec16<T>::load(src + c * VEC, lo);
            Vec16<T>::load(src + half + c * VEC, hi);
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
                const float2 w = cs[t][c * VEC + e];
                rotate(lo[e], hi[e], w.x, w.y, rlo[e], rhi[e]);
            }
            Vec16<T>::store(dst + c * VEC, rlo);
            Vec16<T>::store(dst + half + c * VEC, rhi);
            if (ranged) {
#pragma unroll
                for (int e = 0; e < VEC; ++e) amax = fmaxf(amax, fmaxf(fabsf(rlo[e]), fabsf(rhi[e])));
            }
        } else {
            float x[VEC], r[VEC];
            Vec16<T>::load(src + c * VEC, x);
#pragma unroll
            for (int e = 0; e < VEC; e += 2) {
                const float2 w = cs[t][(c * VEC + e) / 2];
                rotate(x[e], x[e + 1], w.x, w.y, r[e], r[e + 1]);
            }
            Vec16<T>::store(dst + c * VEC, r);
            if (ranged) {
#pragma unroll
                for (int e = 0; e < VEC; ++e) amax = fmaxf(amax, fabsf(r[e]));
            }
        }
    }
    if (ranged && amax > a.range_limit) atomicCAS(a.status, 0, 7);
}

}  // namespace

cudaError_t launch_rope_append(const RopeAppendArgs &a, int dtype, bool interleaved, int batch, cudaStream_t s) {
    int blocks = (a.n + kTok - 1) / kTok;
    if (a.zero_rows > 0) {
        int64_t vecs = (int64_t)a.zero_rows * a.Hkv * (a.d / (dtype == 0 ? 8 : 4));
        blocks += (int)((vecs + kThreads - 1) / kThreads);
    }
    if (dtype == 0) {
        if (interleaved) return launch_pdl(rope_append_kernel<__nv_bfloat16, true>, dim3(blocks, batch), dim3(kThreads), 0, s, a);
        else return launch_pdl(rope_append_kernel<__nv_bfloat16, false>, dim3(blocks, batch), dim3(kThreads), 0, s, a);
    } else {
        if (interleaved) return launch_pdl(rope_append_kernel<float, true>, dim3(blocks, batch), dim3(kThreads), 0, s, a);
        else return launch_pdl(rope_append_kernel<float, false>, dim3(blocks, batch), dim3(kThreads), 0, s, a);
    }
    return cudaGetLastError();
}

}  // namespace kvf
