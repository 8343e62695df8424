// CUDA-core (FFMA) prefix + chunk attention and the split combine kernel.
//
// This is the fp32-cache path (fp32 inputs need fp32-accurate products, which single-pass
// tensor-core formats do not give) and the bisecting reference for the tensor-core kernel.
// It computes Section 2's attention of the chunk's queries over [K_0;...;K_t], [V_0;...;V_t]:
// rows of earlier chunks are all visible, rows of the chunk itself causally, query head h reads
// KV head h / G.  Scores never leave the CTA: a running max / running sum softmax in fp32.
//
// Tiling: one CTA = 64 query rows (row = token * G + head-in-group, so the G heads that share a
// KV head share each K/V tile) x 64 keys per iteration; 256 threads as a 16 x 16 grid, each thread
// a 4 x 4 block of scores and a 4 x (d/16) block of the output.
#include "kvfold_internal.h"

namespace kvf {
namespace {

constexpr int BM = 64, BN = 64, kThreads = 256;

template <typename T> struct Ld;
template <> struct Ld<float> {
    static constexpr int N = 4;   // elements per 16-byte vector
    static __device__ __forceinline__ void load(const float *p, float *dst) {
        *reinterpret_cast<float4 *>(dst) = *reinterpret_cast<const float4 *>(p);
    }
};
template <> struct Ld<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ void load(const __nv_bfloat16 *p, float *dst) {
        uint4 v = *reinterpret_cast<const uint4 *>(p);
        float4 a, b;
        a.x = __uint_as_float(v.x << 16); a.y = __uint_as_float(v.x & 0xFFFF0000u);
        a.z = __uint_as_float(v.y << 16); a.w = __uint_as_float(v.y & 0xFFFF0000u);
        b.x = __uint_as_float(v.z << 16); b.y = __uint_as_float(v.z & 0xFFFF0000u);
        b.z = __uint_as_float(v.w << 16); b.w = __uint_as_float(v.w & 0xFFFF0000u);
        reinterpret_cast<float4 *>(dst)[0] = a;
        reinterpret_cast<float4 *>(dst)[1] = b;
    }
};

template <typename T, int D>
__global__ void __launch_bounds__(kThreads, 2) attn_simt_kernel(const AttnArgs a) {
    constexpr int QS = D + 4;            // padded row stride of the Q and K tiles (floats)
    constexpr int SS = BN + 4;           // padded row stride of the probability tile
    constexpr int NC = D / 64;           // float4 output columns per thread
    constexpr int VEC = Ld<T>::N;
    extern __shared__ __align__(16) float smem[];
    float *Qs = smem;                    // [BM][QS]
    float *Ks = Qs + BM * QS;            // [BN][QS]; reused as the probability tile [BM][SS]
    float *Vs = Ks + BN * QS;            // [BN][D]
    float *Ps = Ks;

    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int tile = blockIdx.x, kvh = blockIdx.y, split = blockIdx.z;
    const int G = a.G, n = a.n;
    const int64_t P = a.prefix, L = P + n * a.self_rows;
    const T *q = reinterpret_cast<const T *>(a.q_rot);
    const T *Kp = reinterpret_cast<const T *>(a.k_plane) + (int64_t)kvh * a.capacity * D;
    const T *Vp = reinterpret_cast<const T *>(a.v_plane) + (int64_t)kvh * a.capacity * D;

    // key-tile range of this split; the row tile needs keys below P + (last token + 1)
    const int row0 = tile * BM;
    const int tok_last = min(n - 1, (row0 + BM - 1) / G);
    const int64_t need = P + (tok_last + 1) * a.self_rows;
    // (virtual key tiles: without a window they are the key tiles themselves)
    const WindowTiles wt(a.win_lo, a.n_sink, BN);
    const int nt_need = (int)((need + BN - 1) / BN) - wt.skip;
    const int nt_all = (int)((L + BN - 1) / BN) - wt.skip;
    const int per = (nt_all + a.splits - 1) / a.splits;
    const int kt_begin = split * per;
    const int kt_end = min(nt_need, kt_begin + per);

    // Q tile -> shared (fp32)
    for (int idx = tid; idx < BM * (D / VEC); idx += kThreads) {
        int r = idx / (D / VEC), c = idx % (D / VEC);
        int R = row0 + r, tok = R / G, gi = R % G;
        float *dst = Qs + r * QS + c * VEC;
        if (tok < n) {
            Ld<T>::load(q + ((int64_t)tok * a.H + kvh * G + gi) * D + c * VEC, dst);
        } else {
#pragma unroll
            for (int e = 0; e < VEC; ++e) dst[e] = 0.f;
        }
    }

    int64_t limit[4];   // keys with index < limit are visible to row 4*ty + i
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int tok = (row0 + 4 * ty + i) / G;
        limit[i] = tok < n ? P + (tok + 1) * a.self_rows : 0;
    }

    float m[4], l[4], acc[4][NC * 4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        m[i] = -INFINITY;
        l[i] = 0.f;
#pragma unroll
        for (int c = 0; c < NC * 4; ++c) acc[i][c] = 0.f;
    }

    for (int kt = kt_begin; kt < kt_end; ++kt) {
        const int64_t key0 = (int64_t)wt.actual(kt) * BN;
        __syncthreads();   // previous iteration is done with Ks / Vs (and Q is in place)
        for (int idx = tid; idx < BN * (D / VEC); idx += kThreads) {
            int r = idx / (D / VEC), c = idx % (D / VEC);
            float *dk = Ks + r * QS + c * VEC;
            float *dv = Vs + r * D + c * VEC;
            if (key0 + r < L) {
                Ld<T>::load(Kp + (key0 + r) * D + c * VEC, dk);
                Ld<T>::load(Vp + (key0 + r) * D + c * VEC, dv);
            } else {
#pragma unroll
                for (int e = 0; e < VEC; ++e) { dk[e] = 0.f; dv[e] = 0.f; }
            }
        }
        __syncthreads();

        float s[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) s[i][j] = 0.f;
#pragma unroll 4
        for (int k4 = 0; k4 < D / 4; ++k4) {
            float4 qa[4], kb[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) qa[i] = *reinterpret_cast<const float4 *>(Qs + (4 * ty + i) * QS + k4 * 4);
#pragma unroll
            for (int j = 0; j < 4; ++j) kb[j] = *reinterpret_cast<const float4 *>(Ks + (tx + 16 * j) * QS + k4 * 4);
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    s[i][j] = fmaf(qa[i].x, kb[j].x, s[i][j]);
                    s[i][j] = fmaf(qa[i].y, kb[j].y, s[i][j]);
                    s[i][j] = fmaf(qa[i].z, kb[j].z, s[i][j]);
                    s[i][j] = fmaf(qa[i].w, kb[j].w, s[i][j]);
                }
        }
        __syncthreads();   // everyone has read Ks; it becomes the probability tile

        float alpha[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int64_t key = key0 + tx + 16 * j;
                bool vis = key < limit[i] && (key >= a.win_lo || key < a.n_sink);
                s[i][j] = vis ? s[i][j] * a.scale_log2 : -INFINITY;
                mx = fmaxf(mx, s[i][j]);
            }
#pragma unroll
            for (int o = 1; o < 16; o <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            float m_new = fmaxf(m[i], mx);
            float m_safe = m_new == -INFINITY ? 0.f : m_new;
            alpha[i] = exp2f(m[i] - m_safe);
            float sum = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float p = exp2f(s[i][j] - m_safe);
                sum += p;
                Ps[(4 * ty + i) * SS + tx + 16 * j] = p;
            }
#pragma unroll
            for (int o = 1; o < 16; o <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            l[i] = l[i] * alpha[i] + sum;
            m[i] = m_new;
#pragma unroll
            for (int c = 0; c < NC * 4; ++c) acc[i][c] *= alpha[i];
        }
        __syncthreads();

#pragma unroll 2
        for (int k4 = 0; k4 < BN / 4; ++k4) {
            float4 p4[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) p4[i] = *reinterpret_cast<const float4 *>(Ps + (4 * ty + i) * SS + k4 * 4);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
                for (int c = 0; c < NC; ++c) {
                    float4 vv = *reinterpret_cast<const float4 *>(Vs + (k4 * 4 + kk) * D + c * 64 + tx * 4);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        float p = kk == 0 ? p4[i].x : kk == 1 ? p4[i].y : kk == 2 ? p4[i].z : p4[i].w;
                        acc[i][c * 4 + 0] = fmaf(p, vv.x, acc[i][c * 4 + 0]);
                        acc[i][c * 4 + 1] = fmaf(p, vv.y, acc[i][c * 4 + 1]);
                        acc[i][c * 4 + 2] = fmaf(p, vv.z, acc[i][c * 4 + 2]);
                        acc[i][c * 4 + 3] = fmaf(p, vv.w, acc[i][c * 4 + 3]);
                    }
                }
            }
        }
    }

    // epilogue
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int R = row0 + 4 * ty + i, tok = R / G, gi = R % G;
        if (tok >= n) continue;
        int h = kvh * G + gi;
        float inv = l[i] > 0.f ? 1.f / l[i] : 0.f;
        float lse2 = l[i] > 0.f ? m[i] + log2f(l[i]) : -INFINITY;
        int64_t row = (int64_t)tok * a.H + h;
        if (a.splits > 1) {
            float *po = a.part_o + ((int64_t)split * n * a.H + row) * D;
#pragma unroll
            for (int c = 0; c < NC; ++c)
                *reinterpret_cast<float4 *>(po + c * 64 + tx * 4) =
                    make_float4(acc[i][c * 4] * inv, acc[i][c * 4 + 1] * inv, acc[i][c * 4 + 2] * inv, acc[i][c * 4 + 3] * inv);
            if (tx == 0) a.part_lse[(int64_t)split * n * a.H + row] = lse2;
        } else {
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                float o0 = acc[i][c * 4] * inv, o1 = acc[i][c * 4 + 1] * inv, o2 = acc[i][c * 4 + 2] * inv, o3 = acc[i][c * 4 + 3] * inv;
                int col = c * 64 + tx * 4;
                if (a.out_f32) {
                    *reinterpret_cast<float4 *>(reinterpret_cast<float *>(a.out) + row * D + col) = make_float4(o0, o1, o2, o3);
                } else {
                    __nv_bfloat162 b0 = __floats2bfloat162_rn(o0, o1), b1 = __floats2bfloat162_rn(o2, o3);
                    uint2 pk;
                    pk.x = *reinterpret_cast<uint32_t *>(&b0);
                    pk.y = *reinterpret_cast<uint32_t *>(&b1);
                    *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(a.out) + row * D + col) = pk;
                }
            }
            if (tx == 0 && a.lse) a.lse[row] = lse2 * 0.6931471805599453f;
        }
    }
}

// Merge the per-split results: with lse_s = log2 of split s's softmax denominator (its own
// maximum folded in) and O_s its normalised output,
//   O = sum_s 2^(lse_s - M) O_s / sum_s 2^(lse_s - M),  M = max_s lse_s,
// in split order (no atomics).
template <int D>
__global__ void __launch_bounds__(256) combine_kernel(const AttnArgs a) {
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;   // (row, float4 column)
    const int64_t rows = (int64_t)a.n * a.H;
    if (idx >= rows * (D / 4)) return;
    const int64_t row = idx / (D / 4);
    const int c = (int)(idx % (D / 4));
    float M = -INFINITY;
    for (int s = 0; s < a.splits; ++s) M = fmaxf(M, a.part_lse[(int64_t)s * rows + row]);
    float den = 0.f;
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < a.splits; ++s) {
        float ls = a.part_lse[(int64_t)s * rows + row];
        if (ls == -INFINITY) continue;
        float w = exp2f(ls - M);
        float4 p = *reinterpret_cast<const float4 *>(a.part_o + ((int64_t)s * rows + row) * D + c * 4);
        den += w;
        o.x = fmaf(w, p.x, o.x); o.y = fmaf(w, p.y, o.y); o.z = fmaf(w, p.z, o.z); o.w = fmaf(w, p.w, o.w);
    }
    float inv = den > 0.f ? 1.f / den : 0.f;
    o.x *= inv; o.y *= inv; o.z *= inv; o.w *= inv;
    if (a.out_f32) {
        *reinterpret_cast<float4 *>(reinterpret_cast<float *>(a.out) + row * D + c * 4) = o;
    } else {
        __nv_bfloat162 b0 = __floats2bfloat162_rn(o.x, o.y), b1 = __floats2bfloat162_rn(o.z, o.w);
        uint2 pk;
        pk.x = *reinterpret_cast<uint32_t *>(&b0);
        pk.y = *reinterpret_cast<uint32_t *>(&b1);
        *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(a.out) + row * D + c * 4) = pk;
    }
    if (c == 0 && a.lse) a.lse[row] = (M + log2f(den)) * 0.6931471805599453f;
}

template <typename T, int D>
cudaError_t launch_simt_t(const AttnArgs &a, cudaStream_t s, int *grid_out) {
    constexpr size_t smem = sizeof(float) * (size_t)(BM * (D + 4) + BN * (D + 4) + BN * D);
    static_assert(BM * (BN + 4) <= BN * (D + 4), "probability tile must fit in the K tile");
    cudaError_t e = raise_smem_limit_once(reinterpret_cast<const void *>(attn_simt_kernel<T, D>), (int)smem);
    if (e != cudaSuccess) return e;
    dim3 grid((a.n * a.G + BM - 1) / BM, a.Hkv, a.splits);
    if (grid_out) *grid_out = grid.x * grid.y * grid.z;
    attn_simt_kernel<T, D><<<grid, kThreads, smem, s>>>(a);
    return cudaGetLastError();
}

}  // namespace

int attn_simt_ctas(int n, int G, int Hkv, int splits) { return ((n * G + BM - 1) / BM) * Hkv * splits; }

cudaError_t launch_attn_simt(const AttnArgs &a, int dtype, cudaStream_t s, int *grid_out) {
    if (dtype == 0) {
        if (a.d == 128) return launch_simt_t<__nv_bfloat16, 128>(a, s, grid_out);
        if (a.d == 64) return launch_simt_t<__nv_bfloat16, 64>(a, s, grid_out);
    } else {
        if (a.d == 128) return launch_simt_t<float, 128>(a, s, grid_out);
        if (a.d == 64) return launch_simt_t<float, 64>(a, s, grid_out);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_combine(const AttnArgs &a, int dtype, cudaStream_t s) {
    (void)dtype;
    int64_t items = (int64_t)a.n * a.H * (a.d / 4);
    int blocks = (int)((items + 255) / 256);
    if (a.d == 128) combine_kernel<128><<<blocks, 256, 0, s>>>(a);
    else if (a.d == 64) combine_kernel<64><<<blocks, 256, 0, s>>>(a);
    else return cudaErrorInvalidValue;
    return cudaGetLastError();
}

}  // namespace kvf
