// Quantised cache storage: rotate + quantise + append.
//
// The paper's Discussion perturbs the stored K/V by a round trip bf16 -> intN -> bf16 and leaves the
// scheme open.  Here a stored row (one token of one KV head, d elements) is symmetric int8 (Q = 127)
// or int4 (Q = 7) with one fp32 scale, decided once when the row is appended:
//     amax = max |x_j|     inv = Q / amax       scale = amax / Q          (fp32, round to nearest)
//     code_j = clamp(rint(x_j * inv), -Q, Q)                               (ties to even)
//     value seen by the attention = bf16(code_j * scale)                   (fp32 product, one rounding)
// For a key row x is the rotated row in fp32 (same operation order as the bf16 path, before any
// rounding to bf16); a value row is quantised as given.  amax = 0 gives codes 0 and scale 0.
// The cache then holds d + 4 (int8) or d / 2 + 4 (int4: code + 8, two to a byte, element 2i in the low
// nibble of byte i) bytes per row instead of 2 d; the attention kernel expands code tiles to bf16 tiles
// in shared memory.  Paged caches keep codes and scales of 128 tokens of every KV head in one page
// (see QuantPlanes); a batch of paged caches is one launch (blockIdx.y = cache).
#include "kvfold_internal.h"

namespace kvf {
namespace {

// One token per CTA of 16 warps: a warp then has three of the token's 48 rows to do, one after the
// other (each a load, a warp reduction and a store), instead of twelve.
constexpr int kTok = 1;        // tokens per CTA
constexpr int kThreads = 512;

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ void rotate(float a, float b, float c, float s, float &ra, float &rb) {
    float cross_a = __fmul_rn(b, s);
    float cross_b = __fmul_rn(a, s);
    ra = __fmaf_rn(a, c, -cross_a);
    rb = __fmaf_rn(b, c, cross_b);
}

// codes of four values of a row held by one lane; the row's scale comes back in `scale`
template <int BITS>
__device__ __forceinline__ void quantise4(const float (&x)[4], int (&code)[4], float &scale) {
    constexpr float Q = BITS == 4 ? 7.f : 127.f;
    float amax = fmaxf(fmaxf(fabsf(x[0]), fabsf(x[1])), fmaxf(fabsf(x[2]), fabsf(x[3])));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    const float inv = amax > 0.f ? __fdiv_rn(Q, amax) : 0.f;
    scale = __fdiv_rn(amax, Q);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        float r = rintf(__fmul_rn(x[e], inv));
        r = fminf(fmaxf(r, -Q), Q);
        code[e] = (int)r;
    }
}

// One warp per row (d = 128: four elements per lane).  Query rows are rotated and written as bf16;
// key rows are rotated in fp32, quantised and appended; value rows are quantised and appended.
template <bool INTERLEAVED, int BITS>
__global__ void __launch_bounds__(kThreads) rope_append_q8_kernel(const RopeAppendArgs a, const QuantPlanes qp) {
    constexpr int RB = 128 * BITS / 8;          // bytes of a stored row
    __shared__ float2 cs[kTok][kMaxHalfDim];   // (cos, sin) per (token, pair)
    constexpr int d = 128, half = 64;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tok0 = blockIdx.x * kTok;
    const int b = blockIdx.y;      // cache of a batch (0 when there is one cache)

    pdl_launch_dependents();
    // (the per-cache arrays of a ragged batch were written by an earlier kernel of the stream: under
    // a dependent launch they are visible only after the wait)
    if (a.prefixes || a.pos0s) pdl_wait();
    const int64_t prefix = a.prefixes ? a.prefixes[b] : a.prefix;
    const int64_t pos0 = a.pos0s ? a.pos0s[b] : a.pos0;
    const int n = a.ns ? (int)a.ns[b] : a.n;               // tokens this cache folds (a.n: the longest chunk, the stride)
    const int ntok = max(0, min(kTok, n - tok0));
    const int32_t *page_table = a.page_tables ? a.page_tables[b] : a.page_table;
    // where row `row` of KV head g lives: byte offset of its codes from the code block, index of its scale
    auto code_off = [&](int g, int64_t row) -> int64_t {
        if (qp.page_bytes == 0) return ((int64_t)g * a.capacity + row) * RB;
        return (int64_t)page_table[row / kKvTile] * qp.page_bytes + ((int64_t)g * kKvTile + row % kKvTile) * RB;
    };
    auto scale_idx = [&](int g, int64_t row) -> int64_t {
        if (qp.page_bytes == 0) return (int64_t)g * qp.scale_stride + row;
        return (int64_t)page_table[row / kKvTile] * (qp.page_bytes / 4) + (int64_t)g * kKvTile + row % kKvTile;
    };
    for (int idx = threadIdx.x; idx < ntok * half; idx += kThreads) {
        int t = idx / half, j = idx % half;
        double theta = (double)(pos0 + tok0 + t) * a.table.inv_freq[j];
        double sn, cn;
        sincos(theta, &sn, &cn);
        cs[t][j] = make_float2((float)cn, (float)sn);
    }
    __syncthreads();
    pdl_wait();   // the table above needs nothing from earlier kernels; the writes below do

    // Rows between the new end of the cache and the next key-tile boundary get value scale 0: the
    // attention expands them to zeros whatever their codes are, so a zero probability never
    // multiplies non-finite bits.
    if (blockIdx.x == 0 && n > 0 && a.k_new) {
        const int zero_rows = a.prefixes ? (int)((kKvTile - (prefix + n) % kKvTile) % kKvTile) : a.zero_rows;
        for (int i = threadIdx.x; i < zero_rows * a.Hkv; i += kThreads)
            qp.v_scales[scale_idx(i / zero_rows, prefix + n + i % zero_rows)] = 0.f;
    }

    const int64_t qoff = (int64_t)b * a.n * a.H * d, koff = (int64_t)b * a.n * a.Hkv * d;
    const __nv_bfloat16 *q = reinterpret_cast<const __nv_bfloat16 *>(a.q) + qoff;
    const __nv_bfloat16 *k = reinterpret_cast<const __nv_bfloat16 *>(a.k_new) + koff;
    const __nv_bfloat16 *v = reinterpret_cast<const __nv_bfloat16 *>(a.v_new) + koff;
    __nv_bfloat16 *qr = reinterpret_cast<__nv_bfloat16 *>(a.q_rot) + qoff;
    const int heads = a.H + (a.k_new ? 2 * a.Hkv : 0);     // query rows, key rows, value rows (queries only: kvf_attend)
    for (int row = warp; row < ntok * heads; row += kThreads / 32) {
        const int t = row / heads, hh = row % heads;
        const int64_t tok = tok0 + t;
        const int64_t cache_row = prefix + tok;
        if (hh >= a.H + a.Hkv) {
            // ---- value row: elements 4 lane .. 4 lane + 3
            const int g = hh - a.H - a.Hkv;
            const uint2 w = *reinterpret_cast<const uint2 *>(v + (tok * a.Hkv + g) * d + 4 * lane);
            const float x[4] = {bf16_lo(w.x), bf16_hi(w.x), bf16_lo(w.y), bf16_hi(w.y)};
            int code[4];
            float scale;
            quantise4<BITS>(x, code, scale);
            const int64_t r = code_off(g, cache_row);
            if (BITS == 8) {
                const uint32_t packed = (uint32_t)(code[0] & 0xFF) | ((uint32_t)(code[1] & 0xFF) << 8) |
                                        ((uint32_t)(code[2] & 0xFF) << 16) | ((uint32_t)(code[3] & 0xFF) << 24);
                *reinterpret_cast<uint32_t *>(qp.v_codes + r + 4 * lane) = packed;
            } else {
                *reinterpret_cast<uint16_t *>(qp.v_codes + r + 2 * lane) =
                    (uint16_t)((code[0] + 8) | ((code[1] + 8) << 4) | ((code[2] + 8) << 8) | ((code[3] + 8) << 12));
            }
            if (lane == 0) qp.v_scales[scale_idx(g, cache_row)] = scale;
            continue;
        }
        const bool is_q = hh < a.H;
        const __nv_bfloat16 *src = is_q ? q + (tok * a.H + hh) * d : k + (tok * a.Hkv + (hh - a.H)) * d;
        float x[4];
        int e0, e1;     // where x[0..1] and x[2..3] sit in the row
        if (!INTERLEAVED) {
            // pairs (j, j + 64) for j = 2 lane, 2 lane + 1
            e0 = 2 * lane; e1 = half + 2 * lane;
            const uint32_t lo = *reinterpret_cast<const uint32_t *>(src + e0);
            const uint32_t hi = *reinterpret_cast<const uint32_t *>(src + e1);
            const float2 w0 = cs[t][2 * lane], w1 = cs[t][2 * lane + 1];
            rotate(bf16_lo(lo), bf16_lo(hi), w0.x, w0.y, x[0], x[2]);
            rotate(bf16_hi(lo), bf16_hi(hi), w1.x, w1.y, x[1], x[3]);
        } else {
            // pairs (2 j, 2 j + 1) for j = 2 lane, 2 lane + 1
            e0 = 4 * lane; e1 = 4 * lane + 2;
            const uint2 w = *reinterpret_cast<const uint2 *>(src + e0);
            const float2 w0 = cs[t][2 * lane], w1 = cs[t][2 * lane + 1];
            rotate(bf16_lo(w.x), bf16_hi(w.x), w0.x, w0.y, x[0], x[1]);
            rotate(bf16_lo(w.y), bf16_hi(w.y), w1.x, w1.y, x[2], x[3]);
        }
        if (is_q) {
            __nv_bfloat16 *dst = qr + (tok * a.H + hh) * d;
            __nv_bfloat162 p0 = __floats2bfloat162_rn(x[0], x[1]), p1 = __floats2bfloat162_rn(x[2], x[3]);
            *reinterpret_cast<__nv_bfloat162 *>(dst + e0) = p0;
            *reinterpret_cast<__nv_bfloat162 *>(dst + e1) = p1;
        } else {
            const int g = hh - a.H;
            int code[4];
            float scale;
            quantise4<BITS>(x, code, scale);
            const int64_t r = code_off(g, cache_row);
            if (BITS == 8) {
                *reinterpret_cast<uint16_t *>(qp.k_codes + r + e0) = (uint16_t)((code[0] & 0xFF) | ((code[1] & 0xFF) << 8));
                *reinterpret_cast<uint16_t *>(qp.k_codes + r + e1) = (uint16_t)((code[2] & 0xFF) | ((code[3] & 0xFF) << 8));
            } else {
                // elements e0, e0 + 1 share byte e0 / 2 (e0 and e1 are even)
                qp.k_codes[r + e0 / 2] = (int8_t)((code[0] + 8) | ((code[1] + 8) << 4));
                qp.k_codes[r + e1 / 2] = (int8_t)((code[2] + 8) | ((code[3] + 8) << 4));
            }
            if (lane == 0) qp.k_scales[scale_idx(g, cache_row)] = scale;
        }
    }
}

}  // namespace

cudaError_t launch_rope_append_q8(const RopeAppendArgs &a, const QuantPlanes &qp, bool interleaved, int batch, cudaStream_t s) {
    const dim3 grid((a.n + kTok - 1) / kTok, batch);
    if (qp.bits == 4) {
        if (interleaved) return launch_pdl(rope_append_q8_kernel<true, 4>, grid, dim3(kThreads), 0, s, a, qp);
        return launch_pdl(rope_append_q8_kernel<false, 4>, grid, dim3(kThreads), 0, s, a, qp);
    }
    if (interleaved) return launch_pdl(rope_append_q8_kernel<true, 8>, grid, dim3(kThreads), 0, s, a, qp);
    return launch_pdl(rope_append_q8_kernel<false, 8>, grid, dim3(kThreads), 0, s, a, qp);
}

}  // namespace kvf
