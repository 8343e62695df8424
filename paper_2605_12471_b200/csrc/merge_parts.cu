// Merging attention results that were computed over disjoint sets of cache rows.
//
// Section 2 of the paper: a chunk's queries attend to the concatenation [K_0; ...; K_t].  The softmax
// over a union of key sets follows from the parts' normalised outputs o_r and log-sum-exps lse_r:
//     lse = log sum_r exp(lse_r),   out = sum_r exp(lse_r - lse) o_r,
// which is what lets one sequence's cache be split by row range over several GPUs (each holds the rows
// of some chunks and answers every chunk's queries over what it holds: kvf_fold_step on the GPU that
// takes the chunk, kvf_attend on the others), with one all-gather of (o_r, lse_r) per step.
// The parts are taken in index order, so the result is bitwise reproducible.
#include "kvfold_internal.h"

namespace kvf {
namespace {

template <typename T> struct Elem4;
template <> struct Elem4<float> {
    static __device__ __forceinline__ float4 load(const float *p) { return *reinterpret_cast<const float4 *>(p); }
    static __device__ __forceinline__ void store(float *p, float4 v) { *reinterpret_cast<float4 *>(p) = v; }
};
template <> struct Elem4<__nv_bfloat16> {
    static __device__ __forceinline__ float4 load(const __nv_bfloat16 *p) {
        const uint2 w = *reinterpret_cast<const uint2 *>(p);
        return make_float4(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xFFFF0000u),
                           __uint_as_float(w.y << 16), __uint_as_float(w.y & 0xFFFF0000u));
    }
    static __device__ __forceinline__ void store(__nv_bfloat16 *p, float4 v) {
        const __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
        uint2 w;
        w.x = *reinterpret_cast<const uint32_t *>(&a);
        w.y = *reinterpret_cast<const uint32_t *>(&b);
        *reinterpret_cast<uint2 *>(p) = w;
    }
};

// One warp per row (a token of a query head); lane l holds elements 4 l .. 4 l + 3 of it (head_dim 128:
// all 32 lanes, head_dim 64: the first 16).
template <typename T>
__global__ void __launch_bounds__(256) merge_parts_kernel(int n_parts, int64_t n_rows, int d, const T *parts_out,
                                                          const float *parts_lse, T *out, float *lse) {
    const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= n_rows) return;
    float M = -INFINITY;
    for (int r = 0; r < n_parts; ++r) M = fmaxf(M, parts_lse[(int64_t)r * n_rows + row]);
    float den = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    const bool mine = 4 * lane < d;
    for (int r = 0; r < n_parts; ++r) {
        const float l = parts_lse[(int64_t)r * n_rows + row];
        if (l == -INFINITY) continue;                       // this part saw no key
        const float w = expf(l - M);
        den += w;
        if (mine) {
            const float4 v = Elem4<T>::load(parts_out + ((int64_t)r * n_rows + row) * d + 4 * lane);
            acc.x = fmaf(w, v.x, acc.x); acc.y = fmaf(w, v.y, acc.y);
            acc.z = fmaf(w, v.z, acc.z); acc.w = fmaf(w, v.w, acc.w);
        }
    }
    const float inv = den > 0.f ? 1.f / den : 0.f;
    if (mine) Elem4<T>::store(out + row * d + 4 * lane, make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv));
    if (lane == 0 && lse) lse[row] = den > 0.f ? M + logf(den) : -INFINITY;
}

}  // namespace

cudaError_t launch_merge_parts(int n_parts, int64_t n_rows, int d, bool f32, const void *parts_out, const float *parts_lse,
                               void *out, float *lse, cudaStream_t s) {
    const unsigned blocks = (unsigned)((n_rows + 7) / 8);
    if (f32)
        merge_parts_kernel<float><<<blocks, 256, 0, s>>>(n_parts, n_rows, d, static_cast<const float *>(parts_out), parts_lse,
                                                         static_cast<float *>(out), lse);
    else
        merge_parts_kernel<__nv_bfloat16><<<blocks, 256, 0, s>>>(n_parts, n_rows, d, static_cast<const __nv_bfloat16 *>(parts_out),
                                                                 parts_lse, static_cast<__nv_bfloat16 *>(out), lse);
    return cudaGetLastError();
}

}  // namespace kvf
