// Decode-shaped steps on a quantised cache: at most 16 query rows (n_tokens * G <= 16, i.e. one to
// four tokens at the Llama group size) against a long prefix stored as int8 or int4 codes.
//
// Section 2 of the paper: the chunk's queries attend to every row of the earlier chunks and,
// causally, to the chunk itself; query head h reads KV head h / G.  The trials of Section 4 end
// with 30 tokens decoded one at a time, each of them such a step.  The paper's Discussion stores
// K/V through a round trip bf16 -> intN -> bf16: the attention sees bf16(code * row scale).
//
// Such a step has almost no arithmetic and is bound by how fast the codes leave HBM.  The
// tensor-core kernel for long chunks expands every code tile into a bf16 tile in shared memory,
// which costs it the shared memory it would need to keep enough bytes in flight, and runs the
// expansion on four warps.  Here the codes never get a bf16 image in shared memory: the whole of
// it is a ring of raw code tiles (K codes, V codes and their row scales: 33 KiB a stage for int8,
// six stages; 17 KiB and ten stages for int4) filled by TMA, with one consumer warp per stage:
// warp w takes every tile that lands in stage w (so it sees every phase of that stage's barriers, which
// is what a parity wait needs), expands codes straight into the register fragments of mma.sync
// m16n8k16 (bf16 in, fp32 accumulate) and keeps its own running softmax and output; the warps'
// results are merged at the end.  Both contractions are free in how they number what they sum
// over or put out, which is what makes the expansion cheap:
//   S = Q K^T sums over d: thread (g, q) of a warp (g = lane / 4, q = lane % 4) takes the 32 codes
//     d = 32 q .. 32 q + 31 of key row g of an 8-key block - one contiguous 32 bytes - as its
//     B elements of the eight k-steps, and Q's fragments are loaded once in the same order;
//   O = P V puts out d: the same 32 codes of a V row become, after one 8 x 8 register transpose
//     (movmatrix) per fragment, the B elements of sixteen 8-column blocks whose columns are, for
//     thread q, again d = 32 q .. 32 q + 31; P comes straight from the score accumulators.
//
// Work: the key tiles (128 keys) of each KV head are cut into ngroups / Hkv ranges (the group
// count is a multiple of the KV heads, so a CTA stays inside one head); every CTA leaves a
// normalised partial and its log2 denominator in slot (group + KV head), which
// combine_groups_kernel merges (or writes the output itself when there is one range per head).
// Every mbarrier wait is bounded and reports through the status word.
#include "kvfold_internal.h"
#include "sm100_ptx.cuh"
#include "quant_expand.cuh"

namespace kvf {
namespace {

constexpr int kKeysPerTile = 128;
constexpr int kD = 128;
constexpr int kMaxRows = 16;                   // one m16 tile of query rows

struct Ctl {
    unsigned long long full[12], empty[12];
    int abort;
};

template <int BITS> struct Geo {
    static constexpr int RB = kD * BITS / 8;                       // bytes of a row of codes
    static constexpr uint32_t kCodes = kKeysPerTile * RB;          // one tile of codes
    static constexpr uint32_t kStage = 2 * kCodes + 1024;          // K codes, V codes, K scales, V scales
    static constexpr int kStages = BITS == 4 ? 10 : 6;
    static constexpr uint32_t kOffCtl = kStages * kStage;
    static constexpr uint32_t kSmem = kOffCtl + 1024 + 1024;       // + control block + alignment slack
    static constexpr int kWarps = kStages;                         // consumer warps, one per stage; one more warp produces
    static constexpr int kThreads = (kWarps + 1) * 32;
};
// what the warps leave for the merge: 16 rows x 128 fp32 and per row a maximum and a sum
constexpr uint32_t kMergeWarp = kMaxRows * kD * 4 + kMaxRows * 8;
static_assert(Geo<4>::kWarps * kMergeWarp <= Geo<4>::kOffCtl && Geo<8>::kWarps * kMergeWarp <= Geo<8>::kOffCtl, "the merge area reuses the ring");

__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    // (not volatile: a pure function of its register operands, so the compiler may interleave independent chains)
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// transpose of an 8 x 8 matrix of 16-bit elements held one row pair per thread
__device__ __forceinline__ uint32_t transpose8x8(uint32_t x) {
    uint32_t y;
    asm("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}

// The 32 codes d = 32 q .. 32 q + 31 of code row `row` of a tile at shared address `tile`
// (rows of RB bytes, swizzled over their 16-byte chunks as the TMA left them) -> 16 registers of
// two bf16 each, bf16(code * scale), in element order.
template <int BITS>
__device__ __forceinline__ void expand_segment(uint32_t tile, int row, int q, float scale, uint32_t (&out)[16]) {
    const float2 sc = make_float2(scale, scale);
    if (BITS == 8) {
        // 128-byte rows, 128-byte swizzle: chunk c of row r sits at c ^ (r & 7); my chunks are 2 q and 2 q + 1
        const uint32_t base = tile + (uint32_t)row * 128u, sw = (uint32_t)row & 7u;
        uint32_t w[8];
#pragma unroll
        for (uint32_t c = 0; c < 2; ++c)
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(w[4 * c]), "=r"(w[4 * c + 1]), "=r"(w[4 * c + 2]), "=r"(w[4 * c + 3]) : "r"(base + (((2u * (uint32_t)q + c) ^ sw) << 4)));   // (volatile: the tile is rewritten by later TMA copies)
#pragma unroll
        for (int i = 0; i < 8; ++i) expand4(w[i] ^ 0x80808080u, sc, out[2 * i], out[2 * i + 1]);
    } else {
        // 64-byte rows, 64-byte swizzle: chunk c of row r sits at c ^ ((r >> 1) & 3); my chunk is q
        const uint32_t base = tile + (uint32_t)row * 64u, sw = ((uint32_t)row >> 1) & 3u;
        uint32_t w[4];
        asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(base + (((uint32_t)q ^ sw) << 4)));
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t o[4];
            expand8(w[i], sc, o);
            out[4 * i] = o[0]; out[4 * i + 1] = o[1]; out[4 * i + 2] = o[2]; out[4 * i + 3] = o[3];
        }
    }
}

template <int BITS>
__global__ void __launch_bounds__(Geo<BITS>::kThreads, 1)
attn_q8_decode_kernel(const AttnArgs a, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v) {
    using Gm = Geo<BITS>;
    constexpr int NST = Gm::kStages, kWarps = Gm::kWarps;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - smem_u32(smem_raw));
    Ctl *ctl = reinterpret_cast<Ctl *>(smem + Gm::kOffCtl);
    const uint32_t bar_full = base + Gm::kOffCtl, bar_empty = bar_full + 12 * 8;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, q = lane & 3;
    const int group = blockIdx.x;
    const int G = a.G, n = a.n, nG = n * G;
    const int64_t P = a.prefix, L = P + n;
    const bool direct = a.ngroups == a.Hkv;

    // this CTA's range of its KV head's key tiles (the same line arithmetic as the other kernels)
    const int nt_all = (int)((L + kKeysPerTile - 1) / kKeysPerTile);
    const int64_t line = (int64_t)a.Hkv * nt_all;
    const int64_t lin0 = group * line / a.ngroups, lin1 = (group + 1) * line / a.ngroups;
    const int kvh = (int)(lin0 / nt_all);
    const int kt0 = (int)(lin0 - (int64_t)kvh * nt_all);
    const int ntiles = (int)(lin1 - lin0);         // a multiple of the KV heads cuts the line inside heads

    if (threadIdx.x == 0) {
        for (int s = 0; s < NST; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        ctl->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    pdl_launch_dependents();
    __syncthreads();
    pdl_wait();   // nothing above reads what an earlier kernel wrote; from here on the rotated chunk and the cache are read

    // what a consumer warp carries through its tiles (declared here so that every warp reaches the
    // merge below by the same path)
    float o[16][4];            // output: 8-column block vb, rows g / g + 8; columns d = 32 q + 2 vb + {0, 1}
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};      // rows g and g + 8; log2 units
#pragma unroll
    for (int vb = 0; vb < 16; ++vb)
#pragma unroll
        for (int e = 0; e < 4; ++e) o[vb][e] = 0.f;

    if (warp == kWarps) {
        if (lane == 0) {
            // ------------------------------------------------------------------ TMA producer
            bool ok = true;
            const int32_t *page_table = a.page_table;
            for (int t = 0; t < ntiles && ok; ++t) {
                const int s = t % NST;
                ok = mbar_wait(bar_empty + 8 * s, ((t / NST) & 1) ^ 1, ctl, a.status);
                if (!ok) break;
                const int ktile = kt0 + t;
                const int key0 = ktile * kKeysPerTile;
                const uint32_t dst = base + (uint32_t)s * Gm::kStage;
                if (page_table) {
                    // paged cache: a key tile is one page, which always holds its 128 rows and their scales
                    const int page = page_table[ktile];
                    mbar_expect_tx(bar_full + 8 * s, 2 * Gm::kCodes + 1024u);
                    tma_load_4d(dst, &map_k, bar_full + 8 * s, 0, 0, kvh, page);
                    tma_load_4d(dst + Gm::kCodes, &map_v, bar_full + 8 * s, 0, 0, kvh, page);
                    bulk_load(dst + 2 * Gm::kCodes, a.k_scales + (int64_t)page * a.scale_page_stride + kvh * kKeysPerTile, 512u, bar_full + 8 * s);
                    bulk_load(dst + 2 * Gm::kCodes + 512u, a.v_scales + (int64_t)page * a.scale_page_stride + kvh * kKeysPerTile, 512u, bar_full + 8 * s);
                } else {
                    // the rows' scales come with the tile (as many as the plane still holds)
                    const int64_t left = a.scale_stride - key0;
                    const uint32_t sbytes = (uint32_t)(left < kKeysPerTile ? left : kKeysPerTile) * 4u;
                    mbar_expect_tx(bar_full + 8 * s, 2 * Gm::kCodes + 2 * sbytes);
                    tma_load_3d(dst, &map_k, bar_full + 8 * s, 0, key0, kvh);
                    tma_load_3d(dst + Gm::kCodes, &map_v, bar_full + 8 * s, 0, key0, kvh);
                    bulk_load(dst + 2 * Gm::kCodes, a.k_scales + (int64_t)kvh * a.scale_stride + key0, sbytes, bar_full + 8 * s);
                    bulk_load(dst + 2 * Gm::kCodes + 512u, a.v_scales + (int64_t)kvh * a.scale_stride + key0, sbytes, bar_full + 8 * s);
                }
            }
            // do not leave while a copy may still be writing into this CTA's shared memory
            for (int t = max(0, ntiles - NST); t < ntiles; ++t) mbar_wait_drain(bar_full + 8 * (t % NST), (t / NST) & 1, a.status);
        }
    } else {
        // ------------------------------------------------------------------ consumers: whole key tiles, one warp each
        // Q fragments of the eight k-steps, in the order the key codes are taken: k-step s of thread q
        // covers d = 32 q + 4 s .. + 3 (first pair: a0 / a1 for rows g / g + 8, second pair: a2 / a3)
        uint32_t aq[8][4];
        {
            const __nv_bfloat16 *q_rot = reinterpret_cast<const __nv_bfloat16 *>(a.q_rot);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int R = g + 8 * h, tok = R / G, gi = R % G;
                const __nv_bfloat16 *src = q_rot + ((int64_t)tok * a.H + kvh * G + gi) * kD + 32 * q;
#pragma unroll
                for (int s = 0; s < 8; ++s) {
                    uint2 w = make_uint2(0u, 0u);
                    if (R < nG) w = *reinterpret_cast<const uint2 *>(src + 4 * s);
                    aq[s][h] = w.x;
                    aq[s][2 + h] = w.y;
                }
            }
        }
        // keys below the limit are visible (rows past the chunk's end are never written; each row of S, P
        // and O depends on that row alone, so they are left unmasked)
        int64_t limit[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int R = g + 8 * h;
            limit[h] = R < nG ? P + R / G + 1 : ((int64_t)1 << 62);
        }
        const float sl2 = a.scale_log2;
        bool ok = true;
        for (int t = warp; t < ntiles && ok; t += kWarps) {
            const int s = warp;          // = t % NST: this warp is the only reader of its stage
            ok = mbar_wait(bar_full + 8 * s, (t / NST) & 1, ctl, a.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const uint32_t k_tile = base + (uint32_t)s * Gm::kStage, v_tile = k_tile + Gm::kCodes;
            const float *k_sc = reinterpret_cast<const float *>(smem + (uint32_t)s * Gm::kStage + 2 * Gm::kCodes);
            const float *v_sc = k_sc + 128;
            const int64_t key_base = (int64_t)(kt0 + t) * kKeysPerTile;
#pragma unroll 1
            for (int half = 0; half < 2; ++half) {
                // ---- scores of 64 keys: eight 8-key blocks, S[kb] = rows g / g + 8, keys 2 q, 2 q + 1 of the block
                float sacc[8][4];
#pragma unroll
                for (int kb = 0; kb < 8; kb += 2) {
                    // two key blocks at a time, each with a second accumulator for its odd k-steps: four
                    // independent chains of four MMAs instead of one chain of eight per block
                    float odd[2][4];
                    uint32_t b[2][16];
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) { sacc[kb + i][e] = 0.f; odd[i][e] = 0.f; }
                        const int row = half * 64 + (kb + i) * 8 + g;
                        // (rows past the end of the planes were not copied: they count as zero)
                        const float scale = key_base + row < a.capacity ? k_sc[row] : 0.f;
                        expand_segment<BITS>(k_tile, row, q, scale, b[i]);
                    }
#pragma unroll
                    for (int ks = 0; ks < 8; ks += 2)
#pragma unroll
                        for (int i = 0; i < 2; ++i) {
                            mma_bf16(sacc[kb + i], aq[ks], b[i][2 * ks], b[i][2 * ks + 1]);
                            mma_bf16(odd[i], aq[ks + 1], b[i][2 * ks + 2], b[i][2 * ks + 3]);
                        }
#pragma unroll
                    for (int i = 0; i < 2; ++i)
#pragma unroll
                        for (int e = 0; e < 4; ++e) sacc[kb + i][e] += odd[i][e];
                }
                // ---- mask, running maximum, probabilities
                const int64_t key_h = key_base + half * 64;
                float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
                for (int kb = 0; kb < 8; ++kb)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int64_t key = key_h + kb * 8 + 2 * q + (e & 1);
                        const float v = key < limit[e >> 1] ? sacc[kb][e] * sl2 : -INFINITY;
                        sacc[kb][e] = v;
                        mx[e >> 1] = fmaxf(mx[e >> 1], v);
                    }
                float alpha[2], m_safe[2];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
                    mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
                    const float m_new = fmaxf(m_run[h], mx[h]);
                    m_safe[h] = m_new == -INFINITY ? 0.f : m_new;
                    alpha[h] = ex2(m_run[h] - m_safe[h]);                   // m_run = -inf -> 0
                    m_run[h] = m_new;
                    l_run[h] *= alpha[h];
                }
                uint32_t pa[4][4];         // P as A fragments of the four 16-key steps
#pragma unroll
                for (int kb = 0; kb < 8; ++kb) {
                    const float p0 = ex2(sacc[kb][0] - m_safe[0]), p1 = ex2(sacc[kb][1] - m_safe[0]);
                    const float p2 = ex2(sacc[kb][2] - m_safe[1]), p3 = ex2(sacc[kb][3] - m_safe[1]);
                    l_run[0] += p0 + p1;
                    l_run[1] += p2 + p3;
                    pa[kb >> 1][2 * (kb & 1)] = pack_bf16_pair(p0, p1);           // a0 / a2: row g
                    pa[kb >> 1][2 * (kb & 1) + 1] = pack_bf16_pair(p2, p3);       // a1 / a3: row g + 8
                }
                if (__any_sync(0xffffffffu, alpha[0] != 1.f || alpha[1] != 1.f)) {
#pragma unroll
                    for (int vb = 0; vb < 16; ++vb) {
                        o[vb][0] *= alpha[0]; o[vb][1] *= alpha[0];
                        o[vb][2] *= alpha[1]; o[vb][3] *= alpha[1];
                    }
                }
                // ---- O += P V, 16 keys at a time
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint32_t bt0[16], bt1[16];
#pragma unroll
                    for (int blk = 0; blk < 2; ++blk) {
                        const int row = half * 64 + j * 16 + blk * 8 + g;
                        const float scale = key_base + row < a.capacity ? v_sc[row] : 0.f;
                        uint32_t b[16];
                        expand_segment<BITS>(v_tile, row, q, scale, b);
                        // register i holds V[key g of the block][d = 32 q + 2 i, + 1]: block i of eight columns
                        // as an 8 x 8 matrix [key][column 2 q, 2 q + 1]; transposed it is that block's B fragment
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const uint32_t tr = transpose8x8(b[i]);
                            if (blk == 0) bt0[i] = tr; else bt1[i] = tr;
                        }
                    }
#pragma unroll
                    for (int vb = 0; vb < 16; ++vb) mma_bf16(o[vb], pa[j], bt0[vb], bt1[vb]);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty + 8 * s);
        }
    }

    // ---------------------------------------------------------------------- merge of the warps' results
    // (every thread comes here, whatever happened above; the ring is free once the consumers are through
    // and the producer has seen its last copies land)
    __syncthreads();
    float *mrg = reinterpret_cast<float *>(smem);
    if (warp < kWarps) {
        float *mo = mrg + (size_t)warp * (kMergeWarp / 4);
        float *mm = mo + kMaxRows * kD;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float l = l_run[h];
            l += __shfl_xor_sync(0xffffffffu, l, 1);
            l += __shfl_xor_sync(0xffffffffu, l, 2);
            const int r = g + 8 * h;
#pragma unroll
            for (int vb = 0; vb < 16; ++vb)
                *reinterpret_cast<float2 *>(mo + r * kD + 32 * q + 2 * vb) = make_float2(o[vb][2 * h], o[vb][2 * h + 1]);
            if (q == 0) {
                mm[2 * r] = m_run[h];
                mm[2 * r + 1] = l;
            }
        }
    }
    __syncthreads();
    for (int item = threadIdx.x; item < kMaxRows * 16; item += kWarps * 32) {
        if (warp >= kWarps) break;
        // item = (row, eight columns)
        const int r = item >> 4, c0 = (item & 15) * 8;
        if (r < nG) {
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) M = fmaxf(M, mrg[(size_t)w * (kMergeWarp / 4) + kMaxRows * kD + 2 * r]);
            float den = 0.f, acc[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) acc[c] = 0.f;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {               // warp order: deterministic
                const float *wo = mrg + (size_t)w * (kMergeWarp / 4);
                const float mw = wo[kMaxRows * kD + 2 * r], lw = wo[kMaxRows * kD + 2 * r + 1];
                const float f = mw == -INFINITY ? 0.f : exp2f(mw - M);
                den += f * lw;
                const float4 x = *reinterpret_cast<const float4 *>(wo + r * kD + c0), y = *reinterpret_cast<const float4 *>(wo + r * kD + c0 + 4);
                acc[0] = fmaf(f, x.x, acc[0]); acc[1] = fmaf(f, x.y, acc[1]); acc[2] = fmaf(f, x.z, acc[2]); acc[3] = fmaf(f, x.w, acc[3]);
                acc[4] = fmaf(f, y.x, acc[4]); acc[5] = fmaf(f, y.y, acc[5]); acc[6] = fmaf(f, y.z, acc[6]); acc[7] = fmaf(f, y.w, acc[7]);
            }
            const float inv = den > 0.f ? 1.f / den : 0.f;
            const float lse2 = den > 0.f ? M + log2f(den) : -INFINITY;
            const int tok = r / G, gi = r % G;
            const int64_t row = (int64_t)tok * a.H + kvh * G + gi;
            if (!direct) {
                const int64_t prow = (int64_t)(group + kvh) * nG + r;
                float4 *dst = reinterpret_cast<float4 *>(a.part_o + prow * kD + c0);
                dst[0] = make_float4(acc[0] * inv, acc[1] * inv, acc[2] * inv, acc[3] * inv);
                dst[1] = make_float4(acc[4] * inv, acc[5] * inv, acc[6] * inv, acc[7] * inv);
                if (c0 == 0) a.part_lse[prow] = lse2;
            } else {
                if (a.out_f32) {
                    float4 *dst = reinterpret_cast<float4 *>(reinterpret_cast<float *>(a.out) + row * kD + c0);
                    dst[0] = make_float4(acc[0] * inv, acc[1] * inv, acc[2] * inv, acc[3] * inv);
                    dst[1] = make_float4(acc[4] * inv, acc[5] * inv, acc[6] * inv, acc[7] * inv);
                } else {
                    *reinterpret_cast<uint4 *>(reinterpret_cast<__nv_bfloat16 *>(a.out) + row * kD + c0) =
                        make_uint4(pack_bf16_pair(acc[0] * inv, acc[1] * inv), pack_bf16_pair(acc[2] * inv, acc[3] * inv),
                                   pack_bf16_pair(acc[4] * inv, acc[5] * inv), pack_bf16_pair(acc[6] * inv, acc[7] * inv));
                }
                if (c0 == 0 && a.lse) a.lse[row] = lse2 * 0.6931471805599453f;
            }
        }
    }
}

}  // namespace

// Rows of query (n * G) one CTA of the decode kernel takes.
int attn_q8_decode_max_rows() { return kMaxRows; }

cudaError_t launch_attn_q8_decode(const AttnArgs &a, const TcMaps &maps, cudaStream_t s) {
    static_assert(sizeof(Ctl) <= 1024, "control block");
    static_assert(Geo<8>::kSmem <= 232448 && Geo<4>::kSmem <= 232448, "shared memory budget of one CTA");
    static_assert(Geo<8>::kStages <= 12 && Geo<4>::kStages <= 12, "control block holds 12 stages");
    auto kernel = a.quant_bits == 4 ? attn_q8_decode_kernel<4> : attn_q8_decode_kernel<8>;
    const uint32_t smem = a.quant_bits == 4 ? Geo<4>::kSmem : Geo<8>::kSmem;
    cudaError_t e = raise_smem_limit_once(reinterpret_cast<const void *>(kernel), (int)smem);
    if (e != cudaSuccess) return e;
    const int threads = a.quant_bits == 4 ? Geo<4>::kThreads : Geo<8>::kThreads;
    return launch_pdl(kernel, dim3(a.ngroups), dim3(threads), smem, s, a, maps.k, maps.v);
}

}  // namespace kvf
