// Decode-shaped steps: at most 16 query rows (n_tokens * G <= 16, i.e. one to four tokens at the
// Llama group size) against a long prefix stored as int8 or int4 codes - or as plain bf16 rows, which
// take the same kernel without the expansion (BITS = 16 below).
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
// it is a ring of raw code tiles (K codes, V codes and their row scales of 128 keys: 33 KiB a
// stage for int8, 17 KiB for int4) filled by TMA, and two consumer warps per stage, each taking
// 64 of the tile's keys (a warp always reads the same stage, so it sees every phase of that
// stage's barriers, which is what a parity wait needs).  A warp expands codes straight into the
// register fragments of mma.sync m16n8k16 (bf16 in, fp32 accumulate) and keeps its own running
// softmax and output; the warps' results are merged at the end.
//
// With so few query rows the KEYS take the 16-row side of the MMA and the query rows the 8-column
// side (one or two column blocks), so no MMA row is wasted on padding and V needs no transpose:
//   S^T = K Q^T (16 keys x 8 rows, summed over d): thread (g, t) of a warp (g = lane / 4,
//     t = lane % 4) takes the 32 codes d = 32 t .. 32 t + 31 of key rows g and g + 8 of a 16-key
//     block - contiguous bytes - as its A elements of the eight k-steps; the contraction is free in
//     how it numbers d, and Q's B fragments are loaded once in the same order;
//   O^T = V^T P^T (128 d x 8 rows, summed over 16 keys): an A element pairs two KEYS of one d, and
//     since every code is expanded on its own, thread (g, t) builds its pairs from the 16 codes
//     d = 16 g .. 16 g + 15 of key rows 2 t, 2 t + 1, 2 t + 8, 2 t + 9 (the MMA's row index is
//     free in how it numbers d as well).  P^T's B fragment is the transposed score fragment:
//     two 8 x 8 register transposes (movmatrix) per 16 keys.
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
constexpr int kMaxRows = 16;                   // two 8-column blocks of query rows

struct Ctl {
    unsigned long long full[12], empty[12];
    int abort;
};

// NB = 8-row blocks of query rows (1: up to 8 rows, 2: up to 16).  A scheduler of the SM holds 16 K
// registers: with 13 warps one of them has four (128 registers a thread, enough for one block of
// rows), with 11 none has more than three (168, what two blocks need without spilling).
// BITS = 16 stands for a cache of plain bf16 rows: the same kernel without the expansion (a tile is then two
// 128-byte-swizzled panels of 64 columns, 32 KiB; three stages of 64 KiB, six consumer warps).
template <int BITS, int NB> struct Geo {
    static constexpr int RB = kD * BITS / 8;                       // bytes of a row of codes
    static constexpr uint32_t kCodes = kKeysPerTile * RB;          // one tile of codes
    static constexpr uint32_t kScales = BITS == 16 ? 0 : 1024;     // K scales, V scales
    static constexpr uint32_t kStage = 2 * kCodes + kScales;       // K codes, V codes, scales
    static constexpr int kStages = BITS == 16 ? 3 : NB == 2 ? 5 : 6;
    static constexpr uint32_t kOffCtl = kStages * kStage;
    static constexpr uint32_t kSmem = kOffCtl + 1024 + 1024;       // + control block + alignment slack
    static constexpr int kWarps = 2 * kStages;                     // consumer warps, two per stage; one more warp produces
    static constexpr int kThreads = (kWarps + 1) * 32;
};
// what the warps leave for the merge: 16 rows x 128 fp32 and per row a maximum and a sum
constexpr uint32_t kMergeWarp = kMaxRows * kD * 4 + kMaxRows * 8;
static_assert(Geo<4, 1>::kWarps * kMergeWarp <= Geo<4, 1>::kOffCtl && Geo<4, 2>::kWarps * kMergeWarp <= Geo<4, 2>::kOffCtl, "the merge area reuses the ring");

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
// (volatile, here and below: the tiles are rewritten by later TMA copies)
__device__ __forceinline__ void lds128(uint32_t addr, uint32_t (&w)[4]) {
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(addr));
}
__device__ __forceinline__ void lds64(uint32_t addr, uint32_t (&w)[2]) {
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(w[0]), "=r"(w[1]) : "r"(addr));
}

// A fragments of S^T = K Q^T for one 16-key block: the 32 codes d = 32 t .. 32 t + 31 of key rows
// `row` and `row + 8` of the code tile at shared address `tile` (rows swizzled over their 16-byte
// chunks as the TMA left them).  k-step s covers d = 32 t + 4 s .. + 3: a0 / a2 from the first row,
// a1 / a3 from the second, each bf16(code * scale) in element order.
template <int BITS>
__device__ __forceinline__ void key_fragments(uint32_t tile, int row, int t, float sc_a, float sc_b, uint32_t (&ka)[8][4]) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int r = row + 8 * h;
        if (BITS == 16) {
            // bf16 rows: two panels of [128 rows][64 columns], 128-byte swizzle; my 32 columns are four 16-byte
            // chunks (t & 1) * 4 .. + 3 of panel t >> 1, each two k-steps' worth
            const uint32_t base = tile + (uint32_t)(t >> 1) * (kKeysPerTile * 128u) + (uint32_t)r * 128u, sw = (uint32_t)r & 7u;
#pragma unroll
            for (uint32_t c = 0; c < 4; ++c) {
                uint32_t w[4];
                lds128(base + (((((uint32_t)t & 1u) << 2) + c) ^ sw) * 16u, w);
                ka[2 * c][h] = w[0]; ka[2 * c][2 + h] = w[1];
                ka[2 * c + 1][h] = w[2]; ka[2 * c + 1][2 + h] = w[3];
            }
            continue;
        }
        const float s1 = h ? sc_b : sc_a;
        const float2 sc = make_float2(s1, s1);
        if (BITS == 8) {
            // 128-byte rows, 128-byte swizzle: chunk c of row r sits at c ^ (r & 7); my chunks are 2 t and 2 t + 1
            const uint32_t base = tile + (uint32_t)r * 128u, sw = (uint32_t)r & 7u;
#pragma unroll
            for (uint32_t c = 0; c < 2; ++c) {
                uint32_t w[4];
                lds128(base + (((2u * (uint32_t)t + c) ^ sw) << 4), w);
#pragma unroll
                for (int i = 0; i < 4; ++i) expand4(w[i] ^ 0x80808080u, sc, ka[4 * c + i][h], ka[4 * c + i][2 + h]);
            }
        } else {
            // 64-byte rows, 64-byte swizzle: chunk c of row r sits at c ^ ((r >> 1) & 3); my chunk is t
            const uint32_t base = tile + (uint32_t)r * 64u, sw = ((uint32_t)r >> 1) & 3u;
            uint32_t w[4];
            lds128(base + (((uint32_t)t ^ sw) << 4), w);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint32_t o[4];
                expand8(w[i], sc, o);
                ka[2 * i][h] = o[0]; ka[2 * i][2 + h] = o[1];
                ka[2 * i + 1][h] = o[2]; ka[2 * i + 1][2 + h] = o[3];
            }
        }
    }
}

// bf16 pair (x(wa), x(wb)) * sc of byte `byte` of two words whose bytes hold code + `bias`
// (2^23 + byte is exact in fp32, as is the difference that follows)
__device__ __forceinline__ uint32_t pair_of_rows(uint32_t wa, uint32_t wb, int byte, float2 off, float2 sc) {
    float2 x = make_float2(__uint_as_float(__byte_perm(wa, 0x4B000000u, 0x7650 + byte)),
                           __uint_as_float(__byte_perm(wb, 0x4B000000u, 0x7650 + byte)));
    x = __fmul2_rn(__fadd2_rn(x, off), sc);
    return pack_bf16_pair(x.x, x.y);
}

// The codes d = 16 g .. 16 g + 15 of key rows row0 + 2 t + {0, 1, 8, 9} of the V code tile, ready
// for pair_of_rows: int8 as four words of four codes (each byte code + 128), int4 as two words of
// low nibbles (elements 16 g + 2 i) and two of high nibbles (elements 16 g + 2 i + 1), each code + 8.
// (bf16 rows: the 16 values themselves, eight words of two.)
template <int BITS>
__device__ __forceinline__ void value_codes(uint32_t tile, int row0, int g, int t, uint32_t (&w)[4][BITS == 16 ? 8 : 4]) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = row0 + 2 * t + (i & 1) + 8 * (i >> 1);
        if constexpr (BITS == 16) {
            // columns 16 g .. 16 g + 15: chunks (g & 3) * 2, + 1 of panel g >> 2
            const uint32_t base = tile + (uint32_t)(g >> 2) * (kKeysPerTile * 128u) + (uint32_t)r * 128u, sw = (uint32_t)r & 7u;
#pragma unroll
            for (uint32_t c = 0; c < 2; ++c) {
                uint32_t x[4];
                lds128(base + (((((uint32_t)g & 3u) << 1) + c) ^ sw) * 16u, x);
#pragma unroll
                for (int k = 0; k < 4; ++k) w[i][4 * c + k] = x[k];
            }
        } else if constexpr (BITS == 8) {
            lds128(tile + (uint32_t)r * 128u + (((uint32_t)g ^ ((uint32_t)r & 7u)) << 4), w[i]);
#pragma unroll
            for (int k = 0; k < 4; ++k) w[i][k] ^= 0x80808080u;
        } else {
            uint32_t x[2];
            lds64(tile + (uint32_t)r * 64u + (((((uint32_t)g >> 1) ^ (((uint32_t)r >> 1) & 3u)) << 4) | (((uint32_t)g & 1u) << 3)), x);
            w[i][0] = x[0] & 0x0F0F0F0Fu; w[i][1] = x[1] & 0x0F0F0F0Fu;
            w[i][2] = (x[0] >> 4) & 0x0F0F0F0Fu; w[i][3] = (x[1] >> 4) & 0x0F0F0F0Fu;
        }
    }
}
// A fragment jp of O^T = V^T P^T: MMA rows g / g + 8 are d = 16 g + 2 jp / + 1, columns the 16 keys.
template <int BITS>
__device__ __forceinline__ void value_fragment(const uint32_t (&w)[4][BITS == 16 ? 8 : 4], int jp, float2 sc01, float2 sc89, uint32_t (&va)[4]) {
    if constexpr (BITS == 16) {
        // word jp of a row holds the row's values at d = 16 g + 2 jp (low half) and + 1 (high half)
        va[0] = __byte_perm(w[0][jp], w[1][jp], 0x5410);
        va[1] = __byte_perm(w[0][jp], w[1][jp], 0x7632);
        va[2] = __byte_perm(w[2][jp], w[3][jp], 0x5410);
        va[3] = __byte_perm(w[2][jp], w[3][jp], 0x7632);
    } else if constexpr (BITS == 8) {
        const float2 off = make_float2(-8388736.f, -8388736.f);          // 2^23 + 128
        const int word = jp >> 1, b = 2 * (jp & 1);
        va[0] = pair_of_rows(w[0][word], w[1][word], b, off, sc01);
        va[1] = pair_of_rows(w[0][word], w[1][word], b + 1, off, sc01);
        va[2] = pair_of_rows(w[2][word], w[3][word], b, off, sc89);
        va[3] = pair_of_rows(w[2][word], w[3][word], b + 1, off, sc89);
    } else {
        const float2 off = make_float2(-8388616.f, -8388616.f);          // 2^23 + 8
        const int word = jp >> 2, b = jp & 3;
        va[0] = pair_of_rows(w[0][word], w[1][word], b, off, sc01);
        va[1] = pair_of_rows(w[0][2 + word], w[1][2 + word], b, off, sc01);
        va[2] = pair_of_rows(w[2][word], w[3][word], b, off, sc89);
        va[3] = pair_of_rows(w[2][2 + word], w[3][2 + word], b, off, sc89);
    }
}

template <int BITS, int NB>
__global__ void __launch_bounds__(Geo<BITS, NB>::kThreads, 1)
attn_q8_decode_kernel(const AttnArgs a, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v) {
    using Gm = Geo<BITS, NB>;
    constexpr int NST = Gm::kStages, kWarps = Gm::kWarps;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - smem_u32(smem_raw));
    Ctl *ctl = reinterpret_cast<Ctl *>(smem + Gm::kOffCtl);
    const uint32_t bar_full = base + Gm::kOffCtl, bar_empty = bar_full + 12 * 8;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t4 = lane & 3;
    const int group = blockIdx.x;
    const int cb = blockIdx.y;     // cache of a batch (0 when there is one cache)
    const int G = a.G;
    // (a ragged batch keeps its members' row counts in device memory, written by an earlier kernel of the
    // stream: those are the one thing read before the set-up below, so wait first there)
    if (a.prefixes) pdl_wait();
    // tokens this cache folds; a.n is the longest chunk of the launch and the stride of the caches' blocks
    const int n = a.ns ? (int)a.ns[cb] : a.n, nmax = a.n, nG = n * G;
    if (n <= 0) return;                                   // a member that sits the step out
    const int64_t P = a.prefixes ? a.prefixes[cb] : a.prefix, L = P + n * a.self_rows;
    const bool direct = a.ngroups == a.Hkv;
    // rows of a partial slot; the slots keep the row layout of the tensor-core kernels, row = token * Gp +
    // head-in-group with Gp = G rounded up to a power of two, because the same merge kernel reads both
    const int64_t slot_rows = (int64_t)nmax * a.Gp;

    // this CTA's range of its KV head's key tiles (the same line arithmetic as the other kernels)
    const int nt_all = (int)((L + kKeysPerTile - 1) / kKeysPerTile);
    const int64_t line = (int64_t)a.Hkv * nt_all;
    const int64_t lin0 = group * line / a.ngroups, lin1 = (group + 1) * line / a.ngroups;
    const int kvh = (int)(lin0 / nt_all);
    const int kt0 = (int)(lin0 - (int64_t)kvh * nt_all);
    const int ntiles = (int)(lin1 - lin0);         // a multiple of the KV heads cuts the line inside heads
    if (ntiles <= 0) {
        // A shorter member of a ragged batch (or a forced split count) can leave a range without a tile: an
        // empty partial, for the merge reads every slot between a head's first and last range.
        pdl_wait();   // (the partial area may still be read by the merge of the step before)
        if (!direct && kvh < a.Hkv)
            for (int item = threadIdx.x; item < nG * (kD / 4); item += blockDim.x) {
                const int r = item / (kD / 4), c4 = item % (kD / 4);
                const int64_t prow = (int64_t)cb * a.part_rows + (int64_t)(group + kvh) * slot_rows + (r / G) * a.Gp + r % G;
                reinterpret_cast<float4 *>(a.part_o + prow * kD)[c4] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (c4 == 0) a.part_lse[prow] = -INFINITY;
            }
        return;
    }

    if (threadIdx.x == 0) {
        for (int s = 0; s < NST; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 2);       // the stage's two consumer warps
        }
        ctl->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    pdl_launch_dependents();
    __syncthreads();
    pdl_wait();   // nothing above reads what an earlier kernel wrote; from here on the rotated chunk and the cache are read

    // what a consumer warp carries through its keys (declared here so that every warp reaches the
    // merge below by the same path): O^T[d = 16 g + 2 jp + {0, 1}][row 8 nb + 2 t + {0, 1}] as
    // ot[nb][jp][{0, 1}] (first d) and [{2, 3}] (second d); maxima and sums of rows 8 nb + 2 t + {0, 1}
    float ot[NB][8][4];
    float m_run[NB][2], l_run[NB][2];
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
        m_run[nb][0] = m_run[nb][1] = -INFINITY;
        l_run[nb][0] = l_run[nb][1] = 0.f;
#pragma unroll
        for (int jp = 0; jp < 8; ++jp)
#pragma unroll
            for (int e = 0; e < 4; ++e) ot[nb][jp][e] = 0.f;
    }

    if (warp == kWarps) {
        if (lane == 0) {
            // ------------------------------------------------------------------ TMA producer
            bool ok = true;
            const int32_t *page_table = a.page_tables ? a.page_tables[cb] : a.page_table;
            for (int t = 0; t < ntiles && ok; ++t) {
                const int s = t % NST;
                ok = mbar_wait(bar_empty + 8 * s, ((t / NST) & 1) ^ 1, ctl, a.status);
                if (!ok) break;
                const int ktile = kt0 + t;
                const int key0 = ktile * kKeysPerTile;
                const uint32_t dst = base + (uint32_t)s * Gm::kStage;
                if (BITS == 16) {
                    // bf16 rows: each tile as two panels of 64 columns (rows past the end of a plane are filled with zeros)
                    constexpr uint32_t kPanel = kKeysPerTile * 128u;
                    mbar_expect_tx(bar_full + 8 * s, 2 * Gm::kCodes);
                    if (page_table) {
                        const int page = page_table[ktile];
                        tma_load_4d(dst, &map_k, bar_full + 8 * s, 0, 0, kvh, page);
                        tma_load_4d(dst + kPanel, &map_k, bar_full + 8 * s, 64, 0, kvh, page);
                        tma_load_4d(dst + Gm::kCodes, &map_v, bar_full + 8 * s, 0, 0, kvh, page);
                        tma_load_4d(dst + Gm::kCodes + kPanel, &map_v, bar_full + 8 * s, 64, 0, kvh, page);
                    } else {
                        tma_load_3d(dst, &map_k, bar_full + 8 * s, 0, key0, kvh);
                        tma_load_3d(dst + kPanel, &map_k, bar_full + 8 * s, 64, key0, kvh);
                        tma_load_3d(dst + Gm::kCodes, &map_v, bar_full + 8 * s, 0, key0, kvh);
                        tma_load_3d(dst + Gm::kCodes + kPanel, &map_v, bar_full + 8 * s, 64, key0, kvh);
                    }
                } else if (page_table) {
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
        // ------------------------------------------------------------------ consumers: 64 keys of every tile of one stage
        const int s = warp >> 1, half = warp & 1;
        // Q^T's B fragments of the eight k-steps, in the order the key codes are taken: k-step ks of
        // thread t covers d = 32 t + 4 ks .. + 3 of query row 8 nb + g
        uint32_t bq[NB][8][2];
        {
            const __nv_bfloat16 *q_rot = reinterpret_cast<const __nv_bfloat16 *>(a.q_rot);
#pragma unroll
            for (int nb = 0; nb < NB; ++nb) {
                const int R = g + 8 * nb, tok = R / G, gi = R % G;
                const __nv_bfloat16 *src = q_rot + (((int64_t)cb * nmax + tok) * a.H + kvh * G + gi) * kD + 32 * t4;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    uint2 w = make_uint2(0u, 0u);
                    if (R < nG) w = *reinterpret_cast<const uint2 *>(src + 4 * ks);
                    bq[nb][ks][0] = w.x;
                    bq[nb][ks][1] = w.y;
                }
            }
        }
        // keys below the limit are visible (rows past the chunk's end are never written; each row of S, P
        // and O depends on that row alone, so they are left unmasked)
        // (counted from the chunk's first key, P)
        int limit[NB][2];
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int R = 8 * nb + 2 * t4 + e;
                limit[nb][e] = R < nG ? (R / G + 1) * a.self_rows : (1 << 30);
            }
        const float sl2 = a.scale_log2;
        bool ok = true;
        for (int t = s; t < ntiles && ok; t += NST) {
            ok = mbar_wait(bar_full + 8 * s, (t / NST) & 1, ctl, a.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const uint32_t k_tile = base + (uint32_t)s * Gm::kStage, v_tile = k_tile + Gm::kCodes;
            // (bf16 rows have no scales: the pointers are then never read)
            const float *k_sc = reinterpret_cast<const float *>(smem + (uint32_t)s * Gm::kStage + 2 * Gm::kCodes);
            const float *v_sc = k_sc + 128;
            const int64_t key_h = (int64_t)(kt0 + t) * kKeysPerTile + half * 64;      // my 64 keys
            // (rows past the end of the planes were not copied: they count as zero)
            const int in_planes = (int)min((int64_t)64, a.capacity - key_h);

            // ---- scores of the 64 keys: four 16-key blocks, sacc[j][nb] = keys g / g + 8 of block j, rows 8 nb + 2 t + {0, 1}
            float sacc[4][NB][4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int rl = 16 * j + g;                       // my first key row within the 64
                uint32_t ka[8][4];
                key_fragments<BITS>(k_tile, half * 64 + rl, t4, BITS != 16 && rl < in_planes ? k_sc[half * 64 + rl] : 0.f,
                                    BITS != 16 && rl + 8 < in_planes ? k_sc[half * 64 + rl + 8] : 0.f, ka);
#pragma unroll
                for (int nb = 0; nb < NB; ++nb) {
                    // a second accumulator for the odd k-steps: two chains of four MMAs instead of one of eight
                    float odd[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) { sacc[j][nb][e] = 0.f; odd[e] = 0.f; }
#pragma unroll
                    for (int ks = 0; ks < 8; ks += 2) {
                        mma_bf16(sacc[j][nb], ka[ks], bq[nb][ks][0], bq[nb][ks][1]);
                        mma_bf16(odd, ka[ks + 1], bq[nb][ks + 1][0], bq[nb][ks + 1][1]);
                    }
#pragma unroll
                    for (int e = 0; e < 4; ++e) sacc[j][nb][e] += odd[e];
                }
            }
            // ---- mask (only where the chunk's own keys are near), running maximum, probabilities
            const bool masked = key_h + 64 > P;
            const int rel = masked ? (int)(key_h - P) + g : 0;      // my first key, counted from P (> -64 where it matters)
            uint32_t pb[4][NB][2];         // P^T as B fragments of the four 16-key steps
            float alpha[NB][2];
            bool rescale = false;
#pragma unroll
            for (int nb = 0; nb < NB; ++nb) {
                float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
                for (int j = 0; j < 4; ++j)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float v = sacc[j][nb][e] * sl2;
                        if (masked && rel + 16 * j + 8 * (e >> 1) >= limit[nb][e & 1]) v = -INFINITY;
                        sacc[j][nb][e] = v;
                        mx[e & 1] = fmaxf(mx[e & 1], v);
                    }
                float m_safe[2];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    mx[e] = fmaxf(mx[e], __shfl_xor_sync(0xffffffffu, mx[e], 4));
                    mx[e] = fmaxf(mx[e], __shfl_xor_sync(0xffffffffu, mx[e], 8));
                    mx[e] = fmaxf(mx[e], __shfl_xor_sync(0xffffffffu, mx[e], 16));
                    const float m_new = fmaxf(m_run[nb][e], mx[e]);
                    m_safe[e] = m_new == -INFINITY ? 0.f : m_new;
                    alpha[nb][e] = ex2(m_run[nb][e] - m_safe[e]);                   // m_run = -inf -> 0
                    m_run[nb][e] = m_new;
                    l_run[nb][e] *= alpha[nb][e];
                    rescale = rescale || alpha[nb][e] != 1.f;
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float p0 = ex2(sacc[j][nb][0] - m_safe[0]), p1 = ex2(sacc[j][nb][1] - m_safe[1]);
                    const float p2 = ex2(sacc[j][nb][2] - m_safe[0]), p3 = ex2(sacc[j][nb][3] - m_safe[1]);
                    l_run[nb][0] += p0 + p2;
                    l_run[nb][1] += p1 + p3;
                    // (key g, rows 2 t, 2 t + 1) transposed: (keys 2 t, 2 t + 1; row g) - P^T's b0; keys + 8: b1
                    pb[j][nb][0] = transpose8x8(pack_bf16_pair(p0, p1));
                    pb[j][nb][1] = transpose8x8(pack_bf16_pair(p2, p3));
                }
            }
            if (__any_sync(0xffffffffu, rescale)) {
#pragma unroll
                for (int nb = 0; nb < NB; ++nb)
#pragma unroll
                    for (int jp = 0; jp < 8; ++jp) {
                        ot[nb][jp][0] *= alpha[nb][0]; ot[nb][jp][1] *= alpha[nb][1];
                        ot[nb][jp][2] *= alpha[nb][0]; ot[nb][jp][3] *= alpha[nb][1];
                    }
            }
            // ---- O^T += V^T P^T, 16 keys at a time
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int r0 = 16 * j + 2 * t4;                  // my first key row within the 64
                float2 sc01, sc89;
                sc01.x = BITS != 16 && r0 < in_planes ? v_sc[half * 64 + r0] : 0.f;
                sc01.y = BITS != 16 && r0 + 1 < in_planes ? v_sc[half * 64 + r0 + 1] : 0.f;
                sc89.x = BITS != 16 && r0 + 8 < in_planes ? v_sc[half * 64 + r0 + 8] : 0.f;
                sc89.y = BITS != 16 && r0 + 9 < in_planes ? v_sc[half * 64 + r0 + 9] : 0.f;
                uint32_t w[4][BITS == 16 ? 8 : 4];
                value_codes<BITS>(v_tile, half * 64 + 16 * j, g, t4, w);
#pragma unroll
                for (int jp = 0; jp < 8; ++jp) {
                    uint32_t va[4];
                    value_fragment<BITS>(w, jp, sc01, sc89, va);
#pragma unroll
                    for (int nb = 0; nb < NB; ++nb) mma_bf16(ot[nb][jp], va, pb[j][nb][0], pb[j][nb][1]);
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
        for (int nb = 0; nb < NB; ++nb)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                float l = l_run[nb][e];          // my keys' share; the other keys sit in the threads of the other g
                l += __shfl_xor_sync(0xffffffffu, l, 4);
                l += __shfl_xor_sync(0xffffffffu, l, 8);
                l += __shfl_xor_sync(0xffffffffu, l, 16);
                const int r = 8 * nb + 2 * t4 + e;
#pragma unroll
                for (int jp = 0; jp < 8; ++jp)
                    *reinterpret_cast<float2 *>(mo + r * kD + 16 * g + 2 * jp) = make_float2(ot[nb][jp][e], ot[nb][jp][2 + e]);
                if (g == 0) {
                    mm[2 * r] = m_run[nb][e];
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
            const int64_t row = ((int64_t)cb * nmax + tok) * a.H + kvh * G + gi;
            if (!direct) {
                const int64_t prow = (int64_t)cb * a.part_rows + (int64_t)(group + kvh) * slot_rows + (r / G) * a.Gp + r % G;
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
    static_assert(Geo<8, 1>::kSmem <= 232448 && Geo<8, 2>::kSmem <= 232448 && Geo<16, 1>::kSmem <= 232448, "shared memory budget of one CTA");
    static_assert(Geo<8, 1>::kStages <= 12, "control block holds 12 stages");
    static_assert(Geo<16, 1>::kWarps * kMergeWarp <= Geo<16, 1>::kOffCtl, "the merge area reuses the ring");
    const bool wide = a.n * a.G > 8;
    const int bits = a.quant_bits ? a.quant_bits : 16;              // 16: plain bf16 rows
    auto kernel = bits == 4 ? (wide ? attn_q8_decode_kernel<4, 2> : attn_q8_decode_kernel<4, 1>)
                : bits == 8 ? (wide ? attn_q8_decode_kernel<8, 2> : attn_q8_decode_kernel<8, 1>)
                            : (wide ? attn_q8_decode_kernel<16, 2> : attn_q8_decode_kernel<16, 1>);
    const uint32_t smem = bits == 4 ? (wide ? Geo<4, 2>::kSmem : Geo<4, 1>::kSmem)
                        : bits == 8 ? (wide ? Geo<8, 2>::kSmem : Geo<8, 1>::kSmem) : (wide ? Geo<16, 2>::kSmem : Geo<16, 1>::kSmem);
    cudaError_t e = raise_smem_limit_once(reinterpret_cast<const void *>(kernel), (int)smem);
    if (e != cudaSuccess) return e;
    const int threads = bits == 16 ? Geo<16, 1>::kThreads : wide ? Geo<8, 2>::kThreads : Geo<8, 1>::kThreads;
    return launch_pdl(kernel, dim3(a.ngroups, a.batch), dim3(threads), smem, s, a, maps.k, maps.v);
}

}  // namespace kvf
