// Tensor-core prefix + chunk attention for fp32 caches with head_dim 128 (sm_100a: tcgen05.mma, TMEM).
//
// Section 2 of the paper: the chunk's queries attend to [K_0;...;K_t], [V_0;...;V_t]; rows of
// earlier chunks are fully visible, rows of the chunk itself causally; query head h reads KV
// head h / G.  The paper's precision ablation (Section 3, "Source of the drift") runs the same
// fold in bf16 and in fp32; this is the fp32 side on the tensor pipe.
//
// fp32 accuracy from 16-bit tensor-core operands.  A single tensor-core pass over fp32 data
// (tf32, bf16, fp16) keeps 8 to 11 significant bits and cannot meet a 1e-5 absolute tolerance.
// Here every fp32 operand x is split into two fp16 numbers, hi = fp16(x) and lo = fp16(x - hi),
// which together carry 22 significant bits (elements below 2^-3 are kept to an absolute 2^-25,
// the spacing of fp16 subnormals), and every product A B becomes three MMAs,
//     A_hi B_hi + A_hi B_lo + A_lo B_hi          (the dropped A_lo B_lo term is below 2^-22),
// each sum over a 64-key step only (scores) or over its 64 keys (output), in fp32 accumulators.  The accumulator of a tensor-core MMA is not rounded to nearest when it is
// updated, which matters once thousands of updates pile up: O = P V is therefore accumulated in
// tensor memory over ONE 64-key step only and then added, in round-to-nearest fp32, to the
// running output row that the softmax thread keeps in registers.  Scores take 16 MMA updates
// per 64-key step, the output 12.  fp16 holds magnitudes up to 65 504: the rotate + append kernel
// checks every rotated key and query and every value it writes for such a cache and sets code 7
// (KVF_ERR_RANGE) in the device status word when one is larger; such caches belong on the
// CUDA-core kernel (KVF_FORCE_SIMT).
//
// Work decomposition (as for the bf16 kernel, with 128-row blocks instead of 256-row pairs): row
// = token * G + head-in-group; the (KV head, 128-key tile) pairs of a step form one line that is
// cut into `ngroups` contiguous ranges; CTA (x = row block, y = group) runs its 128 rows over its
// range, at most two KV heads ("pieces"), in steps of 64 keys.  With ngroups == Hkv the CTA
// writes final outputs, otherwise each piece leaves a normalised partial and its log2
// denominator in slot (group + KV head) for combine_groups_kernel.
//
// Roles (512 threads, one CTA per SM):
//   warps 0-3   softmax, one thread per row (TMEM lane = row): scores of a step from tensor memory
//               (read twice: maximum, then exponentials), probabilities split into fp16 hi / lo and
//               written back to tensor memory, the step's P V added to the 128 output registers
//   warps 4-7   K converters: 16 rows of the step's K tile per warp, fp32 from global memory (one
//               coalesced 512-byte row per warp instruction), split, written as 128-byte-swizzled
//               K-major fp16 tiles into a ring of three slots; in a slot the 64 rows of K_lo follow
//               the 64 rows of K_hi inside each 64-column panel, so [K_hi; K_lo] is ONE 128-row operand
//   warps 8-11  V converters: the same for V (ring of two slots, V_hi then V_lo; a V tile is read
//               MN-major, so its rows are laid out as a K tile's); both converter groups also split
//               the piece's 128 x 128 Q tile
//   warp 12     issuer of the score MMAs (one thread) and owner of the tensor-memory allocation
//   warp 13     issuer of the output MMAs (one thread)
// One tcgen05.mma costs its issuing thread about as long as a 128 x 128 x 16 MMA runs, whatever its
// N, so the kernel is built to issue few, wide MMAs from two threads: per 64-key step and 16
// elements of d, Q_hi [K_hi; K_lo]^T is one MMA with N = 128 (its columns 0-63 are Q_hi K_hi, 64-127
// the small term Q_hi K_lo) and Q_lo K_hi^T one with N = 64 added onto columns 0-63; the softmax
// adds the two halves of a score.  16 score MMAs and 12 output MMAs per step (a first version with
// 24 + 12 from one thread spent ~120 cycles per MMA on issue alone and left the tensor pipe 70 % idle).
// Tensor memory: S0 | S1 (128 fp32 columns each: 64 scores + 64 small terms) | P0 | P1 (hi: 32
// columns, lo: 32 columns) | O (128).  The score issuer runs ahead of the softmax by one step (S is
// double-buffered), the output issuer starts a step's P V as soon as its probabilities are
// written and the previous P V has been added to the registers.
//
// Every wait on an mbarrier is bounded and reports through the status word, as in the bf16 kernel.
#include "kvfold_internal.h"
#include "sm100_ptx.cuh"

#include <cuda_fp16.h>

namespace kvf {
namespace {

constexpr int kRows = 128;                     // query rows of a CTA
constexpr int kD = 128;                        // head_dim
constexpr int kKeys = 64;                      // keys of one step
constexpr int kTileKeys = 128;                 // keys of one tile of the plan's line = two steps
constexpr int kThreads = 512;
constexpr uint32_t kQPanel = kRows * 128;      // [128 rows][64 fp16], 128-byte swizzle
constexpr uint32_t kQPart = 2 * kQPanel;       // hi or lo of the Q tile
constexpr uint32_t kKPanel = kKeys * 128;      // [64 keys][64 fp16]
constexpr uint32_t kKPart = 2 * kKPanel;       // hi or lo of a K (or V) step tile
constexpr uint32_t kKSlot = 2 * kKPart;        // hi + lo
constexpr int kKSlots = 3, kVSlots = 2;
constexpr uint32_t kOffQ = 0;                                  // Q hi, Q lo
constexpr uint32_t kOffK = 2 * kQPart;
constexpr uint32_t kOffV = kOffK + kKSlots * kKSlot;
constexpr uint32_t kOffCtl = kOffV + kVSlots * kKSlot;
constexpr uint32_t kSmemBytes = kOffCtl + 512 + 1024;          // + control block + alignment slack
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0, kColP = 256, kColO = 384;        // S0|S1 at 0, 128; P0|P1 at 256, 320; O at 384
constexpr uint32_t kKOperand = 2 * kKPanel;                    // one 64-column panel of [K_hi; K_lo]: 128 rows
constexpr float kRescaleThreshold = 8.0f;                      // log2 units

enum { B_QFULL = 0, B_QEMPTY = 1, B_KFULL0 = 2, B_KEMPTY0 = B_KFULL0 + kKSlots, B_VFULL0 = B_KEMPTY0 + kKSlots,
       B_VEMPTY0 = B_VFULL0 + kVSlots, B_SFULL0 = B_VEMPTY0 + kVSlots, B_SFREE0 = B_SFULL0 + 2, B_PFULL0 = B_SFREE0 + 2,
       B_OFULL = B_PFULL0 + 2, B_OFREE = B_OFULL + 1, B_DRAIN0 = B_OFREE + 1, B_COUNT = B_DRAIN0 + 2 };

struct Ctl {
    unsigned long long bars[32];
    uint32_t tmem_base;
    int abort;
    long long clk0;                // start of the CTA in SM cycles and in nanoseconds (the timed CTA only)
    unsigned long long ns0;
};
static_assert(B_COUNT <= 32, "control block holds 32 barriers");

// K-major operand: [rows][64 fp16] panels, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t addr) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// MN-major operand (V: [keys][64 fp16 of d] panels of 64 keys; the next 64 columns of d are one
// panel further, the next 8 keys 1024 bytes further).
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t addr) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)(kKPanel >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Instruction descriptors: D fp32, A and B fp16 (format 0), M = 128; scores N = 64, output N = 128
// with B MN-major (bit 16).
constexpr uint32_t kIdescQK64 = (1u << 4) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescQK128 = (1u << 4) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescPV = (1u << 4) | (1u << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ uint32_t half2_bits(__half2 h) { return *reinterpret_cast<uint32_t *>(&h); }

// x = hi + lo with hi = fp16(x), lo = fp16(x - hi), two elements at a time.
__device__ __forceinline__ void split2(float a, float b, uint32_t &hi, uint32_t &lo) {
    const __half2 h = __floats2half2_rn(a, b);
    const float2 f = __half22float2(h);
    hi = half2_bits(h);
    lo = half2_bits(__floats2half2_rn(a - f.x, b - f.y));
}

// One fp32 row segment of four elements -> 8 bytes of hi and 8 bytes of lo at the swizzled place
// of (row r, elements 4 * lane .. 4 * lane + 3) in a K-major tile whose panels hold `panel` bytes.
// (Plain stores: the rows of a tile are independent, and the compiler may interleave their
// conversions; the proxy fence and the barrier arrive behind the tile order them for the MMAs.)
__device__ __forceinline__ void store_split4(uint8_t *part_hi, uint8_t *part_lo, uint32_t panel, int r, int lane, float4 x) {
    uint32_t h0, l0, h1, l1;
    split2(x.x, x.y, h0, l0);
    split2(x.z, x.w, h1, l1);
    const uint32_t off = (uint32_t)(lane >> 4) * panel + (uint32_t)r * 128u +
                         ((((uint32_t)(lane & 15) >> 1) ^ ((uint32_t)r & 7u)) << 4) + ((uint32_t)lane & 1u) * 8u;
    *reinterpret_cast<uint2 *>(part_hi + off) = make_uint2(h0, h1);
    *reinterpret_cast<uint2 *>(part_lo + off) = make_uint2(l0, l1);
}

// 16 columns x (32-bit) of this thread's TMEM lane <-> registers
#define KVF_TMEM_LD16(a, o, taddr)                                                              \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 "                                      \
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];" \
                 : "=r"(a[o + 0]), "=r"(a[o + 1]), "=r"(a[o + 2]), "=r"(a[o + 3]), "=r"(a[o + 4]), "=r"(a[o + 5]), "=r"(a[o + 6]), "=r"(a[o + 7]), \
                   "=r"(a[o + 8]), "=r"(a[o + 9]), "=r"(a[o + 10]), "=r"(a[o + 11]), "=r"(a[o + 12]), "=r"(a[o + 13]), "=r"(a[o + 14]), "=r"(a[o + 15]) \
                 : "r"(taddr) : "memory")
#define KVF_TMEM_ST8(a, o, taddr)                                                               \
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%8], {%0, %1, %2, %3, %4, %5, %6, %7};" \
                 ::"r"(a[o + 0]), "r"(a[o + 1]), "r"(a[o + 2]), "r"(a[o + 3]), "r"(a[o + 4]), "r"(a[o + 5]), "r"(a[o + 6]), "r"(a[o + 7]), \
                   "r"(taddr) : "memory")

// kPair: the CTAs of row blocks 2k and 2k + 1 form a cluster of two that walks the same 64-key steps.  Each
// converts 32 of a step's 64 key rows (K and V) into its own slot and, with bulk copies that complete on the
// partner's FULL barrier, into the partner's; a slot is free once the issuers of BOTH CTAs have committed their
// reads of it.  Each SM then loads and converts half the fp32 rows.  The host launches this variant only when
// the row blocks come in twos (a chunk of a multiple of 256 / G tokens).
template <bool kWindow, bool kPair = false>
__global__ void __launch_bounds__(kThreads, 1) attn_tc32_kernel(const AttnArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    Ctl *ctl = reinterpret_cast<Ctl *>(smem_raw + (base - smem_u32(smem_raw)) + kOffCtl);
    const uint32_t bar0 = base + kOffCtl;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rblock = blockIdx.x, group = blockIdx.y;
    const uint32_t rank = kPair ? cluster_cta_rank() : 0u;
    const int G = a.Gp, Gq = a.G, n = a.n;      // rows per token in the row layout (a power of two), query heads per KV head
    const int64_t P = a.prefix, L = P + n * a.self_rows;
    const bool direct = a.ngroups == a.Hkv;
    const int row0 = rblock * kRows;
    // (paired variant: both CTAs of a cluster take the steps the later row block needs; the earlier one finds
    // nothing visible in the last of them, and its rows' limits mask those keys out)
    const int tok_last = min(n - 1, ((kPair ? (rblock | 1) * kRows : row0) + kRows - 1) / G);
    const int64_t need = P + (tok_last + 1) * a.self_rows;            // keys below `need` are visible to some row of this CTA
    // (virtual key tiles: without a window they are the key tiles themselves)
    const WindowTiles wt(kWindow ? a.win_lo : 0, kWindow ? a.n_sink : 0, kTileKeys);
    const int nt_need = (int)((need + kTileKeys - 1) / kTileKeys) - wt.skip;
    const int nt_all = (int)((L + kTileKeys - 1) / kTileKeys) - wt.skip;
    const int64_t line = (int64_t)a.Hkv * nt_all;
    const int64_t lin0 = group * line / a.ngroups, lin1 = (group + 1) * line / a.ngroups;
    const int kvh_first = (int)(lin0 / nt_all);
    // piece of this CTA on KV head kvh: tiles [kt0, kt0 + ntiles) of the line, walked as nsteps
    // 64-key steps (the second half of the last tile is left out if no row of the CTA sees it)
    auto piece = [&](int kvh, int &kt0, int &ntiles, int &nsteps) -> bool {
        const int64_t b = (int64_t)kvh * nt_all;
        if (kvh >= a.Hkv || b >= lin1) return false;
        kt0 = (int)(max(lin0, b) - b);
        const int kt1 = (int)min(min(lin1, b + nt_all) - b, (int64_t)nt_need);
        ntiles = kt1 - kt0;
        nsteps = 0;
        if (ntiles > 0) {
            const int64_t last_half = (int64_t)wt.actual(kt1 - 1) * kTileKeys + kKeys;
            nsteps = 2 * ntiles - (last_half >= need ? 1 : 0);
        }
        return true;
    };
    auto step_key0 = [&](int kt0, int s) { return (int64_t)wt.actual(kt0 + (s >> 1)) * kTileKeys + (s & 1) * kKeys; };

    if (threadIdx.x == 0) {
        mbar_init(bar(B_QFULL), 8);
        mbar_init(bar(B_QEMPTY), 1);
        for (int s = 0; s < kKSlots; ++s) { mbar_init(bar(B_KFULL0 + s), 4); mbar_init(bar(B_KEMPTY0 + s), kPair ? 2 : 1); }
        for (int s = 0; s < kVSlots; ++s) { mbar_init(bar(B_VFULL0 + s), 4); mbar_init(bar(B_VEMPTY0 + s), kPair ? 2 : 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(B_SFULL0 + i), 1);
            mbar_init(bar(B_SFREE0 + i), 4);
            mbar_init(bar(B_PFULL0 + i), 4);
        }
        mbar_init(bar(B_OFULL), 1);
        mbar_init(bar(B_OFREE), 4);
        mbar_init(bar(B_DRAIN0), 1);
        mbar_init(bar(B_DRAIN0 + 1), 1);
        ctl->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 12) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    pdl_launch_dependents();
    tc_fence_before();
    __syncthreads();
    if (kPair) cluster_sync_all();      // the partner's barriers exist before anything is sent to them
    tc_fence_after();
    pdl_wait();   // nothing above reads what an earlier kernel wrote; from here on the rotated chunk and the cache are read
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(&ctl->tmem_base);
    // One CTA times itself in SM cycles and in nanoseconds: the ratio is the clock the launch ran at
    // (the last row block: it sees the most keys of the chunk itself, so no CTA of the launch runs longer)
    const bool clocked = blockIdx.x == gridDim.x - 1 && blockIdx.y == 0 && threadIdx.x == 0;
    if (clocked) {
        ctl->clk0 = clock64();
        ctl->ns0 = global_ns();
    }

    if (warp >= 12) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 48;");
        if (warp == 12 && lane == 0) {
            // ------------------------------------------------------------------ issuer of the score MMAs
            const uint64_t dqh = desc_kmajor(base + kOffQ), dql = desc_kmajor(base + kOffQ + kQPart);
            int g = 0;                   // steps so far, all pieces = load number of the K ring
            int pc = 0;                  // pieces so far
            bool ok = true;
            int kt0, ntiles, nsteps;
            for (int kvh = kvh_first; ok && piece(kvh, kt0, ntiles, nsteps); ++kvh) {
                if (nsteps <= 0) continue;
                ok = mbar_wait(bar(B_QFULL), pc & 1, ctl, a.status);
                if (!ok) break;
                for (int j = 0; j < nsteps; ++j, ++g) {
                    const int b = g & 1, slot = g % kKSlots;
                    ok = mbar_wait(bar(B_SFREE0 + b), ((g >> 1) & 1) ^ 1, ctl, a.status);
                    if (ok) ok = mbar_wait(bar(B_KFULL0 + slot), (g / kKSlots) & 1, ctl, a.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t dk = desc_kmajor(base + kOffK + (uint32_t)slot * kKSlot);
                    const uint32_t t_s = tmem + kColS + 128u * (uint32_t)b;
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {          // 16 elements of d per MMA: Q_hi [K_hi; K_lo]^T, 128 columns
                        const uint64_t qo = (uint64_t)(((kk >> 2) * kQPanel + (kk & 3) * 32) >> 4);
                        const uint64_t ko = (uint64_t)(((kk >> 2) * kKOperand + (kk & 3) * 32) >> 4);
                        tc_mma(t_s, dqh + qo, dk + ko, kIdescQK128, kk > 0);
                    }
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {          // Q_lo K_hi^T onto columns 0-63
                        const uint64_t qo = (uint64_t)(((kk >> 2) * kQPanel + (kk & 3) * 32) >> 4);
                        const uint64_t ko = (uint64_t)(((kk >> 2) * kKOperand + (kk & 3) * 32) >> 4);
                        tc_mma(t_s, dql + qo, dk + ko, kIdescQK64, 1);
                    }
                    tc_commit(bar(B_SFULL0 + b));
                    if (kPair) tc_commit_pair(bar(B_KEMPTY0 + slot));     // the partner's converters write my slot too
                    else tc_commit(bar(B_KEMPTY0 + slot));
                }
                if (!ok) break;
                tc_commit(bar(B_QEMPTY));                     // every Q K^T of this piece has been issued
                ++pc;
            }
            // tensor memory is released only after every MMA issued here has run
            tc_commit(bar(B_DRAIN0));
            mbar_wait_drain(bar(B_DRAIN0), 0, a.status);
        } else if (warp == 13 && lane == 0) {
            // ------------------------------------------------------------------ issuer of the output MMAs
            int g = 0;                   // steps so far, all pieces = load number of the V ring
            bool ok = true;
            int kt0, ntiles, nsteps;
            for (int kvh = kvh_first; ok && piece(kvh, kt0, ntiles, nsteps); ++kvh) {
                for (int j = 0; j < nsteps; ++j, ++g) {
                    const int b = g & 1, slot = g % kVSlots;
                    ok = mbar_wait(bar(B_VFULL0 + slot), (g / kVSlots) & 1, ctl, a.status);
                    if (ok) ok = mbar_wait(bar(B_PFULL0 + b), (g >> 1) & 1, ctl, a.status);
                    if (ok && g > 0) ok = mbar_wait(bar(B_OFREE), (g - 1) & 1, ctl, a.status);   // the previous P V has been added
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t v_hi = base + kOffV + (uint32_t)slot * kKSlot;
                    const uint32_t p_hi = tmem + kColP + 64u * (uint32_t)b, p_lo = p_hi + 32u, t_o = tmem + kColO;
                    const uint64_t dvh = desc_mnmajor(v_hi), dvl = desc_mnmajor(v_hi + kKPart);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {          // 16 keys = 8 packed columns of P per MMA; small terms first
                        const uint64_t vo = (uint64_t)((kk * 2048) >> 4);
                        tc_mma_ts(t_o, p_hi + kk * 8, dvl + vo, kIdescPV, kk > 0);
                        tc_mma_ts(t_o, p_lo + kk * 8, dvh + vo, kIdescPV, 1);
                    }
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        tc_mma_ts(t_o, p_hi + kk * 8, dvh + (uint64_t)((kk * 2048) >> 4), kIdescPV, 1);
                    tc_commit(bar(B_OFULL));
                    if (kPair) tc_commit_pair(bar(B_VEMPTY0 + slot));
                    else tc_commit(bar(B_VEMPTY0 + slot));
                }
            }
            tc_commit(bar(B_DRAIN0 + 1));
            mbar_wait_drain(bar(B_DRAIN0 + 1), 0, a.status);
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ converters: fp32 rows -> fp16 hi / lo tiles
        asm volatile("setmaxnreg.dec.sync.aligned.u32 104;");
        const bool is_v = warp >= 8;
        const int w4 = (warp - 4) & 3;                       // warp within its converter group
        const int w8 = warp - 4;                             // warp among all converters (Q tile)
        const float *plane = reinterpret_cast<const float *>(is_v ? a.v_plane : a.k_plane);
        const float *q_rot = reinterpret_cast<const float *>(a.q_rot);
        const int nslots = is_v ? kVSlots : kKSlots;
        const uint32_t ring = is_v ? kOffV : kOffK;
        uint8_t *smem = smem_raw + (base - smem_u32(smem_raw));        // the 1024-byte aligned tile area
        const int b_full = is_v ? B_VFULL0 : B_KFULL0, b_empty = is_v ? B_VEMPTY0 : B_KEMPTY0;
        int lc = 0, pc = 0;                                  // ring loads and pieces so far
        bool ok = true;
        int kt0, ntiles, nsteps;
        for (int kvh = kvh_first; ok && piece(kvh, kt0, ntiles, nsteps); ++kvh) {
            if (nsteps <= 0) continue;
            {
                // the piece's Q tile: 16 rows per converter warp, row = token * G + head-in-group
                float4 x[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int R = row0 + w8 * 16 + i, tok = R / G, gi = R % G;
                    x[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (tok < n && gi < Gq) x[i] = *reinterpret_cast<const float4 *>(q_rot + ((int64_t)tok * a.H + kvh * Gq + gi) * kD + lane * 4);
                }
                if (pc > 0) ok = mbar_wait(bar(B_QEMPTY), (pc - 1) & 1, ctl, a.status);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    store_split4(smem + kOffQ, smem + kOffQ + kQPart, kQPanel, w8 * 16 + i, lane, x[i]);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the MMAs read through the async proxy
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B_QFULL));
                ++pc;
            }
            const float *head = plane + (int64_t)kvh * a.capacity * kD;
            // rows of a step this warp converts: 16 of the 64, or 8 of this CTA's 32 in the paired variant
            constexpr int NR = kPair ? 8 : 16;
            const int r0 = kPair ? (int)rank * 32 + w4 * 8 : w4 * 16;
            for (int s = 0; s < nsteps; ++s, ++lc) {
                const int64_t key0 = step_key0(kt0, s);
                // rows past the end of the cache are not content (and may hold anything): they count as zero
                float4 x[NR];
#pragma unroll
                for (int i = 0; i < NR; ++i) {
                    const int64_t key = key0 + r0 + i;
                    x[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (key < L) x[i] = *reinterpret_cast<const float4 *>(head + key * kD + lane * 4);
                }
                const int slot = lc % nslots;
                ok = mbar_wait(bar(b_empty + slot), ((lc / nslots) & 1) ^ 1, ctl, a.status);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                // K: lo rows behind the hi rows inside each panel (one 128-row operand); V: hi tile, then lo tile
                uint8_t *dst = smem + ring + (uint32_t)slot * kKSlot;
                uint8_t *dst_lo = dst + (is_v ? kKPart : kKPanel);
                const uint32_t panel = is_v ? kKPanel : kKOperand;
#pragma unroll
                for (int i = 0; i < NR; ++i) store_split4(dst, dst_lo, panel, r0 + i, lane, x[i]);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the MMAs (and the copies below) read through the async proxy
                __syncwarp();
                if (lane == 0) {
                    if (kPair) {
                        // The partner's 32 rows are on their way: my warp's arrival on the FULL barrier of MY slot (one
                        // of them also books the 16 KiB), then my warp's 8 rows of the four blocks (hi and lo of both
                        // panels) to the same place in the partner's slot, completing on the partner's barrier.  The slot
                        // is free in both CTAs (the EMPTY barrier counts the issuers of both), and neither rewrites it
                        // before the other's issuer has committed, which it does after these bytes have landed.
                        if (w4 == 0) mbar_expect_tx(bar(b_full + slot), kKSlot / 2);
                        else mbar_arrive(bar(b_full + slot));
                        const uint32_t peer_bar = peer_smem(bar(b_full + slot), rank ^ 1u);
                        const uint32_t s_hi = base + ring + (uint32_t)slot * kKSlot + (uint32_t)r0 * 128u;
                        const uint32_t s_lo = s_hi + (is_v ? kKPart : kKPanel);
#pragma unroll
                        for (uint32_t pnl = 0; pnl < 2; ++pnl) {
                            bulk_push(peer_smem(s_hi + pnl * panel, rank ^ 1u), s_hi + pnl * panel, 8u * 128u, peer_bar);
                            bulk_push(peer_smem(s_lo + pnl * panel, rank ^ 1u), s_lo + pnl * panel, 8u * 128u, peer_bar);
                        }
                    } else {
                        mbar_arrive(bar(b_full + slot));
                    }
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax and output rows, one thread per row
        asm volatile("setmaxnreg.inc.sync.aligned.u32 248;");
        const int r = warp * 32 + lane;                  // row of the CTA = TMEM lane
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        const int R = row0 + r, tok = R / G, gi = R % G;
        const bool valid = tok < n && gi < Gq;       // (gi >= Gq: padding of a group that is no power of two)
        // keys below `limit` are visible; a row past the chunk's end is never written, and each
        // row of S, P and O depends on that row alone, so such rows are left unmasked
        const int64_t limit = valid ? P + (tok + 1) * a.self_rows : ((int64_t)1 << 62);
        const float sl2 = a.scale_log2;
        const int64_t nG = (int64_t)n * G;
        const uint32_t t_o = tmem + lane_addr + kColO;

        int g = 0;                     // steps so far, all pieces
        bool ok = true;
        int kt0, ntiles, nsteps;
        for (int kvh = kvh_first; ok && piece(kvh, kt0, ntiles, nsteps); ++kvh) {
            const int64_t prow = (int64_t)(group + kvh) * nG + R;      // my partial row
            if (nsteps <= 0) {
                // no visible key for these rows in this range: an empty partial
                if (!direct && valid) {
                    float4 *po = reinterpret_cast<float4 *>(a.part_o + prow * kD);
#pragma unroll 4
                    for (int c = 0; c < kD / 4; ++c) po[c] = make_float4(0.f, 0.f, 0.f, 0.f);
                    a.part_lse[prow] = -INFINITY;
                }
                continue;
            }
            float m_ref = -INFINITY;   // reference maximum (raw score units) the probabilities are scaled by
            float l = 0.f;
            float o[kD];               // the running output row, unnormalised, in round-to-nearest fp32
#pragma unroll
            for (int c = 0; c < kD; ++c) o[c] = 0.f;
            float alpha = 1.f;         // factor the reference moved by at the current step: owed to the P V of the step before

            // adds the finished P V of the step before (computed under the old reference) and applies alpha
            auto add_pv = [&](float scale) -> bool {
                bool got = mbar_wait(bar(B_OFULL), (g - 1) & 1, ctl, a.status);
                got = __all_sync(0xffffffffu, got);
                if (!got) return false;
                tc_fence_after();
                const bool rescale = __any_sync(0xffffffffu, scale != 1.f);      // rare: the reference moved at this step
                const float2 sv = make_float2(scale, scale);
#pragma unroll
                for (int c0 = 0; c0 < kD; c0 += 32) {
                    uint32_t t[32];
                    KVF_TMEM_LD32(t, 0, t_o + c0);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        float2 v = __fadd2_rn(make_float2(o[c0 + c], o[c0 + c + 1]), make_float2(__uint_as_float(t[c]), __uint_as_float(t[c + 1])));
                        if (rescale) v = __fmul2_rn(v, sv);
                        o[c0 + c] = v.x;
                        o[c0 + c + 1] = v.y;
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B_OFREE));
                return true;
            };

            for (int j = 0; j < nsteps; ++j, ++g) {
                const int b = g & 1;
                const uint32_t t_s = tmem + lane_addr + kColS + 128u * (uint32_t)b;     // 64 scores, then their 64 small terms
                const uint32_t t_p = tmem + lane_addr + kColP + 64u * (uint32_t)b;
                ok = mbar_wait(bar(B_SFULL0 + b), (g >> 1) & 1, ctl, a.status);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                const int64_t key0 = step_key0(kt0, j);
                const int nvis = (int)max((int64_t)0, min((int64_t)kKeys, limit - key0));
                // a step that starts before the window holds hidden columns (the sink tile, the window's first)
                const bool masked = __any_sync(0xffffffffu, nvis < kKeys) || (kWindow && key0 < a.win_lo);
                const int lo_c = kWindow ? (int)max((int64_t)0, min((int64_t)kKeys, a.win_lo - key0)) : 0;
                const int sink_c = kWindow ? (int)max((int64_t)0, min((int64_t)kKeys, (int64_t)a.n_sink - key0)) : 0;

                // first reading of the scores: the row maximum
                // the step's 64 scores (columns c and 64 + c added up) into registers, and the row maximum
                float v[64];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t sc[32], sx[32];
                    KVF_TMEM_LD32(sc, 0, t_s + 32 * h);
                    KVF_TMEM_LD32(sx, 0, t_s + 64 + 32 * h);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        const float2 t = __fadd2_rn(make_float2(__uint_as_float(sc[c]), __uint_as_float(sc[c + 1])),
                                                    make_float2(__uint_as_float(sx[c]), __uint_as_float(sx[c + 1])));
                        v[32 * h + c] = t.x;
                        v[32 * h + c + 1] = t.y;
                    }
                }
                // the scores are in registers: the issuer may overwrite them with the step after next
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B_SFREE0 + b));
                if (masked) {
#pragma unroll
                    for (int c = 0; c < 64; ++c) v[c] = (c < nvis && (c >= lo_c || c < sink_c)) ? v[c] : -INFINITY;
                }
                float mx[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) mx[q] = fmaxf(v[2 * q], v[2 * q + 1]);
#pragma unroll
                for (int c = 16; c < 64; c += 16)
#pragma unroll
                    for (int q = 0; q < 8; ++q) mx[q] = max3(mx[q], v[c + 2 * q], v[c + 2 * q + 1]);
                const float m_tile = fmaxf(max3(mx[0], mx[1], mx[2]), max3(max3(mx[3], mx[4], mx[5]), mx[6], mx[7]));
                // move the reference only when the maximum grew by more than the threshold: the
                // probabilities then stay below 2^threshold and the output row is rarely rescaled
                const bool grow = (m_tile - m_ref) * sl2 > kRescaleThreshold;   // also true when m_ref = -inf < m_tile
                alpha = 1.f;
                if (grow) {
                    alpha = ex2((m_ref - m_tile) * sl2);                         // m_ref = -inf -> 0
                    l *= alpha;
                    m_ref = m_tile;
                }
                const float m_safe = m_ref == -INFINITY ? 0.f : m_ref;
                const float neg = -m_safe * sl2;

                // probabilities, split into fp16 hi / lo, written 16 keys at a time
                float2 acc = make_float2(0.f, 0.f);
                const float2 sl2v = make_float2(sl2, sl2), negv = make_float2(neg, neg);
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    uint32_t ph[8], pl[8];
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const float2 x = __ffma2_rn(make_float2(v[16 * h + 2 * c], v[16 * h + 2 * c + 1]), sl2v, negv);
                        float2 e;
                        e.x = ex2(x.x);
                        e.y = ex2(x.y);
                        acc = __fadd2_rn(acc, e);
                        const __half2 hh = __floats2half2_rn(e.x, e.y);
                        const float2 back = __half22float2(hh);
                        const float2 rest = __fadd2_rn(e, make_float2(-back.x, -back.y));
                        ph[c] = half2_bits(hh);
                        pl[c] = half2_bits(__floats2half2_rn(rest.x, rest.y));
                    }
                    KVF_TMEM_ST8(ph, 0, t_p + 8 * h);
                    KVF_TMEM_ST8(pl, 0, t_p + 32 + 8 * h);
                }
                l += acc.x + acc.y;
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B_PFULL0 + b));

                // the P V of the step before has had this step's softmax to finish in
                if (j > 0) {                  // (first step of a piece: nothing accumulated yet, o is zero)
                    ok = add_pv(alpha);
                    if (!ok) break;
                }
            }
            if (!ok) break;
            // the last step's P V (g was advanced past it)
            ok = add_pv(1.f);
            if (!ok) break;

            const float inv = l > 0.f ? 1.f / l : 0.f;
            const float lse2 = l > 0.f ? m_ref * sl2 + log2f(l) : -INFINITY;
            if (valid) {
                const int64_t row = (int64_t)tok * a.H + kvh * Gq + gi;
                float4 *dst = direct ? reinterpret_cast<float4 *>(reinterpret_cast<float *>(a.out) + row * kD)
                                     : reinterpret_cast<float4 *>(a.part_o + prow * kD);
#pragma unroll
                for (int c = 0; c < kD / 4; ++c)
                    dst[c] = make_float4(o[4 * c] * inv, o[4 * c + 1] * inv, o[4 * c + 2] * inv, o[4 * c + 3] * inv);
                if (!direct) a.part_lse[prow] = lse2;
                else if (a.lse) a.lse[row] = lse2 * 0.6931471805599453f;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    // (paired variant: neither CTA leaves while the partner may still send tiles or commits its way)
    if (kPair) cluster_sync_all();
    if (warp == 12) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
    if (clocked) add_clock_counters(a.status, clock64() - ctl->clk0, global_ns() - ctl->ns0);
}

}  // namespace

bool attn_tc32_supported(int dtype, int d, int G) {
    return dtype == 1 && d == kD && G >= 1 && G <= 64;     // (any group size: rows are laid out with the padded group)
}

int attn_tc32_row_blocks(int n, int G) { return (n * G + kRows - 1) / kRows; }

// Can the row blocks 2k and 2k + 1 of this launch share their conversions (paired variant)?  The row blocks
// must come in twos (the two of a cluster then take the steps of the later one).
static bool pair_launch_ok32(const AttnArgs &a) {
    return a.win_lo <= 0 && ((int64_t)a.n * a.Gp) % (2 * kRows) == 0;
}

// Do the clusters of two fill the device as single CTAs do (queried once per device)?
static bool pair_clusters_fit32(const void *kernel) {
    static std::mutex mu;
    static std::vector<std::pair<int, bool>> seen;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    std::lock_guard<std::mutex> lock(mu);
    for (auto &d : seen)
        if (d.first == dev) return d.second;
    int sms = 0, clusters = 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2, 1024, 1);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    bool fit = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess &&
               cudaOccupancyMaxActiveClusters(&clusters, kernel, &cfg) == cudaSuccess && 2 * clusters >= sms - sms % 2;
    if (!fit) cudaGetLastError();
    seen.push_back({dev, fit});
    return fit;
}

cudaError_t launch_attn_tc32(const AttnArgs &a, cudaStream_t s) {
    static_assert(sizeof(Ctl) <= 512, "control block");
    static_assert(kSmemBytes <= 232448, "shared memory budget of one CTA");
    dim3 grid(attn_tc32_row_blocks(a.n, a.Gp), a.ngroups, 1);
    if (pair_launch_ok32(a)) {
        auto paired = attn_tc32_kernel<false, true>;
        cudaError_t e = raise_smem_limit_once(reinterpret_cast<const void *>(paired), (int)kSmemBytes);
        if (e != cudaSuccess) return e;
        if (pair_clusters_fit32(reinterpret_cast<const void *>(paired)))
            return launch_pdl_cluster2(paired, grid, dim3(kThreads), kSmemBytes, s, a);
    }
    auto kernel = a.win_lo > 0 ? attn_tc32_kernel<true> : attn_tc32_kernel<false>;
    cudaError_t e = raise_smem_limit_once(reinterpret_cast<const void *>(kernel), (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    return launch_pdl(kernel, grid, dim3(kThreads), kSmemBytes, s, a);
}

}  // namespace kvf
