// Tensor-core prefix + chunk attention for bf16 caches (sm_100a: TMA, tcgen05.mma, TMEM).
//
// Section 2 of the paper: the chunk's queries attend to [K_0;...;K_t], [V_0;...;V_t]; rows of
// earlier chunks are fully visible, rows of the chunk itself causally; query head h reads KV
// head h / G.  Scores are never written to memory: S = Q K^T lands in tensor memory, a running
// max / running sum softmax turns it into bf16 probabilities, and O += P V accumulates in tensor
// memory in fp32.
//
// Work decomposition.  A row pair is 256 query rows of one KV head (row = token * G +
// head-in-group, so the G query heads that share a KV head share every K/V tile; a group size that
// is no power of two - the 28 / 4 heads of Qwen2.5-7B - is laid out with G rounded up, the padding
// rows computed and never written), handled as two
// 128-row tiles that take turns on the tensor pipe.  Keys come in 128-row tiles.  The (KV head,
// key tile) pairs of a step are laid out on one line and cut into `ngroups` equal contiguous
// ranges; CTA (x = row pair, y = group) runs its row pair against its group's range, which
// touches at most two KV heads ("pieces").  The CTAs of a group stream the same tiles at the
// same time, so a tile leaves HBM once and the other row pairs hit L2.  With ngroups == Hkv a
// group is exactly one KV head and the CTA writes final outputs; otherwise every piece writes a
// normalised partial output and its log2 denominator to slot (group + KV head) and the combine
// kernel below merges the slots of each KV head in order.
//
// Roles (384 threads): warps 0-3 / 4-7 softmax of row tile 0 / 1 (one thread per row; TMEM lane
// = row), warp 8 TMA producer (Q per piece, then K(j), V(j), ... through a 5-slot ring), warps 9
// and 10 tcgen05.mma issuers of row tile 0 and 1 (warp 9 owns the TMEM allocation); warp 11 only
// completes the third warpgroup, which hands registers to the softmax warpgroups (setmaxnreg
// 80 / 208) so that a whole 128-column score row stays in registers after one tensor-memory load.
// Tensor memory (512 columns): S0 | S1 | O0 | O1, 128 fp32 columns each.  The bf16 probabilities
// overwrite the first 64 columns of their own S tile, in two halves that are handed to the
// second MMA separately, and feed it straight from tensor memory; the tensor pipe runs one
// thread's MMAs in issue order, so the next Q K^T of a row tile cannot overtake the P V that
// still reads those columns.  A single issuing thread for both tiles spends ~126 cycles per MMA
// (measured) against 64 cycles of tensor work, hence one issuer per row tile.
//
// Softmax arithmetic.  p = 2^(s * scale * log2(e) - m) with the reference maximum m moved only
// when the tile maximum exceeds it by more than 2^8 (then the accumulator is rescaled), packed
// two-wide fp32 multiply-adds, one special-function exponential per score.  (The special-function
// unit needs 1024 cycles per 128 x 128 tile and scheduler, as long as the tile's two MMAs; moving
// a share of the exponentials to an FMA-pipe polynomial was measured and did not pay here: the
// scheduler's issue port, not the special-function unit alone, is what the softmax saturates.)
//
// The exponential phases of the two row tiles are sequenced per scheduler (warp w of tile 0 and
// warp w of tile 1 alternate strictly), which keeps the tiles in antiphase: one tile's softmax
// runs under the other tile's MMAs.
//
// Short chunks (at most 128 / G tokens: decode, question chunk) have one row tile only.  The two
// tile slots then work on the same 128 rows and take alternate key tiles ("two streams"), each
// with its own accumulator, K/V ring of three slots and partial result, so the overlap of one
// stream's softmax with the other's MMAs survives and the step runs at HBM speed.
//
// Every wait on an mbarrier is bounded (about one second): on expiry the thread raises the
// CTA's abort flag and records the wait in the device status word, all roles leave their loops,
// copies and MMAs still in flight are waited for (bounded again), tensor memory is released and
// the kernel returns.  A parity wait is sound only for a thread that sees every phase of its
// barrier in order and is never more than one phase away from it; the ring, the hand-over and
// the turn protocols below are all built to that rule.
//
// The kernel may be launched while the kernel before it in the stream is finishing (programmatic
// dependent launch): everything up to pdl_wait() touches only launch arguments and the CTA's own
// shared and tensor memory (a ragged batch, whose row counts live in device memory, waits first).
#include "kvfold_internal.h"
#include "sm100_ptx.cuh"
#include "quant_expand.cuh"

namespace kvf {
namespace {

constexpr int kRows = 128;                    // rows of a Q tile = keys of a K/V tile
constexpr int kD = 128;                       // head_dim
constexpr uint32_t kPanel = 128 * 128;        // bytes of a [128 rows][64 bf16] swizzled panel
constexpr uint32_t kTileBytes = 2 * kPanel;   // a 128 x 128 bf16 tile = two panels
constexpr int kSlots = 5;
constexpr int kThreads = 384;
constexpr uint32_t kOffQ = 0;                         // 2 tiles
constexpr uint32_t kOffKV = 2 * kTileBytes;           // kSlots tiles
constexpr uint32_t kOffCtl = kOffKV + kSlots * kTileBytes;
constexpr uint32_t kSmemBytes = kOffCtl + 512 + 1024; // + control block + alignment slack
// int8 cache storage (kQuant): 512 threads (warps 12-15 expand code tiles to bf16 tiles), three
// bf16 K/V slots, three 16 KiB slots of raw int8 tiles (each with its 128 row scales) behind them
constexpr int kThreadsQ8 = 512;
constexpr int kSlotsQ8 = 3;
constexpr int kRawSlots = 3;
constexpr uint32_t kRawBytes = 128 * 128;             // a 128 x 128 int8 tile
constexpr uint32_t kOffRawQ8 = kOffKV + kSlotsQ8 * kTileBytes;
constexpr uint32_t kOffScaleQ8 = kOffRawQ8 + kRawSlots * kRawBytes;      // 128 fp32 row scales per raw slot
constexpr uint32_t kOffCtlQ8 = (kOffScaleQ8 + kRawSlots * 512 + 1023) / 1024 * 1024;
constexpr uint32_t kSmemBytesQ8 = kOffCtlQ8 + 512 + 1024;
constexpr uint32_t kTmemCols = 512;
constexpr float kRescaleThreshold = 8.0f;             // log2 units

// barrier indices inside the control block
constexpr int kRingBars = 6;                  // 5 slots of the shared ring, or 2 x 3 slots of the per-stream rings
enum { B_QFULL = 0, B_QEMPTY = 1, B_FULL0 = 2, B_EMPTY0 = B_FULL0 + kRingBars, B_SFULL0 = B_EMPTY0 + kRingBars,
       B_PA0 = B_SFULL0 + 2, B_PB0 = B_PA0 + 2, B_OFINAL0 = B_PB0 + 2, B_TURN0 = B_OFINAL0 + 2,
       B_DRAIN0 = B_TURN0 + 8, B_RAWFULL0 = B_DRAIN0 + 2, B_RAWEMPTY0 = B_RAWFULL0 + kRawSlots,
       B_COUNT = B_RAWEMPTY0 + kRawSlots };

struct Ctl {
    unsigned long long bars[40];
    uint32_t tmem_base;
    int abort;
    long long clk0;                // start of the CTA in SM cycles and in nanoseconds (the timed CTA only)
    unsigned long long ns0;
};
static_assert(B_COUNT <= 40, "control block holds 40 barriers");

// Shared-memory matrix descriptors (128-byte swizzle, descriptor version 1).
// K-major operand ([rows][64 bf16] panels, 8-row groups 1024 bytes apart):
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t addr) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// MN-major operand (V: [keys][64 bf16] panels; the next 64 columns of d are one panel further,
// the next 8 keys 1024 bytes further):
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t addr) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)(kPanel >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Instruction descriptor: D fp32, A and B bf16, M = 128, N = 128; bit 16 = B is MN-major.
constexpr uint32_t kIdescQK = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescPV = kIdescQK | (1u << 16);

// 64 scores of a row -> 32 packed bf16 probability pairs in p[0..31]; their sum goes to acc.
__device__ __forceinline__ void exp_half(const uint32_t *v, uint32_t *p, float2 sl2v, float2 negv, float2 &acc0, float2 &acc1) {
#pragma unroll
    for (int c = 0; c < 32; ++c) {
        const float2 x = __ffma2_rn(make_float2(__uint_as_float(v[2 * c]), __uint_as_float(v[2 * c + 1])), sl2v, negv);
        float2 e;
        e.x = ex2(x.x);
        e.y = ex2(x.y);
        if (c & 1) acc1 = __fadd2_rn(acc1, e);
        else acc0 = __fadd2_rn(acc0, e);
        p[c] = pack_bf16(e.x, e.y);
    }
}

// kWindow = false compiles the sink + window arithmetic out (launched whenever win_lo == 0).
// kQuant (0, 8 or 4 bits): map_k / map_v describe int8 or int4 code planes; the producer brings raw code tiles into their own
// ring and warps 12-15 (one thread per key row) expand each to the swizzled bf16 tile the MMAs read,
// value = bf16(code * row scale), which is what the FULL barriers then announce.
// kPair (quantised caches only): the CTAs of row pairs 2k and 2k + 1 form a cluster of two that walks
// the same key tiles.  Each expands 64 of a tile's 128 key rows into its own slot and, with a bulk copy that
// completes on the partner's FULL barrier, into the partner's; a slot is free once the issuers of BOTH CTAs
// have committed their reads of it.  Each SM then expands half the codes.  The host launches this variant only
// when every row pair has two row tiles (a chunk of a multiple of 512 / G tokens).
template <bool kWindow, int kQuant, bool kPair = false>
__global__ void __launch_bounds__(kQuant ? kThreadsQ8 : kThreads, 1)
attn_tc_kernel(const AttnArgs a, const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v) {
    constexpr int NS = kQuant ? kSlotsQ8 : kSlots;        // slots of the shared ring
    constexpr int SR = kQuant ? 2 : 3;                     // slots of each stream's own ring
    constexpr uint32_t offCtl = kQuant ? kOffCtlQ8 : kOffCtl;
    constexpr uint32_t rawBytes = kQuant == 4 ? kRawBytes / 2 : kRawBytes;   // bytes of a 128-row code tile
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    Ctl *ctl = reinterpret_cast<Ctl *>(smem_raw + (base - smem_u32(smem_raw)) + offCtl);
    const uint32_t bar0 = base + offCtl;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    static_assert(!kPair || (kQuant != 0 && !kWindow), "the paired variant is for quantised caches without a window");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int qpair = blockIdx.x, group = blockIdx.y;
    const uint32_t rank = kPair ? cluster_cta_rank() : 0u;     // which of K (0) and V (1) this CTA expands
    const int cb = blockIdx.z;     // cache of a batch (0 when there is one cache)
    const int G = a.Gp;     // rows per token in the row layout (a power of two >= a.G, the query heads per KV head)
    // (a ragged batch keeps its members' row counts in device memory, written by an earlier kernel
    // of the stream: those are the one thing read before the set-up below, so wait first there)
    if (a.prefixes) pdl_wait();
    // tokens this cache folds; a.n is the longest chunk of the launch and the stride of the caches' blocks
    const int n = a.ns ? (int)a.ns[cb] : a.n, nmax = a.n;
    if (blockIdx.x * 2 * kRows >= n * G) return;          // a shorter member of a batch: no row of this row pair exists
    const int64_t P = a.prefixes ? a.prefixes[cb] : a.prefix, L = P + n * a.self_rows;
    // streams == 2 (chunks of at most 128 / G tokens, i.e. one row tile): the two tile slots work on
    // the SAME 128 rows and take alternate key tiles, so that one stream's softmax still runs under
    // the other stream's MMAs; each stream leaves its own partial result.
    const int streams = a.streams;
    const bool direct = a.ngroups == a.Hkv && streams == 1;

    // key tiles: this row pair needs tiles below nt_need; the group's share of the
    // (KV head, tile) line is [lin0, lin1)
    const int row0 = qpair * 2 * kRows;
    // short chunks (at most 128 / G tokens in this row pair) leave the second row tile without a
    // valid row: its issuer and softmax warps then sit the kernel out
    const int tiles = (streams == 2 || row0 + kRows < n * G) ? 2 : 1;
    // (paired variant: both CTAs of a cluster walk the key tiles the later row pair needs; the earlier one
    // finds nothing visible in the last of them, and its rows' limits mask that tile out)
    const int tok_last = min(n - 1, ((kPair ? (qpair | 1) * 2 * kRows : row0) + 2 * kRows - 1) / G);
    // (virtual key tiles: without a window they are the key tiles themselves)
    const WindowTiles wt(kWindow ? a.win_lo : 0, kWindow ? a.n_sink : 0, kRows);
    const int nt_need = (int)((P + (tok_last + 1) * a.self_rows + kRows - 1) / kRows) - wt.skip;
    const int nt_all = (int)((L + kRows - 1) / kRows) - wt.skip;
    // (the line holds a.piece_cost virtual tiles in front of every KV head's key tiles: a range that runs into the
    // next head spends them on what its second piece costs and takes that many key tiles fewer)
    const int pcost = a.piece_cost, ntv = nt_all + pcost;
    const int64_t line = (int64_t)a.Hkv * ntv;
    const int64_t lin0 = group * line / a.ngroups, lin1 = (group + 1) * line / a.ngroups;
    const int kvh_first = (int)(lin0 / ntv);
    // piece k of this CTA: KV head kvh_first + k, tiles [kt0, kt0 + ntiles)
    auto piece = [&](int kvh, int &kt0, int &ntiles) -> bool {
        const int64_t b = (int64_t)kvh * ntv;
        if (kvh >= a.Hkv || b >= lin1) return false;
        kt0 = max((int)(max(lin0, b) - b) - pcost, 0);
        const int kt1 = min(max((int)(min(lin1, b + ntv) - b) - pcost, 0), nt_need);
        ntiles = kt1 - kt0;
        return true;
    };

    if (threadIdx.x == 0) {
        mbar_init(bar(B_QFULL), 1);
        mbar_init(bar(B_QEMPTY), tiles);                                  // both issuers read Q
        for (int s = 0; s < kRingBars; ++s) { mbar_init(bar(B_FULL0 + s), kQuant ? 4 : 1); mbar_init(bar(B_EMPTY0 + s), kPair ? 2 * tiles : streams == 2 ? 1 : tiles); }   // consumers of a K/V tile
        if (kQuant)
            for (int s = 0; s < kRawSlots; ++s) { mbar_init(bar(B_RAWFULL0 + s), 1); mbar_init(bar(B_RAWEMPTY0 + s), 4); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(B_SFULL0 + i), 1);
            mbar_init(bar(B_PA0 + i), 4);
            mbar_init(bar(B_PB0 + i), 4);
            mbar_init(bar(B_OFINAL0 + i), 1);
        }
        for (int w = 0; w < 8; ++w) mbar_init(bar(B_TURN0 + w), 1);
        mbar_init(bar(B_DRAIN0), 1);
        mbar_init(bar(B_DRAIN0 + 1), 1);
        ctl->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 9) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    pdl_launch_dependents();
    tc_fence_before();
    __syncthreads();
    if (kPair) cluster_sync_all();      // the partner's barriers exist before anything is sent to them
    tc_fence_after();
    pdl_wait();   // nothing above reads what an earlier kernel wrote; from here on the rotated chunk is read
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(&ctl->tmem_base);
    // One CTA times itself in SM cycles and in nanoseconds: the ratio is the clock the launch ran at
    // (the last row pair: it sees the most keys of the chunk itself, so no CTA of the launch runs longer)
    const bool clocked = blockIdx.x == gridDim.x - 1 && (blockIdx.y | blockIdx.z) == 0 && threadIdx.x == 0;
    if (clocked) {
        ctl->clk0 = clock64();
        ctl->ns0 = global_ns();
    }
    // K/V tile slots.  Two row tiles: one ring of 5 that both issuers walk in step.  Two streams:
    // each stream owns a ring of 3 (the sixth slot is the second Q tile, unused there), because a
    // parity wait is only sound for a thread that watches every use of its barrier in order.
    auto slot_addr = [&](int sl) { return base + (sl < NS ? kOffKV + (uint32_t)sl * kTileBytes : kOffQ + kTileBytes); };

    if (kQuant && warp >= 12) {
        // ------------------------------------------------------------------ int8 -> bf16 tile expansion
        asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
        // One thread per key row; in the paired variant two threads per row (64 codes each: the thread's
        // half of d is one panel of the bf16 tile) and this CTA's 64 of the tile's 128 rows.
        const int t = kPair ? (int)rank * 64 + (warp - 12) * 16 + (lane >> 1) : (warp - 12) * 32 + lane;   // key row of the tile
        const uint32_t hd = kPair ? (uint32_t)(lane & 1) : 0u;                                           // my half of d
        const uint32_t sw = (uint32_t)(t & 7);
        int tg = 0, rg = 0;
        int rc[2] = {0, 0};
        bool ok = true;
        int kt0, ntiles;
        for (int kvh = kvh_first; ok && piece(kvh, kt0, ntiles); ++kvh) {
            if (ntiles <= 0) continue;
            for (int tt = 0; tt < 2 * ntiles; ++tt, ++tg, ++rg) {
                int slot = tg % NS, use = tg / NS;
                if (streams == 2) {
                    const int st = (tt >> 1) & 1;
                    slot = st * SR + rc[st] % SR;
                    use = rc[st] / SR;
                    ++rc[st];
                }
                const int r = rg % kRawSlots;
                const int64_t key = (int64_t)wt.actual(kt0 + (tt >> 1)) * kRows + t;
                ok = mbar_wait(bar(B_RAWFULL0 + r), (rg / kRawSlots) & 1, ctl, a.status);
                if (ok) ok = mbar_wait(bar(B_EMPTY0 + slot), (use & 1) ^ 1, ctl, a.status);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                // the row's scale arrived with the tile (rows past the end of the planes were not copied)
                float scale = 0.f;
                if (key < a.capacity)
                    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(scale) : "r"(base + kOffScaleQ8 + (uint32_t)r * 512u + (uint32_t)t * 4u));
                const uint32_t dst = slot_addr(slot) + (uint32_t)t * 128u + hd * kPanel;
                const float2 sc = make_float2(scale, scale);
                if (kQuant == 4) {
                    // 64-byte code rows, 64-byte swizzle: chunk c of row t sits at c ^ ((t >> 1) & 3)
                    constexpr uint32_t NC = kPair ? 2 : 4;               // 16-byte chunks of codes I expand
                    const uint32_t src = base + kOffRawQ8 + (uint32_t)r * kRawBytes + (uint32_t)t * 64u;
                    const uint32_t sw4 = (uint32_t)((t >> 1) & 3);
                    uint32_t w[4 * NC];
#pragma unroll
                    for (uint32_t c = 0; c < NC; ++c)
                        asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                                     : "=r"(w[4 * c]), "=r"(w[4 * c + 1]), "=r"(w[4 * c + 2]), "=r"(w[4 * c + 3]) : "r"(src + (((c + NC * hd) ^ sw4) << 4)));
#pragma unroll
                    for (uint32_t k = 0; k < 4 * NC; ++k) {        // word k = 8 codes = one 16-byte chunk of the bf16 row
                        uint32_t o[4];
                        expand8(w[k], sc, o);
                        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (k >> 3) * kPanel + (((k & 7) ^ sw) << 4)),
                                     "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]) : "memory");
                    }
                } else {
                    constexpr uint32_t NC = kPair ? 4 : 8;               // 16-byte chunks of codes I expand
                    const uint32_t src = base + kOffRawQ8 + (uint32_t)r * kRawBytes + (uint32_t)t * 128u;
                    // all 16-byte chunks of the code row first, then the arithmetic: the chunks are
                    // independent, which is what gives one thread enough work in flight
                    uint32_t w[4 * NC];
#pragma unroll
                    for (uint32_t c = 0; c < NC; ++c)
                        asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                                     : "=r"(w[4 * c]), "=r"(w[4 * c + 1]), "=r"(w[4 * c + 2]), "=r"(w[4 * c + 3]) : "r"(src + (((c + NC * hd) ^ sw) << 4)));
#pragma unroll
                    for (uint32_t c = 0; c < NC; ++c) {
                        uint32_t o[8];
                        expand4(w[4 * c] ^ 0x80808080u, sc, o[0], o[1]);
                        expand4(w[4 * c + 1] ^ 0x80808080u, sc, o[2], o[3]);
                        expand4(w[4 * c + 2] ^ 0x80808080u, sc, o[4], o[5]);
                        expand4(w[4 * c + 3] ^ 0x80808080u, sc, o[6], o[7]);
                        const uint32_t k0 = 2 * c, k1 = 2 * c + 1;     // 16-byte chunks of the bf16 row (of my panel, when paired)
                        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (k0 >> 3) * kPanel + (((k0 & 7) ^ sw) << 4)),
                                     "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]) : "memory");
                        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (k1 >> 3) * kPanel + (((k1 & 7) ^ sw) << 4)),
                                     "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]) : "memory");
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the MMAs (and the copy below) read through the async proxy
                __syncwarp();
                if (lane == 0) {
                    if (kPair) {
                        // The partner's 64 rows are on their way: my warp's arrival on the FULL barrier of MY slot
                        // (one of them also books the 16 KiB), then my warp's 16 rows of both panels to the same place
                        // in the partner's slot, completing on the partner's barrier.  The slot is free in both CTAs
                        // (the EMPTY barrier counts the issuers of both), and neither rewrites it before the other's
                        // issuers have committed, which they do after these bytes have landed.
                        if (warp == 12) mbar_expect_tx(bar(B_FULL0 + slot), kTileBytes / 2);
                        else mbar_arrive(bar(B_FULL0 + slot));
                        const uint32_t peer_bar = peer_smem(bar(B_FULL0 + slot), rank ^ 1u);
#pragma unroll
                        for (uint32_t p = 0; p < 2; ++p) {
                            const uint32_t src = slot_addr(slot) + p * kPanel + ((uint32_t)rank * 64u + (uint32_t)(warp - 12) * 16u) * 128u;
                            bulk_push(peer_smem(src, rank ^ 1u), src, 16u * 128u, peer_bar);
                        }
                    } else {
                        mbar_arrive(bar(B_FULL0 + slot));
                    }
                    mbar_arrive(bar(B_RAWEMPTY0 + r));
                }
            }
        }
    } else if (warp >= 8) {
        if (kQuant) asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
        else asm volatile("setmaxnreg.dec.sync.aligned.u32 80;");
        if (warp == 8 && lane == 0) {
            // ------------------------------------------------------------------ TMA producer
            int tg = 0, pc = 0;          // ring loads and pieces so far
            int rc[2] = {0, 0};          // loads so far into each stream's ring
            int rg = 0;                  // int8 storage: loads so far into the ring of raw tiles
            int page = 0;                // paged cache: page of the key tile being loaded
            const int32_t *page_table = a.page_tables ? a.page_tables[cb] : a.page_table;
            const int qtok0 = cb * nmax; // the caches' rotated chunks follow one another
            bool ok = true;
            int kt0, ntiles;
            for (int kvh = kvh_first; ok && piece(kvh, kt0, ntiles); ++kvh) {
                if (ntiles <= 0) continue;
                if (pc > 0) ok = mbar_wait(bar(B_QEMPTY), (pc - 1) & 1, ctl, a.status);
                if (!ok) break;
                mbar_expect_tx(bar(B_QFULL), (streams == 2 ? 1 : 2) * kTileBytes);
                for (int i = 0; i < (streams == 2 ? 1 : 2); ++i)
                    for (int p = 0; p < 2; ++p)
                        tma_load_3d(base + kOffQ + i * kTileBytes + p * kPanel, &map_q, bar(B_QFULL), p * 64, kvh * a.G,
                                    qtok0 + (row0 + i * kRows) / G);
                ++pc;
                for (int t = 0; t < 2 * ntiles; ++t, ++tg) {
                    const CUtensorMap *m = (t & 1) ? &map_v : &map_k;
                    const int ktile = wt.actual(kt0 + (t >> 1));
                    const int key0 = ktile * kRows;
                    if (kQuant) {
                        // a raw code tile (128 rows of 128 bytes, 128-byte swizzle) into the next raw slot
                        const int r = rg % kRawSlots;
                        ok = mbar_wait(bar(B_RAWEMPTY0 + r), ((rg / kRawSlots) & 1) ^ 1, ctl, a.status);
                        if (!ok) break;
                        // ... and the rows' scales behind it (as many as the plane still holds)
                        if (page_table) {
                            // paged cache: a key tile is one page, which always holds its 128 rows and their scales
                            if (kPair || !(t & 1)) page = page_table[ktile];       // K then V of the same tile
                            const float *scales = ((t & 1) ? a.v_scales : a.k_scales) + (int64_t)page * a.scale_page_stride + kvh * kRows;
                            mbar_expect_tx(bar(B_RAWFULL0 + r), rawBytes + kRows * 4u);
                            tma_load_4d(base + kOffRawQ8 + (uint32_t)r * kRawBytes, m, bar(B_RAWFULL0 + r), 0, 0, kvh, page);
                            bulk_load(base + kOffScaleQ8 + (uint32_t)r * 512u, scales, kRows * 4u, bar(B_RAWFULL0 + r));
                            ++rg;
                            continue;
                        }
                        const int64_t left = a.scale_stride - key0;
                        const uint32_t sbytes = (uint32_t)(left < kRows ? left : kRows) * 4u;
                        const float *scales = ((t & 1) ? a.v_scales : a.k_scales) + (int64_t)kvh * a.scale_stride + key0;
                        mbar_expect_tx(bar(B_RAWFULL0 + r), rawBytes + sbytes);
                        tma_load_3d(base + kOffRawQ8 + (uint32_t)r * kRawBytes, m, bar(B_RAWFULL0 + r), 0, key0, kvh);
                        bulk_load(base + kOffScaleQ8 + (uint32_t)r * 512u, scales, sbytes, bar(B_RAWFULL0 + r));
                        ++rg;
                        continue;
                    }
                    int slot = tg % NS, use = tg / NS;
                    if (streams == 2) {
                        const int st = (t >> 1) & 1;          // key tile j goes to stream j & 1
                        slot = st * SR + rc[st] % SR;
                        use = rc[st] / SR;
                        ++rc[st];
                    }
                    ok = mbar_wait(bar(B_EMPTY0 + slot), (use & 1) ^ 1, ctl, a.status);
                    if (!ok) break;
                    mbar_expect_tx(bar(B_FULL0 + slot), kTileBytes);
                    if (page_table) {
                        // paged cache: a key tile is one page; the maps are (d, row in page, KV head, page)
                        if (!(t & 1)) page = page_table[ktile];                // K then V of the same tile
                        tma_load_4d(slot_addr(slot), m, bar(B_FULL0 + slot), 0, 0, kvh, page);
                        tma_load_4d(slot_addr(slot) + kPanel, m, bar(B_FULL0 + slot), 64, 0, kvh, page);
                    } else {
                        tma_load_3d(slot_addr(slot), m, bar(B_FULL0 + slot), 0, key0, kvh);
                        tma_load_3d(slot_addr(slot) + kPanel, m, bar(B_FULL0 + slot), 64, key0, kvh);
                    }
                }
            }
            // do not leave while a copy may still be writing into this CTA's shared memory
            if (pc > 0) mbar_wait_drain(bar(B_QFULL), (pc - 1) & 1, a.status);
            if (kQuant) {
                for (int c = max(0, rg - kRawSlots); c < rg; ++c)
                    mbar_wait_drain(bar(B_RAWFULL0 + c % kRawSlots), (c / kRawSlots) & 1, a.status);
            } else if (streams == 2) {
                for (int st = 0; st < 2; ++st)
                    for (int c = max(0, rc[st] - SR); c < rc[st]; ++c)
                        mbar_wait_drain(bar(B_FULL0 + st * SR + c % SR), (c / SR) & 1, a.status);
            } else {
                for (int t = max(0, tg - NS); t < tg; ++t)
                    mbar_wait_drain(bar(B_FULL0 + t % NS), (t / NS) & 1, a.status);
            }
        } else if ((warp == 9 || (warp == 10 && tiles == 2)) && lane == 0) {
            // ------------------------------------------------------------------ MMA issuer of row tile i
            // One issuing thread per row tile: each thread's MMAs run in its issue order (P V (j)
            // before the Q K^T (j+1) that overwrites the probabilities), the two tiles' streams
            // interleave freely on the tensor pipe, and neither waits on the other's softmax.
            const int i = warp - 9;
            const uint32_t t_s = tmem + i * 128, t_o = tmem + 256 + i * 128;
            const uint64_t qdesc = desc_kmajor(base + kOffQ + (streams == 2 ? 0 : i) * kTileBytes);
            const int j0 = streams == 2 ? i : 0, jstep = streams;    // my key tiles of a piece: j0, j0 + jstep, ...
            auto issue_qk = [&](int slot) {
                const uint64_t kdesc = desc_kmajor(slot_addr(slot));
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint64_t off = (uint64_t)(((kk >> 2) * kPanel + (kk & 3) * 32) >> 4);   // start-address field
                    tc_mma(t_s, qdesc + off, kdesc + off, kIdescQK, kk > 0);
                }
            };
            // 16 keys = 8 packed columns of P per MMA; half h covers keys 64h .. 64h+63
            auto issue_pv_half = [&](int slot, int h, bool accumulate) {
                const uint64_t vdesc = desc_mnmajor(slot_addr(slot));
#pragma unroll
                for (int kk = 4 * h; kk < 4 * h + 4; ++kk)
                    tc_mma_ts(t_o, t_s + kk * 8, vdesc + (uint64_t)((kk * 2048) >> 4), kIdescPV,
                              (accumulate || kk > 4 * h) ? 1u : 0u);
            };
            // a K/V slot is free once its readers have run: in the paired variant the partner's expansion warps
            // wait for my reads as well (they write my slot), so the commit goes to both CTAs' barriers
            auto commit_empty = [&](int slot) {
                if (kPair) tc_commit_pair(bar(B_EMPTY0 + slot));
                else tc_commit(bar(B_EMPTY0 + slot));
            };
            int tg = 0, it = 0, pc = 0;   // ring loads before this piece, my key tiles issued, pieces so far
            bool ok = true;
            // load number -> slot and parity: shared ring (number counts every load) or my own ring
            // (number counts my loads: K of my m-th tile is 2m, its V 2m + 1)
            auto ring = [&](int num, int &slot, uint32_t &par) {
                if (streams == 2) { slot = i * SR + num % SR; par = (num / SR) & 1; }
                else { slot = num % NS; par = (num / NS) & 1; }
            };
            int kt0, ntiles;
            for (int kvh = kvh_first; ok && piece(kvh, kt0, ntiles); ++kvh) {
                if (ntiles <= 0) continue;
                ok = mbar_wait(bar(B_QFULL), pc & 1, ctl, a.status);
                if (!ok) break;
                tc_fence_after();
                int jlast = -1;
                for (int j = j0; j < ntiles && ok; j += jstep, ++it) {
                    const int tk = streams == 2 ? 2 * it : tg + 2 * j;
                    int kslot, vslot;
                    uint32_t kpar, vpar;
                    ring(tk, kslot, kpar);
                    if (j > j0) {
                        ring(tk - 1, vslot, vpar);                               // V of my previous tile
                        ok = mbar_wait(bar(B_FULL0 + vslot), vpar, ctl, a.status);
                        if (ok) ok = mbar_wait(bar(B_PA0 + i), (it - 1) & 1, ctl, a.status);
                        if (!ok) break;
                        tc_fence_after();
                        issue_pv_half(vslot, 0, j - jstep > j0);
                        ok = mbar_wait(bar(B_PB0 + i), (it - 1) & 1, ctl, a.status);
                        if (!ok) break;
                        tc_fence_after();
                        issue_pv_half(vslot, 1, true);
                        commit_empty(vslot);
                    }
                    ok = mbar_wait(bar(B_FULL0 + kslot), kpar, ctl, a.status);
                    if (!ok) break;
                    tc_fence_after();
                    issue_qk(kslot);
                    tc_commit(bar(B_SFULL0 + i));
                    commit_empty(kslot);
                    jlast = j;
                }
                if (!ok) break;
                tc_commit(bar(B_QEMPTY));          // every Q K^T of mine in this piece has been issued
                if (jlast >= 0) {
                    int vslot;
                    uint32_t vpar;
                    ring(streams == 2 ? 2 * it - 1 : tg + 2 * jlast + 1, vslot, vpar);
                    ok = mbar_wait(bar(B_FULL0 + vslot), vpar, ctl, a.status);
                    if (ok) ok = mbar_wait(bar(B_PA0 + i), (it - 1) & 1, ctl, a.status);
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv_half(vslot, 0, jlast > j0);
                    ok = mbar_wait(bar(B_PB0 + i), (it - 1) & 1, ctl, a.status);
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv_half(vslot, 1, true);
                    tc_commit(bar(B_OFINAL0 + i));
                    commit_empty(vslot);
                }
                tg += 2 * ntiles;
                ++pc;
            }
            // whatever made this thread leave its loop, tensor memory is released only after every
            // MMA it issued has run
            tc_commit(bar(B_DRAIN0 + i));
            mbar_wait_drain(bar(B_DRAIN0 + i), 0, a.status);
        }
    } else {
        // ------------------------------------------------------------------ softmax, one thread per row
        if (kQuant) asm volatile("setmaxnreg.inc.sync.aligned.u32 192;");
        else asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
        const int i = warp >> 2;                        // row tile
        const int r = (warp & 3) * 32 + lane;           // row in the tile = TMEM lane
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_s = tmem + lane_addr + i * 128;
        const uint32_t t_o = tmem + lane_addr + 256 + i * 128;
        const int R = row0 + (streams == 2 ? 0 : i * kRows) + r, tok = R / G, gi = R % G;
        const bool valid = tok < n && gi < a.G;     // (gi >= a.G: padding of a group that is no power of two)
        // a warp none of whose 32 rows is a row of the chunk (decode-shaped steps: most warps) keeps
        // every barrier protocol going but skips the loads, the arithmetic and the stores
        const bool warp_live = __any_sync(0xffffffffu, valid);
        const int j0 = streams == 2 ? i : 0, jstep = streams;        // my key tiles of a piece
        // keys below `limit` are visible; a row past the chunk's end is never written, and each
        // row of S, P and O depends on that row alone, so such rows are left unmasked
        const int64_t limit = valid ? P + (tok + 1) * a.self_rows : ((int64_t)1 << 62);
        const float sl2 = a.scale_log2;
        const float2 sl2v = make_float2(sl2, sl2);
        const int64_t nG = (int64_t)nmax * G;                 // rows of a partial slot

        int it = 0, oc = 0;            // my key tiles and my finished pieces so far
        int turn_base = 0;             // turns (see below) both tile slots have taken before this piece
        bool ok = i < tiles;
        int kt0, ntiles;
        for (int kvh = kvh_first; ok && piece(kvh, kt0, ntiles); ++kvh) {
            const int64_t prow = cb * a.part_rows + ((int64_t)(group + kvh) * streams + (streams == 2 ? i : 0)) * nG + R;   // my partial row
            // Turns on the exponentials: in every piece both tile slots take the same number of
            // turns, slot 0 then slot 1, alternating strictly (a slot with fewer key tiles, which
            // happens with two streams, passes its spare turns without doing anything).  Strict
            // alternation is what a parity wait can follow: neither barrier is ever more than one
            // phase away from what its waiter expects.
            const int nturns = ntiles <= 0 ? 0 : (streams == 2 ? (ntiles + 1) / 2 : ntiles);
            const int mine = ntiles > j0 ? (ntiles - j0 + jstep - 1) / jstep : 0;
            auto take_turn = [&](int g) -> bool {      // wait until turn g of this slot may start
                bool got = true;
                if (i == 0) {
                    if (g > 0) got = mbar_wait(bar(B_TURN0 + (warp & 3)), (g - 1) & 1, ctl, a.status);
                } else {
                    got = mbar_wait(bar(B_TURN0 + 4 + (warp & 3)), g & 1, ctl, a.status);
                }
                return __all_sync(0xffffffffu, got);
            };
            auto pass_spare_turns = [&]() -> bool {
                for (int t = mine; t < nturns && tiles == 2; ++t) {
                    if (!take_turn(turn_base + t)) return false;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(B_TURN0 + (i == 0 ? 4 : 0) + (warp & 3)));
                }
                turn_base += nturns;
                return true;
            };
            if (ntiles <= j0) {
                // no visible key for these rows in this range: an empty partial
                if (!direct && valid) {
                    float4 *po = reinterpret_cast<float4 *>(a.part_o + prow * kD);
#pragma unroll 4
                    for (int c = 0; c < kD / 4; ++c) po[c] = make_float4(0.f, 0.f, 0.f, 0.f);
                    a.part_lse[prow] = -INFINITY;
                }
                ok = pass_spare_turns();
                continue;
            }
            float m_ref = -INFINITY;   // reference maximum (raw score units) the probabilities are scaled by
            float l = 0.f;
            for (int j = j0, k = 0; j < ntiles; j += jstep, ++it, ++k) {
                ok = mbar_wait(bar(B_SFULL0 + i), it & 1, ctl, a.status);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                if (!warp_live) {
                    if (tiles == 2) ok = take_turn(turn_base + k);
                    if (!ok) break;
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(bar(B_PA0 + i));
                        mbar_arrive(bar(B_PB0 + i));
                        mbar_arrive(bar(B_TURN0 + (i == 0 ? 4 : 0) + (warp & 3)));
                    }
                    continue;
                }
                const int64_t key0 = (int64_t)wt.actual(kt0 + j) * kRows;
                const int nvis = (int)max((int64_t)0, min((int64_t)kRows, limit - key0));
                // a tile that starts before the window holds hidden columns (the sink tile, the window's first)
                const bool masked = __any_sync(0xffffffffu, nvis < kRows) || (kWindow && key0 < a.win_lo);

                // the whole score row in registers after one load
                uint32_t sc[128];
                KVF_TMEM_LD32(sc, 0, t_s);
                KVF_TMEM_LD32(sc, 32, t_s + 32);
                KVF_TMEM_LD32(sc, 64, t_s + 64);
                KVF_TMEM_LD32(sc, 96, t_s + 96);
                tmem_wait_ld();
                if (masked) {
                    // columns below lo_c lie before the window and count only if they are sinks
                    const int lo_c = kWindow ? (int)max((int64_t)0, min((int64_t)kRows, a.win_lo - key0)) : 0;
                    const int sink_c = kWindow ? (int)max((int64_t)0, min((int64_t)kRows, a.n_sink - key0)) : 0;
#pragma unroll
                    for (int c = 0; c < 128; ++c) sc[c] = (c < nvis && (c >= lo_c || c < sink_c)) ? sc[c] : 0xFF800000u;   // -inf
                }
                float mx[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) mx[q] = fmaxf(__uint_as_float(sc[2 * q]), __uint_as_float(sc[2 * q + 1]));
#pragma unroll
                for (int c = 16; c < 128; c += 16)
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        mx[q] = max3(mx[q], __uint_as_float(sc[c + 2 * q]), __uint_as_float(sc[c + 2 * q + 1]));
                const float m_tile = fmaxf(max3(mx[0], mx[1], mx[2]), max3(max3(mx[3], mx[4], mx[5]), mx[6], mx[7]));
                // move the reference only when the maximum grew by more than the threshold: the
                // probabilities then stay below 2^threshold and the accumulator is rarely rescaled
                const bool grow = (m_tile - m_ref) * sl2 > kRescaleThreshold;   // also true when m_ref = -inf < m_tile
                if (__any_sync(0xffffffffu, grow)) {
                    const float m_new = grow ? m_tile : m_ref;
                    const float alpha = grow ? ex2((m_ref - m_new) * sl2) : 1.f;   // m_ref = -inf -> 0
                    l *= alpha;
                    m_ref = m_new;
                    if (k > 0) {
                        // the commit that completed this S also covers my previous P V: O is quiescent here
                        const float2 av = make_float2(alpha, alpha);
#pragma unroll 1
                        for (int c0 = 0; c0 < 128; c0 += 32) {
                            uint32_t o[32];
                            KVF_TMEM_LD32(o, 0, t_o + c0);
                            tmem_wait_ld();
#pragma unroll
                            for (int c = 0; c < 32; c += 2) {
                                const float2 v = __fmul2_rn(make_float2(__uint_as_float(o[c]), __uint_as_float(o[c + 1])), av);
                                o[c] = __float_as_uint(v.x);
                                o[c + 1] = __float_as_uint(v.y);
                            }
                            KVF_TMEM_ST32(o, 0, t_o + c0);
                        }
                        tmem_wait_st();
                    }
                }
                const float m_safe = m_ref == -INFINITY ? 0.f : m_ref;
                const float neg = -m_safe * sl2;
                const float2 negv = make_float2(neg, neg);
                float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);

                // The two row tiles' warps that share a scheduler take turns on the exponentials:
                // run side by side they halve each other's special-function rate and both tiles
                // fall into step, leaving the tensor pipe idle while both are in their softmax.
                if (tiles == 2) ok = take_turn(turn_base + k);
                if (!ok) break;

                // probabilities; the first 64 keys are handed over before the rest is computed
                uint32_t p[32];
                exp_half(sc, p, sl2v, negv, acc0, acc1);
                KVF_TMEM_ST32(p, 0, t_s);
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B_PA0 + i));
                exp_half(sc + 64, p, sl2v, negv, acc0, acc1);
                KVF_TMEM_ST32(p, 0, t_s + 32);
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(bar(B_PB0 + i));
                    mbar_arrive(bar(B_TURN0 + (i == 0 ? 4 : 0) + (warp & 3)));   // the other tile's turn
                }
                const float2 acc = __fadd2_rn(acc0, acc1);
                l += acc.x + acc.y;
            }
            if (!ok) break;
            ok = pass_spare_turns();
            if (!ok) break;

            ok = mbar_wait(bar(B_OFINAL0 + i), oc & 1, ctl, a.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            ++oc;
            tc_fence_after();
            if (!warp_live) continue;
            const float inv = l > 0.f ? 1.f / l : 0.f;
            const float lse2 = l > 0.f ? m_ref * sl2 + log2f(l) : -INFINITY;
            const int64_t row = ((int64_t)cb * nmax + tok) * a.H + kvh * a.G + gi;
#pragma unroll
            for (int c0 = 0; c0 < 128; c0 += 32) {
                uint32_t o[32];
                KVF_TMEM_LD32(o, 0, t_o + c0);
                tmem_wait_ld();
                if (!valid) continue;
                if (!direct) {
                    float4 *dst = reinterpret_cast<float4 *>(a.part_o + prow * kD + c0);
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        dst[c] = make_float4(__uint_as_float(o[4 * c]) * inv, __uint_as_float(o[4 * c + 1]) * inv,
                                             __uint_as_float(o[4 * c + 2]) * inv, __uint_as_float(o[4 * c + 3]) * inv);
                } else if (a.out_f32) {
                    float4 *dst = reinterpret_cast<float4 *>(reinterpret_cast<float *>(a.out) + row * kD + c0);
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        dst[c] = make_float4(__uint_as_float(o[4 * c]) * inv, __uint_as_float(o[4 * c + 1]) * inv,
                                             __uint_as_float(o[4 * c + 2]) * inv, __uint_as_float(o[4 * c + 3]) * inv);
                } else {
                    uint4 *dst = reinterpret_cast<uint4 *>(reinterpret_cast<__nv_bfloat16 *>(a.out) + row * kD + c0);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            w[e] = pack_bf16(__uint_as_float(o[8 * c + 2 * e]) * inv, __uint_as_float(o[8 * c + 2 * e + 1]) * inv);
                        dst[c] = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
            if (valid) {
                if (!direct) a.part_lse[prow] = lse2;
                else if (a.lse) a.lse[row] = lse2 * 0.6931471805599453f;
            }
            // the next piece's first P V (which overwrites O) is issued only after all 128 rows
            // have handed over its probabilities, i.e. after these loads
        }
    }

    tc_fence_before();
    __syncthreads();
    // (paired variant: neither CTA leaves while the partner may still send tiles or commits its way)
    if (kPair) cluster_sync_all();
    if (warp == 9) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
    if (clocked) add_clock_counters(a.status, clock64() - ctl->clk0, global_ns() - ctl->ns0);
}

// Merge the pieces of each KV head.  Group g owns [g * line / ngroups, (g+1) * line / ngroups) of
// the (KV head, key tile) line, its piece for KV head h sits in slot g + h.  With lse_s = log2 of
// a piece's softmax denominator and O_s its normalised output,
//   O = sum_s 2^(lse_s - M) O_s / sum_s 2^(lse_s - M),  M = max_s lse_s,  in group order.
// One block = kCombineTokens tokens of one KV head; one warp per row, lane = float4 column, so a
// row of a piece is one coalesced 512-byte read and the weights are computed once per row.  The
// groups that touch a KV head come with the launch arguments when the host knows the row count
// (AttnArgs::g_first / g_last); a ragged batch works them out per cache.  Up to eight pieces (the
// usual case) are fetched together with their denominators, so a row costs one trip to memory.
// (64 registers per thread: four blocks per SM, so that the blocks of a 256-token chunk - 512 of them -
// are all resident at once instead of taking turns in waves)
constexpr int kCombineTokens = 4;
template <bool kFew>   // kFew: every KV head has at most eight parts (known on the host), the loops below run once
__global__ void __launch_bounds__(256, kFew ? 4 : 2) combine_groups_kernel(const __grid_constant__ AttnArgs a) {
    __shared__ int g_range[2];
    const int kvh = blockIdx.y, G = a.G;     // (a.Gp >= G: rows a token takes in the slots)
    const int cb = blockIdx.z;     // cache of a batch
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_launch_dependents();
    int g0, g1;
    if (kFew || (a.range_valid && kvh < kRangeHeads)) {      // (kFew is chosen only when the host worked the ranges out)
        g0 = a.g_first[kvh];
        g1 = a.g_last[kvh];
    } else {
        if (a.prefixes) pdl_wait();   // ragged batch: the row counts were written by an earlier kernel of the stream
        const int n_b = a.ns ? (int)a.ns[cb] : a.n;
        if (n_b == 0) return;         // this cache sat the step out
        if (threadIdx.x == 0) {
            const int64_t P = a.prefixes ? a.prefixes[cb] : a.prefix;
            const int nt_all = (int)((P + n_b * a.self_rows + kRows - 1) / kRows) - WindowTiles(a.win_lo, a.n_sink, kRows).skip;
            group_range(a.Hkv, nt_all + a.piece_cost, a.ngroups, kvh, g_range[0], g_range[1]);
        }
        __syncthreads();
        g0 = g_range[0];
        g1 = g_range[1];
    }
    pdl_wait();   // the parts are the attention kernel's output
    // tokens this cache folded (a.n: the longest chunk, the stride); members of different length come
    // with a ragged batch only, which never takes the kFew variant
    const int n = (!kFew && a.ns) ? (int)a.ns[cb] : a.n;
    const int st = a.streams;
    const int np = (g1 - g0 + 1) * st;   // parts of this KV head: st per piece
    // part s of the KV head sits in slot (g0 + s / st + kvh) * st + s % st = (g0 + kvh) * st + s
    const int64_t nG = (int64_t)a.n * a.Gp;
    const int64_t slot0 = (int64_t)(g0 + kvh) * st;
    const float *part_o = a.part_o + (cb * a.part_rows + slot0 * nG) * kD + lane * 4;
    const float *part_lse = a.part_lse + cb * a.part_rows + slot0 * nG;
    const int Gp = a.Gp;                                      // rows a token takes in the slots (>= G: the rest is padding)
    const int rows = kCombineTokens * Gp;                     // rows of this block, row = token * Gp + head-in-group
    const int lgp = __ffs(Gp) - 1;
    for (int rr = warp; rr < rows; rr += 8) {
        const int tok = blockIdx.x * kCombineTokens + (rr >> lgp), gi = rr & (Gp - 1);     // (Gp is a power of two)
        if (tok >= n) break;
        if (gi >= G) continue;
        const int64_t R = (int64_t)tok * Gp + gi;
        const int64_t row = ((int64_t)cb * a.n + tok) * a.H + kvh * G + gi;
        const float *po = part_o + R * kD;                    // part s: po + s * nG * kD
        const float *pl = part_lse + R;                       //         pl + s * nG
        // the first eight pieces (usually all of them) are fetched together with the denominators,
        // so a row costs one trip to memory
        float4 pv[8];
#pragma unroll
        for (int s = 0; s < 8; ++s)
            if (s < np) pv[s] = *reinterpret_cast<const float4 *>(po + s * nG * kD);
        float ls = lane < np ? pl[lane * nG] : -INFINITY;     // lane s holds the denominator of piece s (s < 32)
        float M = ls;
        if (!kFew)
            for (int s = 32 + lane; s < np; s += 32) M = fmaxf(M, pl[s * nG]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
        float den = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s0 = 0; s0 < (kFew ? 1 : np); s0 += 8) {     // 8 pieces at a time, in group order: deterministic
            const int cnt = min(8, np - s0);
            if (!kFew && s0 > 0) {
#pragma unroll
                for (int s = 0; s < 8; ++s)
                    if (s < cnt) pv[s] = *reinterpret_cast<const float4 *>(po + (s0 + s) * nG * kD);
                if ((s0 & 31) == 0) ls = s0 + lane < np ? pl[(s0 + lane) * nG] : -INFINITY;
            }
            const float wl = ls == -INFINITY ? 0.f : exp2f(ls - M);
#pragma unroll
            for (int s = 0; s < 8; ++s) {
                if (s < cnt) {
                    const float w = __shfl_sync(0xffffffffu, wl, (s0 + s) & 31);
                    den += w;
                    acc.x = fmaf(w, pv[s].x, acc.x); acc.y = fmaf(w, pv[s].y, acc.y);
                    acc.z = fmaf(w, pv[s].z, acc.z); acc.w = fmaf(w, pv[s].w, acc.w);
                }
            }
        }
        const float inv = den > 0.f ? 1.f / den : 0.f;
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
        if (a.out_f32) {
            *reinterpret_cast<float4 *>(reinterpret_cast<float *>(a.out) + row * kD + lane * 4) = acc;
        } else {
            uint2 pk;
            pk.x = pack_bf16(acc.x, acc.y);
            pk.y = pack_bf16(acc.z, acc.w);
            *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(a.out) + row * kD + lane * 4) = pk;
        }
        if (lane == 0 && a.lse) a.lse[row] = (M + log2f(den)) * 0.6931471805599453f;
    }
}

}  // namespace

// Any group size up to 64: the kernels lay rows out with the group rounded up to a power of two
// (attn_tc_padded_group), so that a 128-row tile holds whole tokens; the rows of the padding cost
// tensor-core work (1/8 of it for the 28 / 4 heads of Qwen2.5-7B) and are never written.
bool attn_tc_supported(int dtype, int d, int G) {
    return dtype == 0 && d == kD && G >= 1 && G <= 64;
}

int attn_tc_padded_group(int G) {
    int p = 1;
    while (p < G) p *= 2;
    return p;
}

int attn_tc_row_pairs(int n, int G) { return (n * G + 2 * kRows - 1) / (2 * kRows); }

int attn_tc_streams(int n, int G) { return n * G <= kRows ? 2 : 1; }

// Can the row pairs 2k and 2k + 1 of this launch share their expansions (paired variant)?  Every row pair
// must have both row tiles (the two of a cluster then walk the key tiles of the later one).
static bool pair_launch_ok(const AttnArgs &a) {
    // (members of a batch that take fewer tokens than the launch's chunk may lack a row tile: no pairs then)
    if (!a.quant_bits || a.win_lo > 0 || a.streams != 1 || a.ns) return false;
    return ((int64_t)a.n * a.Gp) % (4 * kRows) == 0;
}

// Do the clusters of two fill the device as single CTAs do (queried once per device)?
static bool pair_clusters_fit(const void *kernel, uint32_t smem) {
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
    cfg.blockDim = dim3(kThreadsQ8);
    cfg.dynamicSmemBytes = smem;
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

cudaError_t launch_attn_tc(const AttnArgs &a, const TcMaps &maps, cudaStream_t s) {
    static_assert(sizeof(Ctl) <= 512, "control block");
    static_assert(kSmemBytes <= 232448, "shared memory budget of one CTA");
    static_assert(kSmemBytesQ8 <= 232448, "shared memory budget of one CTA (int8 storage)");
    const bool quant = a.quant_bits != 0;
    auto kernel = a.quant_bits == 8 ? (a.win_lo > 0 ? attn_tc_kernel<true, 8> : attn_tc_kernel<false, 8>)
                : a.quant_bits == 4 ? (a.win_lo > 0 ? attn_tc_kernel<true, 4> : attn_tc_kernel<false, 4>)
                                    : (a.win_lo > 0 ? attn_tc_kernel<true, 0> : attn_tc_kernel<false, 0>);
    const uint32_t smem = quant ? kSmemBytesQ8 : kSmemBytes;
    dim3 grid(attn_tc_row_pairs(a.n, a.Gp), a.ngroups, a.batch);
    if (pair_launch_ok(a)) {
        auto paired = a.quant_bits == 8 ? attn_tc_kernel<false, 8, true> : attn_tc_kernel<false, 4, true>;
        cudaError_t e = raise_smem_limit_once(reinterpret_cast<const void *>(paired), (int)smem);
        if (e != cudaSuccess) return e;
        if (pair_clusters_fit(reinterpret_cast<const void *>(paired), smem))
            return launch_pdl_cluster2(paired, grid, dim3(kThreadsQ8), smem, s, a, maps.q, maps.k, maps.v);
    }
    cudaError_t e = raise_smem_limit_once(reinterpret_cast<const void *>(kernel), (int)smem);
    if (e != cudaSuccess) return e;
    return launch_pdl(kernel, grid, dim3(quant ? kThreadsQ8 : kThreads), smem, s, a, maps.q, maps.k, maps.v);
}

cudaError_t launch_combine_groups(const AttnArgs &a, cudaStream_t s) {
    dim3 grid((a.n + kCombineTokens - 1) / kCombineTokens, a.Hkv, a.batch);
    // at most eight parts per KV head (two streams x four pieces, or eight pieces)?  The host knows when it
    // worked out the groups of each head.
    bool few = a.range_valid != 0 && a.Hkv <= kRangeHeads;
    for (int h = 0; few && h < a.Hkv; ++h) few = (a.g_last[h] - a.g_first[h] + 1) * a.streams <= 8;
    if (few) return launch_pdl(combine_groups_kernel<true>, grid, dim3(256), 0, s, a);
    return launch_pdl(combine_groups_kernel<false>, grid, dim3(256), 0, s, a);
}

}  // namespace kvf
