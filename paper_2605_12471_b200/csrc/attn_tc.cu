// Tensor-core prefix + chunk attention for bf16 caches (sm_100a: TMA, tcgen05.mma, TMEM).
//
// Section 2 of the paper: the chunk's queries attend to [K_0;...;K_t], [V_0;...;V_t]; rows of
// earlier chunks are fully visible, rows of the chunk itself causally; query head h reads KV
// head h / G.  Scores are never written to memory: S = Q K^T lands in tensor memory, a running
// max / running sum softmax turns it into bf16 probabilities, and O += P V accumulates in tensor
// memory in fp32.
//
// One CTA = 256 query rows of one KV head (row = token * G + head-in-group, so the G query heads
// that share a KV head share every K/V tile), processed as two 128-row tiles that take turns on
// the tensor pipe, against 128-key tiles streamed through a 5-slot shared-memory ring by TMA.
//   warps 0-3 / 4-7 : softmax of row tile 0 / 1 (one thread per row; TMEM lane = row)
//   warp 8          : TMA producer (Q once, then K(j), V(j), K(j+1), ...)
//   warp 9          : tcgen05.mma issuer, owns the TMEM allocation
// Tensor memory (512 columns): S0 | S1 | O0 | O1, 128 fp32 columns each.  The bf16 probabilities
// overwrite the first 64 columns of their own S tile (two per 32-bit cell) and feed the second
// MMA straight from tensor memory; the tensor pipe runs one thread's MMAs in issue order, so the
// next Q K^T of a row tile cannot overtake the P V that still reads those columns.
// Split over the key range: blockIdx.z takes a contiguous range of key tiles and writes a
// normalised partial output plus its log2 denominator; the combine kernel merges them.
//
// Every wait on an mbarrier is bounded (about one second): on expiry the thread raises the
// CTA's abort flag and the device status word, all roles leave their loops, tensor memory is
// released and the kernel returns.
#include "kvfold_internal.h"

namespace kvf {
namespace {

constexpr int kRows = 128;                    // rows of a Q tile = keys of a K/V tile
constexpr int kD = 128;                       // head_dim
constexpr uint32_t kPanel = 128 * 128;        // bytes of a [128 rows][64 bf16] swizzled panel
constexpr uint32_t kTileBytes = 2 * kPanel;   // a 128 x 128 bf16 tile = two panels
constexpr int kSlots = 5;
constexpr int kThreads = 320;
constexpr uint32_t kOffQ = 0;                         // 2 tiles
constexpr uint32_t kOffKV = 2 * kTileBytes;           // kSlots tiles
constexpr uint32_t kOffCtl = kOffKV + kSlots * kTileBytes;
constexpr uint32_t kSmemBytes = kOffCtl + 256 + 1024; // + control block + alignment slack
constexpr uint32_t kTmemCols = 512;
constexpr float kRescaleThreshold = 8.0f;             // log2 units
constexpr unsigned long long kWaitLimitNs = 1000000000ull;

// barrier indices inside the control block
enum { B_QFULL = 0, B_FULL0 = 1, B_EMPTY0 = 1 + kSlots, B_SFULL0 = 1 + 2 * kSlots, B_PFULL0 = B_SFULL0 + 2,
       B_OFINAL0 = B_PFULL0 + 2, B_COUNT = B_OFINAL0 + 2 };

struct Ctl {
    unsigned long long bars[24];
    uint32_t tmem_base;
    int abort;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait.  Returns false if the CTA is aborting or the limit ran out.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, Ctl *ctl, int *status) {
    const unsigned long long t0 = global_ns();
    unsigned spins = 0;
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 63u) == 0) {
            if (*reinterpret_cast<volatile int *>(&ctl->abort)) return false;
            if (global_ns() - t0 > kWaitLimitNs) {
                *reinterpret_cast<volatile int *>(&ctl->abort) = 1;
                atomicExch(status, 5);   // KVF_ERR_TIMEOUT
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, Ctl *ctl, int *status) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, ctl, status);
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// A operand from tensor memory (lane = row, each 32-bit column holds two consecutive bf16 of K)
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

#define KVF_R32(a, o) "=r"(a[o + 0]), "=r"(a[o + 1]), "=r"(a[o + 2]), "=r"(a[o + 3]), "=r"(a[o + 4]), "=r"(a[o + 5]), "=r"(a[o + 6]), "=r"(a[o + 7]), \
                      "=r"(a[o + 8]), "=r"(a[o + 9]), "=r"(a[o + 10]), "=r"(a[o + 11]), "=r"(a[o + 12]), "=r"(a[o + 13]), "=r"(a[o + 14]), "=r"(a[o + 15]), \
                      "=r"(a[o + 16]), "=r"(a[o + 17]), "=r"(a[o + 18]), "=r"(a[o + 19]), "=r"(a[o + 20]), "=r"(a[o + 21]), "=r"(a[o + 22]), "=r"(a[o + 23]), \
                      "=r"(a[o + 24]), "=r"(a[o + 25]), "=r"(a[o + 26]), "=r"(a[o + 27]), "=r"(a[o + 28]), "=r"(a[o + 29]), "=r"(a[o + 30]), "=r"(a[o + 31])
#define KVF_W32(a, o) "r"(a[o + 0]), "r"(a[o + 1]), "r"(a[o + 2]), "r"(a[o + 3]), "r"(a[o + 4]), "r"(a[o + 5]), "r"(a[o + 6]), "r"(a[o + 7]), \
                      "r"(a[o + 8]), "r"(a[o + 9]), "r"(a[o + 10]), "r"(a[o + 11]), "r"(a[o + 12]), "r"(a[o + 13]), "r"(a[o + 14]), "r"(a[o + 15]), \
                      "r"(a[o + 16]), "r"(a[o + 17]), "r"(a[o + 18]), "r"(a[o + 19]), "r"(a[o + 20]), "r"(a[o + 21]), "r"(a[o + 22]), "r"(a[o + 23]), \
                      "r"(a[o + 24]), "r"(a[o + 25]), "r"(a[o + 26]), "r"(a[o + 27]), "r"(a[o + 28]), "r"(a[o + 29]), "r"(a[o + 30]), "r"(a[o + 31])

// 32 consecutive fp32 columns of this thread's TMEM lane -> registers a[o .. o+31]
#define KVF_TMEM_LD32(a, o, taddr)                                                              \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                      \
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "      \
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];" \
                 : KVF_R32(a, o) : "r"(taddr) : "memory")
#define KVF_TMEM_ST32(a, o, taddr)                                                              \
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "                               \
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "      \
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};" \
                 ::KVF_W32(a, o), "r"(taddr) : "memory")
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

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

__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const AttnArgs a, const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    Ctl *ctl = reinterpret_cast<Ctl *>(smem_raw + (base - smem_u32(smem_raw)) + kOffCtl);
    const uint32_t bar0 = base + kOffCtl;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int qpair = blockIdx.x, kvh = blockIdx.y, split = blockIdx.z;
    const int G = a.G, n = a.n;
    const int64_t P = a.prefix, L = P + n;

    // key tiles of this CTA
    const int row0 = qpair * 2 * kRows;
    const int tok_last = min(n - 1, (row0 + 2 * kRows - 1) / G);
    const int nt_need = (int)((P + tok_last + 1 + kRows - 1) / kRows);
    const int nt_all = (int)((L + kRows - 1) / kRows);
    const int per = (nt_all + a.splits - 1) / a.splits;
    const int kt0 = split * per;
    const int kt1 = min(nt_need, kt0 + per);
    const int ntiles = kt1 - kt0;

    if (ntiles <= 0) {
        // this split has no visible key for these rows: an empty partial
        if (warp < 8 && a.splits > 1) {
            int R = row0 + threadIdx.x, tok = R / G, gi = R % G;
            if (tok < n) {
                int64_t row = (int64_t)tok * a.H + kvh * G + gi;
                float4 *po = reinterpret_cast<float4 *>(a.part_o + ((int64_t)split * n * a.H + row) * kD);
#pragma unroll 4
                for (int c = 0; c < kD / 4; ++c) po[c] = make_float4(0.f, 0.f, 0.f, 0.f);
                a.part_lse[(int64_t)split * n * a.H + row] = -INFINITY;
            }
        }
        return;
    }

    if (threadIdx.x == 0) {
        mbar_init(bar(B_QFULL), 1);
        for (int s = 0; s < kSlots; ++s) { mbar_init(bar(B_FULL0 + s), 1); mbar_init(bar(B_EMPTY0 + s), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(bar(B_SFULL0 + i), 1); mbar_init(bar(B_PFULL0 + i), 128); mbar_init(bar(B_OFINAL0 + i), 1); }
        ctl->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 9) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(&ctl->tmem_base);

    if (warp == 8) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            mbar_expect_tx(bar(B_QFULL), 2 * kTileBytes);
            for (int i = 0; i < 2; ++i)
                for (int p = 0; p < 2; ++p)
                    tma_load_3d(base + kOffQ + i * kTileBytes + p * kPanel, &map_q, bar(B_QFULL), p * 64, kvh * G,
                                (row0 + i * kRows) / G);
            int issued = 0;
            bool ok = true;
            for (int t = 0; t < 2 * ntiles && ok; ++t) {
                const int slot = t % kSlots, use = t / kSlots;
                ok = mbar_wait(bar(B_EMPTY0 + slot), (use & 1) ^ 1, ctl, a.status);
                if (!ok) break;
                const CUtensorMap *m = (t & 1) ? &map_v : &map_k;
                const int key0 = (kt0 + (t >> 1)) * kRows;
                mbar_expect_tx(bar(B_FULL0 + slot), kTileBytes);
                tma_load_3d(base + kOffKV + slot * kTileBytes, m, bar(B_FULL0 + slot), 0, key0, kvh);
                tma_load_3d(base + kOffKV + slot * kTileBytes + kPanel, m, bar(B_FULL0 + slot), 64, key0, kvh);
                issued = t + 1;
            }
            // do not leave while a copy may still be writing into this CTA's shared memory
            mbar_wait(bar(B_QFULL), 0, ctl, a.status);
            for (int t = max(0, issued - kSlots); t < issued; ++t)
                mbar_wait_slow(bar(B_FULL0 + t % kSlots), (t / kSlots) & 1, ctl, a.status);
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            bool ok = mbar_wait(bar(B_QFULL), 0, ctl, a.status);
            tc_fence_after();
            auto issue_qk = [&](int i, int slot) {
                const uint32_t qa = base + kOffQ + i * kTileBytes, kb = base + kOffKV + slot * kTileBytes;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint32_t off = (kk >> 2) * kPanel + (kk & 3) * 32;
                    tc_mma(tmem + i * 128, desc_kmajor(qa + off), desc_kmajor(kb + off), kIdescQK, kk > 0);
                }
            };
            auto issue_pv = [&](int i, int slot, bool accumulate) {
                const uint32_t vb = base + kOffKV + slot * kTileBytes;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)   // 16 keys = 8 packed columns of P per MMA
                    tc_mma_ts(tmem + 256 + i * 128, tmem + i * 128 + kk * 8, desc_mnmajor(vb + kk * 2048), kIdescPV,
                              (accumulate || kk > 0) ? 1u : 0u);
            };
            for (int j = 0; j < ntiles && ok; ++j) {
                const int tk = 2 * j, kslot = tk % kSlots;
                ok = mbar_wait(bar(B_FULL0 + kslot), (tk / kSlots) & 1, ctl, a.status);
                if (!ok) break;
                tc_fence_after();
                for (int i = 0; i < 2 && ok; ++i) {
                    if (j > 0) {
                        const int tv = 2 * (j - 1) + 1, vslot = tv % kSlots;
                        if (i == 0) ok = mbar_wait(bar(B_FULL0 + vslot), (tv / kSlots) & 1, ctl, a.status);
                        if (ok) ok = mbar_wait(bar(B_PFULL0 + i), (j - 1) & 1, ctl, a.status);
                        if (!ok) break;
                        tc_fence_after();
                        issue_pv(i, vslot, j - 1 > 0);
                        if (i == 1) tc_commit(bar(B_EMPTY0 + vslot));
                    }
                    issue_qk(i, kslot);
                    tc_commit(bar(B_SFULL0 + i));
                    if (i == 1) tc_commit(bar(B_EMPTY0 + kslot));
                }
            }
            if (ok) {
                const int j = ntiles - 1, tv = 2 * j + 1, vslot = tv % kSlots;
                ok = mbar_wait(bar(B_FULL0 + vslot), (tv / kSlots) & 1, ctl, a.status);
                for (int i = 0; i < 2 && ok; ++i) {
                    ok = mbar_wait(bar(B_PFULL0 + i), j & 1, ctl, a.status);
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv(i, vslot, j > 0);
                    tc_commit(bar(B_OFINAL0 + i));
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax, one thread per row
        const int i = warp >> 2;                        // row tile
        const int r = (warp & 3) * 32 + lane;           // row in the tile = TMEM lane
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_s = tmem + lane_addr + i * 128;
        const uint32_t t_o = tmem + lane_addr + 256 + i * 128;
        const int R = row0 + i * kRows + r, tok = R / G, gi = R % G;
        const bool valid = tok < n;
        const int64_t limit = valid ? P + tok + 1 : 0;  // keys below `limit` are visible
        const float sl2 = a.scale_log2;

        float m_ref = -INFINITY;   // reference maximum (raw score units) the probabilities are scaled by
        float l = 0.f;
        bool ok = true;
        for (int j = 0; j < ntiles; ++j) {
            ok = mbar_wait(bar(B_SFULL0 + i), j & 1, ctl, a.status);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            uint32_t s[128];
            KVF_TMEM_LD32(s, 0, t_s);
            KVF_TMEM_LD32(s, 32, t_s + 32);
            KVF_TMEM_LD32(s, 64, t_s + 64);
            KVF_TMEM_LD32(s, 96, t_s + 96);
            tmem_wait_ld();

            const int64_t key0 = (int64_t)(kt0 + j) * kRows;
            const int nvis = (int)max((int64_t)0, min((int64_t)kRows, limit - key0));
            if (nvis < kRows) {
#pragma unroll
                for (int c = 0; c < 128; ++c) s[c] = c < nvis ? s[c] : 0xFF800000u;   // -inf
            }
            float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
            for (int c = 0; c < 128; c += 4) {
                mx0 = fmaxf(mx0, __uint_as_float(s[c]));
                mx1 = fmaxf(mx1, __uint_as_float(s[c + 1]));
                mx2 = fmaxf(mx2, __uint_as_float(s[c + 2]));
                mx3 = fmaxf(mx3, __uint_as_float(s[c + 3]));
            }
            const float m_tile = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
            // move the reference only when the maximum grew by more than the threshold: the
            // probabilities then stay below 2^threshold and the accumulator is rarely rescaled
            const bool grow = (m_tile - m_ref) * sl2 > kRescaleThreshold;   // also true when m_ref = -inf < m_tile
            if (__any_sync(0xffffffffu, grow)) {
                const float m_new = grow ? m_tile : m_ref;
                const float alpha = grow ? ex2((m_ref - m_new) * sl2) : 1.f;   // m_ref = -inf -> 0
                l *= alpha;
                m_ref = m_new;
                if (j > 0) {
                    // the commit that completed S(j) also covers PV(j-1): O is quiescent here
#pragma unroll
                    for (int c0 = 0; c0 < 128; c0 += 32) {
                        uint32_t o[32];
                        KVF_TMEM_LD32(o, 0, t_o + c0);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
                        KVF_TMEM_ST32(o, 0, t_o + c0);
                    }
                    tmem_wait_st();
                }
            }
            const float m_safe = m_ref == -INFINITY ? 0.f : m_ref;
            const float neg = -m_safe * sl2;
            float sum0 = 0.f, sum1 = 0.f, sum2 = 0.f, sum3 = 0.f;
#pragma unroll
            for (int c4 = 0; c4 < 32; ++c4) {
                const float p0 = ex2(fmaf(__uint_as_float(s[c4 * 4 + 0]), sl2, neg));
                const float p1 = ex2(fmaf(__uint_as_float(s[c4 * 4 + 1]), sl2, neg));
                const float p2 = ex2(fmaf(__uint_as_float(s[c4 * 4 + 2]), sl2, neg));
                const float p3 = ex2(fmaf(__uint_as_float(s[c4 * 4 + 3]), sl2, neg));
                sum0 += p0; sum1 += p1; sum2 += p2; sum3 += p3;
                __nv_bfloat162 b0 = __floats2bfloat162_rn(p0, p1), b1 = __floats2bfloat162_rn(p2, p3);
                s[c4 * 2 + 0] = *reinterpret_cast<uint32_t *>(&b0);   // packed pair (2c, 2c+1) -> column c
                s[c4 * 2 + 1] = *reinterpret_cast<uint32_t *>(&b1);
            }
            l += (sum0 + sum1) + (sum2 + sum3);
            KVF_TMEM_ST32(s, 0, t_s);
            KVF_TMEM_ST32(s, 32, t_s + 32);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar(B_PFULL0 + i));
        }

        if (ok) {
            ok = mbar_wait(bar(B_OFINAL0 + i), 0, ctl, a.status);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            tc_fence_after();
            const float inv = l > 0.f ? 1.f / l : 0.f;
            const float lse2 = l > 0.f ? m_ref * sl2 + log2f(l) : -INFINITY;
            const int64_t row = (int64_t)tok * a.H + kvh * G + gi;
#pragma unroll
            for (int c0 = 0; c0 < 128; c0 += 32) {
                uint32_t o[32];
                KVF_TMEM_LD32(o, 0, t_o + c0);
                tmem_wait_ld();
                if (!valid) continue;
                if (a.splits > 1) {
                    float4 *dst = reinterpret_cast<float4 *>(a.part_o + ((int64_t)split * n * a.H + row) * kD + c0);
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
                        for (int e = 0; e < 4; ++e) {
                            __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(o[8 * c + 2 * e]) * inv,
                                                                     __uint_as_float(o[8 * c + 2 * e + 1]) * inv);
                            w[e] = *reinterpret_cast<uint32_t *>(&b);
                        }
                        dst[c] = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
            if (valid) {
                if (a.splits > 1) a.part_lse[(int64_t)split * n * a.H + row] = lse2;
                else if (a.lse) a.lse[row] = lse2 * 0.6931471805599453f;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 9) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

}  // namespace

bool attn_tc_supported(int dtype, int d, int G) {
    return dtype == 0 && d == kD && G >= 1 && G <= 64 && (G & (G - 1)) == 0;
}

int attn_tc_ctas(int n, int G, int Hkv, int splits) { return ((n * G + 2 * kRows - 1) / (2 * kRows)) * Hkv * splits; }

cudaError_t launch_attn_tc(const AttnArgs &a, const TcMaps &maps, cudaStream_t s) {
    static_assert(sizeof(Ctl) <= 256, "control block");
    static_assert(kSmemBytes <= 232448, "shared memory budget of one CTA");
    cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    dim3 grid((a.n * a.G + 2 * kRows - 1) / (2 * kRows), a.Hkv, a.splits);
    attn_tc_kernel<<<grid, kThreads, kSmemBytes, s>>>(a, maps.q, maps.k, maps.v);
    return cudaGetLastError();
}

}  // namespace kvf
