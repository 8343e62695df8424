// Internal declarations shared by the host layer and the kernel launchers.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>
#include <vector>

namespace kvf {

// Programmatic dependent launch: a kernel launched with launch_pdl may be scheduled while the
// kernel before it in the stream is still finishing; it must call pdl_wait() before it touches
// anything an earlier kernel reads or writes (the wait returns when all earlier work in the
// stream has completed and its memory is visible).  pdl_launch_dependents() lets the kernel
// after this one be scheduled early in the same way.  Both are no-ops in a plain launch.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Whether the launches of the calling thread ask for it.  Overlapping a kernel's set-up with the tail of the one
// before pays where a step is short (decode-shaped steps, short prefixes, the sink + window chain: 1.5 - 5 %);
// a long chain of long tensor-bound steps runs at the power cap, where the idle gap between plain launches comes
// back as clock (measured on the 131 072-token chain: 148.3 ms with plain launches against 150.1 ms, the
// attention kernels at 1.53 instead of 1.505 GHz).  The host layer sets this per step (PdlScope).
inline thread_local bool g_pdl_allowed = true;
struct PdlScope {
    bool saved;
    explicit PdlScope(bool allow) : saved(g_pdl_allowed) { g_pdl_allowed = allow; }
    ~PdlScope() { g_pdl_allowed = saved; }
};

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = g_pdl_allowed ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
// The same with the grid's CTAs grouped into clusters of two along x.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl_cluster2(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = g_pdl_allowed ? 1 : 0;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// Raises a kernel's dynamic shared-memory limit, once per kernel and device (the attribute
// belongs to the device's copy of the function): launches after the first skip the runtime call.
inline cudaError_t raise_smem_limit_once(const void *kernel, int bytes) {
    struct Done { const void *kernel; int dev; };
    static std::mutex mu;
    static std::vector<Done> done;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    for (const Done &d : done)
        if (d.kernel == kernel && d.dev == dev) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) done.push_back({kernel, dev});
    return e;
}

constexpr int kMaxHalfDim = 64;       // head_dim <= 128
constexpr int kKvTile = 128;          // key rows per tensor-core tile; V rows are zero-padded to it
constexpr int kPartTokens = 4096;     // the partial area holds kPartTokens * H rows of head_dim floats
constexpr int kMaxSplits = 64;        // CUDA-core path: most splits of the key range

struct RopeTable {
    double inv_freq[kMaxHalfDim];
};

// Where cache row `row` of KV head `g` lives, in elements from the plane's base pointer.
// Contiguous cache: planes are [Hkv][capacity][d].  Paged cache: a page is kKvTile tokens of every
// KV head, K block then V block ([2][Hkv][kKvTile][d]); the K "plane" pointer is the pool's base,
// the V one is one block further, and page_table[row / kKvTile] names the page.
struct RowMap {
    const int32_t *page_table;   // null = contiguous
    int64_t capacity;            // contiguous: rows per head
    int64_t page_elems;          // paged: elements of one page (2 * Hkv * kKvTile * d)
    int32_t d;
#ifdef __CUDACC__
    __device__ __forceinline__ int64_t offset(int g, int64_t row) const {
        if (page_table == nullptr) return ((int64_t)g * capacity + row) * d;
        const int64_t page = page_table[row / kKvTile];
        return page * page_elems + ((int64_t)g * kKvTile + row % kKvTile) * d;
    }
#endif
};

// Arguments of the fused rotate + append kernel (one launch per step).
struct RopeAppendArgs {
    const void *q, *k_new, *v_new;   // [n][H][d], [n][Hkv][d], [n][Hkv][d]; k_new = v_new = null: only the queries
                                     // are rotated, nothing is appended (kvf_attend)
    void *q_rot;                     // [n][H][d]
    void *k_plane, *v_plane;         // [Hkv][capacity][d]
    int64_t capacity, prefix, pos0;  // prefix = rows already held
    int32_t n, H, Hkv, d;
    int32_t zero_rows;               // value rows [prefix+n, prefix+n+zero_rows) are cleared
    const int32_t *page_table;       // paged cache: device table of page numbers, else null
    int64_t page_elems;              // paged cache: elements per page
    // batch of caches advancing together (blockIdx.y = cache b): q, k_new, v_new, q_rot hold the
    // caches' chunks one after the other; cache b's rows go where page_tables[b] says
    const int32_t *const *page_tables;   // device array of device tables, or null (one cache)
    // ragged batch: cache b holds prefixes[b] rows and its chunk starts at position pos0s[b]
    // (device arrays, or null: prefix and pos0 above hold for every cache)
    const int64_t *prefixes, *pos0s;
    // ... and, if its members' chunks differ in length too, cache b folds ns[b] tokens (0 = it sits the step
    // out); n above is then the longest chunk and the stride of the members' blocks in q, k_new, v_new, q_rot
    const int64_t *ns;
    // fp32 cache whose attention runs on fp16 halves of its operands: a rotated query or key or a value
    // above range_limit in magnitude sets code 7 in *status (range_limit = 0: no check)
    int *status;
    float range_limit;
    RopeTable table;
};

// Arguments shared by the attention kernels and the combine kernel.
struct AttnArgs {
    const void *q_rot;               // [n][H][d]
    const void *k_plane, *v_plane;   // [Hkv][capacity][d]
    void *out;                       // [n][H][d], dtype or fp32
    float *lse;                      // [n][H] or null (natural log)
    float *part_o;                   // partial outputs, fp32, normalised per part: CUDA-core path
                                     // [splits][n][H][d]; tensor-core path [slot][n * Gp][d]
    float *part_lse;                 // log2 denominators of the parts, same order; -inf = no key seen
    int *status;                     // device status word
    const int32_t *page_table;       // paged cache: device table of page numbers (one per key tile), else null
    // batch of caches advancing together (blockIdx.z = cache b): q_rot, out, lse hold the caches'
    // chunks one after the other, cache b's partial results start part_rows rows into the partial
    // area per cache before it, its pages are named by page_tables[b]
    const int32_t *const *page_tables;   // device array of device tables, or null (one cache)
    int64_t part_rows;               // rows of the partial area per cache of a batch
    int32_t batch;                   // caches in the launch (1 = one cache)
    const int64_t *prefixes;         // ragged batch: device array of the caches' row counts, else null
    const int64_t *ns;               // ragged batch with chunks of different length: device array of the caches'
                                     // token counts (n below is then the longest chunk = stride of the blocks), else null
    const float *k_scales, *v_scales; // int8 storage: fp32 row scales [Hkv][scale_stride] (the tensor maps then
                                     // describe the int8 code planes), else null; paged: the scale blocks of page 0
    int64_t scale_stride;            // capacity rounded up to a multiple of 4 (16-byte aligned rows of scales)
    int64_t scale_page_stride;       // paged quantised cache: floats from one page's scale block to the next page's
    int32_t quant_bits;              // 0, 8 or 4
    // sink + window variant: of the rows before the chunk only those below n_sink or from win_lo on
    // are visible (win_lo = 0: all of them); see WindowTiles
    int32_t n_sink;
    int64_t win_lo;
    int64_t capacity, prefix;
    int32_t n, H, Hkv, G, d;
    int32_t Gp;                      // rows a token takes in the row layout of the tensor-core kernels and of the partial
                                     // slots (row = token * Gp + head-in-group): G, or for the tcgen05 kernels G rounded up
                                     // to a power of two so that a 128-row tile holds whole tokens (rows with
                                     // head-in-group >= G are padding: computed, never written)
    int32_t splits;                  // CUDA-core path: equal splits of the key range
    int32_t ngroups;                 // tensor-core path: contiguous ranges of the (KV head, key tile) line
    int32_t streams;                 // tensor-core path: 2 = one row tile, its key tiles dealt to two streams
    int32_t piece_cost;              // tensor-core path: the line the groups cut holds, in front of every KV head's key
                                     // tiles, this many virtual tiles that stand for what a second piece costs a CTA
                                     // (another Q load, another drain and set of partial rows): a CTA whose range
                                     // runs into the next KV head gets that many key tiles fewer (0: plain line)
    int32_t out_f32;
    int32_t self_rows;               // 1: a fold step - the chunk's own rows are in the cache, token i sees rows < prefix + i + 1;
                                     // 0: queries only (kvf_attend) - nothing was appended, every token sees rows < prefix
    float scale_log2;                // softmax scale * log2(e)
    // tensor-core paths, when the host knows the row count (no ragged batch): first and last group whose
    // range of the (KV head, key tile) line touches KV head h, for h < kRangeHeads (see group_range)
    int32_t range_valid;
    int16_t g_first[64], g_last[64];
};
constexpr int kRangeHeads = 64;

// Groups cut the line of Hkv * nt_all (KV head, key tile) pairs into ngroups ranges, group g owning
// [g * line / ngroups, (g + 1) * line / ngroups).  First and last group that own a tile of KV head kvh.
// (With AttnArgs::piece_cost the line holds nt_all + piece_cost entries per KV head: callers pass that sum,
// and a group that owns only virtual tiles of a head still counts - it leaves an empty partial.)
__host__ __device__ inline void group_range(int Hkv, int nt_all, int ngroups, int kvh, int &g_first, int &g_last) {
    const int64_t line = (int64_t)Hkv * nt_all;
    auto start = [&](int64_t g) { return g * line / ngroups; };
    auto group_of = [&](int64_t lin) {
        int64_t g = lin * ngroups / line;
        while (g > 0 && start(g) > lin) --g;
        while (g + 1 < ngroups && start(g + 1) <= lin) ++g;
        return (int)g;
    };
    g_first = group_of((int64_t)kvh * nt_all);
    g_last = group_of((int64_t)(kvh + 1) * nt_all - 1);
}

// Key tiles of the sink + window variant.  Tiles that hold no visible row are never loaded: the
// kernels walk "virtual" tiles v = 0, 1, ... and read tile actual(v).  With T0 the tile that holds
// row win_lo, the virtual line is [tile 0, if it holds sinks and T0 > 0] followed by T0, T0 + 1, ...
struct WindowTiles {
    int sink_tiles;   // 1 if tile 0 is walked only for its sink rows
    int skip;         // tiles left out between the sink tile and the window
    __host__ __device__ WindowTiles(int64_t win_lo, int n_sink, int tile_rows) {
        const int t0 = (int)(win_lo / tile_rows);
        sink_tiles = (n_sink > 0 && t0 > 0) ? 1 : 0;
        skip = t0 - sink_tiles;
    }
    __host__ __device__ int actual(int v) const { return v < sink_tiles ? v : v + skip; }
};
constexpr int kMaxSinks = 64;         // sink rows sit in the first key tile of either kernel

// Quantised storage: int8 codes [Hkv][capacity][d] and one fp32 scale per row [Hkv][scale_stride],
// scale_stride = capacity rounded up to a multiple of 4.
// Paged: a page is kKvTile tokens of every KV head, [K codes | V codes][Hkv][kKvTile][row bytes] followed
// by [K scales | V scales][Hkv][kKvTile] fp32; the pointers below are those blocks of page 0.
struct QuantPlanes {
    int8_t *k_codes, *v_codes;       // int4: two codes to a byte (code + 8, element 2i in the low nibble of byte i)
    float *k_scales, *v_scales;
    int64_t scale_stride;
    int32_t bits;                    // 8 or 4
    int64_t page_bytes;              // paged: bytes of one page (0 = contiguous planes)
};
cudaError_t launch_rope_append_q8(const RopeAppendArgs &a, const QuantPlanes &qp, bool interleaved, int batch, cudaStream_t s);

cudaError_t launch_rope_append(const RopeAppendArgs &a, int dtype, bool interleaved, int batch, cudaStream_t s);
cudaError_t launch_attn_simt(const AttnArgs &a, int dtype, cudaStream_t s, int *grid_out);
cudaError_t launch_combine(const AttnArgs &a, int dtype, cudaStream_t s);
int attn_simt_ctas(int n, int G, int Hkv, int splits);

// Tensor-core path (bf16, head_dim 128).
struct TcMaps {
    CUtensorMap q, k, v;
};
bool attn_tc_supported(int dtype, int d, int G);
int attn_tc_padded_group(int G);       // G rounded up to a power of two: rows a token takes in the tcgen05 kernels' row layout
int attn_tc_row_pairs(int n, int G);   // 256-row pairs per KV head = grid.x (G: the padded group, as below)
int attn_tc_streams(int n, int G);     // 2 when the chunk fits one 128-row tile
cudaError_t launch_attn_tc(const AttnArgs &a, const TcMaps &maps, cudaStream_t s);   // grid (row pairs, ngroups)
cudaError_t launch_combine_groups(const AttnArgs &a, cudaStream_t s);                // needed when ngroups != Hkv

// Decode-shaped steps (at most attn_q8_decode_max_rows() query rows) on a quantised cache: codes are
// expanded into mma.sync register fragments, shared memory is all ring.  Grid = ngroups CTAs, ngroups a
// multiple of the KV heads; partial results as for the other tensor-core kernels (streams = 1).
int attn_q8_decode_max_rows();
cudaError_t launch_attn_q8_decode(const AttnArgs &a, const TcMaps &maps, cudaStream_t s);

// Tensor-core path for fp32 caches (head_dim 128): operands split into fp16 halves, three MMAs per
// product; contiguous planes, read straight from global memory (no tensor maps).
// Merge of attention results over disjoint sets of cache rows (merge_parts.cu).
cudaError_t launch_merge_parts(int n_parts, int64_t n_rows, int d, bool f32, const void *parts_out, const float *parts_lse,
                               void *out, float *lse, cudaStream_t s);

bool attn_tc32_supported(int dtype, int d, int G);
int attn_tc32_row_blocks(int n, int G);   // 128-row blocks per KV head = grid.x
cudaError_t launch_attn_tc32(const AttnArgs &a, cudaStream_t s);                     // grid (row blocks, ngroups)

}  // namespace kvf
