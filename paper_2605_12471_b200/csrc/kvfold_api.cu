// Host layer of the C ABI declared in include/kvfold.h: handle, validation, workspace carving,
// TMA descriptor creation, launch planning.  Every step of the fold runs in the kernels this file
// launches; there is no CPU fallback.
#include "../../include/kvfold.h"
#include "kvfold_internal.h"

#include <cmath>
#include <cstdio>
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

using namespace kvf;

namespace {

thread_local char g_cuda_err[256] = "";

kvf_status cuda_fail(cudaError_t e, const char *what) {
    snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", what, cudaGetErrorString(e));
    return KVF_ERR_CUDA;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

size_t elem_bytes(int dtype) { return dtype == KVF_BF16 ? 2 : 4; }

bool pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }

kvf_status check_config(const kvf_config *c) {
    if (!c) return KVF_ERR_INVALID_ARG;
    if (c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->capacity <= 0 || c->max_chunk <= 0)
        return KVF_ERR_INVALID_ARG;
    if (c->n_q_heads % c->n_kv_heads != 0) return KVF_ERR_INVALID_ARG;
    if (c->dtype != KVF_BF16 && c->dtype != KVF_F32) return KVF_ERR_UNSUPPORTED;
    if (c->head_dim != 64 && c->head_dim != 128) return KVF_ERR_UNSUPPORTED;
    int G = c->n_q_heads / c->n_kv_heads;
    if (G > 64) return KVF_ERR_UNSUPPORTED;
    if (c->rope_base <= 0.0 && !c->inv_freq) return KVF_ERR_INVALID_ARG;
    if (c->softmax_scale < 0.0) return KVF_ERR_INVALID_ARG;
    if ((int64_t)c->max_chunk > c->capacity) return KVF_ERR_INVALID_ARG;
    if (c->capacity > (int64_t)1 << 31) return KVF_ERR_UNSUPPORTED;
    if ((c->flags & KVF_CACHE_INT8) && (c->flags & KVF_CACHE_INT4)) return KVF_ERR_INVALID_ARG;
    if ((c->flags & (KVF_CACHE_INT8 | KVF_CACHE_INT4)) &&
        (c->dtype != KVF_BF16 || (c->flags & KVF_FORCE_SIMT) || !attn_tc_supported(c->dtype, c->head_dim, G)))
        return KVF_ERR_UNSUPPORTED;
    return KVF_OK;
}

struct Layout {
    size_t status, q_rot, st_q, st_k, st_v, st_out, st_lse, part_o, part_lse, total;
    size_t st_q2, st_k2, st_v2;   // second staging set (KVF_HOST_UPLOAD_AHEAD)
    size_t st_out2, st_lse2;      // second result staging set (KVF_HOST_DOWNLOAD_BEHIND)
    size_t part_o2, part_lse2;    // second set of partial results (KVF_COMBINE_BEHIND)
};

Layout workspace_layout(const kvf_config *c) {
    Layout l;
    const size_t eb = elem_bytes(c->dtype);
    const size_t qb = (size_t)c->max_chunk * c->n_q_heads * c->head_dim * eb;
    const size_t kb = (size_t)c->max_chunk * c->n_kv_heads * c->head_dim * eb;
    const size_t ob = (size_t)c->max_chunk * c->n_q_heads * c->head_dim *
                      ((c->flags & KVF_OUT_F32) ? 4 : eb);
    size_t off = 0;
    l.status = off;   off = align_up(off + 256, 1024);
    l.q_rot = off;    off = align_up(off + qb, 1024);
    l.st_q = off;     off = align_up(off + qb, 1024);
    l.st_k = off;     off = align_up(off + kb, 1024);
    l.st_v = off;     off = align_up(off + kb, 1024);
    l.st_q2 = l.st_k2 = l.st_v2 = 0;
    if (c->flags & KVF_HOST_UPLOAD_AHEAD) {
        l.st_q2 = off; off = align_up(off + qb, 1024);
        l.st_k2 = off; off = align_up(off + kb, 1024);
        l.st_v2 = off; off = align_up(off + kb, 1024);
    }
    l.st_out = off;   off = align_up(off + ob, 1024);
    l.st_lse = off;   off = align_up(off + (size_t)c->max_chunk * c->n_q_heads * 4, 1024);
    l.st_out2 = l.st_lse2 = 0;
    if (c->flags & KVF_HOST_DOWNLOAD_BEHIND) {
        l.st_out2 = off; off = align_up(off + ob, 1024);
        l.st_lse2 = off; off = align_up(off + (size_t)c->max_chunk * c->n_q_heads * 4, 1024);
    }
    l.part_o = off;   off = align_up(off + (size_t)kPartTokens * c->n_q_heads * c->head_dim * 4, 1024);
    l.part_lse = off; off = align_up(off + (size_t)kPartTokens * c->n_q_heads * 4, 1024);
    l.part_o2 = l.part_lse2 = 0;
    if (c->flags & KVF_COMBINE_BEHIND) {
        l.part_o2 = off;   off = align_up(off + (size_t)kPartTokens * c->n_q_heads * c->head_dim * 4, 1024);
        l.part_lse2 = off; off = align_up(off + (size_t)kPartTokens * c->n_q_heads * 4, 1024);
    }
    l.total = off;
    return l;
}

struct ProfRec {
    cudaEvent_t a, b;
    int kind;
};

}  // namespace

struct kvf_cache {
    kvf_config cfg;
    RopeTable table;
    int device;
    int sm_count;
    char *storage;
    char *workspace;
    size_t plane_bytes;
    Layout lay;
    int64_t len;
    int G;                   // query heads per KV head
    int Gp;                  // rows a token takes in the tcgen05 kernels' row layout: G rounded up to a power of two
    float scale_log2;
    bool tc;                 // bf16, head_dim 128: the tcgen05 kernel fed by TMA
    bool tc32;               // fp32, head_dim 128: the tcgen05 kernel on fp16 halves of the operands
    TcMaps maps;
    int force_splits;
    int64_t part_rows_cap;   // rows of head_dim floats the partial area holds
    uint64_t launches;
    bool profile;
    const int32_t *page_table = nullptr;   // paged cache: device table, one page number per 128 tokens
    int64_t page_elems = 0;                // paged cache: elements per page
    int32_t n_pool_pages = 0;
    // KVF_HOST_UPLOAD_AHEAD: the library's upload stream, "upload done" and "staging set read" events
    cudaStream_t up_stream = nullptr;
    cudaEvent_t ev_up[2] = {nullptr, nullptr}, ev_read[2] = {nullptr, nullptr};
    bool ev_read_set[2] = {false, false};
    uint64_t host_steps = 0;
    // KVF_HOST_DOWNLOAD_BEHIND: the library's download stream, "step done" (caller's stream) and "results
    // copied" (download stream) events of the two result staging sets
    cudaStream_t down_stream = nullptr;
    cudaEvent_t ev_step[2] = {nullptr, nullptr}, ev_down[2] = {nullptr, nullptr};
    bool ev_down_set[2] = {false, false};
    uint64_t host_down_steps = 0;
    // KVF_COMBINE_BEHIND: the library's stream for the merge of the partial results, "attention launched"
    // (caller's stream) and "merged" (that stream) events, which capture, if any, the open merge belongs to,
    // and which of the two sets of partial results the next step with a merge writes
    cudaStream_t comb_stream = nullptr;
    cudaEvent_t ev_attn = nullptr, ev_comb = nullptr;
    bool comb_pending = false;
    unsigned long long comb_capture = 0;
    int part_set = 0;
    bool quant = false;                    // int8 storage: codes + scales in `storage`, bf16 image in the workspace
    QuantPlanes qp = {};
    int32_t n_sink = 0;                    // sink + window variant: rows always visible
    int64_t window = 0;                    // and the rows before the chunk that stay visible (0 = all)
    std::vector<ProfRec> recs;
    std::vector<cudaEvent_t> pool;
};

// Caches that advance together: one launch of each kernel folds one chunk into every member.
struct kvf_batch {
    std::vector<kvf_cache *> caches;
    char *workspace;
    size_t off_status, off_tables, off_lens, off_q_rot, off_part_o, off_part_lse;
    int64_t part_rows;       // rows of the partial area per cache
    CUtensorMap map_q;       // rotated chunks of all members: [n_caches * max_chunk][H][d]
    uint64_t launches;
};

namespace {

struct BatchLayout {
    size_t status, tables, lens, q_rot, part_o, part_lse, total;
    int64_t part_rows;
};

BatchLayout batch_layout(const kvf_config *c, int n_caches) {
    BatchLayout l;
    // per cache: what two streams of a one-tile chunk can leave (2 * (2 Hkv - 1) slots of 128 rows),
    // or its share of one cache's partial area if that is more
    int64_t rows = (int64_t)2 * (2 * c->n_kv_heads - 1) * kKvTile;
    const int64_t share = ((int64_t)kPartTokens * c->n_q_heads + n_caches - 1) / n_caches;
    if (share > rows) rows = share;
    l.part_rows = rows;
    size_t off = 0;
    l.status = off;   off = align_up(off + 256, 1024);
    l.tables = off;   off = align_up(off + (size_t)n_caches * sizeof(void *), 1024);
    l.lens = off;     off = align_up(off + (size_t)n_caches * 3 * sizeof(int64_t), 1024);   // row counts, first positions, chunk lengths
    l.q_rot = off;    off = align_up(off + (size_t)n_caches * c->max_chunk * c->n_q_heads * c->head_dim * elem_bytes(c->dtype), 1024);
    l.part_o = off;   off = align_up(off + (size_t)n_caches * rows * c->head_dim * 4, 1024);
    l.part_lse = off; off = align_up(off + (size_t)n_caches * rows * 4, 1024);
    l.total = off;
    return l;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

// 3-D bf16 tensor map (x = head_dim, y, z) with a 64-element (128-byte) swizzled inner box.
kvf_status make_map(EncodeTiledFn fn, CUtensorMap *m, void *base, uint64_t dim_y, uint64_t dim_z,
                    uint64_t stride_y_bytes, uint64_t stride_z_bytes, int d, uint32_t box_y, uint32_t box_z) {
    cuuint64_t dims[3] = {(cuuint64_t)d, dim_y, dim_z};
    cuuint64_t strides[2] = {stride_y_bytes, stride_z_bytes};
    cuuint32_t box[3] = {64u, box_y, box_z};
    cuuint32_t estr[3] = {1u, 1u, 1u};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(g_cuda_err, sizeof(g_cuda_err), "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
        return KVF_ERR_CUDA;
    }
    return KVF_OK;
}

// 4-D bf16 tensor map of a page pool: (x = head_dim, row in page, KV head, page); `base` is the K or
// the V block of page 0, consecutive pages are page_bytes apart.
kvf_status make_page_map(EncodeTiledFn fn, CUtensorMap *m, void *base, int d, int Hkv, uint64_t n_pages,
                         uint64_t page_bytes) {
    const uint64_t row = (uint64_t)d * 2;
    cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)kKvTile, (cuuint64_t)Hkv, n_pages};
    cuuint64_t strides[3] = {row, row * kKvTile, page_bytes};
    cuuint32_t box[4] = {64u, (cuuint32_t)kKvTile, 1u, 1u};
    cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(g_cuda_err, sizeof(g_cuda_err), "cuTensorMapEncodeTiled (page pool) failed with CUresult %d", (int)r);
        return KVF_ERR_CUDA;
    }
    return KVF_OK;
}

// cuTensorMapEncodeTiled, looked up in the driver once per process (a failed lookup is retried).
kvf_status encode_fn(EncodeTiledFn *fn) {
    static std::mutex mu;
    static EncodeTiledFn cached = nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!cached) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetDriverEntryPoint");
        if (qres != cudaDriverEntryPointSuccess || !sym) {
            snprintf(g_cuda_err, sizeof(g_cuda_err), "driver has no cuTensorMapEncodeTiled");
            return KVF_ERR_CUDA;
        }
        cached = reinterpret_cast<EncodeTiledFn>(sym);
    }
    *fn = cached;
    return KVF_OK;
}

kvf_status build_maps(kvf_cache *c) {
    EncodeTiledFn fn = nullptr;
    kvf_status es = encode_fn(&fn);
    if (es != KVF_OK) return es;
    const kvf_config &f = c->cfg;
    const int d = f.head_dim;
    const uint64_t row = (uint64_t)d * 2;
    // rotated queries [max_chunk][H][d]: one box = (128/Gp tokens) x (Gp heads from the first of one KV head on) x 64
    // (Gp > G: the box runs into the next KV head's queries, or past the last head, where it reads zeros - padding rows)
    kvf_status s = make_map(fn, &c->maps.q, c->workspace + c->lay.q_rot, (uint64_t)f.n_q_heads,
                            (uint64_t)f.max_chunk, row, row * f.n_q_heads, d, (uint32_t)c->Gp,
                            (uint32_t)(128 / c->Gp));
    if (s != KVF_OK) return s;
    if (c->page_table && c->quant) {
        // pages of codes: (row bytes, row in page, KV head, page), the K and the V block of a page apart
        const cuuint64_t rb = (cuuint64_t)d * c->qp.bits / 8;
        for (int kv = 0; kv < 2; ++kv) {
            cuuint64_t dims[4] = {rb, (cuuint64_t)kKvTile, (cuuint64_t)f.n_kv_heads, (cuuint64_t)c->n_pool_pages};
            cuuint64_t strides[3] = {rb, rb * kKvTile, (cuuint64_t)c->qp.page_bytes};
            cuuint32_t box[4] = {(cuuint32_t)rb, (cuuint32_t)kKvTile, 1u, 1u};
            cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
            CUresult r = fn(kv ? &c->maps.v : &c->maps.k, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, kv ? (void *)c->qp.v_codes : (void *)c->qp.k_codes,
                            dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                            c->qp.bits == 4 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) {
                snprintf(g_cuda_err, sizeof(g_cuda_err), "cuTensorMapEncodeTiled (paged codes) failed with CUresult %d", (int)r);
                return KVF_ERR_CUDA;
            }
        }
        return KVF_OK;
    }
    if (c->page_table) {
        const uint64_t page_bytes = (uint64_t)c->page_elems * 2;
        s = make_page_map(fn, &c->maps.k, c->storage, d, f.n_kv_heads, (uint64_t)c->n_pool_pages, page_bytes);
        if (s != KVF_OK) return s;
        return make_page_map(fn, &c->maps.v, c->storage + c->plane_bytes, d, f.n_kv_heads, (uint64_t)c->n_pool_pages,
                             page_bytes);
    }
    if (c->quant) {
        // code planes [Hkv][capacity][row bytes]: one box = 128 rows of one head x 128 (int8) or 64 (int4)
        // bytes, swizzled over the row's 16-byte chunks
        const cuuint64_t rb = (cuuint64_t)d * c->qp.bits / 8;
        for (int kv = 0; kv < 2; ++kv) {
            cuuint64_t dims[3] = {rb, (cuuint64_t)f.capacity, (cuuint64_t)f.n_kv_heads};
            cuuint64_t strides[2] = {rb, rb * f.capacity};
            cuuint32_t box[3] = {(cuuint32_t)rb, (cuuint32_t)kKvTile, 1u};
            cuuint32_t estr[3] = {1u, 1u, 1u};
            CUresult r = fn(kv ? &c->maps.v : &c->maps.k, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, kv ? (void *)c->qp.v_codes : (void *)c->qp.k_codes,
                            dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                            c->qp.bits == 4 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) {
                snprintf(g_cuda_err, sizeof(g_cuda_err), "cuTensorMapEncodeTiled (int8 codes) failed with CUresult %d", (int)r);
                return KVF_ERR_CUDA;
            }
        }
        return KVF_OK;
    }
    // planes [Hkv][capacity][d]: one box = 128 rows of one head x 64
    char *kbase = c->storage;
    char *vbase = c->storage + c->plane_bytes;
    s = make_map(fn, &c->maps.k, kbase, (uint64_t)f.capacity, (uint64_t)f.n_kv_heads, row,
                 row * f.capacity, d, (uint32_t)kKvTile, 1u);
    if (s != KVF_OK) return s;
    return make_map(fn, &c->maps.v, vbase, (uint64_t)f.capacity,
                    (uint64_t)f.n_kv_heads, row, row * f.capacity, d, (uint32_t)kKvTile, 1u);
}

struct Plan {
    bool qdec;     // a few query rows on a bf16 or quantised cache: the decode kernel that feeds MMAs from registers
    bool tc;
    int splits;    // CUDA-core path: splits of the key range; tensor-core path: ranges per KV head (rounded up)
    int ngroups;   // tensor-core path: ranges of the (KV head, key tile) line
    int ctas, kernels;
};

// `batch` caches share the launch (their CTAs fill the SMs together) and `part_rows_cap` is the
// partial area of ONE cache.
// First row of the window for a chunk that starts at row `prefix` (0 = every earlier row is visible).
int64_t window_lo(const kvf_cache *c, int64_t prefix) {
    if (c->window <= 0) return 0;
    const int64_t lo = prefix - c->window;
    return lo <= c->n_sink ? 0 : lo;       // the window reaches the sinks: nothing is hidden
}

Plan make_plan(const kvf_cache *c, int n, int64_t prefix, int batch = 1, int64_t part_rows_cap = -1) {
    if (part_rows_cap < 0) part_rows_cap = c->part_rows_cap;
    Plan p;
    p.qdec = false;
    p.tc = c->tc || c->tc32;
    p.ngroups = 0;
    const int64_t L = prefix + n;
    const int Hkv = c->cfg.n_kv_heads;
    if ((c->quant || c->tc) && c->window <= 0 && n * c->G <= attn_q8_decode_max_rows()) {
        // one CTA per SM (all caches of a batch together), each inside one KV head (a multiple of the KV heads),
        // at least two key tiles each; a forced split count is the number of ranges per KV head
        const int64_t nt = (L + kKvTile - 1) / kKvTile;
        int64_t per_head = c->force_splits > 0 ? c->force_splits : c->sm_count / (Hkv * batch);
        if (c->force_splits <= 0 && per_head > nt / 2) per_head = nt / 2;
        if (per_head > nt) per_head = nt;
        const int64_t slots_cap = part_rows_cap / ((int64_t)n * c->Gp);           // slots = groups + Hkv - 1
        if (per_head * Hkv + Hkv - 1 > slots_cap) per_head = (slots_cap - (Hkv - 1)) / Hkv;
        if (per_head < 1) per_head = 1;
        p.qdec = true;
        p.ngroups = (int)(per_head * Hkv);
        p.splits = (int)per_head;
        p.ctas = p.ngroups * batch;
        p.kernels = 2 + (per_head > 1 ? 1 : 0);
        return p;
    }
    if (p.tc) {
        // one CTA per (row pair, group); the groups cut the Hkv * nt line of (KV head, key tile)
        // into equal ranges.  Whole KV heads if that fills the SMs, else as many groups as give
        // one CTA per SM, with at least 4 key tiles each and within the partial area.
        const int64_t nt = (L + kKvTile - 1) / kKvTile - WindowTiles(window_lo(c, prefix), c->n_sink, kKvTile).skip;
        // (row blocks of a KV head: 256-row pairs in the bf16 kernel, 128-row blocks in the fp32 one)
        const int pairs = c->tc32 ? attn_tc32_row_blocks(n, c->Gp) : attn_tc_row_pairs(n, c->Gp);
        int64_t groups = Hkv;
        if (c->force_splits > 0) {
            groups = (int64_t)Hkv * c->force_splits;
        } else if ((int64_t)pairs * Hkv * batch < c->sm_count) {
            groups = c->sm_count / (pairs * batch);
            if (groups > Hkv * nt / 4) groups = Hkv * nt / 4;
            // A group count that is a multiple of the KV heads keeps every CTA inside one KV head: one Q load
            // and one set of partial rows instead of two.  Measured at C = 256 (Llama shape): the second
            // piece costs a CTA about as long as 3.3 key tiles, so while the line is short - here below
            // ~12 K tokens - 128 aligned CTAs beat 148 that straddle KV heads.
            const int64_t aligned = groups / Hkv * Hkv;
            if (aligned >= Hkv && aligned < groups) {
                const double line = (double)Hkv * (double)nt;
                if (line / (double)aligned - line / (double)groups < 3.3) groups = aligned;
            }
        } else {
            // whole KV heads fill the SMs, but the last wave may be half empty (256 CTAs on 148 SMs):
            // cut a little finer - up to twice the KV heads - if that fills the waves at least 5 %
            // better; the price is the partial results of one chunk and the combine kernel
            auto fill = [&](int64_t g) {
                const int64_t ctas = (int64_t)pairs * g * batch;
                const int64_t waves = (ctas + c->sm_count - 1) / c->sm_count;
                return (double)ctas / (double)(waves * c->sm_count);
            };
            double best = fill(Hkv) + 0.05;
            for (int64_t g = Hkv + 1; g <= 2 * Hkv && g * 4 <= Hkv * nt; ++g)
                if (fill(g) > best) { best = fill(g); groups = g; }
        }
        const int streams = c->tc32 ? 1 : attn_tc_streams(n, c->Gp);
        const int64_t slots_cap = part_rows_cap / ((int64_t)n * c->Gp) / streams;   // slots = streams * (groups + Hkv - 1)
        if (groups + Hkv - 1 > slots_cap) groups = slots_cap - (Hkv - 1);
        if (groups > Hkv * nt) groups = Hkv * nt;
        if (groups < Hkv) groups = Hkv;
        p.ngroups = (int)groups;
        p.splits = (int)((groups + Hkv - 1) / Hkv);
        p.ctas = pairs * p.ngroups * batch;
        p.kernels = 2 + ((p.ngroups != Hkv || streams == 2) ? 1 : 0);   // short chunks always leave two parts
        return p;
    }
    const int64_t nt = (L + 63) / 64 - WindowTiles(window_lo(c, prefix), c->n_sink, 64).skip;
    const int units = attn_simt_ctas(n, c->G, Hkv, 1);
    const int target = c->sm_count * 2;
    int64_t max_splits = part_rows_cap / ((int64_t)n * c->cfg.n_q_heads);
    if (max_splits > kMaxSplits) max_splits = kMaxSplits;
    if (max_splits < 1) max_splits = 1;
    int splits = 1;
    if (c->force_splits > 0) {
        splits = c->force_splits;
    } else if (units < target) {
        // one wave: as many splits as still fit the machine at once (a second, partly filled
        // wave would double the time), but keep at least 4 key tiles per split
        int want = target / units;
        int64_t cap = nt / 4;
        if (want > cap) want = (int)cap;
        splits = want;
    }
    if (splits > max_splits) splits = (int)max_splits;
    if ((int64_t)splits > nt) splits = (int)nt;
    if (splits < 1) splits = 1;
    p.splits = splits;
    p.ctas = units * splits;
    p.kernels = 2 + (splits > 1 ? 1 : 0);
    return p;
}

cudaEvent_t get_event(kvf_cache *c) {
    if (!c->pool.empty()) {
        cudaEvent_t e = c->pool.back();
        c->pool.pop_back();
        return e;
    }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
}

struct ProfScope {
    kvf_cache *c;
    cudaStream_t s;
    ProfRec r;
    bool on;
    ProfScope(kvf_cache *c_, cudaStream_t s_, int kind) : c(c_), s(s_), on(false) {
        if (c->profile && c->recs.size() < 65536) {
            r.a = get_event(c);
            r.b = get_event(c);
            r.kind = kind;
            on = r.a && r.b;
            if (on) cudaEventRecord(r.a, s);
        }
    }
    ~ProfScope() {
        if (on) {
            cudaEventRecord(r.b, s);
            c->recs.push_back(r);
        }
    }
};

kvf_status check_ptr(const void *p) {
    if (!p) return KVF_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(p) & 15u) return KVF_ERR_INVALID_ARG;
    return KVF_OK;
}

// What a second piece costs a CTA of the bf16 / quantised tcgen05 kernel, in key tiles (measured at C = 256 on
// the Llama shape: ~3.3): the line the groups cut carries that many virtual tiles in front of every KV head, so a
// CTA whose range runs into the next head takes as many key tiles fewer and all CTAs of a launch finish
// together.  Only where ranges do run across heads (a group count that is no multiple of the KV heads) and for
// chunks of two row tiles; the fp32 kernel and the decode kernel cut the plain line.
#ifndef KVF_PIECE_COST
#define KVF_PIECE_COST 3
#endif
int piece_cost_of(const kvf_cache *c, const Plan &plan, int streams) {
    if (!c->tc || plan.qdec || streams != 1 || plan.ngroups % c->cfg.n_kv_heads == 0) return 0;
    return KVF_PIECE_COST;
}

// A step whose attention kernel is long enough for a chain of such steps to run at the power cap: bf16 rows, full
// row tiles on the tensor cores and at least KVF_PDL_MAX_TILES key tiles per CTA.
#ifndef KVF_PDL_MAX_TILES
#define KVF_PDL_MAX_TILES 32
#endif
bool long_step(const kvf_cache *c, const Plan &plan, int streams, int64_t L) {
    // KVF_DEPENDENT_LAUNCH=always / never in the environment overrides the rule (read once; for measurements)
    static const int forced = [] {
        const char *e = std::getenv("KVF_DEPENDENT_LAUNCH");
        return !e ? 0 : std::strcmp(e, "always") == 0 ? 1 : std::strcmp(e, "never") == 0 ? 2 : 0;
    }();
    if (forced) return forced == 2;
    // (bf16 rows only: the quantised kernels are bound by issue slots and the fp32 kernel by its softmax thread,
    // not by the power cap - measured, they keep 0.2 - 0.5 % with dependent launches)
    if (!c->tc || c->quant || plan.qdec || streams != 1 || plan.ngroups <= 0 || c->window > 0) return false;
    const int64_t nt = (L + kKvTile - 1) / kKvTile;
    return nt * c->cfg.n_kv_heads >= (int64_t)KVF_PDL_MAX_TILES * plan.ngroups;
}

// The groups that touch each KV head, worked out once on the host for the combine kernel.
void fill_group_ranges(AttnArgs &aa, int64_t nt_all) {
    aa.range_valid = 0;
    if (aa.ngroups <= 0 || aa.ngroups > 32767 || nt_all <= 0 || nt_all > (int64_t)1 << 30) return;
    for (int h = 0; h < aa.Hkv && h < kRangeHeads; ++h) {
        int g0, g1;
        group_range(aa.Hkv, (int)nt_all, aa.ngroups, h, g0, g1);
        aa.g_first[h] = (int16_t)g0;
        aa.g_last[h] = (int16_t)g1;
    }
    aa.range_valid = 1;
}

// The capture `st` is part of (0: none).  An event recorded in one capture cannot be waited for
// from outside it or from another one.
kvf_status capture_of(cudaStream_t st, unsigned long long *id) {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    unsigned long long cid = 0;
    cudaError_t e = cudaStreamGetCaptureInfo(st, &cs, &cid);
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamGetCaptureInfo");
    *id = cs == cudaStreamCaptureStatusActive ? cid : 0;
    return KVF_OK;
}

// Makes `st` wait for a merge that still runs on the library's stream.
kvf_status join_combine(kvf_cache *c, cudaStream_t st) {
    if (!c->comb_pending) return KVF_OK;
    cudaError_t e = cudaStreamWaitEvent(st, c->ev_comb, 0);
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamWaitEvent(merge)");
    c->comb_pending = false;
    return KVF_OK;
}

kvf_status step_impl(kvf_cache *c, const void *q, const void *k_new, const void *v_new, int32_t n,
                     int64_t pos0, void *out, float *lse, cudaStream_t st) {
    const kvf_config &f = c->cfg;
    const int64_t P = c->len;
    // k_new == null: queries only (kvf_attend) - nothing is appended, every query row sees the P rows held
    const bool attend = k_new == nullptr;
    const int64_t L = attend ? P : P + n;                     // rows the step's queries can see at most
    const Plan plan = make_plan(c, n, L - n);
    const bool behind = c->comb_stream != nullptr;
    unsigned long long capture = 0;
    if (behind) {
        kvf_status s = capture_of(st, &capture);
        if (s != KVF_OK) return s;
        if (c->comb_pending && capture != c->comb_capture) return KVF_ERR_INVALID_ARG;    // flush first
    }

    RopeAppendArgs ra;
    ra.q = q; ra.k_new = k_new; ra.v_new = v_new;
    ra.q_rot = c->workspace + c->lay.q_rot;
    ra.k_plane = c->storage;
    ra.v_plane = c->storage + c->plane_bytes;
    ra.capacity = f.capacity; ra.prefix = P; ra.pos0 = pos0;
    ra.n = n; ra.H = f.n_q_heads; ra.Hkv = f.n_kv_heads; ra.d = f.head_dim;
    {
        int64_t pad_end = (L + kKvTile - 1) / kKvTile * kKvTile;
        if (pad_end > f.capacity && !c->page_table) pad_end = f.capacity;   // a page always has its 128 rows
        ra.zero_rows = attend ? 0 : (int32_t)(pad_end - L);
    }
    ra.page_table = c->page_table;
    ra.page_elems = c->page_elems;
    ra.page_tables = nullptr;
    ra.prefixes = nullptr; ra.pos0s = nullptr; ra.ns = nullptr;
    ra.status = reinterpret_cast<int *>(c->workspace + c->lay.status);
    ra.range_limit = c->tc32 ? 65504.f : 0.f;      // the fp32 tensor-core kernel computes on fp16 halves
    ra.table = c->table;

    AttnArgs aa;
    aa.q_rot = ra.q_rot;
    aa.k_plane = ra.k_plane; aa.v_plane = ra.v_plane;
    aa.out = out; aa.lse = lse;
    // (with the merge behind the step, this step's attention kernel fills one set of partial results while
    // the merge of the step before may still read the other)
    const bool second = behind && c->part_set == 1;
    aa.part_o = reinterpret_cast<float *>(c->workspace + (second ? c->lay.part_o2 : c->lay.part_o));
    aa.part_lse = reinterpret_cast<float *>(c->workspace + (second ? c->lay.part_lse2 : c->lay.part_lse));
    aa.status = reinterpret_cast<int *>(c->workspace + c->lay.status);
    aa.page_table = c->page_table;
    aa.page_tables = nullptr; aa.part_rows = 0; aa.batch = 1; aa.prefixes = nullptr; aa.ns = nullptr;
    aa.n_sink = c->n_sink; aa.win_lo = window_lo(c, P);
    aa.k_scales = c->quant ? c->qp.k_scales : nullptr;
    aa.v_scales = c->quant ? c->qp.v_scales : nullptr;
    aa.scale_stride = c->qp.scale_stride;
    aa.scale_page_stride = c->qp.page_bytes / 4;
    aa.quant_bits = c->quant ? c->qp.bits : 0;
    aa.capacity = f.capacity; aa.prefix = P;
    aa.n = n; aa.H = f.n_q_heads; aa.Hkv = f.n_kv_heads; aa.G = c->G; aa.d = f.head_dim;
    aa.Gp = c->Gp;
    aa.splits = plan.tc ? 1 : plan.splits;
    aa.ngroups = plan.ngroups;
    aa.streams = (c->tc && !plan.qdec) ? attn_tc_streams(n, c->Gp) : 1;
    aa.out_f32 = (f.dtype == KVF_F32 || (f.flags & KVF_OUT_F32)) ? 1 : 0;
    aa.scale_log2 = c->scale_log2;
    aa.range_valid = 0;
    aa.piece_cost = piece_cost_of(c, plan, aa.streams);
    aa.self_rows = attend ? 0 : 1;
    if (plan.tc && plan.kernels > 2)
        fill_group_ranges(aa, (L + kKvTile - 1) / kKvTile - WindowTiles(aa.win_lo, aa.n_sink, kKvTile).skip + aa.piece_cost);

    // plain launches for long tensor-bound steps, dependent launches for short ones (see g_pdl_allowed)
    const PdlScope pdl(!long_step(c, plan, aa.streams, L));
    cudaError_t e;
    if (c->quant) {
        // int8 storage: rotate + quantise + append (the attention kernel expands the code tiles itself)
        ProfScope ps(c, st, 0);
        e = launch_rope_append_q8(ra, c->qp, (f.flags & KVF_ROPE_INTERLEAVED) != 0, 1, st);
    } else {
        ProfScope ps(c, st, 0);
        e = launch_rope_append(ra, f.dtype, (f.flags & KVF_ROPE_INTERLEAVED) != 0, 1, st);
    }
    if (e != cudaSuccess) return cuda_fail(e, "rope_append launch");
    c->launches++;
    {
        ProfScope ps(c, st, 1);
        if (plan.qdec) e = launch_attn_q8_decode(aa, c->maps, st);
        else if (c->tc) e = launch_attn_tc(aa, c->maps, st);
        else if (c->tc32) e = launch_attn_tc32(aa, st);
        else e = launch_attn_simt(aa, f.dtype, st, nullptr);
    }
    if (e != cudaSuccess) return cuda_fail(e, "attention launch");
    c->launches++;
    if (behind && plan.kernels > 2) {
        // the merge goes behind the attention kernel on the library's stream; the caller's stream
        // meets it again at the end of the next step, or in kvf_cache_flush
        e = cudaEventRecord(c->ev_attn, st);
        if (e != cudaSuccess) return cuda_fail(e, "cudaEventRecord(attention)");
    }
    // the merge of the step before: behind this step's attention kernel on the caller's stream, which by
    // now has had that whole kernel to hide under (its set of partial results is written again in the next step)
    if (kvf_status s = join_combine(c, st)) return s;
    if (plan.kernels > 2) {
        cudaStream_t cs = st;
        if (behind) {
            cs = c->comb_stream;
            e = cudaStreamWaitEvent(cs, c->ev_attn, 0);
            if (e != cudaSuccess) return cuda_fail(e, "merge stream hand-over");
        }
        {
            ProfScope ps(c, cs, 2);
            e = plan.tc ? launch_combine_groups(aa, cs) : launch_combine(aa, f.dtype, cs);
        }
        if (e != cudaSuccess) return cuda_fail(e, "combine launch");
        c->launches++;
        if (behind) {
            e = cudaEventRecord(c->ev_comb, cs);
            if (e != cudaSuccess) return cuda_fail(e, "cudaEventRecord(merge)");
            c->comb_pending = true;
            c->comb_capture = capture;
            c->part_set ^= 1;
        }
    }
    c->len = L;
    return KVF_OK;
}

// What every handle starts from: shape, device, buffers, rotation table, softmax scale, counters.
kvf_status init_handle(kvf_cache *c, const kvf_config *cfg, void *storage, void *workspace) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
    c->cfg = *cfg;
    c->cfg.inv_freq = nullptr;
    c->device = dev;
    c->sm_count = sms;
    c->storage = static_cast<char *>(storage);
    c->workspace = static_cast<char *>(workspace);
    c->len = 0;
    c->G = cfg->n_q_heads / cfg->n_kv_heads;
    c->Gp = attn_tc_padded_group(c->G);
    const double scale = cfg->softmax_scale > 0.0 ? cfg->softmax_scale : 1.0 / std::sqrt((double)cfg->head_dim);
    c->scale_log2 = (float)(scale * 1.4426950408889634);
    for (int j = 0; j < cfg->head_dim / 2; ++j)
        c->table.inv_freq[j] = cfg->inv_freq ? cfg->inv_freq[j]
                                             : std::pow(cfg->rope_base, -2.0 * (double)j / (double)cfg->head_dim);
    for (int j = cfg->head_dim / 2; j < kMaxHalfDim; ++j) c->table.inv_freq[j] = 0.0;
    c->force_splits = 0;
    c->part_rows_cap = (int64_t)kPartTokens * cfg->n_q_heads;
    c->launches = 0;
    c->profile = false;
    c->tc = !(cfg->flags & KVF_FORCE_SIMT) && attn_tc_supported(cfg->dtype, cfg->head_dim, c->G);
    c->tc32 = !(cfg->flags & KVF_FORCE_SIMT) && attn_tc32_supported(cfg->dtype, cfg->head_dim, c->G);
    return KVF_OK;
}

// KVF_COMBINE_BEHIND: the stream and the events are made with the handle, so that a step inside a
// stream capture creates nothing.
kvf_status setup_combine_behind(kvf_cache *c) {
    if (!(c->cfg.flags & KVF_COMBINE_BEHIND)) return KVF_OK;
    cudaError_t e = cudaStreamCreateWithFlags(&c->comb_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_attn, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_comb, cudaEventDisableTiming);
    return e == cudaSuccess ? KVF_OK : cuda_fail(e, "merge stream setup");
}

// Bytes of one page: 128 tokens of every KV head, K block then V block; quantised caches keep the rows'
// codes there and behind them one fp32 scale per row, K then V.
size_t page_bytes_of(const kvf_config *cfg) {
    const size_t rows = 2 * (size_t)cfg->n_kv_heads * kKvTile;
    if (cfg->flags & (KVF_CACHE_INT8 | KVF_CACHE_INT4))
        return rows * ((cfg->flags & KVF_CACHE_INT4) ? (size_t)cfg->head_dim / 2 : (size_t)cfg->head_dim) + rows * 4;
    return rows * (size_t)cfg->head_dim * elem_bytes(cfg->dtype);
}

kvf_status check_step(kvf_cache *c, int32_t n, int64_t pos0) {
    if (!c) return KVF_ERR_INVALID_ARG;
    if (n < 1 || n > c->cfg.max_chunk) return KVF_ERR_INVALID_ARG;
    if (pos0 < 0) return KVF_ERR_INVALID_ARG;
    if (c->len + n > c->cfg.capacity) return KVF_ERR_CAPACITY;
    if ((c->cfg.flags & KVF_STRICT_POS) && pos0 != c->len) return KVF_ERR_POS;
    return KVF_OK;
}

}  // namespace

extern "C" {

size_t kvf_cache_storage_bytes(const kvf_config *cfg) {
    if (check_config(cfg) != KVF_OK) return 0;
    if (cfg->flags & (KVF_CACHE_INT8 | KVF_CACHE_INT4)) {
        // codes and one fp32 scale per row (rows of scales padded to 16 bytes), K and V
        const size_t row = (cfg->flags & KVF_CACHE_INT4) ? (size_t)cfg->head_dim / 2 : (size_t)cfg->head_dim;
        return 2 * (size_t)cfg->n_kv_heads * ((size_t)cfg->capacity * row + align_up((size_t)cfg->capacity, 4) * 4);
    }
    return 2 * (size_t)cfg->n_kv_heads * (size_t)cfg->capacity * (size_t)cfg->head_dim * elem_bytes(cfg->dtype);
}

size_t kvf_workspace_bytes(const kvf_config *cfg) {
    if (check_config(cfg) != KVF_OK) return 0;
    return workspace_layout(cfg).total;
}

kvf_status kvf_cache_create(const kvf_config *cfg, void *dev_storage, size_t storage_bytes,
                            void *dev_workspace, size_t workspace_bytes, kvf_cache **out) {
    if (!out) return KVF_ERR_INVALID_ARG;
    *out = nullptr;
    kvf_status s = check_config(cfg);
    if (s != KVF_OK) return s;
    if (!dev_storage || !dev_workspace) return KVF_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(dev_storage) & 255u) || (reinterpret_cast<uintptr_t>(dev_workspace) & 255u))
        return KVF_ERR_INVALID_ARG;
    if (storage_bytes < kvf_cache_storage_bytes(cfg)) return KVF_ERR_CAPACITY;
    if (workspace_bytes < kvf_workspace_bytes(cfg)) return KVF_ERR_CAPACITY;

    kvf_cache *c = new (std::nothrow) kvf_cache();
    if (!c) return KVF_ERR_INVALID_ARG;
    s = init_handle(c, cfg, dev_storage, dev_workspace);
    if (s != KVF_OK) { delete c; return s; }
    c->plane_bytes = kvf_cache_storage_bytes(cfg) / 2;
    c->lay = workspace_layout(cfg);
    if (cfg->flags & (KVF_CACHE_INT8 | KVF_CACHE_INT4)) {
        c->qp.bits = (cfg->flags & KVF_CACHE_INT4) ? 4 : 8;
        const size_t codes = (size_t)cfg->n_kv_heads * cfg->capacity * cfg->head_dim * c->qp.bits / 8;
        c->quant = true;
        c->plane_bytes = codes;
        c->qp.k_codes = reinterpret_cast<int8_t *>(c->storage);
        c->qp.v_codes = c->qp.k_codes + codes;
        c->qp.k_scales = reinterpret_cast<float *>(c->storage + 2 * codes);
        c->qp.scale_stride = (int64_t)align_up((size_t)cfg->capacity, 4);
        c->qp.v_scales = c->qp.k_scales + (size_t)cfg->n_kv_heads * c->qp.scale_stride;
    }
    if (c->tc) {
        s = build_maps(c);
        if (s != KVF_OK) { delete c; return s; }
    }
    cudaError_t e = cudaMemset(c->workspace + c->lay.status, 0, 256);
    if (e != cudaSuccess) { delete c; return cuda_fail(e, "cudaMemset(status)"); }
    s = setup_combine_behind(c);
    if (s != KVF_OK) { kvf_cache_destroy(c); return s; }
    *out = c;
    return KVF_OK;
}

size_t kvf_paged_pool_bytes(const kvf_config *cfg, int32_t n_pages) {
    if (check_config(cfg) != KVF_OK || n_pages <= 0) return 0;
    return (size_t)n_pages * page_bytes_of(cfg);
}

kvf_status kvf_paged_cache_create(const kvf_config *cfg, void *dev_pool, size_t pool_bytes, int32_t n_pool_pages,
                                  const int32_t *dev_page_table, void *dev_workspace, size_t workspace_bytes,
                                  kvf_cache **out) {
    if (!out) return KVF_ERR_INVALID_ARG;
    *out = nullptr;
    kvf_status s = check_config(cfg);
    if (s != KVF_OK) return s;
    const int G = cfg->n_q_heads / cfg->n_kv_heads;
    if ((cfg->flags & KVF_FORCE_SIMT) || !attn_tc_supported(cfg->dtype, cfg->head_dim, G)) return KVF_ERR_UNSUPPORTED;
    if (!dev_pool || !dev_workspace || !dev_page_table || n_pool_pages <= 0) return KVF_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(dev_pool) & 255u) || (reinterpret_cast<uintptr_t>(dev_workspace) & 255u) ||
        (reinterpret_cast<uintptr_t>(dev_page_table) & 3u))
        return KVF_ERR_INVALID_ARG;
    if (pool_bytes < kvf_paged_pool_bytes(cfg, n_pool_pages)) return KVF_ERR_CAPACITY;
    if (workspace_bytes < kvf_workspace_bytes(cfg)) return KVF_ERR_CAPACITY;

    kvf_cache *c = new (std::nothrow) kvf_cache();
    if (!c) return KVF_ERR_INVALID_ARG;
    s = init_handle(c, cfg, dev_pool, dev_workspace);
    if (s != KVF_OK) { delete c; return s; }
    c->page_table = dev_page_table;
    c->n_pool_pages = n_pool_pages;
    c->page_elems = (int64_t)2 * cfg->n_kv_heads * kKvTile * cfg->head_dim;
    c->plane_bytes = (size_t)cfg->n_kv_heads * kKvTile * cfg->head_dim * elem_bytes(cfg->dtype);   // V block inside a page
    if (cfg->flags & (KVF_CACHE_INT8 | KVF_CACHE_INT4)) {
        // quantised pages: [K codes | V codes][Hkv][128][row bytes], then [K scales | V scales][Hkv][128] fp32
        c->quant = true;
        c->qp.bits = (cfg->flags & KVF_CACHE_INT4) ? 4 : 8;
        const size_t codes = (size_t)cfg->n_kv_heads * kKvTile * cfg->head_dim * c->qp.bits / 8;   // one block of codes
        c->plane_bytes = codes;
        c->qp.page_bytes = (int64_t)page_bytes_of(cfg);
        c->qp.k_codes = reinterpret_cast<int8_t *>(c->storage);
        c->qp.v_codes = c->qp.k_codes + codes;
        c->qp.k_scales = reinterpret_cast<float *>(c->storage + 2 * codes);
        c->qp.v_scales = c->qp.k_scales + (size_t)cfg->n_kv_heads * kKvTile;
        c->qp.scale_stride = 0;
    }
    c->lay = workspace_layout(cfg);
    s = build_maps(c);
    if (s != KVF_OK) { delete c; return s; }
    cudaError_t e = cudaMemset(c->workspace + c->lay.status, 0, 256);
    if (e != cudaSuccess) { delete c; return cuda_fail(e, "cudaMemset(status)"); }
    s = setup_combine_behind(c);
    if (s != KVF_OK) { kvf_cache_destroy(c); return s; }
    *out = c;
    return KVF_OK;
}

kvf_status kvf_fold_step(kvf_cache *c, const void *q, const void *k_new, const void *v_new,
                         int32_t n_tokens, int64_t pos0, void *out, float *lse, void *cuda_stream) {
    kvf_status s = check_step(c, n_tokens, pos0);
    if (s != KVF_OK) return s;
    if (check_ptr(q) || check_ptr(k_new) || check_ptr(v_new) || check_ptr(out)) return KVF_ERR_INVALID_ARG;
    if (lse && (reinterpret_cast<uintptr_t>(lse) & 3u)) return KVF_ERR_INVALID_ARG;
    return step_impl(c, q, k_new, v_new, n_tokens, pos0, out, lse, static_cast<cudaStream_t>(cuda_stream));
}

kvf_status kvf_attend(kvf_cache *c, const void *q, int32_t n_tokens, int64_t pos0, void *out, float *lse,
                      void *cuda_stream) {
    if (!c) return KVF_ERR_INVALID_ARG;
    if (n_tokens < 1 || n_tokens > c->cfg.max_chunk || pos0 < 0) return KVF_ERR_INVALID_ARG;
    if (c->len < 1) return KVF_ERR_INVALID_ARG;               // nothing to attend to
    if (c->window > 0) return KVF_ERR_UNSUPPORTED;
    if (check_ptr(q) || check_ptr(out)) return KVF_ERR_INVALID_ARG;
    if (lse && (reinterpret_cast<uintptr_t>(lse) & 3u)) return KVF_ERR_INVALID_ARG;
    return step_impl(c, q, nullptr, nullptr, n_tokens, pos0, out, lse, static_cast<cudaStream_t>(cuda_stream));
}

kvf_status kvf_merge_partials(int32_t n_parts, int64_t n_rows, int32_t head_dim, kvf_dtype dtype, const void *parts_out,
                              const float *parts_lse, void *out, float *lse, void *cuda_stream) {
    if (n_parts < 1 || n_parts > 1024 || n_rows < 1) return KVF_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return KVF_ERR_UNSUPPORTED;
    if (dtype != KVF_BF16 && dtype != KVF_F32) return KVF_ERR_UNSUPPORTED;
    if (check_ptr(parts_out) || check_ptr(out) || !parts_lse) return KVF_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(parts_lse) & 3u) || (lse && (reinterpret_cast<uintptr_t>(lse) & 3u))) return KVF_ERR_INVALID_ARG;
    cudaError_t e = launch_merge_parts(n_parts, n_rows, head_dim, dtype == KVF_F32, parts_out, parts_lse, out, lse,
                                       static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? KVF_OK : cuda_fail(e, "merge_parts launch");
}

kvf_status kvf_fold_step_host(kvf_cache *c, const void *q_host, const void *k_host, const void *v_host,
                              int32_t n_tokens, int64_t pos0, void *out_host, float *lse_host,
                              void *cuda_stream) {
    kvf_status s = check_step(c, n_tokens, pos0);
    if (s != KVF_OK) return s;
    if (!q_host || !k_host || !v_host || !out_host) return KVF_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const kvf_config &f = c->cfg;
    const size_t eb = elem_bytes(f.dtype);
    const size_t qb = (size_t)n_tokens * f.n_q_heads * f.head_dim * eb;
    const size_t kb = (size_t)n_tokens * f.n_kv_heads * f.head_dim * eb;
    const size_t ob = (size_t)n_tokens * f.n_q_heads * f.head_dim * ((f.flags & KVF_OUT_F32) ? 4 : eb);
    char *w = c->workspace;
    cudaError_t e = cudaSuccess;
    size_t oq = c->lay.st_q, ok_ = c->lay.st_k, ov = c->lay.st_v;
    int set = 0;
    if (f.flags & KVF_HOST_UPLOAD_AHEAD) {
        // upload on the library's stream into the staging set the step before last used: it runs
        // while the previous step computes, and starts once that set's last reader (the rotate +
        // append kernel of two steps ago, marked by ev_read) is done
        if (!c->up_stream) {
            e = cudaStreamCreateWithFlags(&c->up_stream, cudaStreamNonBlocking);
            for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
                e = cudaEventCreateWithFlags(&c->ev_up[i], cudaEventDisableTiming);
                if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_read[i], cudaEventDisableTiming);
            }
            if (e != cudaSuccess) return cuda_fail(e, "upload stream setup");
        }
        set = (int)(c->host_steps & 1);
        if (set) { oq = c->lay.st_q2; ok_ = c->lay.st_k2; ov = c->lay.st_v2; }
        cudaStream_t up = c->up_stream;
        if (c->ev_read_set[set]) e = cudaStreamWaitEvent(up, c->ev_read[set], 0);
        if (e == cudaSuccess) e = cudaMemcpyAsync(w + oq, q_host, qb, cudaMemcpyHostToDevice, up);
        if (e == cudaSuccess) e = cudaMemcpyAsync(w + ok_, k_host, kb, cudaMemcpyHostToDevice, up);
        if (e == cudaSuccess) e = cudaMemcpyAsync(w + ov, v_host, kb, cudaMemcpyHostToDevice, up);
        if (e == cudaSuccess) e = cudaEventRecord(c->ev_up[set], up);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(st, c->ev_up[set], 0);
    } else {
        e = cudaMemcpyAsync(w + oq, q_host, qb, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaMemcpyAsync(w + ok_, k_host, kb, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaMemcpyAsync(w + ov, v_host, kb, cudaMemcpyHostToDevice, st);
    }
    if (e != cudaSuccess) return cuda_fail(e, "host-to-device copy");
    const bool behind = (f.flags & KVF_HOST_DOWNLOAD_BEHIND) != 0;
    int oset = 0;
    size_t o_out = c->lay.st_out, o_lse = c->lay.st_lse;
    if (behind) {
        if (!c->down_stream) {
            e = cudaStreamCreateWithFlags(&c->down_stream, cudaStreamNonBlocking);
            for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
                e = cudaEventCreateWithFlags(&c->ev_step[i], cudaEventDisableTiming);
                if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_down[i], cudaEventDisableTiming);
            }
            if (e != cudaSuccess) return cuda_fail(e, "download stream setup");
        }
        oset = (int)(c->host_down_steps & 1);
        if (oset) { o_out = c->lay.st_out2; o_lse = c->lay.st_lse2; }
        // this result set was last copied out two steps ago: the step must not overwrite it before that copy is done
        if (c->ev_down_set[oset]) {
            e = cudaStreamWaitEvent(st, c->ev_down[oset], 0);
            if (e != cudaSuccess) return cuda_fail(e, "cudaStreamWaitEvent(download)");
        }
    }
    float *lse_dev = lse_host ? reinterpret_cast<float *>(w + o_lse) : nullptr;
    s = step_impl(c, w + oq, w + ok_, w + ov, n_tokens, pos0, w + o_out, lse_dev, st);
    if (s != KVF_OK) return s;
    if (f.flags & KVF_HOST_UPLOAD_AHEAD) {
        e = cudaEventRecord(c->ev_read[set], st);      // (after the whole step: later than needed, never too early)
        if (e != cudaSuccess) return cuda_fail(e, "cudaEventRecord");
        c->ev_read_set[set] = true;
        c->host_steps++;
    }
    cudaStream_t ds = behind ? c->down_stream : st;
    if (behind) {
        // the copies of this step's results run on the library's stream, behind the step, while the caller's
        // stream goes on with the next step
        e = cudaEventRecord(c->ev_step[oset], st);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(ds, c->ev_step[oset], 0);
        if (e == cudaSuccess && c->comb_pending) e = cudaStreamWaitEvent(ds, c->ev_comb, 0);   // the merge writes the results
        if (e != cudaSuccess) return cuda_fail(e, "download stream hand-over");
    } else if (kvf_status js = join_combine(c, st)) {
        return js;
    }
    e = cudaMemcpyAsync(out_host, w + o_out, ob, cudaMemcpyDeviceToHost, ds);
    if (e == cudaSuccess && lse_host)
        e = cudaMemcpyAsync(lse_host, lse_dev, (size_t)n_tokens * f.n_q_heads * 4, cudaMemcpyDeviceToHost, ds);
    if (e != cudaSuccess) return cuda_fail(e, "device-to-host copy");
    if (behind) {
        e = cudaEventRecord(c->ev_down[oset], ds);
        if (e != cudaSuccess) return cuda_fail(e, "cudaEventRecord(download)");
        c->ev_down_set[oset] = true;
        c->host_down_steps++;
        // the step BEFORE this one has had this whole step to copy its results out: from here on the
        // caller's stream is behind them
        if (c->ev_down_set[oset ^ 1]) {
            e = cudaStreamWaitEvent(st, c->ev_down[oset ^ 1], 0);
            if (e != cudaSuccess) return cuda_fail(e, "cudaStreamWaitEvent(previous download)");
        }
    }
    return KVF_OK;
}

kvf_status kvf_cache_flush(kvf_cache *c, void *cuda_stream) {
    if (!c) return KVF_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (c->comb_pending) {
        unsigned long long capture = 0;
        kvf_status s = capture_of(st, &capture);
        if (s != KVF_OK) return s;
        if (capture != c->comb_capture) return KVF_ERR_INVALID_ARG;
        s = join_combine(c, st);
        if (s != KVF_OK) return s;
    }
    for (int i = 0; i < 2; ++i) {
        if (!c->ev_down_set[i]) continue;
        cudaError_t e = cudaStreamWaitEvent(st, c->ev_down[i], 0);
        if (e != cudaSuccess) return cuda_fail(e, "cudaStreamWaitEvent(flush)");
    }
    return KVF_OK;
}

kvf_status kvf_cache_host_flush(kvf_cache *c, void *cuda_stream) { return kvf_cache_flush(c, cuda_stream); }

int64_t kvf_cache_len(const kvf_cache *c) { return c ? c->len : -1; }

kvf_status kvf_cache_reset(kvf_cache *c) {
    if (!c) return KVF_ERR_INVALID_ARG;
    c->len = 0;
    return KVF_OK;
}

kvf_status kvf_cache_set_len(kvf_cache *c, int64_t len) {
    if (!c) return KVF_ERR_INVALID_ARG;
    if (len < 0 || len > c->cfg.capacity) return KVF_ERR_CAPACITY;
    c->len = len;
    return KVF_OK;
}

kvf_status kvf_cache_status(kvf_cache *c) {
    if (!c) return KVF_ERR_INVALID_ARG;
    int word = 0;
    cudaError_t e = cudaMemcpy(&word, c->workspace + c->lay.status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpy(status)");
    if (word == 0) return KVF_OK;
    return (word & 0xFF) == KVF_ERR_RANGE ? KVF_ERR_RANGE : KVF_ERR_TIMEOUT;
}

int32_t kvf_cache_status_word(kvf_cache *c) {
    if (!c) return -1;
    int word = 0;
    cudaError_t e = cudaMemcpy(&word, c->workspace + c->lay.status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) { cuda_fail(e, "cudaMemcpy(status)"); return -1; }
    return word;
}

kvf_status kvf_cache_sm_clock(kvf_cache *c, uint64_t cycles_ns[2]) {
    if (!c || !cycles_ns) return KVF_ERR_INVALID_ARG;
    unsigned long long ctr[2] = {0, 0};
    cudaError_t e = cudaMemcpy(ctr, c->workspace + c->lay.status + 16, sizeof(ctr), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpy(clock counters)");
    cycles_ns[0] = ctr[0];
    cycles_ns[1] = ctr[1];
    return KVF_OK;
}

void *kvf_cache_k_plane(const kvf_cache *c) { return c && !c->page_table ? c->storage : nullptr; }
void *kvf_cache_v_plane(const kvf_cache *c) { return c && !c->page_table ? c->storage + c->plane_bytes : nullptr; }
float *kvf_cache_k_scales(const kvf_cache *c) { return c && c->quant && !c->page_table ? c->qp.k_scales : nullptr; }
float *kvf_cache_v_scales(const kvf_cache *c) { return c && c->quant && !c->page_table ? c->qp.v_scales : nullptr; }

kvf_status kvf_cache_plan(const kvf_cache *c, int32_t n_tokens, int64_t prefix_len, int32_t plan[4]) {
    if (!c || !plan || n_tokens < 1 || n_tokens > c->cfg.max_chunk || prefix_len < 0) return KVF_ERR_INVALID_ARG;
    Plan p = make_plan(c, n_tokens, prefix_len);
    plan[0] = p.tc ? 1 : 0;
    plan[1] = p.splits;
    plan[2] = p.ctas;
    plan[3] = p.kernels;
    return KVF_OK;
}

kvf_status kvf_cache_set_splits(kvf_cache *c, int32_t splits) {
    if (!c || splits < 0) return KVF_ERR_INVALID_ARG;
    c->force_splits = splits;
    return KVF_OK;
}

kvf_status kvf_cache_set_window(kvf_cache *c, int32_t n_sink, int64_t window) {
    if (!c || n_sink < 0 || window < 0) return KVF_ERR_INVALID_ARG;
    if (window == 0 && n_sink != 0) return KVF_ERR_INVALID_ARG;   // sinks mean something only beside a window
    if (n_sink > kMaxSinks) return KVF_ERR_UNSUPPORTED;
    c->n_sink = n_sink;
    c->window = window;
    return KVF_OK;
}

uint64_t kvf_cache_launch_count(const kvf_cache *c) { return c ? c->launches : 0; }

kvf_status kvf_cache_profile(kvf_cache *c, int32_t enable) {
    if (!c) return KVF_ERR_INVALID_ARG;
    c->profile = enable != 0;
    return KVF_OK;
}

kvf_status kvf_cache_profile_read(kvf_cache *c, double ms[3], uint64_t launches[3]) {
    if (!c || !ms || !launches) return KVF_ERR_INVALID_ARG;
    kvf_status rc = KVF_OK;
    for (ProfRec &r : c->recs) {
        cudaError_t e = cudaEventSynchronize(r.b);
        float t = 0.f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&t, r.a, r.b);
        if (e != cudaSuccess) rc = cuda_fail(e, "cudaEventElapsedTime");
        else if (r.kind >= 0 && r.kind < 3) { ms[r.kind] += t; launches[r.kind] += 1; }
        c->pool.push_back(r.a);
        c->pool.push_back(r.b);
    }
    c->recs.clear();
    return rc;
}

void kvf_cache_destroy(kvf_cache *c) {
    if (!c) return;
    for (ProfRec &r : c->recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    for (cudaEvent_t e : c->pool) cudaEventDestroy(e);
    for (int i = 0; i < 2; ++i) {
        if (c->ev_up[i]) cudaEventDestroy(c->ev_up[i]);
        if (c->ev_read[i]) cudaEventDestroy(c->ev_read[i]);
    }
    if (c->up_stream) cudaStreamDestroy(c->up_stream);
    for (int i = 0; i < 2; ++i) {
        if (c->ev_step[i]) cudaEventDestroy(c->ev_step[i]);
        if (c->ev_down[i]) cudaEventDestroy(c->ev_down[i]);
    }
    if (c->down_stream) cudaStreamDestroy(c->down_stream);
    if (c->ev_attn) cudaEventDestroy(c->ev_attn);
    if (c->ev_comb) cudaEventDestroy(c->ev_comb);
    if (c->comb_stream) cudaStreamDestroy(c->comb_stream);
    delete c;
}

size_t kvf_batch_workspace_bytes(const kvf_config *cfg, int32_t n_caches) {
    if (check_config(cfg) != KVF_OK || n_caches < 1 || n_caches > 65535) return 0;
    return batch_layout(cfg, n_caches).total;
}

kvf_status kvf_batch_create(kvf_cache *const *caches, int32_t n_caches, void *dev_workspace, size_t workspace_bytes,
                            kvf_batch **out) {
    if (!out) return KVF_ERR_INVALID_ARG;
    *out = nullptr;
    if (!caches || n_caches < 1 || n_caches > 65535 || !dev_workspace) return KVF_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(dev_workspace) & 255u) return KVF_ERR_INVALID_ARG;
    for (int i = 0; i < n_caches; ++i)
        if (!caches[i]) return KVF_ERR_INVALID_ARG;
    const kvf_cache *c0 = caches[0];
    // members: paged caches of one pool, same shape (they then share the pool's tensor maps)
    for (int i = 0; i < n_caches; ++i) {
        const kvf_cache *c = caches[i];
        if (!c->page_table || !c->tc) return KVF_ERR_UNSUPPORTED;
        const kvf_config &x = c->cfg, &y = c0->cfg;
        if (c->storage != c0->storage || c->n_pool_pages != c0->n_pool_pages || c->device != c0->device ||
            x.n_q_heads != y.n_q_heads || x.n_kv_heads != y.n_kv_heads || x.head_dim != y.head_dim ||
            x.dtype != y.dtype || x.capacity != y.capacity || x.max_chunk != y.max_chunk || x.flags != y.flags ||
            c->scale_log2 != c0->scale_log2 ||
            std::memcmp(c->table.inv_freq, c0->table.inv_freq, sizeof(c0->table.inv_freq)) != 0)
            return KVF_ERR_INVALID_ARG;
        for (int j = 0; j < i; ++j)
            if (caches[j] == c) return KVF_ERR_INVALID_ARG;
    }
    const BatchLayout lay = batch_layout(&c0->cfg, n_caches);
    if (workspace_bytes < lay.total) return KVF_ERR_CAPACITY;

    kvf_batch *b = new (std::nothrow) kvf_batch();
    if (!b) return KVF_ERR_INVALID_ARG;
    b->caches.assign(caches, caches + n_caches);
    b->workspace = static_cast<char *>(dev_workspace);
    b->off_status = lay.status; b->off_tables = lay.tables; b->off_lens = lay.lens; b->off_q_rot = lay.q_rot;
    b->off_part_o = lay.part_o; b->off_part_lse = lay.part_lse;
    b->part_rows = lay.part_rows;
    b->launches = 0;

    EncodeTiledFn fn = nullptr;
    kvf_status s = encode_fn(&fn);
    if (s != KVF_OK) { delete b; return s; }
    const kvf_config &f = c0->cfg;
    const uint64_t row = (uint64_t)f.head_dim * 2;
    s = make_map(fn, &b->map_q, b->workspace + lay.q_rot, (uint64_t)f.n_q_heads, (uint64_t)n_caches * f.max_chunk, row,
                 row * f.n_q_heads, f.head_dim, (uint32_t)c0->Gp, (uint32_t)(128 / c0->Gp));
    if (s != KVF_OK) { delete b; return s; }

    std::vector<const int32_t *> tables(n_caches);
    for (int i = 0; i < n_caches; ++i) tables[i] = caches[i]->page_table;
    cudaError_t e = cudaMemcpy(b->workspace + lay.tables, tables.data(), (size_t)n_caches * sizeof(void *),
                               cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemset(b->workspace + lay.status, 0, 256);
    if (e != cudaSuccess) { delete b; return cuda_fail(e, "batch workspace setup"); }
    *out = b;
    return KVF_OK;
}

}  // extern "C"

namespace {

// Per-member row counts and first positions of a ragged step, 64 members per launch, written into
// the batch workspace by a plain (fully stream-ordered) kernel: no host-to-device copy, so a
// ragged step can be captured into a graph like any other.
struct LenChunk {
    int64_t prefix[64], pos0[64];
    int32_t n[64];
    int32_t base, count;
};
__global__ void write_lengths_kernel(const LenChunk c, int64_t *prefixes, int64_t *pos0s, int64_t *ns) {
    const int i = threadIdx.x;
    if (i < c.count) {
        prefixes[c.base + i] = c.prefix[i];
        pos0s[c.base + i] = c.pos0[i];
        ns[c.base + i] = c.n[i];
    }
}

// One step of a batch.  pos0s == nullptr: every member holds the same number of rows and starts at
// pos0; else member i starts at pos0s[i] and the members' row counts may differ.  ns != nullptr
// (ragged only): member i folds ns[i] <= n tokens (0 = it sits the step out) out of blocks of n.
kvf_status batch_step(kvf_batch *b, const void *q, const void *k_new, const void *v_new, int32_t n,
                      int64_t pos0, const int64_t *pos0s, const int32_t *ns, void *out, float *lse,
                      void *cuda_stream) {
    if (!b) return KVF_ERR_INVALID_ARG;
    kvf_cache *c0 = b->caches[0];
    const bool ragged = pos0s != nullptr;
    int64_t P = c0->len;                                      // ragged: the longest member, for the plan
    for (kvf_cache *c : b->caches) {
        if (c->n_sink != c0->n_sink || c->window != c0->window) return KVF_ERR_INVALID_ARG;   // one mask
        if (!ragged && c->len != P) return KVF_ERR_INVALID_ARG;   // the members advance together
        if (c->len > P) P = c->len;
    }
    if (ragged && c0->window > 0) return KVF_ERR_UNSUPPORTED;     // the window is placed per launch
    kvf_status s = KVF_OK;
    bool any = ns == nullptr;
    for (size_t i = 0; i < b->caches.size() && s == KVF_OK; ++i) {
        if (ns && (ns[i] < 0 || ns[i] > n)) return KVF_ERR_INVALID_ARG;
        if (ns && ns[i] == 0) continue;                         // sits the step out: nothing to check
        any = true;
        s = check_step(b->caches[i], ns ? ns[i] : n, ragged ? pos0s[i] : pos0);
    }
    if (s != KVF_OK) return s;
    if (n < 1 || n > c0->cfg.max_chunk || !any) return KVF_ERR_INVALID_ARG;   // (a step nobody takes part in)
    if (check_ptr(q) || check_ptr(k_new) || check_ptr(v_new) || check_ptr(out)) return KVF_ERR_INVALID_ARG;
    if (lse && (reinterpret_cast<uintptr_t>(lse) & 3u)) return KVF_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const kvf_config &f = c0->cfg;
    const int B = (int)b->caches.size();
    const Plan plan = make_plan(c0, n, P, B, b->part_rows);
    int64_t *dev_prefixes = reinterpret_cast<int64_t *>(b->workspace + b->off_lens);
    int64_t *dev_pos0s = dev_prefixes + B;
    int64_t *dev_ns = dev_pos0s + B;
    if (ragged) {
        for (int base = 0; base < B; base += 64) {
            LenChunk ch;
            ch.base = base;
            ch.count = std::min(64, B - base);
            for (int i = 0; i < ch.count; ++i) {
                ch.prefix[i] = b->caches[base + i]->len;
                ch.pos0[i] = pos0s[base + i];
                ch.n[i] = ns ? ns[base + i] : n;
            }
            write_lengths_kernel<<<1, 64, 0, st>>>(ch, dev_prefixes, dev_pos0s, dev_ns);
            cudaError_t e = cudaGetLastError();
            if (e != cudaSuccess) return cuda_fail(e, "write_lengths launch");
            b->launches++;
        }
    }
    const int32_t *const *tables = reinterpret_cast<const int32_t *const *>(b->workspace + b->off_tables);

    RopeAppendArgs ra;
    ra.q = q; ra.k_new = k_new; ra.v_new = v_new;
    ra.q_rot = b->workspace + b->off_q_rot;
    ra.k_plane = c0->storage;
    ra.v_plane = c0->storage + c0->plane_bytes;
    ra.capacity = f.capacity; ra.prefix = P; ra.pos0 = pos0;
    ra.n = n; ra.H = f.n_q_heads; ra.Hkv = f.n_kv_heads; ra.d = f.head_dim;
    // value rows to clear up to the next page boundary; ragged: each member's own count, at most a page less one
    ra.zero_rows = ragged ? kKvTile - 1 : (int32_t)((P + n + kKvTile - 1) / kKvTile * kKvTile - (P + n));
    ra.page_table = c0->page_table;
    ra.page_elems = c0->page_elems;
    ra.page_tables = tables;
    ra.prefixes = ragged ? dev_prefixes : nullptr;
    ra.pos0s = ragged ? dev_pos0s : nullptr;
    ra.ns = ns ? dev_ns : nullptr;
    ra.status = nullptr; ra.range_limit = 0.f;
    ra.table = c0->table;

    AttnArgs aa;
    aa.q_rot = ra.q_rot;
    aa.k_plane = ra.k_plane; aa.v_plane = ra.v_plane;
    aa.out = out; aa.lse = lse;
    aa.part_o = reinterpret_cast<float *>(b->workspace + b->off_part_o);
    aa.part_lse = reinterpret_cast<float *>(b->workspace + b->off_part_lse);
    aa.status = reinterpret_cast<int *>(b->workspace + b->off_status);
    aa.page_table = c0->page_table;
    aa.page_tables = tables; aa.part_rows = b->part_rows; aa.batch = B;
    aa.prefixes = ragged ? dev_prefixes : nullptr;
    aa.ns = ns ? dev_ns : nullptr;
    aa.n_sink = c0->n_sink; aa.win_lo = window_lo(c0, P);
    aa.k_scales = c0->quant ? c0->qp.k_scales : nullptr;
    aa.v_scales = c0->quant ? c0->qp.v_scales : nullptr;
    aa.scale_stride = 0;
    aa.scale_page_stride = c0->qp.page_bytes / 4;
    aa.quant_bits = c0->quant ? c0->qp.bits : 0;
    aa.capacity = f.capacity; aa.prefix = P;
    aa.n = n; aa.H = f.n_q_heads; aa.Hkv = f.n_kv_heads; aa.G = c0->G; aa.d = f.head_dim;
    aa.Gp = c0->Gp;
    aa.splits = 1;
    aa.ngroups = plan.ngroups;
    aa.streams = plan.qdec ? 1 : attn_tc_streams(n, c0->Gp);
    aa.out_f32 = (f.flags & KVF_OUT_F32) ? 1 : 0;
    aa.scale_log2 = c0->scale_log2;
    aa.range_valid = 0;
    aa.piece_cost = piece_cost_of(c0, plan, aa.streams);
    aa.self_rows = 1;
    if (!ragged && plan.kernels > 2)
        fill_group_ranges(aa, (P + n + kKvTile - 1) / kKvTile - WindowTiles(aa.win_lo, aa.n_sink, kKvTile).skip + aa.piece_cost);

    const PdlScope pdl(!long_step(c0, plan, aa.streams, P + n));
    cudaError_t e = c0->quant ? launch_rope_append_q8(ra, c0->qp, (f.flags & KVF_ROPE_INTERLEAVED) != 0, B, st)
                              : launch_rope_append(ra, f.dtype, (f.flags & KVF_ROPE_INTERLEAVED) != 0, B, st);
    if (e != cudaSuccess) return cuda_fail(e, "rope_append launch (batch)");
    b->launches++;
    TcMaps maps = c0->maps;
    maps.q = b->map_q;
    e = plan.qdec ? launch_attn_q8_decode(aa, maps, st) : launch_attn_tc(aa, maps, st);
    if (e != cudaSuccess) return cuda_fail(e, "attention launch (batch)");
    b->launches++;
    if (plan.kernels > 2) {
        e = launch_combine_groups(aa, st);
        if (e != cudaSuccess) return cuda_fail(e, "combine launch (batch)");
        b->launches++;
    }
    for (size_t i = 0; i < b->caches.size(); ++i) b->caches[i]->len += ns ? ns[i] : n;
    return KVF_OK;
}

}  // namespace

extern "C" {

kvf_status kvf_batch_fold_step(kvf_batch *b, const void *q, const void *k_new, const void *v_new, int32_t n,
                               int64_t pos0, void *out, float *lse, void *cuda_stream) {
    return batch_step(b, q, k_new, v_new, n, pos0, nullptr, nullptr, out, lse, cuda_stream);
}

kvf_status kvf_batch_fold_step_ragged(kvf_batch *b, const void *q, const void *k_new, const void *v_new, int32_t n,
                                      const int64_t *pos0_or_null, void *out, float *lse, void *cuda_stream) {
    if (!b) return KVF_ERR_INVALID_ARG;
    std::vector<int64_t> own;
    if (!pos0_or_null) {                                       // positions continue from each member's length
        for (kvf_cache *c : b->caches) own.push_back(c->len);
        pos0_or_null = own.data();
    }
    return batch_step(b, q, k_new, v_new, n, 0, pos0_or_null, nullptr, out, lse, cuda_stream);
}

kvf_status kvf_batch_fold_step_varlen(kvf_batch *b, const void *q, const void *k_new, const void *v_new,
                                      const int32_t *n_tokens, int32_t max_tokens, const int64_t *pos0_or_null,
                                      void *out, float *lse, void *cuda_stream) {
    if (!b || !n_tokens) return KVF_ERR_INVALID_ARG;
    std::vector<int64_t> own;
    if (!pos0_or_null) {                                       // positions continue from each member's length
        for (kvf_cache *c : b->caches) own.push_back(c->len);
        pos0_or_null = own.data();
    }
    return batch_step(b, q, k_new, v_new, max_tokens, 0, pos0_or_null, n_tokens, out, lse, cuda_stream);
}

kvf_status kvf_batch_plan(const kvf_batch *b, int32_t n_tokens, int64_t prefix_len, int32_t plan[4]) {
    if (!b || !plan || n_tokens < 1 || n_tokens > b->caches[0]->cfg.max_chunk || prefix_len < 0) return KVF_ERR_INVALID_ARG;
    Plan p = make_plan(b->caches[0], n_tokens, prefix_len, (int)b->caches.size(), b->part_rows);
    plan[0] = 1;
    plan[1] = p.splits;
    plan[2] = p.ctas;
    plan[3] = p.kernels;
    return KVF_OK;
}

int32_t kvf_batch_status_word(kvf_batch *b) {
    if (!b) return -1;
    int word = 0;
    cudaError_t e = cudaMemcpy(&word, b->workspace + b->off_status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) { cuda_fail(e, "cudaMemcpy(status)"); return -1; }
    return word;
}

uint64_t kvf_batch_launch_count(const kvf_batch *b) { return b ? b->launches : 0; }

void kvf_batch_destroy(kvf_batch *b) { delete b; }

const char *kvf_status_str(kvf_status s) {
    switch (s) {
        case KVF_OK: return "KVF_OK";
        case KVF_ERR_INVALID_ARG: return "KVF_ERR_INVALID_ARG";
        case KVF_ERR_CAPACITY: return "KVF_ERR_CAPACITY";
        case KVF_ERR_UNSUPPORTED: return "KVF_ERR_UNSUPPORTED";
        case KVF_ERR_CUDA: return "KVF_ERR_CUDA";
        case KVF_ERR_TIMEOUT: return "KVF_ERR_TIMEOUT";
        case KVF_ERR_POS: return "KVF_ERR_POS";
        case KVF_ERR_RANGE: return "KVF_ERR_RANGE";
    }
    return "KVF_ERR_UNKNOWN";
}

const char *kvf_last_cuda_error(void) { return g_cuda_err; }

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// kvf_fold_step_static: the fold step for callers that cannot allocate device memory.
//
// Scratch of the step (status word, rotated queries, split partial results) lives in the
// file-scope device array below instead of a caller-provided workspace.  Every device that loads
// this library holds the array (kStaticScratchBytes) from module load until the process exits.
// In host code the array's name is only a handle for the runtime: its device address is asked
// for once per device with cudaGetSymbolAddress, with that device current, and that address is
// what the kernels get.
namespace {

constexpr size_t kStaticStatusBytes = 1024;
constexpr size_t kStaticQRotBytes = (size_t)4 << 20;     // rotated queries of one chunk
constexpr size_t kStaticPartOBytes = (size_t)16 << 20;   // split partial outputs, fp32
constexpr size_t kStaticPartLseBytes = (size_t)256 << 10;
constexpr size_t kStaticScratchBytes = kStaticStatusBytes + kStaticQRotBytes + kStaticPartOBytes + kStaticPartLseBytes;
static_assert(kStaticScratchBytes == KVF_STATIC_SCRATCH_BYTES, "header and library disagree on the scratch size");

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
char *g_static_ptr[kMaxDevices];   // device address of g_static_scratch, per device; null = not asked yet

// Device address of the scratch array on the current device (looked up on the first call).
kvf_status static_scratch(int dev, char **out) {
    if (dev < 0 || dev >= kMaxDevices) return KVF_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(static scratch)");
        if (!p || (reinterpret_cast<uintptr_t>(p) & 255u)) {
            snprintf(g_cuda_err, sizeof(g_cuda_err), "static scratch has no usable device address");
            return KVF_ERR_CUDA;
        }
        g_static_ptr[dev] = static_cast<char *>(p);
    }
    *out = g_static_ptr[dev];
    return KVF_OK;
}

// Tensor maps of recent static calls, so that a loop over the layers of a model encodes each
// layer's maps once: keyed on the device, the planes and the shape (the rotated-query map points
// into the static scratch, which never moves).
struct StaticMaps {
    int dev;
    const void *storage;
    int32_t H, Hkv, d, max_chunk;
    int64_t capacity;
    TcMaps maps;
};
constexpr size_t kStaticMapEntries = 128;
std::vector<StaticMaps> g_static_maps;
size_t g_static_maps_next = 0;

kvf_status static_maps(kvf_cache *c) {
    const kvf_config &f = c->cfg;
    std::lock_guard<std::mutex> lock(g_static_mu);
    for (const StaticMaps &m : g_static_maps)
        if (m.dev == c->device && m.storage == c->storage && m.H == f.n_q_heads && m.Hkv == f.n_kv_heads &&
            m.d == f.head_dim && m.max_chunk == f.max_chunk && m.capacity == f.capacity) {
            c->maps = m.maps;
            return KVF_OK;
        }
    kvf_status s = build_maps(c);
    if (s != KVF_OK) return s;
    const StaticMaps m = {c->device, c->storage, f.n_q_heads, f.n_kv_heads, f.head_dim, f.max_chunk, f.capacity, c->maps};
    if (g_static_maps.size() < kStaticMapEntries) g_static_maps.push_back(m);
    else g_static_maps[g_static_maps_next++ % kStaticMapEntries] = m;
    return KVF_OK;
}

}  // namespace

extern "C" kvf_status kvf_fold_step_static(const kvf_config *cfg, void *dev_storage, size_t storage_bytes,
                                           int64_t len, const void *q, const void *k_new, const void *v_new,
                                           int32_t n_tokens, int64_t pos0, void *out, float *lse,
                                           void *cuda_stream) {
    kvf_status s = check_config(cfg);
    if (s != KVF_OK) return s;
    if (cfg->flags & (KVF_CACHE_INT8 | KVF_CACHE_INT4)) return KVF_ERR_UNSUPPORTED;   // contiguous bf16 / fp32 planes only
    if (!dev_storage || (reinterpret_cast<uintptr_t>(dev_storage) & 255u)) return KVF_ERR_INVALID_ARG;
    if (storage_bytes < kvf_cache_storage_bytes(cfg)) return KVF_ERR_CAPACITY;
    if (len < 0 || n_tokens < 1 || n_tokens > cfg->max_chunk || pos0 < 0) return KVF_ERR_INVALID_ARG;
    if (len + n_tokens > cfg->capacity) return KVF_ERR_CAPACITY;
    if ((cfg->flags & KVF_STRICT_POS) && pos0 != len) return KVF_ERR_POS;
    if (check_ptr(q) || check_ptr(k_new) || check_ptr(v_new) || check_ptr(out)) return KVF_ERR_INVALID_ARG;
    if (lse && (reinterpret_cast<uintptr_t>(lse) & 3u)) return KVF_ERR_INVALID_ARG;

    // sizes the fixed scratch can hold (max_chunk sizes the rotated-query area and its TMA box);
    // all of this is checked before the first CUDA call
    const size_t row_elems = (size_t)cfg->n_q_heads * cfg->head_dim;
    if ((size_t)cfg->max_chunk * row_elems * elem_bytes(cfg->dtype) > kStaticQRotBytes) {
        snprintf(g_cuda_err, sizeof(g_cuda_err), "max_chunk x heads x head_dim exceeds the static scratch");
        return KVF_ERR_CAPACITY;
    }
    const size_t part_tokens = std::min(kStaticPartOBytes / (row_elems * 4), kStaticPartLseBytes / ((size_t)cfg->n_q_heads * 4));
    if (part_tokens < (size_t)n_tokens) {
        snprintf(g_cuda_err, sizeof(g_cuda_err), "n_tokens x heads x head_dim partial rows exceed the static scratch");
        return KVF_ERR_CAPACITY;
    }
    {
        // A chunk that fits one 128-row tile runs as two streams on the tensor-core paths and always
        // leaves 2 * (groups + Hkv - 1) partial slots of n * G rows, with groups >= Hkv: the least the
        // kernel will write has to fit (the plan cuts the key range no finer than the rest allows).
        const int G = cfg->n_q_heads / cfg->n_kv_heads;
        const bool tensor_path = !(cfg->flags & KVF_FORCE_SIMT) && attn_tc_supported(cfg->dtype, cfg->head_dim, G);
        const int Gp = attn_tc_padded_group(G);      // rows a token takes in the partial slots
        if (tensor_path && attn_tc_streams(n_tokens, Gp) == 2) {
            const size_t least = (size_t)2 * (2 * (size_t)cfg->n_kv_heads - 1) * (size_t)n_tokens * Gp;
            if (least > part_tokens * (size_t)cfg->n_q_heads) {
                snprintf(g_cuda_err, sizeof(g_cuda_err),
                         "a short chunk over %d KV heads leaves more partial rows than the static scratch holds",
                         (int)cfg->n_kv_heads);
                return KVF_ERR_CAPACITY;
            }
        }
    }

    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    char *scratch = nullptr;
    s = static_scratch(dev, &scratch);
    if (s != KVF_OK) return s;

    // a handle on the stack that points the ordinary step at the static scratch
    kvf_cache c;
    s = init_handle(&c, cfg, dev_storage, scratch);
    if (s != KVF_OK) return s;
    c.plane_bytes = kvf_cache_storage_bytes(cfg) / 2;
    c.lay = Layout();
    c.lay.status = 0;
    c.lay.q_rot = kStaticStatusBytes;
    c.lay.part_o = kStaticStatusBytes + kStaticQRotBytes;
    c.lay.part_lse = c.lay.part_o + kStaticPartOBytes;
    c.lay.total = kStaticScratchBytes;
    c.len = len;
    c.part_rows_cap = (int64_t)part_tokens * cfg->n_q_heads;   // the plan splits only as far as this holds
    if (c.tc) {
        s = static_maps(&c);
        if (s != KVF_OK) return s;
    }

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // the array keeps what the last call left: the status word has to start at zero
    e = cudaMemsetAsync(scratch, 0, 256, st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(status)");
    return step_impl(&c, q, k_new, v_new, n_tokens, pos0, out, lse, st);
}
