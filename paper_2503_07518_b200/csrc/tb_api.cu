// C ABI of the library: argument validation, host mirrors of the cache lengths, launch glue.
// Nothing here computes; every step of the path runs in the kernels of the other files.
#include <cstdio>
#include <cstring>
#include <new>

#include "tb_internal.h"

using namespace tb;

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int elem_size(int dtype) { return dtype == TB_BF16 ? 2 : 4; }

struct Layout {
    size_t kv_bytes, kimp_bytes;
    size_t off_W, off_idx, off_cnt, off_status, off_counter, off_len, off_len_proj, off_misc, state_bytes;
    size_t off_part_o, off_part_ml, off_sel_idx, off_sel_cnt, off_sel_keys, off_sel_bins, work_bytes;
    int idx_cap, sel_stride;
};

// Heads per (layer, sequence) of the projected-key cache (hi), the index lists (hl) and the
// attention units (ha) under the configuration's selection scope.
void scope_heads(const tb_config* c, int* hi, int* hl, int* ha) {
    *hi = c->list_scope == TB_SCOPE_LAYER ? 1 : c->n_kv_heads;
    *hl = c->list_scope == TB_SCOPE_LAYER ? 1 : c->list_scope == TB_SCOPE_Q_HEAD ? c->n_q_heads : c->n_kv_heads;
    *ha = c->list_scope == TB_SCOPE_Q_HEAD ? c->n_q_heads : c->n_kv_heads;
}

tb_status check_config(const tb_config* c) {
    if (!c) return TB_ERR_INVALID_ARG;
    if (c->n_layers <= 0 || c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->max_batch <= 0 || c->max_seq_len <= 0 ||
        c->max_budget <= 0 || c->max_radius < 0 || c->device < 0)
        return TB_ERR_INVALID_ARG;
    if (c->n_q_heads % c->n_kv_heads != 0) return TB_ERR_INVALID_ARG;
    if (c->kv_dtype != TB_F32 && c->kv_dtype != TB_BF16) return TB_ERR_INVALID_ARG;
    if (c->list_scope != TB_SCOPE_KV_HEAD && c->list_scope != TB_SCOPE_Q_HEAD && c->list_scope != TB_SCOPE_LAYER) return TB_ERR_INVALID_ARG;
    if (c->head_dim != 128) return TB_ERR_UNSUPPORTED;
    if (c->imp_dim != 16 && c->imp_dim != 32) return TB_ERR_UNSUPPORTED;
    if (c->n_q_heads / c->n_kv_heads > kMaxGroup) return TB_ERR_UNSUPPORTED;
    // rows of the 2-D view of the projected-key cache are addressed with 32-bit TMA coordinates
    double rows = (double)c->n_layers * c->max_batch * c->n_kv_heads * c->max_seq_len;
    if (rows >= 2147483648.0) return TB_ERR_UNSUPPORTED;
    if ((double)(2 * c->max_radius + 1) * c->max_budget > 1e9) return TB_ERR_UNSUPPORTED;
    return TB_OK;
}

void compute_layout(const tb_config* c, Layout* l) {
    const size_t es = elem_size(c->kv_dtype);
    int hi, hl, ha;
    scope_heads(c, &hi, &hl, &ha);
    const size_t pairs = (size_t)c->n_layers * c->max_batch;
    const size_t units = pairs * hl;                                   // index lists
    l->kv_bytes = pairs * c->n_kv_heads * c->max_seq_len * 2 * c->head_dim * es;
    l->kimp_bytes = pairs * hi * c->max_seq_len * c->imp_dim * es;
    l->idx_cap = (int)align_up((size_t)(2 * c->max_radius + 1) * c->max_budget, 4);
    l->sel_stride = (int)align_up((size_t)c->max_budget, 4);
    size_t o = 0;
    l->off_W = o, o = align_up(o + (size_t)c->n_layers * c->n_kv_heads * c->head_dim * c->imp_dim * es, 256);
    l->off_idx = o, o = align_up(o + units * l->idx_cap * 4, 256);
    l->off_cnt = o, o = align_up(o + units * 4, 256);
    l->off_status = o, o = align_up(o + 4, 256);
    l->off_counter = o, o = align_up(o + pairs * ha * 4, 256);
    l->off_len = o, o = align_up(o + pairs * 4, 256);
    l->off_len_proj = o, o = align_up(o + pairs * 4, 256);
    l->off_misc = o, o = align_up(o + 8 * 4, 256);
    l->state_bytes = o;
    const size_t units_q = (size_t)c->n_layers * c->max_batch * c->n_q_heads;
    o = 0;
    l->off_part_o = o, o = align_up(o + units_q * kMaxSplits * c->head_dim * 4, 256);
    l->off_part_ml = o, o = align_up(o + units_q * kMaxSplits * 2 * 4, 256);
    l->off_sel_idx = o, o = align_up(o + units * l->sel_stride * 4, 256);
    l->off_sel_cnt = o, o = align_up(o + units * 4, 256);
    const size_t row = align_up((size_t)c->max_seq_len, 256);
    l->off_sel_keys = o, o = align_up(o + units * row * 4, 256);       // one 32-bit key per token
    l->off_sel_bins = o, o = align_up(o + units * row * 2, 256);       // one 16-bit first digit per token
    l->work_bytes = o;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 2-D view of the projected-key cache: one row per token slot, d' columns; boxes of 256 rows whose
// 16-byte chunks are swizzled in shared memory so that one-row-per-thread reads hit distinct banks.
tb_status make_kimp_map(tb_ctx* c) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess)
        return TB_ERR_CUDA;
    const tb_config& g = c->cfg;
    const int es = elem_size(g.kv_dtype);
    const int row_bytes = g.imp_dim * es;
    cuuint64_t dims[2] = {(cuuint64_t)g.imp_dim, (cuuint64_t)g.n_layers * g.max_batch * c->geom.Hi * g.max_seq_len};
    cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
    cuuint32_t box[2] = {(cuuint32_t)g.imp_dim, 256u};
    cuuint32_t estr[2] = {1u, 1u};
    CUtensorMapSwizzle sw = row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                            : row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                              : CU_TENSOR_MAP_SWIZZLE_32B;
    CUresult r = ((EncodeTiledFn)fn)(&c->kimp_map, g.kv_dtype == TB_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                                     2, c->kimp, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? TB_OK : TB_ERR_CUDA;
}

// The reduction the kernels run, or -1.  A list with a single importance query (one list per query
// head, one per layer) has nothing to reduce: every mode means the same there.  TB_PER_QHEAD on a
// context whose lists are per KV head is refused: the lists it asks for do not exist.
int effective_reduce(const tb_ctx* c, int reduce) {
    if (reduce != TB_GROUP_SUM && reduce != TB_GROUP_MAX && reduce != TB_PER_QHEAD) return -1;
    if (c->geom.gl == 1) return TB_GROUP_SUM;
    return reduce == TB_PER_QHEAD ? -1 : reduce;
}

bool bad_layers(const tb_ctx* c, int lb, int lc) { return lb < 0 || lc <= 0 || lb + lc > c->cfg.n_layers; }

// Resolve and validate the sequence list of a call.
tb_status resolve_seqs(const tb_ctx* c, const int32_t* seq_ids, int n_seq, int* out) {
    if (n_seq <= 0) return TB_ERR_INVALID_ARG;
    if (n_seq > kMaxLaunchSeq) return TB_ERR_UNSUPPORTED;
    for (int i = 0; i < n_seq; ++i) {
        int s = seq_ids ? seq_ids[i] : i;
        if (s < 0 || s >= c->cfg.max_batch) return TB_ERR_INVALID_ARG;
        for (int j = 0; j < i; ++j)
            if (out[j] == s) return TB_ERR_INVALID_ARG;   // a sequence may appear once per call
        out[i] = s;
    }
    return TB_OK;
}

// Lengths of a launch's units: the host mirrors, or -- when the kernels read the device counters -- upper
// bounds (mirror + declared growth) that the launchers size grids and shared memory with.
void fill_table(const tb_ctx* c, UnitTable* ut, int lb, int lc, const int* seqs, int n_seq, bool projected = false) {
    ut->layer_begin = lb, ut->layer_count = lc, ut->n_seq = n_seq;
    ut->use_dev_len = c->dev_lengths, ut->len_is_projected = projected;
    ut->len_dev = c->st.len, ut->len_proj_dev = c->st.len_proj;
    for (int i = 0; i < n_seq; ++i) ut->seq_id[i] = seqs[i];
    const std::vector<int>& src = projected ? c->len_proj : c->len;
    for (int l = 0; l < lc; ++l)
        for (int i = 0; i < n_seq; ++i) {
            long long L = src[(size_t)(lb + l) * c->cfg.max_batch + seqs[i]];
            if (c->dev_lengths) L = L + c->growth_reserve < c->cfg.max_seq_len ? L + c->growth_reserve : c->cfg.max_seq_len;
            ut->len[l * n_seq + i] = (int)L;
        }
}

int layers_per_launch(int n_seq) {
    int n = kMaxLaunchUnits / n_seq;
    return n < 1 ? 1 : n;
}

void cand_range(int L, int S, int W, int* lo, int* hi) {
    *lo = S < L ? S : L;
    *hi = L - W > *lo ? L - W : *lo;
}

}  // namespace

extern "C" {

tb_status tb_query_sizes(const tb_config* cfg, size_t* kv_bytes, size_t* kimp_bytes, size_t* state_bytes, size_t* workspace_bytes) {
    tb_status st = check_config(cfg);
    if (st != TB_OK) return st;
    if (!kv_bytes || !kimp_bytes || !state_bytes || !workspace_bytes) return TB_ERR_INVALID_ARG;
    Layout l;
    compute_layout(cfg, &l);
    *kv_bytes = l.kv_bytes, *kimp_bytes = l.kimp_bytes, *state_bytes = l.state_bytes, *workspace_bytes = l.work_bytes;
    return TB_OK;
}

tb_status tb_create(const tb_config* cfg, void* kv, void* kimp, void* state, void* workspace, tb_ctx** out) {
    tb_status st = check_config(cfg);
    if (st != TB_OK) return st;
    if (!kv || !kimp || !state || !workspace || !out) return TB_ERR_INVALID_ARG;
    if (((uintptr_t)kv | (uintptr_t)kimp | (uintptr_t)state | (uintptr_t)workspace) & 255) return TB_ERR_INVALID_ARG;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return TB_ERR_CUDA;
    if (dev != cfg->device) return TB_ERR_INVALID_ARG;
    {
        // kimp, state and workspace must be device memory.  The KV cache may also be page-locked host
        // memory that the device addresses through the same pointer (offloaded KV, paper Sec. 4.4):
        // the attention kernels then fetch just the selected rows over the host link.  Anything else
        // would fault in a kernel later, so it is refused here.
        cudaPointerAttributes pa;
        const void* dev_only[3] = {kimp, state, workspace};
        for (const void* ptr : dev_only) {
            if (cudaPointerGetAttributes(&pa, ptr) != cudaSuccess) { (void)cudaGetLastError(); return TB_ERR_INVALID_ARG; }
            if (pa.type != cudaMemoryTypeDevice && pa.type != cudaMemoryTypeManaged) return TB_ERR_INVALID_ARG;
        }
        if (cudaPointerGetAttributes(&pa, kv) != cudaSuccess) { (void)cudaGetLastError(); return TB_ERR_INVALID_ARG; }
        const bool on_device = pa.type == cudaMemoryTypeDevice || pa.type == cudaMemoryTypeManaged;
        const bool mapped_host = pa.type == cudaMemoryTypeHost && pa.devicePointer == kv;
        if (!on_device && !mapped_host) return TB_ERR_INVALID_ARG;
    }
    tb_ctx* c = new (std::nothrow) tb_ctx();
    if (!c) return TB_ERR_INVALID_ARG;
    c->cfg = *cfg;
    Layout l;
    compute_layout(cfg, &l);
    c->kv = kv, c->kimp = kimp;
    c->state_bytes = l.state_bytes, c->work_bytes = l.work_bytes;
    char* sp = (char*)state;
    c->st.W = sp + l.off_W;
    c->st.idx = (int32_t*)(sp + l.off_idx);
    c->st.cnt = (int32_t*)(sp + l.off_cnt);
    c->st.status = (int32_t*)(sp + l.off_status);
    c->st.attn_counter = (uint32_t*)(sp + l.off_counter);
    c->st.len = (int32_t*)(sp + l.off_len);
    c->st.len_proj = (int32_t*)(sp + l.off_len_proj);
    c->st.misc_counter = (uint32_t*)(sp + l.off_misc);
    char* wp = (char*)workspace;
    c->wk.part_o = (float*)(wp + l.off_part_o);
    c->wk.part_ml = (float*)(wp + l.off_part_ml);
    c->wk.sel_idx = (int32_t*)(wp + l.off_sel_idx);
    c->wk.sel_cnt = (int32_t*)(wp + l.off_sel_cnt);
    c->wk.sel_stride = l.sel_stride;
    c->wk.sel_keys = (uint32_t*)(wp + l.off_sel_keys);
    c->wk.sel_bins = (uint16_t*)(wp + l.off_sel_bins);
    Geom& g = c->geom;
    g.n_layers = cfg->n_layers, g.Hq = cfg->n_q_heads, g.Hkv = cfg->n_kv_heads, g.g = cfg->n_q_heads / cfg->n_kv_heads;
    scope_heads(cfg, &g.Hi, &g.Hl, &g.Ha);
    g.gl = cfg->list_scope == TB_SCOPE_KV_HEAD ? g.g : 1, g.ga = g.Hq / g.Ha;
    g.D = cfg->head_dim, g.dp = cfg->imp_dim, g.max_batch = cfg->max_batch, g.max_seq_len = cfg->max_seq_len;
    g.idx_cap = l.idx_cap, g.dtype = cfg->kv_dtype;
    const size_t n = (size_t)cfg->n_layers * cfg->max_batch;
    c->len.assign(n, 0), c->len_proj.assign(n, 0), c->has_sel.assign(n, 0), c->sel_cnt.assign(n, -1);
    c->last_bytes = 0, c->launches = 0;
    c->wait_poll_limit = 0, c->drop_tile = -1;
    c->dev_lengths = 0, c->growth_reserve = 0;
    c->res_rows = nullptr, c->res_sinks = c->res_window = 0, c->imp_rows = nullptr;
    c->last_cache_write = c->last_list_write = -4;
    c->tile_rows = 256;
    for (int i = 0; i < 17; ++i) c->attn_max_active[i] = 0;
    if (cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { delete c; return TB_ERR_CUDA; }
    // only the small control parts need defined contents; the index lists and partials are always
    // written before they are read
    if (cudaMemset(sp + l.off_cnt, 0, l.state_bytes - l.off_cnt) != cudaSuccess ||
        cudaMemset(sp + l.off_W, 0, l.off_idx - l.off_W) != cudaSuccess) {
        delete c;
        return TB_ERR_CUDA;
    }
    st = make_kimp_map(c);
    if (st != TB_OK) { delete c; return st; }
    *out = c;
    return TB_OK;
}

tb_status tb_destroy(tb_ctx* ctx) {
    if (!ctx) return TB_ERR_INVALID_ARG;
    delete ctx;
    return TB_OK;
}

int32_t tb_index_capacity(const tb_ctx* ctx) { return ctx ? ctx->geom.idx_cap : 0; }

tb_status tb_set_projection(tb_ctx* c, int32_t layer, const void* W_dev, void* stream) {
    if (!c || !W_dev || layer < 0 || layer >= c->cfg.n_layers) return TB_ERR_INVALID_ARG;
    const size_t bytes = (size_t)c->cfg.n_kv_heads * c->cfg.head_dim * c->cfg.imp_dim * elem_size(c->cfg.kv_dtype);
    if (cudaMemcpyAsync((char*)c->st.W + layer * bytes, W_dev, bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)stream) != cudaSuccess)
        return TB_ERR_CUDA;
    c->last_cache_write = (long long)c->launches;   // treat as written by the next launch's predecessor
    return TB_OK;
}

tb_status tb_reset_sequence(tb_ctx* c, int32_t seq) {
    if (!c || seq < 0 || seq >= c->cfg.max_batch) return TB_ERR_INVALID_ARG;
    if (c->dev_lengths) {
        // the device counters of this sequence, one 4-byte entry per layer (a blocking strided clear)
        const size_t pitch = (size_t)c->cfg.max_batch * 4;
        if (cudaMemset2D(c->st.len + seq, pitch, 0, 4, c->cfg.n_layers) != cudaSuccess ||
            cudaMemset2D(c->st.len_proj + seq, pitch, 0, 4, c->cfg.n_layers) != cudaSuccess)
            return TB_ERR_CUDA;
    }
    for (int l = 0; l < c->cfg.n_layers; ++l) {
        const size_t i = (size_t)l * c->cfg.max_batch + seq;
        c->len[i] = c->len_proj[i] = c->has_sel[i] = 0, c->sel_cnt[i] = -1;
    }
    return TB_OK;
}

tb_status tb_get_length(const tb_ctx* c, int32_t layer, int32_t seq, int32_t* len, int32_t* len_projected) {
    if (!c || layer < 0 || layer >= c->cfg.n_layers || seq < 0 || seq >= c->cfg.max_batch) return TB_ERR_INVALID_ARG;
    const size_t i = (size_t)layer * c->cfg.max_batch + seq;
    if (len) *len = c->len[i];
    if (len_projected) *len_projected = c->len_proj[i];
    return TB_OK;
}

tb_status tb_append_kv(tb_ctx* c, int32_t lb, int32_t lc, const int32_t* seq_ids, const int32_t* n_new, int32_t n_seq,
                       const void* k, const void* v, void* stream) {
    if (!c || !n_new || !k || !v || bad_layers(c, lb, lc)) return TB_ERR_INVALID_ARG;
    int seqs[kMaxLaunchSeq];
    tb_status st = resolve_seqs(c, seq_ids, n_seq, seqs);
    if (st != TB_OK) return st;
    int tok_off[kMaxLaunchSeq + 1];
    tok_off[0] = 0;
    for (int i = 0; i < n_seq; ++i) {
        if (n_new[i] < 0) return TB_ERR_INVALID_ARG;
        tok_off[i + 1] = tok_off[i] + n_new[i];
        for (int l = lb; l < lb + lc; ++l)
            if (c->len[(size_t)l * c->cfg.max_batch + seqs[i]] + n_new[i] > c->cfg.max_seq_len) return TB_ERR_CAPACITY;
    }
    const int total = tok_off[n_seq];
    if (total == 0) return TB_OK;
    const size_t es = elem_size(c->cfg.kv_dtype);
    const size_t layer_stride = (size_t)total * c->cfg.n_kv_heads * c->cfg.head_dim * es;
    const int step = layers_per_launch(n_seq);
    for (int l0 = lb; l0 < lb + lc; l0 += step) {
        const int n = l0 + step <= lb + lc ? step : lb + lc - l0;
        UnitTable ut;
        fill_table(c, &ut, l0, n, seqs, n_seq);
        if (launch_append(c, ut, n_new, tok_off, total, (const char*)k + (size_t)(l0 - lb) * layer_stride,
                          (const char*)v + (size_t)(l0 - lb) * layer_stride, (cudaStream_t)stream) != cudaSuccess)
            return TB_ERR_CUDA;
        c->last_cache_write = (long long)c->launches;
        c->launches++;
    }
    for (int l = lb; l < lb + lc; ++l)
        for (int i = 0; i < n_seq; ++i) c->len[(size_t)l * c->cfg.max_batch + seqs[i]] += n_new[i];
    return TB_OK;
}

tb_status tb_project_keys(tb_ctx* c, int32_t lb, int32_t lc, const int32_t* seq_ids, const int32_t* pos_begin,
                          const int32_t* pos_end, int32_t n_seq, void* stream) {
    if (!c || (pos_begin == nullptr) != (pos_end == nullptr) || bad_layers(c, lb, lc)) return TB_ERR_INVALID_ARG;
    int seqs[kMaxLaunchSeq];
    tb_status st = resolve_seqs(c, seq_ids, n_seq, seqs);
    if (st != TB_OK) return st;
    const bool auto_range = pos_begin == nullptr;       // everything cached and not yet projected
    int max_range = 0;
    for (int i = 0; i < n_seq; ++i) {
        if (!auto_range && (pos_begin[i] < 0 || pos_end[i] < pos_begin[i])) return TB_ERR_INVALID_ARG;
        for (int l = lb; l < lb + lc; ++l) {
            const size_t u = (size_t)l * c->cfg.max_batch + seqs[i];
            if (auto_range) {
                int n = c->len[u] - c->len_proj[u] + (c->dev_lengths ? c->growth_reserve : 0);
                if (n > c->cfg.max_seq_len) n = c->cfg.max_seq_len;
                if (n > max_range) max_range = n;
                continue;
            }
            if (pos_end[i] > c->len[u]) return TB_ERR_INVALID_ARG;          // beyond the cached tokens
            if (pos_begin[i] > c->len_proj[u]) return TB_ERR_INVALID_ARG;   // would leave a hole
            if (pos_end[i] - pos_begin[i] > max_range) max_range = pos_end[i] - pos_begin[i];
        }
    }
    if (auto_range && !c->dev_lengths) {
        // lengths are the host's: the ranges are worked out here, layer by layer (they may differ between layers)
        for (int l = lb; l < lb + lc; ++l) {
            int b[kMaxLaunchSeq], e[kMaxLaunchSeq], mr = 0;
            for (int i = 0; i < n_seq; ++i) {
                const size_t u = (size_t)l * c->cfg.max_batch + seqs[i];
                b[i] = c->len_proj[u], e[i] = c->len[u] > c->len_proj[u] ? c->len[u] : c->len_proj[u];
                if (e[i] - b[i] > mr) mr = e[i] - b[i];
            }
            if (mr == 0) continue;
            UnitTable ut;
            fill_table(c, &ut, l, 1, seqs, n_seq);
            if (launch_project(c, ut, b, e, mr, (cudaStream_t)stream) != cudaSuccess) return TB_ERR_CUDA;
            c->last_cache_write = (long long)c->launches;
            c->launches++;
        }
    } else {
        const int step = layers_per_launch(n_seq);
        for (int l0 = lb; l0 < lb + lc; l0 += step) {
            const int n = l0 + step <= lb + lc ? step : lb + lc - l0;
            UnitTable ut;
            fill_table(c, &ut, l0, n, seqs, n_seq);
            if (max_range > 0) {
                if (launch_project(c, ut, pos_begin, pos_end, max_range, (cudaStream_t)stream) != cudaSuccess) return TB_ERR_CUDA;
                c->last_cache_write = (long long)c->launches;
                c->launches++;
            }
        }
    }
    for (int l = lb; l < lb + lc; ++l)
        for (int i = 0; i < n_seq; ++i) {
            const size_t u = (size_t)l * c->cfg.max_batch + seqs[i];
            const int end = auto_range ? c->len[u] : pos_end[i];
            if (end > c->len_proj[u]) c->len_proj[u] = end;
        }
    return TB_OK;
}

tb_status tb_score_tokens(tb_ctx* c, int32_t layer, const int32_t* seq_ids, int32_t n_seq, const float* q_imp, int32_t reduce,
                          float score_scale, float* scores, void* stream) {
    if (!c || !q_imp || !scores || bad_layers(c, layer, 1)) return TB_ERR_INVALID_ARG;
    reduce = effective_reduce(c, reduce);
    if (reduce < 0) return TB_ERR_UNSUPPORTED;
    int seqs[kMaxLaunchSeq];
    tb_status st = resolve_seqs(c, seq_ids, n_seq, seqs);
    if (st != TB_OK) return st;
    UnitTable ut;
    fill_table(c, &ut, layer, 1, seqs, n_seq, /*projected=*/true);   // projected tokens only
    if (launch_score(c, ut, q_imp, reduce, score_scale, scores, (cudaStream_t)stream) != cudaSuccess) return TB_ERR_CUDA;
    c->launches++;
    return TB_OK;
}

tb_status tb_select_topk(tb_ctx* c, int32_t lb, int32_t lc, const int32_t* seq_ids, int32_t n_seq, const float* q_imp,
                         const tb_select_params* p, int32_t* idx_out, int32_t* cnt_out, void* stream) {
    if (!c || !p || bad_layers(c, lb, lc)) return TB_ERR_INVALID_ARG;
    if (p->budget < 0 || p->sinks < 0 || p->recent < 0 || p->radius < 0 || p->interval < 1 || p->step < 0) return TB_ERR_INVALID_ARG;
    if (p->nmode != TB_NEIGHBOR_DILATE && p->nmode != TB_NEIGHBOR_CLUSTER) return TB_ERR_INVALID_ARG;
    const int reduce = effective_reduce(c, p->reduce);
    if (reduce < 0) return TB_ERR_UNSUPPORTED;
    if (p->budget > c->cfg.max_budget || p->radius > c->cfg.max_radius) return TB_ERR_CAPACITY;
    int seqs[kMaxLaunchSeq];
    tb_status st = resolve_seqs(c, seq_ids, n_seq, seqs);
    if (st != TB_OK) return st;
    const bool refresh = p->step % p->interval == 0;
    const int mb = c->cfg.max_batch;
    uint64_t bytes = 0;
    if (refresh) {
        if (!q_imp) return TB_ERR_INVALID_ARG;
        for (int l = lb; l < lb + lc; ++l)
            for (int i = 0; i < n_seq; ++i) {
                const size_t u = (size_t)l * mb + seqs[i];
                if (c->len[u] <= 0) return TB_ERR_INVALID_ARG;
                int lo, hi;
                cand_range(c->len[u], p->sinks, p->recent, &lo, &hi);
                if (c->len_proj[u] < hi) return TB_ERR_UNPROJECTED;
                bytes += (uint64_t)(hi - lo) * c->geom.Hi * c->cfg.imp_dim * elem_size(c->cfg.kv_dtype);   // every key stream once (lists that share one re-read it from L2)
            }
    } else {
        for (int l = lb; l < lb + lc; ++l)
            for (int i = 0; i < n_seq; ++i)
                if (!c->has_sel[(size_t)l * mb + seqs[i]]) return TB_ERR_STATE;
    }
    const int step = layers_per_launch(n_seq);
    // Two passes over the call's chunks: the first only checks that every launch has a configuration
    // (sizes beyond what a kernel takes are refused before anything runs), the second launches.
    for (int pass = 0; pass < 2; ++pass) {
        const bool dry = pass == 0;
        if (dry && !refresh) continue;
        for (int l0 = lb; l0 < lb + lc; l0 += step) {
            const int n = l0 + step <= lb + lc ? step : lb + lc - l0;
            UnitTable ut;
            fill_table(c, &ut, l0, n, seqs, n_seq);
            const size_t unit_off = (size_t)(l0 - lb) * n_seq * c->geom.Hl;
            if (refresh) {
                SelectArgs a;
                a.q_imp = q_imp + (size_t)(l0 - lb) * n_seq * c->geom.Hl * c->geom.gl * c->cfg.imp_dim;
                a.budget = p->budget, a.sinks = p->sinks, a.recent = p->recent, a.reduce = reduce;
                if (p->radius == 0) {
                    a.idx_dst = nullptr, a.cnt_dst = nullptr, a.dst_is_state = 1, a.idx_stride = c->geom.idx_cap;
                } else {
                    a.idx_dst = c->wk.sel_idx, a.cnt_dst = c->wk.sel_cnt, a.dst_is_state = 0, a.idx_stride = c->wk.sel_stride;
                }
                cudaError_t e = launch_select(c, ut, a, (cudaStream_t)stream, dry);
                if (e != cudaSuccess) return dry ? TB_ERR_UNSUPPORTED : TB_ERR_CUDA;
                if (!dry) c->last_list_write = (long long)c->launches, c->launches++;
                if (p->radius > 0) {
                    NeighborArgs na;
                    na.idx_src = c->wk.sel_idx, na.cnt_src = c->wk.sel_cnt, na.src_stride = c->wk.sel_stride;
                    na.radius = p->radius, na.nmode = p->nmode, na.sinks = p->sinks, na.recent = p->recent;
                    e = launch_neighbors(c, ut, na, (cudaStream_t)stream, dry);
                    if (e != cudaSuccess) return dry ? TB_ERR_UNSUPPORTED : TB_ERR_CUDA;
                    if (!dry) c->last_list_write = (long long)c->launches, c->launches++;
                }
                if (!dry && c->imp_rows) {               // KV migration into the Important buffer
                    if (launch_migrate(c, ut, (cudaStream_t)stream) != cudaSuccess) return TB_ERR_CUDA;
                    c->last_list_write = (long long)c->launches, c->launches++;
                }
            }
            if (!dry && (idx_out || cnt_out)) {
                if (launch_copy_lists(c, ut, idx_out ? idx_out + unit_off * c->geom.idx_cap : nullptr,
                                      cnt_out ? cnt_out + unit_off : nullptr, (cudaStream_t)stream) != cudaSuccess)
                    return TB_ERR_CUDA;
                c->launches++;
            }
        }
    }
    if (refresh) {
        for (int l = lb; l < lb + lc; ++l)
            for (int i = 0; i < n_seq; ++i) {
                const size_t u = (size_t)l * mb + seqs[i];
                c->has_sel[u] = 1;
                int lo, hi;
                cand_range(c->len[u], p->sinks, p->recent, &lo, &hi);
                // without neighbour expansion the stored count is known here: min(budget, candidates)
                c->sel_cnt[u] = p->radius == 0 ? (p->budget < hi - lo ? p->budget : hi - lo) : -1;
            }
        c->last_bytes = bytes;
    }
    return TB_OK;
}

tb_status tb_sparse_decode_attention(tb_ctx* c, int32_t lb, int32_t lc, const int32_t* seq_ids, int32_t n_seq, const void* q,
                                     const tb_select_params* p, const int32_t* idx, const int32_t* cnt, float sm_scale,
                                     float* out, float* lse, void* stream) {
    if (!c || !q || !p || !out || bad_layers(c, lb, lc)) return TB_ERR_INVALID_ARG;
    if ((idx == nullptr) != (cnt == nullptr)) return TB_ERR_INVALID_ARG;
    const bool dense = p->budget < 0;
    if (!dense && (p->sinks < 0 || p->recent < 0 || p->radius < 0)) return TB_ERR_INVALID_ARG;
    int seqs[kMaxLaunchSeq];
    tb_status st = resolve_seqs(c, seq_ids, n_seq, seqs);
    if (st != TB_OK) return st;
    const int mb = c->cfg.max_batch;
    uint64_t bytes = 0;
    int bound = c->geom.idx_cap;
    if (!dense && !idx) {
        // DILATE grows a selection to at most (2r+1)B positions, CLUSTER to (1+r)B
        long long b = (long long)(p->nmode == TB_NEIGHBOR_CLUSTER ? 1 + p->radius : 2 * p->radius + 1) * p->budget;
        if (b < bound) bound = (int)b;
    }
    for (int l = lb; l < lb + lc; ++l)
        for (int i = 0; i < n_seq; ++i) {
            const size_t u = (size_t)l * mb + seqs[i];
            const int L = c->len[u];
            if (L <= 0) return TB_ERR_INVALID_ARG;
            if (!dense && !idx && !c->has_sel[u]) return TB_ERR_STATE;
            long long rows = L;
            if (!dense) {
                rows = (long long)(p->sinks < L ? p->sinks : L) + bound + p->recent;
                if (rows > L) rows = L;
            }
            bytes += (uint64_t)rows * c->geom.Ha * 2 * c->cfg.head_dim * elem_size(c->cfg.kv_dtype);
        }
    const int step = layers_per_launch(n_seq);
    const size_t es = elem_size(c->cfg.kv_dtype);
    for (int l0 = lb; l0 < lb + lc; l0 += step) {
        const int n = l0 + step <= lb + lc ? step : lb + lc - l0;
        UnitTable ut;
        fill_table(c, &ut, l0, n, seqs, n_seq);
        const size_t hq_off = (size_t)(l0 - lb) * n_seq * c->cfg.n_q_heads;
        const size_t unit_off = (size_t)(l0 - lb) * n_seq * c->geom.Hl;
        AttnArgs a;
        a.res_rows = c->res_rows, a.res_sinks = c->res_sinks, a.res_window = c->res_window;
        a.imp_rows = (dense || idx) ? nullptr : c->imp_rows;
        a.q = (const char*)q + hq_off * c->cfg.head_dim * es;
        a.idx = idx ? idx + unit_off * c->geom.idx_cap : nullptr;
        a.cnt = cnt ? cnt + unit_off : nullptr;
        a.out = out + hq_off * c->cfg.head_dim;
        a.lse = lse ? lse + hq_off : nullptr;
        a.dense = dense, a.sinks = dense ? 0 : p->sinks, a.recent = dense ? 0 : p->recent;
        a.list_bound = bound;
        for (int l = 0; l < n; ++l)
            for (int i = 0; i < n_seq; ++i)
                a.known_cnt[l * n_seq + i] = (dense || idx || c->dev_lengths) ? -1 : c->sel_cnt[(size_t)(l0 + l) * mb + seqs[i]];
        a.nsplit = 0;
        a.sm_scale = sm_scale > 0.f ? sm_scale : 1.0f / sqrtf((float)c->cfg.head_dim);
        a.early_ok = !idx && (long long)c->launches - c->last_cache_write >= 2 && (long long)c->launches - c->last_list_write >= 2;
        if (launch_attention(c, ut, a, (cudaStream_t)stream) != cudaSuccess) return TB_ERR_CUDA;
        c->launches++;
    }
    c->last_bytes = bytes;
    return TB_OK;
}

tb_status tb_get_status(tb_ctx* c, void* stream, int32_t* device_status) {
    if (!c || !device_status) return TB_ERR_INVALID_ARG;
    int32_t v = 0;
    if (cudaMemcpyAsync(&v, c->st.status, 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess) return TB_ERR_CUDA;
    if (cudaMemsetAsync(c->st.status, 0, 4, (cudaStream_t)stream) != cudaSuccess) return TB_ERR_CUDA;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return TB_ERR_CUDA;
    *device_status = v;
    return TB_OK;
}

size_t tb_resident_rows_bytes(const tb_config* cfg, int32_t sinks, int32_t window) {
    if (check_config(cfg) != TB_OK || sinks < 0 || window < 0) return 0;
    return (size_t)cfg->n_layers * cfg->max_batch * cfg->n_kv_heads * ((size_t)sinks + window) * 2 * cfg->head_dim * elem_size(cfg->kv_dtype);
}

size_t tb_important_buffer_bytes(const tb_config* cfg) {
    if (check_config(cfg) != TB_OK || cfg->list_scope != TB_SCOPE_KV_HEAD) return 0;
    Layout l;
    compute_layout(cfg, &l);
    return (size_t)cfg->n_layers * cfg->max_batch * cfg->n_kv_heads * (size_t)l.idx_cap * 2 * cfg->head_dim * elem_size(cfg->kv_dtype);
}

namespace {
bool device_memory(const void* p) {
    cudaPointerAttributes pa;
    if (cudaPointerGetAttributes(&pa, p) != cudaSuccess) { (void)cudaGetLastError(); return false; }
    return pa.type == cudaMemoryTypeDevice || pa.type == cudaMemoryTypeManaged;
}
bool all_sequences_empty(const tb_ctx* c) {
    for (int v : c->len) if (v) return false;
    return true;
}
}  // namespace

tb_status tb_bind_resident_rows(tb_ctx* c, void* rows_dev, size_t bytes, int32_t sinks, int32_t window) {
    if (!c || sinks < 0 || window < 0) return TB_ERR_INVALID_ARG;
    if (!rows_dev) { c->res_rows = nullptr, c->res_sinks = c->res_window = 0; return TB_OK; }
    if (sinks + window == 0 || ((uintptr_t)rows_dev & 255) || !device_memory(rows_dev)) return TB_ERR_INVALID_ARG;
    if (bytes < tb_resident_rows_bytes(&c->cfg, sinks, window)) return TB_ERR_CAPACITY;
    if (!all_sequences_empty(c)) return TB_ERR_STATE;   // the copies are kept current by the appends: bind before the first one
    c->res_rows = rows_dev, c->res_sinks = sinks, c->res_window = window;
    return TB_OK;
}

tb_status tb_bind_important_buffer(tb_ctx* c, void* buf_dev, size_t bytes) {
    if (!c) return TB_ERR_INVALID_ARG;
    if (!buf_dev) { c->imp_rows = nullptr; return TB_OK; }
    if (c->cfg.list_scope != TB_SCOPE_KV_HEAD) return TB_ERR_UNSUPPORTED;
    if (((uintptr_t)buf_dev & 255) || !device_memory(buf_dev)) return TB_ERR_INVALID_ARG;
    if (bytes < tb_important_buffer_bytes(&c->cfg)) return TB_ERR_CAPACITY;
    for (int& v : c->has_sel) v = 0;                    // stored lists have no rows in the buffer yet: select first
    c->imp_rows = buf_dev;
    return TB_OK;
}

tb_status tb_use_device_lengths(tb_ctx* c, int32_t on, int32_t growth_reserve) {
    if (!c || growth_reserve < 0) return TB_ERR_INVALID_ARG;
    if (on && !c->dev_lengths) {
        // the counters are only kept while they are read: bring them up to the mirrors (blocking copies)
        const size_t n = (size_t)c->cfg.n_layers * c->cfg.max_batch * 4;
        if (cudaMemcpy(c->st.len, c->len.data(), n, cudaMemcpyHostToDevice) != cudaSuccess ||
            cudaMemcpy(c->st.len_proj, c->len_proj.data(), n, cudaMemcpyHostToDevice) != cudaSuccess)
            return TB_ERR_CUDA;
    }
    c->dev_lengths = on ? 1 : 0;
    c->growth_reserve = on ? growth_reserve : 0;
    return TB_OK;
}

tb_status tb_sync_lengths(tb_ctx* c, void* stream) {
    if (!c) return TB_ERR_INVALID_ARG;
    const size_t n = (size_t)c->cfg.n_layers * c->cfg.max_batch;
    std::vector<int32_t> a(n), b(n);
    if (cudaMemcpyAsync(a.data(), c->st.len, n * 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess ||
        cudaMemcpyAsync(b.data(), c->st.len_proj, n * 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess ||
        cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess)
        return TB_ERR_CUDA;
    for (size_t i = 0; i < n; ++i) c->len[i] = a[i], c->len_proj[i] = b[i], c->sel_cnt[i] = -1;
    return TB_OK;
}

tb_status tb_set_wait_diagnostics(tb_ctx* c, int32_t poll_limit, int32_t drop_tile) {
    if (!c || poll_limit < 0) return TB_ERR_INVALID_ARG;
    c->wait_poll_limit = poll_limit;
    c->drop_tile = drop_tile < 0 ? -1 : drop_tile;
    return TB_OK;
}

uint64_t tb_last_step_bytes(const tb_ctx* c) { return c ? c->last_bytes : 0; }
uint64_t tb_launch_count(const tb_ctx* c) { return c ? c->launches : 0; }

const char* tb_status_string(int32_t s) {
    switch (s) {
        case TB_OK: return "ok";
        case TB_ERR_INVALID_ARG: return "invalid argument";
        case TB_ERR_UNSUPPORTED: return "unsupported shape or mode";
        case TB_ERR_CAPACITY: return "capacity exceeded";
        case TB_ERR_UNPROJECTED: return "candidate keys not projected";
        case TB_ERR_STATE: return "no stored selection";
        case TB_ERR_CUDA: return "CUDA runtime error";
        case TB_ERR_TIMEOUT: return "device wait timed out";
        case TB_ERR_BAD_INDEX: return "index outside the cached tokens";
        default: return "unknown status";
    }
}

}  // extern "C"
