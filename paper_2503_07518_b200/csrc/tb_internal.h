// Host-side context and the launch interfaces between the C ABI (tb_api.cu) and the kernel files.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/tokenbutler.h"

namespace tb {

constexpr int kMaxLaunchSeq = 64;     // sequences per launch (larger batches are chunked on the host)
constexpr int kMaxLaunchUnits = 256;  // (layer, sequence) pairs per launch
constexpr int kMaxSplits = 32;        // split-K partitions per (sequence, KV head)
constexpr int kMaxGroup = 8;          // query heads per KV head

// Geometry every kernel needs; passed by value.
struct Geom {
    int n_layers, Hq, Hkv, g, D, dp;
    // Selection scope (tb_list_scope): Hi key streams of the projected-key cache, Hl index lists and
    // Ha attention units per (layer, sequence); gl importance queries are reduced into one list and
    // ga query heads share an attention unit's gathered rows.
    //   per KV head:    Hi = Hl = Ha = Hkv, gl = ga = g
    //   per query head: Hi = Hkv, Hl = Ha = Hq, gl = ga = 1
    int Hi, Hl, Ha, gl, ga;
    int max_batch, max_seq_len;
    int idx_cap;       // entries per index-list row
    int dtype;         // tb_dtype
};

// Per-launch table of (layer-local, sequence) pairs: which cache slot and how many tokens.
// Lengths come two ways.  By default they travel here, as kernel parameters copied from the host's
// mirrors (no dependent load at kernel start; a captured CUDA graph then replays the lengths it was
// captured with).  With use_dev_len the kernels read the context's device counters, which the append
// and projection kernels advance themselves, so a captured graph replays a growing sequence; `len`
// then holds upper bounds (length + the reserve the caller declared) that size grids and shared memory.
struct UnitTable {
    int layer_begin, layer_count, n_seq;
    int use_dev_len;            // 1: kernels read len_dev / len_proj_dev
    int len_is_projected;       // 1: "length" means projected length (materialised scores cover projected tokens)
    const int32_t* len_dev;     // [n_layers * max_batch] tokens cached
    const int32_t* len_proj_dev;   // [n_layers * max_batch] tokens whose keys are projected
    int seq_id[kMaxLaunchSeq];
    int len[kMaxLaunchUnits];   // [layer_local * n_seq + s]
};

struct SelectArgs {
    const float* q_imp;   // [layer_count][n_seq][Hq][dp]
    int32_t* idx_dst;     // rows of `idx_stride` entries, indexed like the stored lists (see below)
    int32_t* cnt_dst;
    int dst_is_state;     // 1: rows indexed by (layer, seq_id, head) in the context's lists; 0: by launch unit
    int idx_stride;
    int budget, sinks, recent;
    int reduce;           // tb_group_reduce: TB_GROUP_SUM or TB_GROUP_MAX
};

struct NeighborArgs {
    const int32_t* idx_src;  // launch-unit indexed rows of `src_stride`
    const int32_t* cnt_src;
    int src_stride;
    int radius, nmode, sinks, recent;
};

// Where an attended row is read from: the K|V cache, or one of two optional copies in device memory.
// A row reference is one int: bits 0..28 the row inside its source, bits 29..30 the source.
constexpr int kRowSrcShift = 29;
constexpr int kRowIdxMask = (1 << kRowSrcShift) - 1;
constexpr int kRowSrcCache = 0, kRowSrcResident = 1, kRowSrcImportant = 2;

struct AttnArgs {
    // Resident rows (offloaded KV): per (layer, sequence, KV head) the first res_sinks tokens and a ring of the
    // res_window most recent ones (token t in slot res_sinks + t % res_window), kept current by the append kernel.
    const void* res_rows;   // NULL = not bound
    int res_sinks, res_window;
    // Important buffer: per (layer, sequence, KV head) the K|V rows of the stored list, in list order,
    // written by the migration kernel at every refresh (NULL = not bound, or caller-supplied lists).
    const void* imp_rows;
    const void* q;          // [layer_count][n_seq][Hq][D]
    const int32_t* idx;     // caller lists (launch-unit indexed) or NULL = stored lists
    const int32_t* cnt;
    float* out;             // [layer_count][n_seq][Hq][D]
    float* lse;             // optional
    int dense, sinks, recent, nsplit;
    int early_ok;           // 1: lists and cache rows were written at least two launches ago
    int cluster_merge;      // 1: the splits of a (sequence, KV head) are one cluster and merge through DSMEM
    int list_bound;         // host-known upper bound of the list length (sizes the split count)
    float sm_scale;
    // Length of the stored list per (layer-local, sequence) when the host knows it exactly (selection
    // without neighbour expansion: min(budget, candidates), equal for all KV heads), else -1: saves
    // the kernels a dependent global load before they can split the rows.
    int known_cnt[kMaxLaunchUnits];
};

constexpr int kStatusCapacity = -3;      // device status: an append in a replayed graph ran past max_seq_len
constexpr int kStatusUnprojected = -4;   // device status: a replayed selection found candidates that are not projected

struct DevState {
    int32_t* len;         // [n_layers * max_batch] device copies of the lengths, advanced by the append kernel
    int32_t* len_proj;    // ... and of the projected lengths, advanced by the projection kernels
    uint32_t* misc_counter;   // arrival counters of the append / projection kernels (self-resetting)
    void* W;              // [n_layers][Hkv][D][dp] kv_dtype
    int32_t* idx;         // [n_layers][max_batch][Hl][idx_cap]
    int32_t* cnt;         // [n_layers][max_batch][Hl]
    int32_t* status;      // device status word
    uint32_t* attn_counter;  // [n_layers*max_batch*Ha] split arrival counters (self-resetting)
};

struct DevWork {
    float* part_o;        // [units_q][kMaxSplits][D]
    float* part_ml;       // [units_q][kMaxSplits][2]
    int32_t* sel_idx;     // [n_layers*max_batch*Hl][max_budget rounded]  pre-expansion selection
    int32_t* sel_cnt;
    int sel_stride;
    uint32_t* sel_keys;   // [n_layers*max_batch*Hl][max_seq_len rounded up to 256]  score keys of a many-problem selection launch
    uint16_t* sel_bins;   // same shape, 2 bytes per token: first digits of a very long problem's rows, when they do not fit on chip
};

}  // namespace tb

struct tb_ctx {
    tb_config cfg;
    tb::Geom geom;
    void* kv;
    void* kimp;
    tb::DevState st;
    tb::DevWork wk;
    size_t state_bytes, work_bytes;
    std::vector<int> len, len_proj;       // [n_layers * max_batch]
    std::vector<int> has_sel;             // [n_layers * max_batch]
    std::vector<int> sel_cnt;             // [n_layers * max_batch] stored list length when the host knows it, else -1
    CUtensorMap kimp_map;                 // 2-D view of kimp: rows = all token slots, cols = d'
    int tile_rows;                        // rows per TMA box of the score pass
    int sm_count;
    int attn_max_active[17];              // co-resident attention clusters per cluster size (0 = not asked yet)
    void* res_rows;                       // resident sink + window rows (tb_bind_resident_rows), or NULL
    int res_sinks, res_window;
    void* imp_rows;                       // Important buffer (tb_bind_important_buffer), or NULL
    int dev_lengths;                      // 1: kernels read the device counters (graph-replayable growth)
    int growth_reserve;                   // tokens a sequence may grow beyond the host mirror while graphs are replayed
    int wait_poll_limit;                  // polls per bounded wait of the selection kernels; 0 = the default (seconds)
    int drop_tile;                        // diagnostics: tile whose copy the next single-block selection leaves out, -1 = none
    uint64_t last_bytes, launches;
    // index (value of `launches` at launch time) of the last kernel that wrote the caches / the stored
    // lists; a kernel may read them before its dependency wait only if that writer is not its predecessor
    long long last_cache_write, last_list_write;
};

namespace tb {

#ifdef __CUDACC__
// Tokens of launch unit (layer-local ll, sequence s): a kernel parameter, or the device counter.
__device__ __forceinline__ int unit_len(const Geom& gm, const UnitTable& ut, int ll, int s) {
    if (!ut.use_dev_len) return ut.len[ll * ut.n_seq + s];
    const size_t pair = (size_t)(ut.layer_begin + ll) * gm.max_batch + ut.seq_id[s];
    return ut.len_is_projected ? ut.len_proj_dev[pair] : ut.len_dev[pair];
}
// Last block of a grid to get here (after its global writes): true for exactly one block, which also
// resets the counter for the next launch.  Called by all threads of the block.
__device__ __forceinline__ bool last_block_arrives(uint32_t* counter, unsigned n_blocks) {
    __shared__ int s_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned prev = atomicAdd(counter, 1u);
        s_last = prev == n_blocks - 1u;
        if (s_last) *counter = 0u;
    }
    __syncthreads();
    return s_last != 0;
}
#endif

// Kernel attributes (dynamic shared-memory limit, non-portable cluster sizes) belong to a device's
// context, so each launcher configures its kernels on first use per device.
inline bool first_use_on_this_device(unsigned char (&seen)[64]) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return true;
    if (seen[dev]) return false;
    seen[dev] = 1;
    return true;
}

// tb_cache.cu
cudaError_t launch_append(const tb_ctx* c, const UnitTable& ut, const int* n_new, const int* tok_off, int total_new,
                          const void* k, const void* v, cudaStream_t s);
// pos_begin == nullptr: every listed sequence's unprojected tokens [projected length, length), taken from the
// device counters; max_range then bounds the tokens of any one (layer, sequence)
cudaError_t launch_project(const tb_ctx* c, const UnitTable& ut, const int* pos_begin, const int* pos_end, int max_range, cudaStream_t s);

// tb_select.cu
cudaError_t launch_score(const tb_ctx* c, const UnitTable& ut, const float* q_imp, int reduce, float scale, float* scores,
                         cudaStream_t s);
// `dry`: work out the launch configuration and report whether it exists, launch nothing, change nothing
// (the entry points check every chunk of a call this way before the first real launch)
cudaError_t launch_select(const tb_ctx* c, const UnitTable& ut, const SelectArgs& a, cudaStream_t s, bool dry = false);
// one block per problem; launch_select hands over to it when a launch holds at least two problems per SM
cudaError_t launch_select_wave(const tb_ctx* c, const UnitTable& ut, const SelectArgs& a, cudaStream_t s, bool dry = false);
// few, long problems: a cluster per problem on parked keys
cudaError_t launch_select_cw(const tb_ctx* c, const UnitTable& ut, const SelectArgs& a, cudaStream_t s, bool dry = false);
cudaError_t launch_neighbors(const tb_ctx* c, const UnitTable& ut, const NeighborArgs& a, cudaStream_t s, bool dry = false);
// copies the rows of the stored lists into the Important buffer (after a refresh)
cudaError_t launch_migrate(const tb_ctx* c, const UnitTable& ut, cudaStream_t s);
cudaError_t launch_copy_lists(const tb_ctx* c, const UnitTable& ut, int32_t* idx_out, int32_t* cnt_out, cudaStream_t s);

// tb_attention.cu
cudaError_t launch_attention(const tb_ctx* c, const UnitTable& ut, const AttnArgs& a, cudaStream_t s);

}  // namespace tb
