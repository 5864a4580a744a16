// Sparse decode attention (paper Sec. 3.3: attention over Sink + Important + Local-Window rows of
// the never-evicted cache; Sec. 3.4: the important rows are gathered by index).
//
// One launch covers (layer, sequence, KV head) x split.  Every gathered K|V row pair (adjacent in
// memory) is loaded once and shared by the g query heads of its KV head.  Each split keeps an online
// softmax (m, l, o) per query head; the last block to arrive for a (sequence, KV head) merges the
// splits in split order, so the result is bit-reproducible.
#include <cooperative_groups.h>
#include <type_traits>

#include "tb_common.cuh"
#include "tb_internal.h"

namespace cg = cooperative_groups;

namespace tb {

constexpr int kAttnThreads = 128;
constexpr int kAttnWarps = kAttnThreads / 32;
constexpr int kRowsPerIter = 4;
constexpr int kAttnMaxCluster = 16;      // splits that can be merged inside a thread-block cluster (16 is non-portable)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Which row does attended row r refer to?  Rows are sinks, then the index list, then the window.  The answer
// is a row reference (see kRowSrcShift): a token of the cache or, when the context has them, a slot of the
// resident sink / window copies or of the Important buffer.
template <bool kSources>           // false: every row comes from the cache (the copies are not bound)
struct RowMap {
    int n_sink, n_list, w_begin, L, dense;
    int res_sinks, res_window;      // 0 = no resident copies
    int use_imp;                    // list rows come from the Important buffer, in list order
    const int32_t* list;
    // token t in the resident copies if they hold it (one of the first res_sinks tokens, else one of the
    // res_window most recent), else in the cache
    __device__ __forceinline__ int res_ref(int t) const {
        if constexpr (!kSources) return t;
        if (t < res_sinks) return (kRowSrcResident << kRowSrcShift) | t;
        return (res_window > 0 && t >= L - res_window) ? (kRowSrcResident << kRowSrcShift) | (res_sinks + t % res_window) : t;
    }
    __device__ __forceinline__ int sink_ref(int t) const { return res_ref(t); }
    __device__ __forceinline__ int window_ref(int t) const { return res_ref(t); }
    __device__ __forceinline__ int token(int r, bool& bad) const {
        bad = false;
        if (dense) return r;
        if (r < n_sink) return sink_ref(r);
        r -= n_sink;
        if (r < n_list) {
            if (kSources && use_imp) return (kRowSrcImportant << kRowSrcShift) | r;
            int t = list[r];
            if (t < 0 || t >= L) { bad = true; return 0; }
            return t;
        }
        return window_ref(w_begin + (r - n_list));
    }
    // the same with a bad list entry reported as -1 (nothing else depends on the loaded value)
    __device__ __forceinline__ int token_or_neg(int r) const {
        if (dense) return r;
        if (r < n_sink) return sink_ref(r);
        r -= n_sink;
        if (r < n_list) {
            if (kSources && use_imp) return (kRowSrcImportant << kRowSrcShift) | r;
            const int t = list[r];
            return (t < 0 || t >= L) ? -1 : t;
        }
        return window_ref(w_begin + (r - n_list));
    }
};

// An attention unit is (layer, sequence, head h < Ha): one KV head with its group of query heads, or,
// with one list per query head, a single query head.  It reads KV head h*Hkv/Ha and list h*Hl/Ha.
struct AttnUnit {
    size_t kv_c;      // unit row of the K|V cache
    size_t list_c;    // row of the context's lists
    int list_l;       // row of caller-supplied lists [layer_count][n_seq][Hl]
    int lu;           // launch-local attention unit
    __device__ __forceinline__ AttnUnit(const Geom& gm, const UnitTable& ut, int ll, int s, int h) {
        const size_t pc = (size_t)(ut.layer_begin + ll) * gm.max_batch + ut.seq_id[s];
        const int pl = ll * ut.n_seq + s;
        // (the usual scopes have Hl == Ha, and Hkv == Ha or Hl: no division on the way to the first load)
        const int lh = gm.Hl == gm.Ha ? h : (h * gm.Hl) / gm.Ha;
        kv_c = pc * gm.Hkv + (gm.Hkv == gm.Ha ? h : (h * gm.Hkv) / gm.Ha);
        list_c = pc * gm.Hl + lh;
        list_l = pl * gm.Hl + lh;
        lu = pl * gm.Ha + h;
    }
};

// Publishes one split's (m, l, o) per query head and lets the last block to arrive for the
// (sequence, KV head) merge all splits in split order:  M = max m_j;  l = sum l_j 2^(m_j-M);
// out = sum o_j 2^(m_j-M) / l;  lse = (M + log2 l) ln 2.  Called by all 128 threads; thread = channel.
struct SplitSink {
    float* part_o;
    float* part_ml;
    uint32_t* counters;
    float* out;
    float* lse;
    size_t hq0;        // first query head of this (layer, sequence, KV head) in the launch
    int lu, split, nsplit;

    __device__ __forceinline__ void publish(int u, float M, float lsum, float o) const {
        const size_t pq = (hq0 + u) * kMaxSplits + split;
        part_o[pq * 128 + threadIdx.x] = o;
        if (threadIdx.x == 0) part_ml[pq * 2] = M, part_ml[pq * 2 + 1] = lsum;
    }
    // the same, for a thread that holds channel `ch` of head u / the head's statistics
    __device__ __forceinline__ void publish_at(int u, int ch, float o) const { part_o[((hq0 + u) * kMaxSplits + split) * 128 + ch] = o; }
    __device__ __forceinline__ void publish_stat(int u, float M, float lsum) const {
        const size_t pq = (hq0 + u) * kMaxSplits + split;
        part_ml[pq * 2] = M, part_ml[pq * 2 + 1] = lsum;
    }
    __device__ __forceinline__ void merge_if_last(int g, int* sh_last) const {
        const int tid = threadIdx.x;
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            unsigned prev = atomicAdd(&counters[lu], 1u);
            *sh_last = prev == (unsigned)nsplit - 1u;
            if (*sh_last) counters[lu] = 0;             // ready for the next launch
        }
        __syncthreads();
        if (!*sh_last) return;
        __threadfence();
        // all (head, split) statistics in one round trip, then weights, then 16-byte wide sums
        __shared__ float mm[kMaxGroup][kMaxSplits], lw[kMaxGroup][kMaxSplits], w[kMaxGroup][kMaxSplits];
        __shared__ float Lsum[kMaxGroup];
        for (int i = tid; i < g * nsplit; i += kAttnThreads) {
            const int u = i / nsplit, j = i % nsplit;
            const size_t pq = (hq0 + u) * kMaxSplits + j;
            mm[u][j] = __ldcg(&part_ml[pq * 2]);
            lw[u][j] = __ldcg(&part_ml[pq * 2 + 1]);
        }
        __syncthreads();
        if (tid < g) {
            float M = -INFINITY;
            for (int j = 0; j < nsplit; ++j) M = fmaxf(M, mm[tid][j]);
            const float Ms = M == -INFINITY ? 0.f : M;
            float lsum = 0.f;
            for (int j = 0; j < nsplit; ++j) {
                const float e = exp2f(mm[tid][j] - Ms);
                w[tid][j] = e;
                lsum += lw[tid][j] * e;
            }
            Lsum[tid] = lsum;
            if (lse) lse[hq0 + tid] = (M + log2f(lsum)) * kLn2;
        }
        __syncthreads();
        for (int item = tid; item < g * 32; item += kAttnThreads) {
            const int u = item >> 5, c4 = item & 31;
            const float4* src = reinterpret_cast<const float4*>(part_o + (hq0 + u) * kMaxSplits * 128) + c4;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
            for (int j = 0; j < nsplit; ++j) {
                const float4 v = __ldcg(src + j * 32);
                const float e = w[u][j];
                acc.x = fmaf(v.x, e, acc.x), acc.y = fmaf(v.y, e, acc.y), acc.z = fmaf(v.z, e, acc.z), acc.w = fmaf(v.w, e, acc.w);
            }
            const float inv = 1.f / Lsum[u];
            reinterpret_cast<float4*>(out + (hq0 + u) * 128)[c4] = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
        }
    }
};

template <typename T>
struct RowVec;   // the 4 channels of a 128-channel row that one lane owns
template <>
struct RowVec<float> {
    float4 v;
    __device__ __forceinline__ void load(const float* row, int lane) { v = __ldg(reinterpret_cast<const float4*>(row) + lane); }
    __device__ __forceinline__ void get(float* f) const { f[0] = v.x, f[1] = v.y, f[2] = v.z, f[3] = v.w; }
};
template <>
struct RowVec<__nv_bfloat16> {
    uint2 v;
    __device__ __forceinline__ void load(const __nv_bfloat16* row, int lane) { v = __ldg(reinterpret_cast<const uint2*>(row) + lane); }
    __device__ __forceinline__ void get(float* f) const { f[0] = bf16_lo(v.x), f[1] = bf16_hi(v.x), f[2] = bf16_lo(v.y), f[3] = bf16_hi(v.y); }
};

template <typename T, int G>
__global__ void __launch_bounds__(kAttnThreads) attn_kernel(Geom gm, UnitTable ut, AttnArgs a, const T* __restrict__ kv,
                                                            const int32_t* __restrict__ state_idx, const int32_t* __restrict__ state_cnt,
                                                            float* __restrict__ part_o, float* __restrict__ part_ml,
                                                            uint32_t* __restrict__ counters, int32_t* __restrict__ status) {
    constexpr int D = 128;
    __shared__ float sh_o[kAttnWarps][G][D];
    __shared__ float sh_m[kAttnWarps][G], sh_l[kAttnWarps][G];
    __shared__ int sh_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int split = blockIdx.x, h = blockIdx.y;
    const int ll = blockIdx.z / ut.n_seq, s = blockIdx.z % ut.n_seq;
    const int L = unit_len(gm, ut, ll, s);
    const int g = gm.ga;
    const AttnUnit au(gm, ut, ll, s, h);
    const int lu = au.lu;

    RowMap<true> rm;
    rm.L = L, rm.dense = a.dense;
    rm.res_sinks = a.res_rows ? a.res_sinks : 0, rm.res_window = a.res_rows ? a.res_window : 0;
    rm.use_imp = a.imp_rows != nullptr && a.idx == nullptr;
    rm.n_sink = a.dense ? 0 : min(a.sinks, L);
    rm.w_begin = a.dense ? 0 : max(rm.n_sink, L - a.recent);
    int n_list = 0;
    if (!a.dense) {
        const int known = a.known_cnt[ll * ut.n_seq + s];
        n_list = a.idx ? a.cnt[au.list_l] : (known >= 0 ? known : state_cnt[au.list_c]);
        n_list = max(0, min(n_list, gm.idx_cap));
    }
    rm.n_list = n_list;
    rm.list = a.idx ? a.idx + (size_t)au.list_l * gm.idx_cap : state_idx + au.list_c * gm.idx_cap;
    const int n_rows = a.dense ? L : rm.n_sink + n_list + (L - rm.w_begin);

    const int r_begin = (int)((long long)n_rows * split / a.nsplit);
    const int r_end = (int)((long long)n_rows * (split + 1) / a.nsplit);
    const int per_warp = (r_end - r_begin + kAttnWarps - 1) / kAttnWarps;
    const int wb = min(r_end, r_begin + warp * per_warp), we = min(r_end, wb + per_warp);

    // this lane's 4 channels of each query head, pre-scaled so that logits are in base-2 units
    const float qscale = a.sm_scale * kLog2e;
    float q[G][4];
    const T* qbase = reinterpret_cast<const T*>(a.q) + ((size_t)(ll * ut.n_seq + s) * gm.Hq + h * g) * D;
#pragma unroll
    for (int u = 0; u < G; ++u) {
        if (u < g) {
            RowVec<T> rv;
            rv.load(qbase + u * D, lane);
            rv.get(q[u]);
        } else {
            q[u][0] = q[u][1] = q[u][2] = q[u][3] = 0.f;
        }
    }

    float m[G], l[G], acc[G][4];
#pragma unroll
    for (int u = 0; u < G; ++u) {
        m[u] = -INFINITY, l[u] = 0.f;
        acc[u][0] = acc[u][1] = acc[u][2] = acc[u][3] = 0.f;
    }

    // the unit's rows in the cache and in the optional copies, indexed by a row reference's source
    const T* src_base[3] = {kv + au.kv_c * gm.max_seq_len * 2 * D,
                            reinterpret_cast<const T*>(a.res_rows) + au.kv_c * (size_t)(a.res_sinks + a.res_window) * 2 * D,
                            reinterpret_cast<const T*>(a.imp_rows) + au.list_c * (size_t)gm.idx_cap * 2 * D};
    bool any_bad = false;
    for (int r0 = wb; r0 < we; r0 += kRowsPerIter) {
        RowVec<T> kr[kRowsPerIter], vr[kRowsPerIter];
        bool valid[kRowsPerIter];
#pragma unroll
        for (int i = 0; i < kRowsPerIter; ++i) {
            bool bad = false;
            valid[i] = r0 + i < we;
            int t = valid[i] ? rm.token(r0 + i, bad) : 0;
            if (bad) valid[i] = false, any_bad = true;
            const int which = t >> kRowSrcShift;
            const T* row = (which == 0 ? src_base[0] : which == 1 ? src_base[1] : src_base[2]) + (size_t)(t & kRowIdxMask) * 2 * D;
            kr[i].load(row, lane);
            vr[i].load(row + D, lane);
        }
        float x[kRowsPerIter][G];
#pragma unroll
        for (int i = 0; i < kRowsPerIter; ++i) {
            float kf[4];
            kr[i].get(kf);
#pragma unroll
            for (int u = 0; u < G; ++u) {
                float p = q[u][0] * kf[0];
                p = fmaf(q[u][1], kf[1], p);
                p = fmaf(q[u][2], kf[2], p);
                p = fmaf(q[u][3], kf[3], p);
                p = warp_sum(p);
                x[i][u] = valid[i] ? p * qscale : -INFINITY;
            }
        }
#pragma unroll
        for (int u = 0; u < G; ++u) {
            float mn = m[u];
#pragma unroll
            for (int i = 0; i < kRowsPerIter; ++i) mn = fmaxf(mn, x[i][u]);
            const float ms = mn == -INFINITY ? 0.f : mn;
            const float corr = exp2f(m[u] - ms);
            m[u] = mn;
            l[u] *= corr;
            acc[u][0] *= corr, acc[u][1] *= corr, acc[u][2] *= corr, acc[u][3] *= corr;
#pragma unroll
            for (int i = 0; i < kRowsPerIter; ++i) {
                const float p = exp2f(x[i][u] - ms);
                float vf[4];
                vr[i].get(vf);
                l[u] += p;
                acc[u][0] = fmaf(p, vf[0], acc[u][0]);
                acc[u][1] = fmaf(p, vf[1], acc[u][1]);
                acc[u][2] = fmaf(p, vf[2], acc[u][2]);
                acc[u][3] = fmaf(p, vf[3], acc[u][3]);
            }
        }
    }
    if (any_bad && lane == 0) atomicExch(status, kStatusBadIndex);

    // ---- combine the block's warps (fixed order) and publish the split's partial ------------------
#pragma unroll
    for (int u = 0; u < G; ++u) {
        if (lane == 0) sh_m[warp][u] = m[u], sh_l[warp][u] = l[u];
        *reinterpret_cast<float4*>(&sh_o[warp][u][lane * 4]) = make_float4(acc[u][0], acc[u][1], acc[u][2], acc[u][3]);
    }
    __syncthreads();
    SplitSink sink{part_o, part_ml, counters, a.out, a.lse, (size_t)(ll * ut.n_seq + s) * gm.Hq + h * g, lu, split, a.nsplit};
    for (int u = 0; u < g; ++u) {
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kAttnWarps; ++w) M = fmaxf(M, sh_m[w][u]);
        const float Ms = M == -INFINITY ? 0.f : M;
        float lsum = 0.f, o = 0.f;
#pragma unroll
        for (int w = 0; w < kAttnWarps; ++w) {
            const float e = exp2f(sh_m[w][u] - Ms);
            lsum += sh_l[w][u] * e;
            o += sh_o[w][u][tid] * e;
        }
        sink.publish(u, M, lsum, o);
    }
    sink.merge_if_last(g, &sh_last);
}

// ---------------------------------------------------------------------------------------------------
// bf16 path: tensor-core tiles of (16 gathered tokens) x (query heads padded to 8).
//
// Each warp owns a ring of shared-memory stages; a stage holds 16 gathered K|V row pairs (512 B each,
// copied by the whole warp with 16-byte cp.async) at a 512-byte pitch with the 16-byte chunks of a row
// permuted by the row number, so that ldmatrix reads are bank-conflict free.  S = K Q^T (tokens x heads) and O^T += V^T P^T (channels x heads) run on
// mma.sync m16n8k16 (bf16 in, fp32 accumulate) with the GQA group's heads as the N = 8 columns --
// the one place where batch x group makes the contraction a real dense tile; P is split into a bf16
// high and low part (two MMAs) so that the probabilities keep ~16 bits, and reaches the B operand
// through movmatrix transposes.  24 MMAs per 16 tokens.

#ifdef TB_PHASE_TIMING
__device__ unsigned long long g_attn_phase_ns[2][16];
__device__ unsigned long long g_attn_blk_ns[2][12][1024];   // per block of the last launches on an even and on an odd layer: every stamp
__device__ long long g_attn_blk_clk[2][12][1024];            // the same stamps in SM cycles (differences inside one block only)
#define attn_stamp(i) attn_stamp_((i), ut.layer_begin & 1)
__device__ __forceinline__ void attn_stamp_(int i, int par) {
    if (threadIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        const int b = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
        if (b < 1024 && i < 12) g_attn_blk_ns[par][i][b] = t;
        if (b < 1024 && i < 12) g_attn_blk_clk[par][i][b] = clock64();
    }
    if (threadIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && (blockIdx.x == 0 || blockIdx.x == gridDim.x - 1)) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        g_attn_phase_ns[blockIdx.x == 0 ? 0 : 1][i] = t;
    }
}
extern "C" int tb_debug_attn_phase_ns(unsigned long long* out) {
    return (int)cudaMemcpyFromSymbol(out, g_attn_phase_ns, sizeof(g_attn_phase_ns));
}
extern "C" int tb_debug_attn_blocks_clk(long long* out) {
    return (int)cudaMemcpyFromSymbol(out, g_attn_blk_clk, sizeof(g_attn_blk_clk));
}
extern "C" int tb_debug_attn_blocks_ns(unsigned long long* out) {
    return (int)cudaMemcpyFromSymbol(out, g_attn_blk_ns, sizeof(g_attn_blk_ns));
}
#else
#define attn_stamp(i) ((void)0)
#endif

constexpr int kTileTok = 16;
// A stage holds 16 K|V rows at a pitch of 512 bytes; the 16-byte chunk c of row i sits at chunk
// c ^ (i & 7), so the eight rows of an ldmatrix tile hit eight different bank groups without padding.
// Every 128-byte line of a source row therefore lands in one 128-byte line of shared memory and the
// copy of a row is four full-line requests.  (With a padded pitch of 528 a source line straddled two
// destination lines and was split: invisible in HBM, but over the host link, where every request is
// its own read transaction, it halved the throughput of a cache in page-locked host memory.)
constexpr int kRowPitch = 512;
constexpr int kStageBytes = kTileTok * kRowPitch;     // 8192

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float* d, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// Transposes an 8x8 matrix of 16-bit elements held one 32-bit pair per lane.
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Shared memory behind the warps' stages for the merge inside a cluster of C blocks: the accumulator slices this
// block owns from every block ([slices per owner][C][32 lanes] float4) and every block's (m, l) ([C][4] float4).
static inline size_t cluster_merge_bytes(int C) { return (size_t)((8 + C - 1) / C) * C * 32 * 16 + (size_t)C * 4 * 16; }

// NW warps per block.  With a.cluster_merge the blocks of one (sequence, KV head) form a thread-block
// cluster (one block per split): the warps of a block fold their results through shared memory, the blocks exchange
// channel slices of theirs through distributed shared memory, one cluster barrier, and every block merges
// and writes the slices it owns -- no partials in global memory, no last-block round trips.  Without it (more splits than a cluster holds) the splits
// go through the global workspace and the last block to arrive merges them (NW must be 4 then).
// kSources: the resident sink / window copies or the Important buffer are bound and a row reference names
// its source; without them (the usual case) the gather carries no trace of the option.
template <int NW, int kMmaStages, bool kSources = false>
__global__ void __launch_bounds__(NW * 32) attn_mma_kernel(Geom gm, UnitTable ut, AttnArgs a, const __nv_bfloat16* __restrict__ kv,
                                                           const int32_t* __restrict__ state_idx,
                                                           const int32_t* __restrict__ state_cnt, float* __restrict__ part_o,
                                                           float* __restrict__ part_ml, uint32_t* __restrict__ counters,
                                                           int32_t* __restrict__ status) {
    constexpr int D = 128;
    extern __shared__ __align__(128) unsigned char smem_dyn[];
    __shared__ int sh_last;

    attn_stamp(0);
    // Dependency wait (see pdl_wait).  When the lists or cache rows may come from the predecessor: before the
    // first read of anything it may have written -- the list entries, or already the lengths and list counts when
    // those are read on the device; what comes from the kernel parameters alone (row map, split, addresses) runs
    // beside the predecessor's tail.  Otherwise only before the queries are read, so that the list fetch and the
    // first gathers overlap the predecessor as well.  The own dependent is released at the start in that case,
    // else right after the wait (see tb_api.cu on why not before).
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gid = lane >> 2, tig = lane & 3;
    const int split = blockIdx.x, h = blockIdx.y;
    const int ll = ut.layer_count == 1 ? 0 : blockIdx.z / ut.n_seq, s = blockIdx.z - ll * ut.n_seq;
    bool waited = a.early_ok != 0;
    if (waited) pdl_launch_dependents();
    if (!waited && (ut.use_dev_len || (!a.dense && (a.idx != nullptr || a.known_cnt[ll * ut.n_seq + s] < 0)))) {
        pdl_wait();
        pdl_launch_dependents();
        waited = true;
    }
    const int L = unit_len(gm, ut, ll, s);
    const int g = gm.ga;
    const AttnUnit au(gm, ut, ll, s, h);
    const int lu = au.lu;

    RowMap<kSources> rm;
    rm.L = L, rm.dense = a.dense;
    rm.res_sinks = a.res_rows ? a.res_sinks : 0, rm.res_window = a.res_rows ? a.res_window : 0;
    rm.use_imp = a.imp_rows != nullptr && a.idx == nullptr;
    rm.n_sink = a.dense ? 0 : min(a.sinks, L);
    rm.w_begin = a.dense ? 0 : max(rm.n_sink, L - a.recent);
    int n_list = 0;
    if (!a.dense) {
        const int known = a.known_cnt[ll * ut.n_seq + s];
        n_list = a.idx ? a.cnt[au.list_l] : (known >= 0 ? known : state_cnt[au.list_c]);
        n_list = max(0, min(n_list, gm.idx_cap));
    }
    rm.n_list = n_list;
    rm.list = a.idx ? a.idx + (size_t)au.list_l * gm.idx_cap : state_idx + au.list_c * gm.idx_cap;
    const int n_rows = a.dense ? L : rm.n_sink + n_list + (L - rm.w_begin);

    // rows of this split, dealt to the warps in whole tiles of 16
    // (32-bit arithmetic whenever it is exact: a 64-bit division costs hundreds of cycles in a prologue that is
    // on the critical path of the cluster that starts late)
    const bool small = n_rows < (1 << 24);             // nsplit <= 32
    const int r_begin = small ? (int)((unsigned)n_rows * (unsigned)split / (unsigned)a.nsplit) : (int)((long long)n_rows * split / a.nsplit);
    const int r_end = small ? (int)((unsigned)n_rows * (unsigned)(split + 1) / (unsigned)a.nsplit) : (int)((long long)n_rows * (split + 1) / a.nsplit);
    const int tiles_all = (r_end - r_begin + kTileTok - 1) / kTileTok;
    // dealt evenly: no warp gets more than one tile above another (a tile beyond a warp's stages waits for
    // a stage to drain and then for its rows, a whole memory latency)
    const int tiles_lo = tiles_all / NW, tiles_rem = tiles_all % NW;
    const int wb = min(r_end, r_begin + (warp * tiles_lo + min(warp, tiles_rem)) * kTileTok);
    const int we = min(r_end, wb + (tiles_lo + (warp < tiles_rem ? 1 : 0)) * kTileTok);
    const int n_tiles = (we - wb + kTileTok - 1) / kTileTok;

    unsigned char* my_stage = smem_dyn + (size_t)warp * kMmaStages * kStageBytes;
    // the unit's rows in the cache and in the optional copies (see RowMap), 512 bytes per K|V row pair
    const unsigned char* kv_unit = reinterpret_cast<const unsigned char*>(kv) + au.kv_c * gm.max_seq_len * 2 * D * 2;
    const unsigned char* res_unit = reinterpret_cast<const unsigned char*>(a.res_rows) + au.kv_c * (size_t)(a.res_sinks + a.res_window) * 2 * D * 2;
    const unsigned char* imp_unit = reinterpret_cast<const unsigned char*>(a.imp_rows) + au.list_c * (size_t)gm.idx_cap * 2 * D * 2;

    if (!waited) {
        pdl_wait();
        pdl_launch_dependents();
    }
    bool any_bad = false;
    // Gather of one tile: the whole warp copies each 512-byte K|V row with one 16-byte cp.async per
    // lane (one warp instruction per row; the per-row TMA bulk copies this replaces queued up at the
    // SM's single TMA port and took ~2 us to issue).  Rows past the end of the warp's range repeat
    // its last row (their probabilities are masked to zero), so a stage always holds finite numbers.
    // Every tile slot commits exactly one group, empty or not, so "all but the newest
    // kMmaStages-1 groups are complete" always means "the tile about to be used has landed".
    const uint32_t stage_u32 = smem_u32(my_stage);
    auto issue_token = [&](int tile, int t) {     // t: lane i < 16 holds the token of row i
        const uint32_t dst = stage_u32 + (tile % kMmaStages) * kStageBytes;
#pragma unroll
        for (int i = 0; i < kTileTok; ++i) {
            const int ti = __shfl_sync(0xffffffffu, t, i);
            const unsigned char* src = kv_unit;
            int row = ti;
            if constexpr (kSources) {
                const int which = ti >> kRowSrcShift;
                src = which == 0 ? kv_unit : which == 1 ? res_unit : imp_unit;
                row = ti & kRowIdxMask;
            }
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + i * kRowPitch + ((lane ^ (i & 7)) << 4)),
                         "l"(src + lane * 16 + (size_t)row * 512) : "memory");
        }
    };
    auto commit = [&]() { asm volatile("cp.async.commit_group;" ::: "memory"); };
    attn_stamp(1);
    // Lane i < 16 keeps, one bit per tile from the current one on, whether its row of that tile is a
    // bad list entry (outside the cached tokens): known when the tile's rows are issued, used when
    // the tile is consumed.  (Reading the entry a second time at consumption, as an earlier version did,
    // cost 5-8% of the kernel; fetching the entries one tile ahead of their issue cost 4% on
    // bandwidth-saturated launches and is not done.)
    uint32_t bad_bits = 0;
    auto tokens_of = [&](int tile) {                // -1 = bad entry
        return (tile < n_tiles && lane < kTileTok) ? rm.token_or_neg(min(wb + tile * kTileTok + lane, we - 1)) : 0;
    };
    {   // the first tiles' list entries are fetched together (one memory round trip), then their rows
        int tok[kMmaStages];
#pragma unroll
        for (int t = 0; t < kMmaStages; ++t) tok[t] = tokens_of(t);
#pragma unroll
        for (int t = 0; t < kMmaStages; ++t) {
            bad_bits |= (uint32_t)(tok[t] < 0) << t;
            if (t < n_tiles) issue_token(t, max(tok[t], 0));
            commit();
        }
    }
    attn_stamp(2);

    if (a.early_ok) pdl_wait();                        // the queries are this call's input
    attn_stamp(7);
    // Q^T as the B operand of S = K Q^T: k = channels, n = query heads (gid; heads >= g are zero padding)
    uint32_t qb[8][2];
    {
        const __nv_bfloat16* qbase = reinterpret_cast<const __nv_bfloat16*>(a.q) + ((size_t)(ll * ut.n_seq + s) * gm.Hq + h * g) * D;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            qb[ks][0] = qb[ks][1] = 0u;
            if (gid < g) {
                qb[ks][0] = __ldg(reinterpret_cast<const uint32_t*>(qbase + gid * D + ks * 16 + tig * 2));
                qb[ks][1] = __ldg(reinterpret_cast<const uint32_t*>(qbase + gid * D + ks * 16 + 8 + tig * 2));
            }
        }
    }
    const float qscale = a.sm_scale * kLog2e;
#ifdef TB_PHASE_TIMING
    if (qb[7][1] == 0x7fc1dead) any_bad = true;            // the stamp below waits for the queries
    attn_stamp(8);
#endif

    // O^T accumulators: 8 tiles of (16 channels x 8 heads); this thread: channels mt*16 + gid (+8),
    // heads 2*tig and 2*tig+1 -- the same two heads as its columns of S.
    float o[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};   // heads 2*tig, 2*tig+1; l over this thread's tokens

    // per-lane ldmatrix row addresses inside a stage
    const int mi = lane >> 3, r8 = lane & 7;
    // row offset + swizzled chunk: chunk 2 ks + (mi >> 1) of the K half, 16 + 2 mt + (mi & 1) of the V half,
    // each xor (row & 7) = r8; the k-step / channel-tile part is xored in at the use
    const uint32_t k_row_off = ((mi & 1) * 8 + r8) * kRowPitch, k_swz = (uint32_t)((mi >> 1) ^ r8) << 4;        // ^ ks * 32   (A of S = K Q^T)
    const uint32_t v_row_off = ((mi >> 1) * 8 + r8) * kRowPitch + 256, v_swz = (uint32_t)((mi & 1) ^ r8) << 4;  // ^ mt * 32   (A of O^T = V^T P^T)

    // A warp whose rows all fit its stages (two or three tiles: the latency-bound launches, where a block holds a
    // few hundred rows) takes its first two tiles as one 32-token tile: the two S = K Q^T chains interleave, there
    // is one softmax update instead of two, and every O^T accumulator gets four MMAs behind two loads.  One tile
    // at a time is a chain of ~1500 dependent cycles per tile with nothing to overlap it in the warp.
    int tile_first = 0;
    if (n_tiles >= 2 && n_tiles <= kMmaStages) {
        const bool inA = lane < kTileTok && wb + lane < we, inB = lane < kTileTok && wb + kTileTok + lane < we;
        const bool badA = inA && (bad_bits & 1u), badB = inB && (bad_bits & 2u);
        any_bad |= badA | badB;
        bad_bits >>= 2;
        const unsigned vmA = __ballot_sync(0xffffffffu, inA && !badA), vmB = __ballot_sync(0xffffffffu, inB && !badB);
        asm volatile("cp.async.wait_group %0;" ::"n"(kMmaStages - 2) : "memory");
        __syncwarp();
        attn_stamp(3);
        const uint32_t sA = stage_u32, sB = stage_u32 + kStageBytes;
        float ca[4] = {0.f, 0.f, 0.f, 0.f}, cb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            uint32_t a0, a1, a2, a3, b0, b1, b2, b3;
            ldmatrix_x4(sA + k_row_off + ((ks * 32) ^ k_swz), a0, a1, a2, a3);
            ldmatrix_x4(sB + k_row_off + ((ks * 32) ^ k_swz), b0, b1, b2, b3);
            mma_bf16(ca, a0, a1, a2, a3, qb[ks][0], qb[ks][1]);
            mma_bf16(cb, b0, b1, b2, b3, qb[ks][0], qb[ks][1]);
        }
        const bool vA0 = (vmA >> gid) & 1u, vA1 = (vmA >> (gid + 8)) & 1u, vB0 = (vmB >> gid) & 1u, vB1 = (vmB >> (gid + 8)) & 1u;
        float x[8];
        x[0] = vA0 ? ca[0] * qscale : -INFINITY, x[1] = vA0 ? ca[1] * qscale : -INFINITY;
        x[2] = vA1 ? ca[2] * qscale : -INFINITY, x[3] = vA1 ? ca[3] * qscale : -INFINITY;
        x[4] = vB0 ? cb[0] * qscale : -INFINITY, x[5] = vB0 ? cb[1] * qscale : -INFINITY;
        x[6] = vB1 ? cb[2] * qscale : -INFINITY, x[7] = vB1 ? cb[3] * qscale : -INFINITY;
        float tmax[2] = {fmaxf(fmaxf(x[0], x[2]), fmaxf(x[4], x[6])), fmaxf(fmaxf(x[1], x[3]), fmaxf(x[5], x[7]))};
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) {
            tmax[0] = fmaxf(tmax[0], __shfl_xor_sync(0xffffffffu, tmax[0], off));
            tmax[1] = fmaxf(tmax[1], __shfl_xor_sync(0xffffffffu, tmax[1], off));
        }
        // these are the warp's first rows: nothing accumulated yet to rescale
        m_run[0] = tmax[0], m_run[1] = tmax[1];
        const float ms0 = tmax[0] == -INFINITY ? 0.f : tmax[0], ms1 = tmax[1] == -INFINITY ? 0.f : tmax[1];
        float p[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) p[i] = exp2f(x[i] - ((i & 1) ? ms1 : ms0));
        l_run[0] = (p[0] + p[2]) + (p[4] + p[6]);
        l_run[1] = (p[1] + p[3]) + (p[5] + p[7]);
        float ph[8], pl[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            ph[i] = __bfloat162float(__float2bfloat16_rn(p[i]));
            pl[i] = p[i] - ph[i];
        }
        const uint32_t hA0 = movmatrix_trans(pack_bf16(ph[0], ph[1])), hA1 = movmatrix_trans(pack_bf16(ph[2], ph[3]));
        const uint32_t lA0 = movmatrix_trans(pack_bf16(pl[0], pl[1])), lA1 = movmatrix_trans(pack_bf16(pl[2], pl[3]));
        const uint32_t hB0 = movmatrix_trans(pack_bf16(ph[4], ph[5])), hB1 = movmatrix_trans(pack_bf16(ph[6], ph[7]));
        const uint32_t lB0 = movmatrix_trans(pack_bf16(pl[4], pl[5])), lB1 = movmatrix_trans(pack_bf16(pl[6], pl[7]));
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) {
            uint32_t a0, a1, a2, a3, b0, b1, b2, b3;
            ldmatrix_x4_trans(sA + v_row_off + ((mt * 32) ^ v_swz), a0, a1, a2, a3);
            ldmatrix_x4_trans(sB + v_row_off + ((mt * 32) ^ v_swz), b0, b1, b2, b3);
            mma_bf16(o[mt], a0, a1, a2, a3, hA0, hA1);
            mma_bf16(o[mt], a0, a1, a2, a3, lA0, lA1);
            mma_bf16(o[mt], b0, b1, b2, b3, hB0, hB1);
            mma_bf16(o[mt], b0, b1, b2, b3, lB0, lB1);
        }
        __syncwarp();
        commit(), commit();                            // the two tile slots' groups of the loop below
        tile_first = 2;
    }
    for (int tile = tile_first; tile < n_tiles; ++tile) {
        const int st = tile % kMmaStages;
        const int r0 = wb + tile * kTileTok;
        // validity of the tile's 16 rows (past-the-end and out-of-range list entries are masked)
        const bool in_range = lane < kTileTok && r0 + lane < we;
        const bool bad = in_range && (bad_bits & 1u);
        any_bad |= bad;
        bad_bits >>= 1;
        const unsigned vmask = __ballot_sync(0xffffffffu, in_range && !bad);
        asm volatile("cp.async.wait_group %0;" ::"n"(kMmaStages - 1) : "memory");
        __syncwarp();                                  // every lane's copies of this tile are visible to the warp
        if (tile == 0) attn_stamp(3);
        const uint32_t sb = stage_u32 + st * kStageBytes;

        // S[token][head]: this thread holds tokens gid (c0,c1) and gid+8 (c2,c3), heads 2*tig, 2*tig+1
        float sc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            uint32_t a0, a1, a2, a3;
            ldmatrix_x4(sb + k_row_off + ((ks * 32) ^ k_swz), a0, a1, a2, a3);
            mma_bf16(sc, a0, a1, a2, a3, qb[ks][0], qb[ks][1]);
        }
#ifdef TB_PHASE_TIMING
        if (tile == 0) { if (sc[0] == 1.2345e33f) any_bad = true; attn_stamp(9); }
#endif
        const bool v0 = (vmask >> gid) & 1u, v1 = (vmask >> (gid + 8)) & 1u;
        float x[4];
        x[0] = v0 ? sc[0] * qscale : -INFINITY, x[1] = v0 ? sc[1] * qscale : -INFINITY;
        x[2] = v1 ? sc[2] * qscale : -INFINITY, x[3] = v1 ? sc[3] * qscale : -INFINITY;
        float tmax[2] = {fmaxf(x[0], x[2]), fmaxf(x[1], x[3])};
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) {       // over the 8 token rows held by lanes with the same tig
            tmax[0] = fmaxf(tmax[0], __shfl_xor_sync(0xffffffffu, tmax[0], off));
            tmax[1] = fmaxf(tmax[1], __shfl_xor_sync(0xffffffffu, tmax[1], off));
        }
        float corr[2], ms[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const float m_new = fmaxf(m_run[e], tmax[e]);
            ms[e] = m_new == -INFINITY ? 0.f : m_new;
            corr[e] = exp2f(m_run[e] - ms[e]);
            m_run[e] = m_new;
        }
        float p[4];
        p[0] = exp2f(x[0] - ms[0]), p[1] = exp2f(x[1] - ms[1]), p[2] = exp2f(x[2] - ms[0]), p[3] = exp2f(x[3] - ms[1]);
        l_run[0] = l_run[0] * corr[0] + p[0] + p[2];
        l_run[1] = l_run[1] * corr[1] + p[1] + p[3];
        if (__any_sync(0xffffffffu, corr[0] != 1.f || corr[1] != 1.f)) {
#pragma unroll
            for (int i = 0; i < 8; ++i) o[i][0] *= corr[0], o[i][1] *= corr[1], o[i][2] *= corr[0], o[i][3] *= corr[1];
        }
        // P = P_hi + P_lo in bf16, transposed into the B operand (k = tokens, n = heads)
        float ph[4], pl[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            ph[i] = __bfloat162float(__float2bfloat16_rn(p[i]));
            pl[i] = p[i] - ph[i];
        }
        const uint32_t bh0 = movmatrix_trans(pack_bf16(ph[0], ph[1])), bh1 = movmatrix_trans(pack_bf16(ph[2], ph[3]));
        const uint32_t bl0 = movmatrix_trans(pack_bf16(pl[0], pl[1])), bl1 = movmatrix_trans(pack_bf16(pl[2], pl[3]));
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) {
            uint32_t a0, a1, a2, a3;
            ldmatrix_x4_trans(sb + v_row_off + ((mt * 32) ^ v_swz), a0, a1, a2, a3);
            mma_bf16(o[mt], a0, a1, a2, a3, bh0, bh1);
            mma_bf16(o[mt], a0, a1, a2, a3, bl0, bl1);
        }
#ifdef TB_PHASE_TIMING
        if (tile == 0) { if (o[7][3] == 1.2345e33f) any_bad = true; attn_stamp(10); }
#endif
        __syncwarp();                                  // the warp is done reading this stage
        if (tile + kMmaStages < n_tiles) {
            const int t = tokens_of(tile + kMmaStages);
            bad_bits |= (uint32_t)(t < 0) << (kMmaStages - 1);         // bit k is tile + 1 + k now
            issue_token(tile + kMmaStages, max(t, 0));
        }
        commit();
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (any_bad && lane < kTileTok) atomicExch(status, kStatusBadIndex);

    // ---- the warps' results become the block's, the blocks' the problem's -------------------------------
    attn_stamp(4);
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
        l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], off);
        l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], off);
    }
    __syncwarp();
    const size_t hq0 = (size_t)(ll * ut.n_seq + s) * gm.Hq + h * g;
    // Every warp parks its accumulators in its own (drained) stages, lane by lane in the MMA layout -- float4
    // number mt * 32 + lane is accumulator tile mt (16 channels) of that lane, number 256 + lane its (m, l) of
    // heads 2 tig and 2 tig + 1 -- so that nothing is transposed and every access is a conflict-free 16 bytes.
    // After one block barrier a thread owns one (tile, lane) slot: it folds the NW warps' values of that slot,
    // all loads independent of one another, and holds a piece of the block's result in registers.
    // (Measured alternatives, all within 0.03 us per launch of this one: a binary tree over the warps with a
    // named barrier per pair; two barriers with the weights computed once.  Parking only the lanes of real heads
    // when the group has at most four -- half the shared-memory traffic, 16 shuffles -- was 0.5 us slower.)
    {
        float4* tbuf = reinterpret_cast<float4*>(my_stage);
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) tbuf[mt * 32 + lane] = make_float4(o[mt][0], o[mt][1], o[mt][2], o[mt][3]);
        tbuf[8 * 32 + lane] = make_float4(m_run[0], l_run[0], m_run[1], l_run[1]);
    }
    __syncthreads();
    auto warp_buf = [&](int w) { return reinterpret_cast<const float4*>(smem_dyn + (size_t)w * kMmaStages * kStageBytes); };
    // block result of slot (mt, ln): acc = (head 2tg ch, head 2tg+1 ch, head 2tg ch+8, head 2tg+1 ch+8), ch = mt*16 + ln/4
    auto fold_slot = [&](int mt, int ln, float4& acc, float4& stat) {
        float4 q[NW];
#pragma unroll
        for (int w = 0; w < NW; ++w) q[w] = warp_buf(w)[8 * 32 + ln];
        float M0 = -INFINITY, M1 = -INFINITY;
#pragma unroll
        for (int w = 0; w < NW; ++w) M0 = fmaxf(M0, q[w].x), M1 = fmaxf(M1, q[w].z);
        const float M0s = M0 == -INFINITY ? 0.f : M0, M1s = M1 == -INFINITY ? 0.f : M1;
        float L0 = 0.f, L1 = 0.f;
        acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            const float e0 = exp2f(q[w].x - M0s), e1 = exp2f(q[w].z - M1s);
            L0 = fmaf(q[w].y, e0, L0), L1 = fmaf(q[w].w, e1, L1);
            const float4 v = warp_buf(w)[mt * 32 + ln];
            acc.x = fmaf(v.x, e0, acc.x), acc.y = fmaf(v.y, e1, acc.y), acc.z = fmaf(v.z, e0, acc.z), acc.w = fmaf(v.w, e1, acc.w);
        }
        stat = make_float4(M0, L0, M1, L1);
    };
    attn_stamp(5);
    if (a.cluster_merge) {
        // Merge of the blocks' results inside the cluster, sliced by channels: the 128 channels are eight slices
        // of 16 (one accumulator tile each), slice j belongs to block j mod C.  The thread that folded a slot sends
        // it to the slice's owner, the block's (m, l) go to every owner -- 4.5 KB per block in all --, one cluster
        // barrier, and every owner merges its 16 channels of all heads from the C partials (blocks in rank order:
        // bit-reproducible) and writes them out.  No single merging block: the work behind the barrier is C terms
        // per output, not C x 8, and their loads are issued together.
        cg::cluster_group cluster = cg::this_cluster();
        const int rank = (int)cluster.block_rank(), C = (int)cluster.num_blocks();
        const int T = (8 + C - 1) / C;                               // slices per owner
        float4* area = reinterpret_cast<float4*>(smem_dyn + (size_t)NW * kMmaStages * kStageBytes);   // [T][C][32 lanes]
        float4* ml = area + (size_t)T * C * 32;                      // [C][4]: (m, l) of heads 2 tig, 2 tig + 1
        // writes one merged piece: (acc, sums ls0 / ls1, maxima M0 / M1) of heads 2 tg, 2 tg + 1 at channels ch, ch + 8
        auto write_piece = [&](int tg, int ch, const float4& acc, float M0, float ls0, float M1, float ls1) {
            const int u0 = 2 * tg, u1 = u0 + 1;
            if (u0 < g) {
                a.out[(hq0 + u0) * D + ch] = acc.x / ls0, a.out[(hq0 + u0) * D + ch + 8] = acc.z / ls0;
                if (a.lse && ch == 0) a.lse[hq0 + u0] = (M0 + log2f(ls0)) * kLn2;
            }
            if (u1 < g) {
                a.out[(hq0 + u1) * D + ch] = acc.y / ls1, a.out[(hq0 + u1) * D + ch + 8] = acc.w / ls1;
                if (a.lse && ch == 0) a.lse[hq0 + u1] = (M1 + log2f(ls1)) * kLn2;
            }
        };
        if (C == 1) {                                                // the block's result is the problem's
            for (int slot = tid; slot < 256; slot += NW * 32) {
                const int mt = slot >> 5, ln = slot & 31;
                float4 acc, stat;
                fold_slot(mt, ln, acc, stat);
                write_piece(ln & 3, mt * 16 + (ln >> 2), acc, stat.x, stat.y, stat.z, stat.w);
            }
            attn_stamp(6);
            return;
        }
        for (int slot = tid; slot < 256; slot += NW * 32) {
            const int mt = slot >> 5, ln = slot & 31;
            float4 acc, stat;
            fold_slot(mt, ln, acc, stat);
            cluster.map_shared_rank(area, mt % C)[((mt / C) * C + rank) * 32 + ln] = acc;
            if (mt == 0 && (ln >> 2) < C) cluster.map_shared_rank(ml, ln >> 2)[rank * 4 + (ln & 3)] = stat;
        }
        cluster.sync();
        // the owners' merge, unrolled to a bound on the cluster size so that the loads go out together
        auto owner_merge = [&](auto bound) {
            constexpr int kC = decltype(bound)::value;
            for (int i = tid; i < T * 32; i += NW * 32) {
                const int ts = i >> 5, ln = i & 31, tg = ln & 3;
                const int j = ts * C + rank;                         // the slice
                if (j >= 8) continue;
                float4 q[kC], v[kC];
#pragma unroll
                for (int r = 0; r < kC; ++r) {
                    q[r] = r < C ? ml[r * 4 + tg] : make_float4(-INFINITY, 0.f, -INFINITY, 0.f);
                    v[r] = r < C ? area[(ts * C + r) * 32 + ln] : make_float4(0.f, 0.f, 0.f, 0.f);
                }
                float M0 = -INFINITY, M1 = -INFINITY;
#pragma unroll
                for (int r = 0; r < kC; ++r) M0 = fmaxf(M0, q[r].x), M1 = fmaxf(M1, q[r].z);
                const float M0s = M0 == -INFINITY ? 0.f : M0, M1s = M1 == -INFINITY ? 0.f : M1;
                float ls0 = 0.f, ls1 = 0.f;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int r = 0; r < kC; ++r) {
                    const float e0 = exp2f(q[r].x - M0s), e1 = exp2f(q[r].z - M1s);
                    ls0 = fmaf(q[r].y, e0, ls0), ls1 = fmaf(q[r].w, e1, ls1);
                    acc.x = fmaf(v[r].x, e0, acc.x), acc.y = fmaf(v[r].y, e1, acc.y);
                    acc.z = fmaf(v[r].z, e0, acc.z), acc.w = fmaf(v[r].w, e1, acc.w);
                }
                write_piece(tg, j * 16 + (ln >> 2), acc, M0, ls0, M1, ls1);
            }
        };
        if (rank < 8) {
            if (C <= 4) owner_merge(std::integral_constant<int, 4>{});
            else if (C <= 9) owner_merge(std::integral_constant<int, 9>{});
            else owner_merge(std::integral_constant<int, kAttnMaxCluster>{});
        }
    } else if constexpr (NW == kAttnWarps) {
        // splits through the global workspace, merged by the last block to arrive
        SplitSink sink{part_o, part_ml, counters, a.out, a.lse, hq0, lu, split, a.nsplit};
        for (int slot = tid; slot < 256; slot += NW * 32) {
            const int mt = slot >> 5, ln = slot & 31, u0 = 2 * (ln & 3), ch = mt * 16 + (ln >> 2);
            float4 acc, stat;
            fold_slot(mt, ln, acc, stat);
            if (u0 < g) {
                sink.publish_at(u0, ch, acc.x), sink.publish_at(u0, ch + 8, acc.z);
                if (mt == 0 && ln < 4) sink.publish_stat(u0, stat.x, stat.y);
            }
            if (u0 + 1 < g) {
                sink.publish_at(u0 + 1, ch, acc.y), sink.publish_at(u0 + 1, ch + 8, acc.w);
                if (mt == 0 && ln < 4) sink.publish_stat(u0 + 1, stat.z, stat.w);
            }
        }
        sink.merge_if_last(g, &sh_last);
    }
    attn_stamp(6);
}

static int pick_nsplit(const tb_ctx* c, int units, int max_rows) {
    // about two blocks per SM and never a thin second wave: with 64 problems of 9.8K rows, 4 splits
    // (256 blocks) ran at 58.5 us, 5 at 63.6, 6 at 61.5, 7 (448 blocks, four more than fit at once) at 75.7,
    // 10 at 65.0
    int n = 2 * c->sm_count / units;
#ifdef TB_FORCE_NSPLIT
    n = TB_FORCE_NSPLIT;
#endif
    int by_rows = max_rows / 64;
    if (n > by_rows) n = by_rows;
    if (n > kMaxSplits) n = kMaxSplits;
    if (n < 1) n = 1;
    return n;
}

cudaError_t launch_attention(const tb_ctx* c, const UnitTable& ut, const AttnArgs& a_in, cudaStream_t s) {
    const Geom& gm = c->geom;
    AttnArgs a = a_in;
    int max_rows = 0;
    for (int i = 0; i < ut.layer_count * ut.n_seq; ++i) {
        int L = ut.len[i];
        int rows = a.dense ? L : (a.sinks < L ? a.sinks : L) + a.list_bound + a.recent;
        if (rows > L) rows = L;
        if (rows > max_rows) max_rows = rows;
    }
    const int units = ut.layer_count * ut.n_seq * gm.Ha;
    a.cluster_merge = 0;
    int nw = kAttnWarps;
    if (gm.dtype == TB_BF16) {
        static unsigned char seen[64];
        int* max_active = const_cast<tb_ctx*>(c)->attn_max_active;
        if (first_use_on_this_device(seen)) {
            cudaError_t e = cudaSuccess;
            auto prepare = [&](auto kernel, int max_kb, bool required) {
                cudaError_t r = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, max_kb * 1024);
                if (r == cudaSuccess) (void)cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
                if (r != cudaSuccess && required && e == cudaSuccess) e = r;
            };
            prepare(attn_mma_kernel<4, 2, false>, 113, true), prepare(attn_mma_kernel<4, 2, true>, 113, true);
            prepare(attn_mma_kernel<8, 2, false>, 220, true), prepare(attn_mma_kernel<8, 2, true>, 220, true);
            prepare(attn_mma_kernel<8, 3, false>, 220, true), prepare(attn_mma_kernel<8, 3, true>, 220, true);
            prepare(attn_mma_kernel<12, 2, false>, 224, false), prepare(attn_mma_kernel<12, 2, true>, 224, false);
            if (e != cudaSuccess) return e;
            (void)cudaGetLastError();
        }
        auto clusters_that_fit = [&](int csize) {     // how many clusters of `csize` 8-warp blocks run at once
            if (max_active[csize] == 0) {
                cudaLaunchConfig_t q = {};
                q.gridDim = dim3(csize, 1, 1), q.blockDim = dim3(256, 1, 1);
                const size_t mb = cluster_merge_bytes(csize);
                const bool three = csize <= 8 && 8 * 3 * kStageBytes + mb <= 220 * 1024;
                q.dynamicSmemBytes = 8 * (three ? 3 : 2) * kStageBytes + mb;
                cudaLaunchAttribute at[1];
                at[0].id = cudaLaunchAttributeClusterDimension;
                at[0].val.clusterDim.x = csize, at[0].val.clusterDim.y = 1, at[0].val.clusterDim.z = 1;
                q.attrs = at, q.numAttrs = 1;
                int n_clusters = 0;
                cudaError_t qe = three ? cudaOccupancyMaxActiveClusters(&n_clusters, attn_mma_kernel<8, 3>, &q)
                                       : cudaOccupancyMaxActiveClusters(&n_clusters, attn_mma_kernel<8, 2>, &q);
                if (qe != cudaSuccess) n_clusters = 0;
                (void)cudaGetLastError();
                max_active[csize] = n_clusters > 0 ? n_clusters : -1;
            }
            return max_active[csize];
        };
        // Few problems (one layer of a small batch): blocks of 8 warps, one per SM, and the largest
        // cluster (up to 16 blocks, sizes above 8 are non-portable) that the device can keep resident
        // for every problem at once; the splits merge inside the cluster.  Many problems: 4-warp
        // blocks, two per SM, clusters of up to 8; splits beyond that go through the global workspace.
        int n = 0;
        const int by_rows = max_rows / (8 * kTileTok) < 1 ? 1 : max_rows / (8 * kTileTok);
#ifdef TB_FORCE_ATTN_CLUSTER
        n = TB_FORCE_ATTN_CLUSTER;
#else
        // First choice: a launch that takes at most half of the SMs, so that the next layer's blocks
        // (programmatic dependent launch) can fetch their lists and first rows on free SMs while this
        // layer still computes (config 2, 8 problems: clusters of 9 run at 7.36 us per layer, the largest
        // that fits, 10, at 7.86, 8 at 8.65).  Otherwise the largest cluster that fits once.
        {
            const int cand = c->sm_count / (2 * units);
            if (cand >= 6 && cand <= 16 && cand <= by_rows && clusters_that_fit(cand) >= units) n = cand;
        }
        for (int cand = 16; cand >= 1 && !n; cand = cand > 8 ? cand - 2 : cand - 1)
            if (cand <= by_rows && units * cand <= c->sm_count && (cand <= 8 || clusters_that_fit(cand) >= units)) n = cand;
#endif
        if (n && max_rows / n <= 1024) {
            a.nsplit = n, nw = 8, a.cluster_merge = 1;
            // more than two tiles per warp would leave the third waiting for a free stage: 12 warps
            // per block when their rings and the merge area still fit the SM
            const int rows_per_block = (max_rows + n - 1) / n;
            if (rows_per_block > 8 * 2 * kTileTok && 12 * 2 * kStageBytes + cluster_merge_bytes(n) <= 224 * 1024) nw = 12;
        } else {
            a.nsplit = pick_nsplit(c, units, max_rows);
            // clusters only when the whole launch is resident at once: in multi-wave launches the
            // co-scheduling constraint costs more than the global merge (measured on the batch-8 workload)
            if (a.nsplit <= 8 && units * a.nsplit <= 2 * c->sm_count) a.cluster_merge = 1;
        }
    } else {
        a.nsplit = pick_nsplit(c, units, max_rows);
    }
    dim3 grid(a.nsplit, gm.Ha, ut.layer_count * ut.n_seq);
#define TB_ATTN(T, G)                                                                                                   \
    attn_kernel<T, G><<<grid, kAttnThreads, 0, s>>>(gm, ut, a, (const T*)c->kv, c->st.idx, c->st.cnt, c->wk.part_o,     \
                                                   c->wk.part_ml, c->st.attn_counter, c->st.status)
#define TB_ATTN_G(T)                                  \
    do {                                              \
        if (gm.ga == 1) TB_ATTN(T, 1);                \
        else if (gm.ga == 2) TB_ATTN(T, 2);           \
        else if (gm.ga <= 4) TB_ATTN(T, 4);           \
        else TB_ATTN(T, 8);                           \
    } while (0)
    if (gm.dtype == TB_BF16) {
        const size_t merge_bytes = a.cluster_merge ? cluster_merge_bytes(a.nsplit) : 0;
        // three stages per warp when the 8-warp block still fits the SM with them
        const int nst = (nw == 8 && 8 * 3 * kStageBytes + merge_bytes <= 220 * 1024 && a.nsplit <= 8) ? 3 : 2;
        size_t smem = (size_t)nw * nst * kStageBytes + merge_bytes;
        // The split count of the 4-warp launches is chosen for two blocks per SM; their 64 KB of stages would let
        // a third one in, and the block scheduler then loads some SMs with three blocks and leaves others with one
        // (batch 8 at 64K: 59 us per launch against 52.6).  Asking for a third of the SM's shared memory plus a
        // little keeps it at two.
        if (nw == 4 && smem < 76 * 1024) smem = 76 * 1024;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = grid;
        cfg.blockDim = dim3(nw * 32, 1, 1);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = s;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = a.cluster_merge ? a.nsplit : 1;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see pdl_wait()
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 2;
        const __nv_bfloat16* kvp = (const __nv_bfloat16*)c->kv;
        const bool sources = a.res_rows != nullptr || a.imp_rows != nullptr;
#define TB_MMA(NW_, ST_)                                                                                                          \
    (sources ? cudaLaunchKernelEx(&cfg, attn_mma_kernel<NW_, ST_, true>, gm, ut, a, kvp, (const int32_t*)c->st.idx,               \
                                  (const int32_t*)c->st.cnt, c->wk.part_o, c->wk.part_ml, c->st.attn_counter, c->st.status)       \
             : cudaLaunchKernelEx(&cfg, attn_mma_kernel<NW_, ST_, false>, gm, ut, a, kvp, (const int32_t*)c->st.idx,              \
                                  (const int32_t*)c->st.cnt, c->wk.part_o, c->wk.part_ml, c->st.attn_counter, c->st.status))
        if (nw == 12) return TB_MMA(12, 2);
        if (nw == 8 && nst == 3) return TB_MMA(8, 3);
        if (nw == 8) return TB_MMA(8, 2);
        return TB_MMA(4, 2);
#undef TB_MMA
    } else {
        TB_ATTN_G(float);
    }
#undef TB_ATTN_G
#undef TB_ATTN
    return cudaGetLastError();
}

}  // namespace tb

// ---------------------------------------------------------------------------------------------------
// Allocation-free attention entry point.
//
// Some callers cannot obtain device memory at the time they need attention: a plugin running inside
// a serving process whose memory pool is fixed at start-up, code on a latency-critical thread where a
// cudaMalloc (which may synchronise the whole device) is forbidden, or a host that has already handed
// all free HBM to its KV cache.  For them the split-K partials and arrival counters live in the
// file-scope device array below instead of a caller-provided workspace.  The array is part of the
// library image: every GPU that loads the library holds it (about 1 MB) until the process exits.

namespace {

constexpr int kStaticMaxQHeads = TB_STATIC_MAX_QHEADS;                 // n_seq * n_q_heads per call
constexpr size_t kStaticPartO = (size_t)kStaticMaxQHeads * tb::kMaxSplits * 128 * sizeof(float);
constexpr size_t kStaticPartMl = (size_t)kStaticMaxQHeads * tb::kMaxSplits * 2 * sizeof(float);
constexpr size_t kStaticCounters = (size_t)kStaticMaxQHeads * sizeof(uint32_t);   // one per (sequence, KV head) at most
constexpr size_t kStaticStatus = 256;
constexpr size_t kStaticBytes = kStaticPartO + kStaticPartMl + kStaticCounters + kStaticStatus;

// In host code this name is only a handle for the runtime, never a device address: the address a
// kernel may use comes from cudaGetSymbolAddress, asked once per device with that device current.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
unsigned char* g_scratch_addr[kMaxDevices];     // per device, filled at first use
int g_sm_count[kMaxDevices];

tb_status static_scratch_for_current_device(unsigned char** out, int* sm_count) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return TB_ERR_CUDA;
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return TB_ERR_CUDA;
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return TB_ERR_CUDA;
        if (cudaFuncSetAttribute(tb::attn_mma_kernel<4, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 113 * 1024) != cudaSuccess)
            return TB_ERR_CUDA;
        g_sm_count[dev] = sms;
        g_scratch_addr[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_scratch_addr[dev];
    *sm_count = g_sm_count[dev];
    return TB_OK;
}

}  // namespace

extern "C" tb_status tb_sparse_decode_attention_static(const void* kv_dev, int32_t kv_dtype, int32_t n_q_heads, int32_t n_kv_heads,
                                                       int32_t head_dim, int32_t max_seq_len, const int32_t* seq_slots,
                                                       const int32_t* seq_lens, int32_t n_seq, const void* q_dev,
                                                       const int32_t* idx_dev, const int32_t* cnt_dev, int32_t idx_stride,
                                                       int32_t sinks, int32_t recent, float sm_scale, float* out_dev,
                                                       float* lse_dev, void* stream) {
    using namespace tb;
    if (!kv_dev || !seq_lens || !q_dev || !out_dev || n_seq <= 0 || n_q_heads <= 0 || n_kv_heads <= 0 || max_seq_len <= 0)
        return TB_ERR_INVALID_ARG;
    if ((idx_dev == nullptr) != (cnt_dev == nullptr) || sinks < 0 || recent < 0) return TB_ERR_INVALID_ARG;
    if (idx_dev && idx_stride <= 0) return TB_ERR_INVALID_ARG;
    if (kv_dtype != TB_F32 && kv_dtype != TB_BF16) return TB_ERR_INVALID_ARG;
    if (n_q_heads % n_kv_heads != 0) return TB_ERR_INVALID_ARG;
    if (head_dim != 128 || n_q_heads / n_kv_heads > kMaxGroup) return TB_ERR_UNSUPPORTED;
    // the fixed scratch bounds the problem: refuse anything larger instead of overrunning it
    if (n_seq > kMaxLaunchSeq || (long long)n_seq * n_q_heads > kStaticMaxQHeads) return TB_ERR_CAPACITY;

    unsigned char* scratch = nullptr;
    int sm_count = 0;
    tb_status st = static_scratch_for_current_device(&scratch, &sm_count);
    if (st != TB_OK) return st;
    {
        // The scratch address belongs to the current device; a cache that lives on another GPU would be
        // read by kernels launched here.  (Page-locked host memory has no owning device and is accepted.)
        cudaPointerAttributes pa;
        int dev = -1;
        if (cudaPointerGetAttributes(&pa, kv_dev) != cudaSuccess || cudaGetDevice(&dev) != cudaSuccess) {
            (void)cudaGetLastError();
            return TB_ERR_INVALID_ARG;
        }
        if ((pa.type == cudaMemoryTypeDevice || pa.type == cudaMemoryTypeManaged) && pa.device != dev) return TB_ERR_INVALID_ARG;
        if (pa.type == cudaMemoryTypeUnregistered) return TB_ERR_INVALID_ARG;
    }
    float* part_o = reinterpret_cast<float*>(scratch);
    float* part_ml = reinterpret_cast<float*>(scratch + kStaticPartO);
    uint32_t* counters = reinterpret_cast<uint32_t*>(scratch + kStaticPartO + kStaticPartMl);
    int32_t* status = reinterpret_cast<int32_t*>(scratch + kStaticPartO + kStaticPartMl + kStaticCounters);

    Geom gm;
    gm.n_layers = 1, gm.Hq = n_q_heads, gm.Hkv = n_kv_heads, gm.g = n_q_heads / n_kv_heads, gm.D = head_dim, gm.dp = 0;
    gm.Hi = gm.Hl = gm.Ha = n_kv_heads, gm.gl = gm.ga = gm.g;
    gm.max_batch = 1 << 20, gm.max_seq_len = max_seq_len, gm.idx_cap = idx_dev ? idx_stride : 0, gm.dtype = kv_dtype;
    UnitTable ut;
    ut.layer_begin = 0, ut.layer_count = 1, ut.n_seq = n_seq;
    ut.use_dev_len = 0, ut.len_is_projected = 0, ut.len_dev = nullptr, ut.len_proj_dev = nullptr;   // lengths are the caller's
    int max_rows = 0;
    for (int i = 0; i < n_seq; ++i) {
        const int slot = seq_slots ? seq_slots[i] : i;
        if (slot < 0 || seq_lens[i] <= 0 || seq_lens[i] > max_seq_len) return TB_ERR_INVALID_ARG;
        ut.seq_id[i] = slot;
        ut.len[i] = seq_lens[i];
        int rows = seq_lens[i];
        if (idx_dev) {
            long long r = (long long)(sinks < rows ? sinks : rows) + idx_stride + recent;
            if (r < rows) rows = (int)r;
        }
        if (rows > max_rows) max_rows = rows;
    }
    AttnArgs a;
    a.res_rows = nullptr, a.res_sinks = a.res_window = 0, a.imp_rows = nullptr;
    a.q = q_dev, a.idx = idx_dev, a.cnt = cnt_dev, a.out = out_dev, a.lse = lse_dev;
    a.dense = idx_dev ? 0 : 1, a.sinks = idx_dev ? sinks : 0, a.recent = idx_dev ? recent : 0;
    a.list_bound = idx_dev ? idx_stride : 0;
    a.cluster_merge = 0;
    a.early_ok = 0;
    for (int i = 0; i < n_seq; ++i) a.known_cnt[i] = -1;
    a.sm_scale = sm_scale > 0.f ? sm_scale : 1.0f / sqrtf((float)head_dim);
    {   // about four 4-warp blocks per SM, at least 64 rows per split; no clusters here: the splits
        // always merge through the scratch array (last block to arrive, fixed order)
        int units = n_seq * n_kv_heads, target = 4 * sm_count;
        int n = (target + units - 1) / units, by_rows = max_rows / 64;
        if (n > by_rows) n = by_rows;
        if (n > kMaxSplits) n = kMaxSplits;
        if (n < 1) n = 1;
        a.nsplit = n;
    }
    cudaStream_t s = (cudaStream_t)stream;
    // the array keeps whatever the previous call left: the arrival counters must start at zero.  The status
    // word is left alone: it collects errors until tb_static_get_status reads and clears it.
    if (cudaMemsetAsync(counters, 0, kStaticCounters, s) != cudaSuccess) return TB_ERR_CUDA;
    dim3 grid(a.nsplit, n_kv_heads, n_seq);
    // the stored-list arguments of the kernels are never read here (caller lists or dense)
    if (kv_dtype == TB_BF16) {
        attn_mma_kernel<4, 2><<<grid, kAttnThreads, kAttnWarps * 2 * kStageBytes, s>>>(
            gm, ut, a, (const __nv_bfloat16*)kv_dev, nullptr, nullptr, part_o, part_ml, counters, status);
    } else {
#define TB_ATTN_S(G) attn_kernel<float, G><<<grid, kAttnThreads, 0, s>>>(gm, ut, a, (const float*)kv_dev, nullptr, nullptr, part_o, part_ml, counters, status)
        if (gm.ga == 1) TB_ATTN_S(1); else if (gm.ga == 2) TB_ATTN_S(2); else if (gm.ga <= 4) TB_ATTN_S(4); else TB_ATTN_S(8);
#undef TB_ATTN_S
    }
    return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}

extern "C" tb_status tb_static_get_status(void* stream, int32_t* device_status) {
    if (!device_status) return TB_ERR_INVALID_ARG;
    unsigned char* scratch = nullptr;
    int sm_count = 0;
    tb_status st = static_scratch_for_current_device(&scratch, &sm_count);
    if (st != TB_OK) return st;
    int32_t* status = reinterpret_cast<int32_t*>(scratch + kStaticPartO + kStaticPartMl + kStaticCounters);
    int32_t v = 0;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemcpyAsync(&v, status, 4, cudaMemcpyDeviceToHost, s) != cudaSuccess) return TB_ERR_CUDA;
    if (cudaMemsetAsync(status, 0, 4, s) != cudaSuccess) return TB_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return TB_ERR_CUDA;
    *device_status = v;
    return TB_OK;
}
