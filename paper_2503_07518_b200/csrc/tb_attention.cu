// Sparse decode attention (paper Sec. 3.3: attention over Sink + Important + Local-Window rows of
// the never-evicted cache; Sec. 3.4: the important rows are gathered by index).
//
// One launch covers (layer, sequence, KV head) x split.  Every gathered K|V row pair (adjacent in
// memory) is loaded once and shared by the g query heads of its KV head.  Each split keeps an online
// softmax (m, l, o) per query head; the last block to arrive for a (sequence, KV head) merges the
// splits in split order, so the result is bit-reproducible.
#include "tb_common.cuh"
#include "tb_internal.h"

namespace tb {

constexpr int kAttnThreads = 128;
constexpr int kAttnWarps = kAttnThreads / 32;
constexpr int kRowsPerIter = 4;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Which token does attended row r refer to?  Rows are sinks, then the index list, then the window.
struct RowMap {
    int n_sink, n_list, w_begin, L, dense;
    const int32_t* list;
    __device__ __forceinline__ int token(int r, bool& bad) const {
        bad = false;
        if (dense || r < n_sink) return r;
        r -= n_sink;
        if (r < n_list) {
            int t = list[r];
            if (t < 0 || t >= L) { bad = true; return 0; }
            return t;
        }
        return w_begin + (r - n_list);
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
    const int L = ut.len[ll * ut.n_seq + s];
    const int g = gm.g;
    const size_t cu = ((size_t)(ut.layer_begin + ll) * gm.max_batch + ut.seq_id[s]) * gm.Hkv + h;
    const int lu = (ll * ut.n_seq + s) * gm.Hkv + h;                 // launch-local unit

    RowMap rm;
    rm.L = L, rm.dense = a.dense;
    rm.n_sink = a.dense ? 0 : min(a.sinks, L);
    rm.w_begin = a.dense ? 0 : max(rm.n_sink, L - a.recent);
    int n_list = 0;
    if (!a.dense) {
        n_list = a.idx ? a.cnt[lu] : state_cnt[cu];
        n_list = max(0, min(n_list, gm.idx_cap));
    }
    rm.n_list = n_list;
    rm.list = a.idx ? a.idx + (size_t)lu * gm.idx_cap : state_idx + cu * gm.idx_cap;
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

    const T* kv_unit = kv + cu * gm.max_seq_len * 2 * D;
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
            const T* row = kv_unit + (size_t)t * 2 * D;
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
        const size_t pq = ((size_t)(ll * ut.n_seq + s) * gm.Hq + h * g + u) * kMaxSplits + split;
        part_o[pq * D + tid] = o;
        if (tid == 0) part_ml[pq * 2] = M, part_ml[pq * 2 + 1] = lsum;
    }

    // ---- last block of this (sequence, KV head) merges the splits ----------------------------------
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        unsigned prev = atomicAdd(&counters[lu], 1u);
        sh_last = prev == (unsigned)a.nsplit - 1u;
        if (sh_last) counters[lu] = 0;                  // ready for the next launch
    }
    __syncthreads();
    if (!sh_last) return;
    __threadfence();
    for (int u = 0; u < g; ++u) {
        const size_t hq = (size_t)(ll * ut.n_seq + s) * gm.Hq + h * g + u;
        const size_t pq = hq * kMaxSplits;
        float M = -INFINITY;
        for (int j = 0; j < a.nsplit; ++j) M = fmaxf(M, __ldcg(&part_ml[(pq + j) * 2]));
        const float Ms = M == -INFINITY ? 0.f : M;
        float lsum = 0.f, o = 0.f;
        for (int j = 0; j < a.nsplit; ++j) {
            const float e = exp2f(__ldcg(&part_ml[(pq + j) * 2]) - Ms);
            lsum += __ldcg(&part_ml[(pq + j) * 2 + 1]) * e;
            o += __ldcg(&part_o[(pq + j) * D + tid]) * e;
        }
        a.out[hq * D + tid] = o / lsum;
        if (a.lse && tid == 0) a.lse[hq] = (M + log2f(lsum)) * kLn2;
    }
}

static int pick_nsplit(const tb_ctx* c, int units, int max_rows) {
    int target = 4 * c->sm_count;
    int n = (target + units - 1) / units;
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
    if (a.nsplit <= 0) a.nsplit = pick_nsplit(c, ut.layer_count * ut.n_seq * gm.Hkv, max_rows);
    dim3 grid(a.nsplit, gm.Hkv, ut.layer_count * ut.n_seq);
#define TB_ATTN(T, G)                                                                                                   \
    attn_kernel<T, G><<<grid, kAttnThreads, 0, s>>>(gm, ut, a, (const T*)c->kv, c->st.idx, c->st.cnt, c->wk.part_o,     \
                                                   c->wk.part_ml, c->st.attn_counter, c->st.status)
#define TB_ATTN_G(T)                                  \
    do {                                              \
        if (gm.g == 1) TB_ATTN(T, 1);                 \
        else if (gm.g == 2) TB_ATTN(T, 2);            \
        else if (gm.g <= 4) TB_ATTN(T, 4);            \
        else TB_ATTN(T, 8);                           \
    } while (0)
    if (gm.dtype == TB_BF16) TB_ATTN_G(__nv_bfloat16); else TB_ATTN_G(float);
#undef TB_ATTN_G
#undef TB_ATTN
    return cudaGetLastError();
}

}  // namespace tb
