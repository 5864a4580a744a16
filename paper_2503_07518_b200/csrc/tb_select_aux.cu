// Selection helpers off the hot streaming kernel: materialised scores (standalone API call),
// neighbour fetching (paper Sec. 3.4 "Neighbor fetching") and copying stored lists out.
#include "tb_select.cuh"

namespace tb {

// ---- standalone scores ---------------------------------------------------------------------------

template <typename T, int DP, int RED>
__global__ void __launch_bounds__(256) score_kernel(Geom gm, UnitTable ut, const float* __restrict__ q_imp, float scale,
                                                    const T* __restrict__ kimp, float* __restrict__ scores) {
    constexpr int NCH = DP / Elem<T>::kPer16;
    __shared__ __align__(16) float qs[kMaxGroup * 32];
    int ll, s, h;
    decode_unit(gm, ut, blockIdx.y, ll, s, h);
    const int L = unit_len(gm, ut, ll, s);
    GroupScorer<T, DP, RED> scorer;
    scorer.load(q_imp + query_row(gm, ut, ll, s, h) * DP, gm.gl, qs);
    if (RED != TB_GROUP_SUM) __syncthreads();
    const uint4* base = reinterpret_cast<const uint4*>(kimp + key_unit(gm, ut, ll, s, h) * gm.max_seq_len * DP);
    float* out = scores + ((size_t)(ll * ut.n_seq + s) * gm.Hl + h) * gm.max_seq_len;
    for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < L; t += gridDim.x * blockDim.x) {
        const uint4* row = base + (size_t)t * NCH;
        float sc = scorer.score([&](int c) { return __ldg(row + c); });
        out[t] = scale * sc;
    }
}

cudaError_t launch_score(const tb_ctx* c, const UnitTable& ut, const float* q_imp, int reduce, float scale, float* scores, cudaStream_t s) {
    const Geom& gm = c->geom;
    int maxL = 0;
    for (int i = 0; i < ut.layer_count * ut.n_seq; ++i) maxL = ut.len[i] > maxL ? ut.len[i] : maxL;
    if (maxL == 0) return cudaSuccess;
    dim3 grid((maxL + 255) / 256, ut.layer_count * ut.n_seq * gm.Hl);
    if (grid.x > 64) grid.x = 64;
#define TB_SCORE(T, DP)                                                                                                   \
    do {                                                                                                                  \
        if (reduce == TB_GROUP_MAX) score_kernel<T, DP, TB_GROUP_MAX><<<grid, 256, 0, s>>>(gm, ut, q_imp, scale, (const T*)c->kimp, scores); \
        else score_kernel<T, DP, TB_GROUP_SUM><<<grid, 256, 0, s>>>(gm, ut, q_imp, scale, (const T*)c->kimp, scores);     \
    } while (0)
    if (gm.dtype == TB_BF16) {
        if (gm.dp == 32) TB_SCORE(__nv_bfloat16, 32); else TB_SCORE(__nv_bfloat16, 16);
    } else {
        if (gm.dp == 32) TB_SCORE(float, 32); else TB_SCORE(float, 16);
    }
#undef TB_SCORE
    return cudaGetLastError();
}

// ---- neighbour fetching ---------------------------------------------------------------------------

constexpr int kNbThreads = 256;

__global__ void __launch_bounds__(kNbThreads) neighbor_kernel(Geom gm, UnitTable ut, NeighborArgs a, int32_t* __restrict__ state_idx,
                                                              int32_t* __restrict__ state_cnt) {
    extern __shared__ uint32_t mask[];               // one bit per candidate position
    __shared__ int warp_tot[kNbThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int ll, s, h;
    decode_unit(gm, ut, blockIdx.x, ll, s, h);
    const int L = unit_len(gm, ut, ll, s);
    const int lo = min(a.sinks, L), hi = max(lo, L - a.recent);
    const int span = hi - lo;
    const int n_words = (span + 31) / 32;
    const int32_t* src = a.idx_src + (size_t)blockIdx.x * a.src_stride;
    const int cnt = a.cnt_src[blockIdx.x];
    const size_t cu = list_unit(gm, ut, ll, s, h);
    int32_t* dst = state_idx + cu * gm.idx_cap;

    for (int i = tid; i < n_words; i += kNbThreads) mask[i] = 0;
    __syncthreads();
    auto mark = [&](int p) {
        if (p >= lo && p < hi) atomicOr(&mask[(p - lo) >> 5], 1u << ((p - lo) & 31));
    };
    const int r = a.radius;
    for (int i = tid; i < cnt; i += kNbThreads) {
        const int p = src[i];
        if (a.nmode == TB_NEIGHBOR_DILATE) {
            for (int d = -r; d <= r; ++d) mark(p + d);
        } else {
            mark(p);
            if (i == 0 || src[i - 1] != p - 1) {       // first token of a run of consecutive positions
                int j = i;
                while (j + 1 < cnt && src[j + 1] == src[j] + 1) ++j;
                const int b = src[j], n = r * (b - p + 1);
                const int right = (n + 1) / 2, left = n / 2;
                for (int x = b + 1; x <= b + right; ++x) mark(x);
                for (int x = p - left; x <= p - 1; ++x) mark(x);
            }
        }
    }
    __syncthreads();

    // ordered compaction of the bitmask: each warp owns a contiguous range of words
    const int wseg = ((n_words + kNbThreads - 1) / kNbThreads) * 32;
    const int wb = min(n_words, warp * wseg), we = min(n_words, (warp + 1) * wseg);
    int tot = 0;
    for (int i = wb + lane; i < we; i += 32) tot += __popc(mask[i]);
    tot = warp_sum_int(tot);
    if (lane == 0) warp_tot[warp] = tot;
    __syncthreads();
    int pos = 0, all = 0;
    for (int w = 0; w < kNbThreads / 32; ++w) {
        if (w < warp) pos += warp_tot[w];
        all += warp_tot[w];
    }
    for (int i0 = wb; i0 < we; i0 += 32) {
        const int i = i0 + lane;
        uint32_t m = i < we ? mask[i] : 0u;
        const int c = __popc(m);
        const int incl = warp_incl_scan(c, lane);
        int o = pos + incl - c;
        while (m) {
            int bit = __ffs(m) - 1;
            m &= m - 1;
            dst[o++] = lo + i * 32 + bit;
        }
        pos += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (tid == 0) state_cnt[cu] = all;
}

cudaError_t launch_neighbors(const tb_ctx* c, const UnitTable& ut, const NeighborArgs& a, cudaStream_t s, bool dry) {
    const Geom& gm = c->geom;
    int max_span = 0;
    for (int i = 0; i < ut.layer_count * ut.n_seq; ++i) {
        int L = ut.len[i], lo = a.sinks < L ? a.sinks : L, hi = L - a.recent > lo ? L - a.recent : lo;
        if (hi - lo > max_span) max_span = hi - lo;
    }
    size_t smem = (size_t)((max_span + 31) / 32) * 4 + 16;
    if (smem > 200 * 1024) return cudaErrorInvalidConfiguration;   // one bit per candidate on chip: up to 1,638,272 candidates
    if (dry) return cudaSuccess;
    static unsigned char seen[64];
    if (first_use_on_this_device(seen)) {
        cudaError_t e = cudaFuncSetAttribute(neighbor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return e;
    }
    neighbor_kernel<<<ut.layer_count * ut.n_seq * gm.Hl, kNbThreads, smem, s>>>(gm, ut, a, c->st.idx, c->st.cnt);
    return cudaGetLastError();
}

// ---- copy stored lists out --------------------------------------------------------------------------

__global__ void copy_lists_kernel(Geom gm, UnitTable ut, const int32_t* __restrict__ state_idx, const int32_t* __restrict__ state_cnt,
                                  int32_t* __restrict__ idx_out, int32_t* __restrict__ cnt_out) {
    int ll, s, h;
    decode_unit(gm, ut, blockIdx.x, ll, s, h);
    const size_t cu = list_unit(gm, ut, ll, s, h);
    const int n = state_cnt[cu];
    if (idx_out)
        for (int i = threadIdx.x; i < n; i += blockDim.x) idx_out[(size_t)blockIdx.x * gm.idx_cap + i] = state_idx[cu * gm.idx_cap + i];
    if (cnt_out && threadIdx.x == 0) cnt_out[blockIdx.x] = n;
}

cudaError_t launch_copy_lists(const tb_ctx* c, const UnitTable& ut, int32_t* idx_out, int32_t* cnt_out, cudaStream_t s) {
    copy_lists_kernel<<<ut.layer_count * ut.n_seq * c->geom.Hl, 256, 0, s>>>(c->geom, ut, c->st.idx, c->st.cnt, idx_out, cnt_out);
    return cudaGetLastError();
}

}  // namespace tb
