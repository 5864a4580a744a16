// Cache maintenance kernels: append new K/V rows to the interleaved KV cache (paper Sec. 3.3: the
// full cache is kept, never evicted) and project key rows into the d'-dimensional importance space
// (Sec. 3.1, K_imp = K W_K), eagerly or in deferred batches (Sec. 3.3).
#include "tb_common.cuh"
#include "tb_internal.h"

namespace tb {

struct AppendTable {
    int tok_off[kMaxLaunchSeq + 1];  // prefix sums of n_new over the listed sequences
};

// One thread per 16-byte chunk of a (token, head) K|V row pair.
template <typename T>
__global__ void append_kernel(Geom gm, UnitTable ut, AppendTable at, int total_new, const T* __restrict__ k_new,
                              const T* __restrict__ v_new, T* __restrict__ kv) {
    constexpr int kPer16 = Elem<T>::kPer16;
    const int chunks_per_row = gm.D / kPer16;          // 16-byte chunks in one K (or V) row
    const int chunks_per_pair = 2 * chunks_per_row;
    const int ll = blockIdx.y;
    const long long work = (long long)total_new * gm.Hkv * chunks_per_pair;
    for (long long w = (long long)blockIdx.x * blockDim.x + threadIdx.x; w < work; w += (long long)gridDim.x * blockDim.x) {
        int chunk = (int)(w % chunks_per_pair);
        long long th = w / chunks_per_pair;
        int h = (int)(th % gm.Hkv);
        int tok = (int)(th / gm.Hkv);                  // index into the concatenated new tokens
        int s = 0;
        while (s + 1 < ut.n_seq && at.tok_off[s + 1] <= tok) ++s;
        int pos = ut.len[ll * ut.n_seq + s] + (tok - at.tok_off[s]);
        int is_v = chunk >= chunks_per_row;
        int c16 = is_v ? chunk - chunks_per_row : chunk;
        const T* src = (is_v ? v_new : k_new) + (((size_t)ll * total_new + tok) * gm.Hkv + h) * gm.D;
        size_t row = (((size_t)(ut.layer_begin + ll) * gm.max_batch + ut.seq_id[s]) * gm.Hkv + h) * gm.max_seq_len + pos;
        T* dst = kv + row * 2 * gm.D + (size_t)is_v * gm.D;
        reinterpret_cast<uint4*>(dst)[c16] = reinterpret_cast<const uint4*>(src)[c16];
    }
}

cudaError_t launch_append(const tb_ctx* c, const UnitTable& ut, const int* n_new, const int* tok_off, int total_new,
                          const void* k, const void* v, cudaStream_t s) {
    (void)n_new;
    AppendTable at;
    for (int i = 0; i <= ut.n_seq; ++i) at.tok_off[i] = tok_off[i];
    const Geom& gm = c->geom;
    int es = gm.dtype == TB_BF16 ? 2 : 4;
    long long work = (long long)total_new * gm.Hkv * (2 * gm.D * es / 16);
    int threads = 256;
    long long blocks = (work + threads - 1) / threads;
    if (blocks > 148 * 16) blocks = 148 * 16;
    dim3 grid((unsigned)blocks, ut.layer_count);
    if (gm.dtype == TB_BF16)
        append_kernel<__nv_bfloat16><<<grid, threads, 0, s>>>(gm, ut, at, total_new, (const __nv_bfloat16*)k,
                                                            (const __nv_bfloat16*)v, (__nv_bfloat16*)c->kv);
    else
        append_kernel<float><<<grid, threads, 0, s>>>(gm, ut, at, total_new, (const float*)k, (const float*)v, (float*)c->kv);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// K_imp[t][j] = round( sum_c K[t][c] * W[c][j] ), channels in ascending order, fp32 FMA chain.

struct ProjectTable {
    int pos_begin[kMaxLaunchSeq];
    int pos_end[kMaxLaunchSeq];
};

constexpr int kProjTokens = 32;   // tokens per block
constexpr int kProjThreads = 128; // 4 threads per token, each owning dp/4 outputs

template <typename T, int DP>
__global__ void __launch_bounds__(kProjThreads) project_kernel(Geom gm, UnitTable ut, ProjectTable pt, const T* __restrict__ kv,
                                                               const T* __restrict__ Wall, T* __restrict__ kimp) {
    constexpr int D = 128;
    constexpr int JPT = DP / 4;                       // outputs per thread
    __shared__ float Ws[D * DP];
    __shared__ float Ks[kProjTokens][D + 1];

    const int ll = blockIdx.z / ut.n_seq, s = blockIdx.z % ut.n_seq, h = blockIdx.y;
    const int layer = ut.layer_begin + ll;
    const int t0 = pt.pos_begin[s] + blockIdx.x * kProjTokens;
    const int t_end = pt.pos_end[s];
    if (t0 >= t_end) return;
    const int nt = min(kProjTokens, t_end - t0);

    const T* W = Wall + ((size_t)layer * gm.Hkv + h) * D * DP;
    for (int i = threadIdx.x; i < D * DP; i += kProjThreads) Ws[i] = Elem<T>::to_f32(W[i]);
    const size_t row0 = (((size_t)layer * gm.max_batch + ut.seq_id[s]) * gm.Hkv + h) * gm.max_seq_len + t0;
    for (int i = threadIdx.x; i < nt * D; i += kProjThreads) {
        int t = i / D, ch = i % D;
        Ks[t][ch] = Elem<T>::to_f32(kv[(row0 + t) * 2 * D + ch]);
    }
    __syncthreads();

    const int t = threadIdx.x / 4, jq = threadIdx.x % 4;
    if (t >= nt) return;
    float acc[JPT];
#pragma unroll
    for (int j = 0; j < JPT; ++j) acc[j] = 0.f;
#pragma unroll 4
    for (int ch = 0; ch < D; ++ch) {
        float kx = Ks[t][ch];
#pragma unroll
        for (int j = 0; j < JPT; ++j) acc[j] = fmaf(kx, Ws[ch * DP + jq * JPT + j], acc[j]);
    }
    T* dst = kimp + (row0 + t) * DP + jq * JPT;
#pragma unroll
    for (int j = 0; j < JPT; ++j) dst[j] = Elem<T>::from_f32(acc[j]);
}

cudaError_t launch_project(const tb_ctx* c, const UnitTable& ut, const int* pos_begin, const int* pos_end, cudaStream_t s) {
    ProjectTable pt;
    int max_range = 0;
    for (int i = 0; i < ut.n_seq; ++i) {
        pt.pos_begin[i] = pos_begin[i];
        pt.pos_end[i] = pos_end[i];
        if (pos_end[i] - pos_begin[i] > max_range) max_range = pos_end[i] - pos_begin[i];
    }
    if (max_range <= 0) return cudaSuccess;
    const Geom& gm = c->geom;
    dim3 grid((max_range + kProjTokens - 1) / kProjTokens, gm.Hkv, ut.layer_count * ut.n_seq);
#define TB_PROJ(T, DP) \
    project_kernel<T, DP><<<grid, kProjThreads, 0, s>>>(gm, ut, pt, (const T*)c->kv, (const T*)c->st.W, (T*)c->kimp)
    if (gm.dtype == TB_BF16) {
        if (gm.dp == 32) TB_PROJ(__nv_bfloat16, 32); else TB_PROJ(__nv_bfloat16, 16);
    } else {
        if (gm.dp == 32) TB_PROJ(float, 32); else TB_PROJ(float, 16);
    }
#undef TB_PROJ
    return cudaGetLastError();
}

}  // namespace tb
