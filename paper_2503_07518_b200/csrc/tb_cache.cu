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
// The last block to finish advances the device length counters (read by every block of this launch at
// its start, so they may only change once all have arrived).
template <typename T>
__global__ void append_kernel(Geom gm, UnitTable ut, AppendTable at, int total_new, const T* __restrict__ k_new,
                              const T* __restrict__ v_new, T* __restrict__ kv, int32_t* __restrict__ len_dev,
                              uint32_t* __restrict__ counter, int32_t* __restrict__ status, T* __restrict__ res_rows,
                              int res_sinks, int res_window) {
    constexpr int kPer16 = Elem<T>::kPer16;
    const int chunks_per_row = gm.D / kPer16;          // 16-byte chunks in one K (or V) row
    const int chunks_per_pair = 2 * chunks_per_row;
    const int ll = blockIdx.y;
    const long long work = (long long)total_new * gm.Hkv * chunks_per_pair;
    // Launched as a programmatic dependent (a decode step appends right after the previous layer's
    // attention): resident early, but the new rows may come from the predecessor and the cache rows
    // written here may still be read by it, so wait first; the successor may then get ready.
    pdl_wait();
    pdl_launch_dependents();
    for (long long w = (long long)blockIdx.x * blockDim.x + threadIdx.x; w < work; w += (long long)gridDim.x * blockDim.x) {
        int chunk = (int)(w % chunks_per_pair);
        long long th = w / chunks_per_pair;
        int h = (int)(th % gm.Hkv);
        int tok = (int)(th / gm.Hkv);                  // index into the concatenated new tokens
        int s = 0;
        while (s + 1 < ut.n_seq && at.tok_off[s + 1] <= tok) ++s;
        const int base = unit_len(gm, ut, ll, s);
        if (base + (at.tok_off[s + 1] - at.tok_off[s]) > gm.max_seq_len) continue;   // only a replayed graph gets here (reported below)
        int pos = base + (tok - at.tok_off[s]);
        int is_v = chunk >= chunks_per_row;
        int c16 = is_v ? chunk - chunks_per_row : chunk;
        const T* src = (is_v ? v_new : k_new) + (((size_t)ll * total_new + tok) * gm.Hkv + h) * gm.D;
        size_t row = (((size_t)(ut.layer_begin + ll) * gm.max_batch + ut.seq_id[s]) * gm.Hkv + h) * gm.max_seq_len + pos;
        T* dst = kv + row * 2 * gm.D + (size_t)is_v * gm.D;
        const uint4 val = reinterpret_cast<const uint4*>(src)[c16];
        reinterpret_cast<uint4*>(dst)[c16] = val;
        if (res_rows) {
            // resident copies (offloaded KV): the first res_sinks tokens, and a ring of the res_window most recent
            const int n_s = at.tok_off[s + 1] - at.tok_off[s];
            int slot = -1;
            if (pos < res_sinks) slot = pos;
            else if (res_window > 0 && pos >= base + n_s - res_window) slot = res_sinks + pos % res_window;
            if (slot >= 0) {
                const size_t unit = ((size_t)(ut.layer_begin + ll) * gm.max_batch + ut.seq_id[s]) * gm.Hkv + h;
                T* rdst = res_rows + (unit * (size_t)(res_sinks + res_window) + slot) * 2 * gm.D + (size_t)is_v * gm.D;
                reinterpret_cast<uint4*>(rdst)[c16] = val;
            }
        }
    }
    // (only when the kernels read the device counters: otherwise the host's mirrors carry the lengths and
    // the counters are brought up to date when that mode is switched on)
    if (ut.use_dev_len && last_block_arrives(counter, gridDim.x * gridDim.y)) {
        for (int i = threadIdx.x; i < ut.layer_count * ut.n_seq; i += blockDim.x) {
            const int l2 = i / ut.n_seq, s2 = i % ut.n_seq;
            const size_t pair = (size_t)(ut.layer_begin + l2) * gm.max_batch + ut.seq_id[s2];
            const int base = unit_len(gm, ut, l2, s2), n = at.tok_off[s2 + 1] - at.tok_off[s2];
            if (base + n > gm.max_seq_len) atomicExch(status, kStatusCapacity);
            else len_dev[pair] = base + n;
        }
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
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks, ut.layer_count, 1), cfg.blockDim = dim3(threads, 1, 1), cfg.dynamicSmemBytes = 0, cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see pdl_wait()
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr, cfg.numAttrs = 1;
    if (gm.dtype == TB_BF16)
        return cudaLaunchKernelEx(&cfg, append_kernel<__nv_bfloat16>, gm, ut, at, total_new, (const __nv_bfloat16*)k,
                                  (const __nv_bfloat16*)v, (__nv_bfloat16*)c->kv, c->st.len, c->st.misc_counter, c->st.status,
                                  (__nv_bfloat16*)c->res_rows, c->res_sinks, c->res_window);
    return cudaLaunchKernelEx(&cfg, append_kernel<float>, gm, ut, at, total_new, (const float*)k, (const float*)v, (float*)c->kv,
                              c->st.len, c->st.misc_counter, c->st.status, (float*)c->res_rows, c->res_sinks, c->res_window);
}

// ---------------------------------------------------------------------------------------------
// KV migration (paper Sec. 3.3: on a prediction step the selected K/V pairs are moved into the contiguous
// Important buffer, from which the following steps attend): rows list[j] of the cache -> row j of the
// unit's buffer, 16 bytes per thread.  One block column per list; the count is read on the device.
template <typename T>
__global__ void __launch_bounds__(256) migrate_kernel(Geom gm, UnitTable ut, const T* __restrict__ kv, const int32_t* __restrict__ state_idx,
                                                      const int32_t* __restrict__ state_cnt, T* __restrict__ imp) {
    constexpr int kPer16 = Elem<T>::kPer16;
    const int chunks = 2 * gm.D / kPer16;              // 16-byte chunks of a K|V row pair
    const int u = blockIdx.y, h = u % gm.Hl, s = (u / gm.Hl) % ut.n_seq, ll = u / (gm.Hl * ut.n_seq);
    const size_t pc = (size_t)(ut.layer_begin + ll) * gm.max_batch + ut.seq_id[s];
    const size_t lc = pc * gm.Hl + h, kc = pc * gm.Hkv + h;               // lists are per KV head here
    const int n = min(state_cnt[lc], gm.idx_cap);
    const int32_t* list = state_idx + lc * gm.idx_cap;
    const uint4* src = reinterpret_cast<const uint4*>(kv + kc * gm.max_seq_len * 2 * gm.D);
    uint4* dst = reinterpret_cast<uint4*>(imp + lc * (size_t)gm.idx_cap * 2 * gm.D);
    for (long long w = (long long)blockIdx.x * blockDim.x + threadIdx.x; w < (long long)n * chunks; w += (long long)gridDim.x * blockDim.x) {
        const int j = (int)(w / chunks), c = (int)(w % chunks);
        dst[(size_t)j * chunks + c] = src[(size_t)list[j] * chunks + c];
    }
}

cudaError_t launch_migrate(const tb_ctx* c, const UnitTable& ut, cudaStream_t s) {
    const Geom& gm = c->geom;
    const int units = ut.layer_count * ut.n_seq * gm.Hl;
    int bx = 2 * c->sm_count / units;                  // about two blocks per SM over the launch
    bx = bx < 1 ? 1 : bx > 64 ? 64 : bx;
    dim3 grid(bx, units);
    if (gm.dtype == TB_BF16)
        migrate_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(gm, ut, (const __nv_bfloat16*)c->kv, c->st.idx, c->st.cnt, (__nv_bfloat16*)c->imp_rows);
    else
        migrate_kernel<float><<<grid, 256, 0, s>>>(gm, ut, (const float*)c->kv, c->st.idx, c->st.cnt, (float*)c->imp_rows);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// K_imp[t][j] = round( sum_c K[t][c] * W[c][j] ), channels in ascending order, fp32 FMA chain.

struct ProjectTable {
    int auto_range;                  // 1: [projected length, length) of every (layer, sequence), from the device counters
    int pos_begin[kMaxLaunchSeq];
    int pos_end[kMaxLaunchSeq];
};

// Token range of a projection block's (layer, sequence).
__device__ __forceinline__ void project_range(const Geom& gm, const UnitTable& ut, const ProjectTable& pt, int ll, int s, int& begin, int& end) {
    if (pt.auto_range) {
        const size_t pair = (size_t)(ut.layer_begin + ll) * gm.max_batch + ut.seq_id[s];
        begin = ut.len_proj_dev[pair], end = ut.len_dev[pair];
    } else {
        begin = pt.pos_begin[s], end = pt.pos_end[s];
    }
}
// The last block of a projection launch to finish advances the device counters of the projected lengths.
__device__ __forceinline__ void project_finish(const Geom& gm, const UnitTable& ut, const ProjectTable& pt, int32_t* len_proj_dev,
                                               uint32_t* counter) {
    if (!ut.use_dev_len || !last_block_arrives(counter, gridDim.x * gridDim.y * gridDim.z)) return;
    for (int i = threadIdx.x; i < ut.layer_count * ut.n_seq; i += blockDim.x) {
        int b, e;
        project_range(gm, ut, pt, i / ut.n_seq, i % ut.n_seq, b, e);
        const size_t pair = (size_t)(ut.layer_begin + i / ut.n_seq) * gm.max_batch + ut.seq_id[i % ut.n_seq];
        if (e > len_proj_dev[pair]) len_proj_dev[pair] = e;
    }
}

constexpr int kProjTokens = 32;   // tokens per block
constexpr int kProjThreads = 128; // 4 threads per token, each owning dp/4 outputs

template <typename T, int DP>
__global__ void __launch_bounds__(kProjThreads) project_kernel(Geom gm, UnitTable ut, ProjectTable pt, const T* __restrict__ kv,
                                                               const T* __restrict__ Wall, T* __restrict__ kimp,
                                                               int32_t* __restrict__ len_proj_dev, uint32_t* __restrict__ counter) {
    constexpr int D = 128;
    constexpr int JPT = DP / 4;                       // outputs per thread
    __shared__ float Ws[D * DP];
    __shared__ float Ks[kProjTokens][D + 1];

    const int ll = blockIdx.z / ut.n_seq, s = blockIdx.z % ut.n_seq, h = blockIdx.y;
    const int layer = ut.layer_begin + ll;
    int r_begin, t_end;
    project_range(gm, ut, pt, ll, s, r_begin, t_end);
    const int t0 = r_begin + blockIdx.x * kProjTokens;
    const int nt = max(0, min(kProjTokens, t_end - t0));               // 0: nothing for this block (it still reports in at the end)

    // One key stream per KV head, or (one list per layer) a single stream that sums the heads'
    // projections: K_imp[t] = sum_h K[t][h] . W[h], heads in ascending order on one fp32 chain.
    const int n_sum = gm.Hkv / gm.Hi;
    const size_t pair = (size_t)layer * gm.max_batch + ut.seq_id[s];
    const int t = threadIdx.x / 4, jq = threadIdx.x % 4;
    float acc[JPT];
#pragma unroll
    for (int j = 0; j < JPT; ++j) acc[j] = 0.f;
    for (int hs = 0; hs < n_sum; ++hs) {
        const int hk = h * n_sum + hs;
        const T* W = Wall + ((size_t)layer * gm.Hkv + hk) * D * DP;
        if (hs) __syncthreads();
        for (int i = threadIdx.x; i < D * DP; i += kProjThreads) Ws[i] = Elem<T>::to_f32(W[i]);
        if (nt == 0) break;
        const size_t krow0 = (pair * gm.Hkv + hk) * gm.max_seq_len + t0;
        for (int i = threadIdx.x; i < nt * D; i += kProjThreads) {
            int tt = i / D, ch = i % D;
            Ks[tt][ch] = Elem<T>::to_f32(kv[(krow0 + tt) * 2 * D + ch]);
        }
        __syncthreads();
        if (t < nt) {
#pragma unroll 4
            for (int ch = 0; ch < D; ++ch) {
                float kx = Ks[t][ch];
#pragma unroll
                for (int j = 0; j < JPT; ++j) acc[j] = fmaf(kx, Ws[ch * DP + jq * JPT + j], acc[j]);
            }
        }
    }
    if (t < nt) {
        const size_t row0 = (pair * gm.Hi + h) * gm.max_seq_len + t0;
        T* dst = kimp + (row0 + t) * DP + jq * JPT;
#pragma unroll
        for (int j = 0; j < JPT; ++j) dst[j] = Elem<T>::from_f32(acc[j]);
    }
    project_finish(gm, ut, pt, len_proj_dev, counter);
}

// bf16 storage: the projection is the one dense contraction of the path ([tokens x 128] . [128 x d']
// per KV head), so it runs on the tensor cores: 128 tokens per block, K rows and the W_K slice staged
// in shared memory with 16-byte cp.async (K rows unpadded with an XOR swizzle of their 16-byte chunks, so
// that a source line is one full-line request and ldmatrix still sees eight bank groups), mma.sync m16n8k16 with fp32
// accumulation, one round-to-nearest-even to bf16.  HBM-bound: 256 B read + 2 d' B written per token.
constexpr int kPmTokens = 128;
constexpr int kPmThreads = 128;
constexpr int kPmKPitch = 256;            // 256 B of K per token, 16-byte chunk c of row t at chunk c ^ (t & 7)

template <int DP>
__global__ void __launch_bounds__(kPmThreads) project_mma_kernel(Geom gm, UnitTable ut, ProjectTable pt,
                                                                 const __nv_bfloat16* __restrict__ kv,
                                                                 const __nv_bfloat16* __restrict__ Wall,
                                                                 __nv_bfloat16* __restrict__ kimp, int32_t* __restrict__ len_proj_dev,
                                                                 uint32_t* __restrict__ counter) {
    constexpr int D = 128;
    constexpr int kWPitch = DP * 2 + 16;  // bytes per W row (one channel, d' outputs) + pad
    constexpr int NT = DP / 8;            // 8-wide output tiles
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* Ks = smem;                                  // [128 tokens][kPmKPitch]
    unsigned char* Ws = smem + kPmTokens * kPmKPitch;          // [128 channels][kWPitch]

    const int ll = blockIdx.z / ut.n_seq, s = blockIdx.z % ut.n_seq, h = blockIdx.y;
    const int layer = ut.layer_begin + ll;
    int r_begin, t_end;
    project_range(gm, ut, pt, ll, s, r_begin, t_end);
    const int t0 = r_begin + blockIdx.x * kPmTokens;
    if (t0 >= t_end) {                                                 // nothing for this block: it only reports in
        project_finish(gm, ut, pt, len_proj_dev, counter);
        return;
    }
    const int nt_valid = min(kPmTokens, t_end - t0);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gid = lane >> 2, tig = lane & 3;

    // One key stream per KV head, or (one list per layer) a single stream that sums the heads'
    // projections in the fp32 accumulators, heads in ascending order.
    const int n_sum = gm.Hkv / gm.Hi;
    const size_t pair = (size_t)layer * gm.max_batch + ut.seq_id[s];
    const uint32_t ks_u32 = smem_u32(Ks), ws_u32 = smem_u32(Ws);
    const int mi = lane >> 3, r8 = lane & 7;
    float acc[2][NT][4];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int n = 0; n < NT; ++n) acc[mt][n][0] = acc[mt][n][1] = acc[mt][n][2] = acc[mt][n][3] = 0.f;

    for (int hs = 0; hs < n_sum; ++hs) {
        const int hk = h * n_sum + hs;
        const size_t krow0 = (pair * gm.Hkv + hk) * gm.max_seq_len + t0;
        const unsigned char* kbase = reinterpret_cast<const unsigned char*>(kv) + krow0 * 2 * D * 2;
        const unsigned char* wbase = reinterpret_cast<const unsigned char*>(Wall + ((size_t)layer * gm.Hkv + hk) * D * DP);
        if (hs) __syncthreads();                                       // the previous head's tiles are consumed
        for (int i = tid; i < kPmTokens * 16; i += kPmThreads) {          // 16 chunks of 16 B per K row
            const int t = i >> 4, ch = i & 15;
            const int tc = min(t, nt_valid - 1);                           // rows past the range repeat the last one
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ks_u32 + t * kPmKPitch + ((ch ^ (t & 7)) << 4)),
                         "l"(kbase + (size_t)tc * 512 + ch * 16) : "memory");
        }
        for (int i = tid; i < D * (DP / 8); i += kPmThreads) {             // DP/8 chunks per W row
            const int r = i / (DP / 8), ch = i % (DP / 8);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ws_u32 + r * kWPitch + ch * 16),
                         "l"(wbase + (size_t)r * DP * 2 + ch * 16) : "memory");
        }
        asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
        __syncthreads();

        // B fragments (W: k = channel, n = output) for every k-step and output tile, loaded once per warp
        uint32_t bw[8][NT][2];
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
#pragma unroll
            for (int np = 0; np < NT / 2; ++np) {
                // matrices: (ch lo, outs np*16+0..7), (ch hi, same), (ch lo, outs +8), (ch hi, outs +8)
                const uint32_t addr = ws_u32 + (ks * 16 + (mi & 1) * 8 + r8) * kWPitch + (np * 16 + (mi >> 1) * 8) * 2;
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                             : "=r"(bw[ks][2 * np][0]), "=r"(bw[ks][2 * np][1]), "=r"(bw[ks][2 * np + 1][0]), "=r"(bw[ks][2 * np + 1][1])
                             : "r"(addr));
            }
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
            const int tok = warp * 32 + mt * 16;                           // first token of this 16-token tile
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                uint32_t a0, a1, a2, a3;
                const uint32_t addr = ks_u32 + (tok + (mi & 1) * 8 + r8) * kPmKPitch + ((ks * 32) ^ (((mi >> 1) ^ r8) << 4));
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3) : "r"(addr));
#pragma unroll
                for (int n = 0; n < NT; ++n)
                    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                                 : "+f"(acc[mt][n][0]), "+f"(acc[mt][n][1]), "+f"(acc[mt][n][2]), "+f"(acc[mt][n][3])
                                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(bw[ks][n][0]), "r"(bw[ks][n][1]));
            }
        }
    }
    __nv_bfloat16* out = kimp + ((pair * gm.Hi + h) * gm.max_seq_len + t0) * DP;
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
        const int tok = warp * 32 + mt * 16;
#pragma unroll
        for (int n = 0; n < NT; ++n) {
            const int j = n * 8 + tig * 2;
            if (tok + gid < nt_valid) {
                __nv_bfloat162 v = __floats2bfloat162_rn(acc[mt][n][0], acc[mt][n][1]);
                *reinterpret_cast<__nv_bfloat162*>(out + (size_t)(tok + gid) * DP + j) = v;
            }
            if (tok + gid + 8 < nt_valid) {
                __nv_bfloat162 v = __floats2bfloat162_rn(acc[mt][n][2], acc[mt][n][3]);
                *reinterpret_cast<__nv_bfloat162*>(out + (size_t)(tok + gid + 8) * DP + j) = v;
            }
        }
    }
    project_finish(gm, ut, pt, len_proj_dev, counter);
}

cudaError_t launch_project(const tb_ctx* c, const UnitTable& ut, const int* pos_begin, const int* pos_end, int max_range, cudaStream_t s) {
    ProjectTable pt;
    pt.auto_range = pos_begin == nullptr;
    for (int i = 0; i < ut.n_seq; ++i) {
        pt.pos_begin[i] = pt.auto_range ? 0 : pos_begin[i];
        pt.pos_end[i] = pt.auto_range ? 0 : pos_end[i];
    }
    if (max_range <= 0) return cudaSuccess;
    const Geom& gm = c->geom;
    if (gm.dtype == TB_BF16) {
        dim3 grid_mma((max_range + kPmTokens - 1) / kPmTokens, gm.Hi, ut.layer_count * ut.n_seq);
        const __nv_bfloat16* kvp = (const __nv_bfloat16*)c->kv;
        const __nv_bfloat16* wp = (const __nv_bfloat16*)c->st.W;
        if (gm.dp == 32) {
            const size_t smem = kPmTokens * kPmKPitch + 128 * (32 * 2 + 16);
            static unsigned char seen[64];
            if (first_use_on_this_device(seen)) {
                cudaError_t e = cudaFuncSetAttribute(project_mma_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
                if (e != cudaSuccess) return e;
            }
            project_mma_kernel<32><<<grid_mma, kPmThreads, smem, s>>>(gm, ut, pt, kvp, wp, (__nv_bfloat16*)c->kimp, c->st.len_proj, c->st.misc_counter + 1);
        } else {
            const size_t smem = kPmTokens * kPmKPitch + 128 * (16 * 2 + 16);
            static unsigned char seen[64];
            if (first_use_on_this_device(seen)) {
                cudaError_t e = cudaFuncSetAttribute(project_mma_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
                if (e != cudaSuccess) return e;
            }
            project_mma_kernel<16><<<grid_mma, kPmThreads, smem, s>>>(gm, ut, pt, kvp, wp, (__nv_bfloat16*)c->kimp, c->st.len_proj, c->st.misc_counter + 1);
        }
        return cudaGetLastError();
    }
    dim3 grid((max_range + kProjTokens - 1) / kProjTokens, gm.Hi, ut.layer_count * ut.n_seq);
#define TB_PROJ(T, DP) \
    project_kernel<T, DP><<<grid, kProjThreads, 0, s>>>(gm, ut, pt, (const T*)c->kv, (const T*)c->st.W, (T*)c->kimp, c->st.len_proj, c->st.misc_counter + 1)
    if (gm.dp == 32) TB_PROJ(float, 32); else TB_PROJ(float, 16);
#undef TB_PROJ
    return cudaGetLastError();
}

}  // namespace tb
