// Importance scoring and token selection (paper Sec. 3.4 "score computation against all projected
// keys ... top-B selection", Sec. 4 "Token Selection Policy", Sec. 3.4 "Neighbor fetching").
//
//   score_kernel      materialises fp32 scores (standalone API call, not on the fast path)
//   select_kernel     fused: streams the projected keys of one (layer, sequence, KV head) through
//                     shared memory with 2-D TMA tiles, scores each row, keeps the scores on chip as
//                     order-preserving 32-bit keys, and finds the exact top-B with a radix select
//                     whose histograms are merged across a thread-block cluster through distributed
//                     shared memory.  Output: ascending positions, ties to the lower position.
//   neighbor_kernel   expands a selection by the DILATE or CLUSTER rule via a bitmask over the
//                     candidate range, compacted in order.
#include <cooperative_groups.h>

#include "tb_common.cuh"
#include "tb_internal.h"

namespace cg = cooperative_groups;

namespace tb {

constexpr int kSelThreads = 256;
constexpr int kTileRows = 256;      // rows per TMA box = one row per thread
constexpr int kStages = 3;
constexpr int kBins = 2048;         // 11-bit digits (the last pass uses 10 bits)
constexpr int kMaxCluster = 8;

// Optional per-phase timestamps of block (0,0) and of the last block, for tuning builds only
// (-DTB_PHASE_TIMING); the product build compiles these away.
#ifdef TB_PHASE_TIMING
__device__ unsigned long long g_phase_ns[2][16];
__device__ __forceinline__ void phase_stamp(int i) {
    if (threadIdx.x == 0 && blockIdx.y == 0 && (blockIdx.x == 0 || blockIdx.x == gridDim.x - 1)) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        g_phase_ns[blockIdx.x == 0 ? 0 : 1][i] = t;
    }
}
extern "C" int tb_debug_phase_ns(unsigned long long* out) {
    return (int)cudaMemcpyFromSymbol(out, g_phase_ns, sizeof(g_phase_ns));
}
#else
__device__ __forceinline__ void phase_stamp(int) {}
#endif

// ---- scoring arithmetic shared by the standalone and the fused kernel --------------------------

// Importance query of KV head h: sum over the g query heads of the group, in head order.
template <int DP>
__device__ __forceinline__ void load_group_query(const float* __restrict__ q_imp_unit, int g, float* qr) {
#pragma unroll
    for (int j = 0; j < DP; ++j) qr[j] = 0.f;
    for (int u = 0; u < g; ++u)
#pragma unroll
        for (int j = 0; j < DP; ++j) qr[j] += q_imp_unit[u * DP + j];
}

// Dot product of one projected-key row (NCH 16-byte chunks fetched by `ld(c)`) with qr.  Two FMA
// chains (even / odd chunks), each in ascending element order, added at the end: the result depends
// only on the row's bytes, never on where the row sits.
template <typename T, int DP, typename LoadChunk>
__device__ __forceinline__ float row_score(const float* qr, LoadChunk ld) {
    constexpr int P = Elem<T>::kPer16;
    constexpr int NCH = DP / P;
    float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
        uint4 v = ld(c);
        float f[P];
        Elem<T>::unpack16(v, f);
        if (c & 1) {
#pragma unroll
            for (int e = 0; e < P; ++e) acc1 = fmaf(qr[c * P + e], f[e], acc1);
        } else {
#pragma unroll
            for (int e = 0; e < P; ++e) acc0 = fmaf(qr[c * P + e], f[e], acc0);
        }
    }
    return acc0 + acc1;
}

__device__ __forceinline__ void decode_unit(const Geom& gm, const UnitTable& ut, int u, int& ll, int& s, int& h) {
    h = u % gm.Hkv;
    s = (u / gm.Hkv) % ut.n_seq;
    ll = u / (gm.Hkv * ut.n_seq);
}
__device__ __forceinline__ size_t cache_unit(const Geom& gm, const UnitTable& ut, int ll, int s, int h) {
    return ((size_t)(ut.layer_begin + ll) * gm.max_batch + ut.seq_id[s]) * gm.Hkv + h;
}

// ---- standalone scores ---------------------------------------------------------------------------

template <typename T, int DP>
__global__ void __launch_bounds__(256) score_kernel(Geom gm, UnitTable ut, const float* __restrict__ q_imp, float scale,
                                                    const T* __restrict__ kimp, float* __restrict__ scores) {
    constexpr int NCH = DP / Elem<T>::kPer16;
    int ll, s, h;
    decode_unit(gm, ut, blockIdx.y, ll, s, h);
    const int L = ut.len[ll * ut.n_seq + s];
    float qr[DP];
    load_group_query<DP>(q_imp + ((size_t)(ll * ut.n_seq + s) * gm.Hq + h * gm.g) * DP, gm.g, qr);
    const uint4* base = reinterpret_cast<const uint4*>(kimp + cache_unit(gm, ut, ll, s, h) * gm.max_seq_len * DP);
    float* out = scores + ((size_t)(ll * ut.n_seq + s) * gm.Hkv + h) * gm.max_seq_len;
    for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < L; t += gridDim.x * blockDim.x) {
        const uint4* row = base + (size_t)t * NCH;
        float sc = row_score<T, DP>(qr, [&](int c) { return __ldg(row + c); });
        out[t] = scale * sc;
    }
}

cudaError_t launch_score(const tb_ctx* c, const UnitTable& ut, const float* q_imp, float scale, float* scores, cudaStream_t s) {
    const Geom& gm = c->geom;
    int maxL = 0;
    for (int i = 0; i < ut.layer_count * ut.n_seq; ++i) maxL = ut.len[i] > maxL ? ut.len[i] : maxL;
    if (maxL == 0) return cudaSuccess;
    dim3 grid((maxL + 255) / 256, ut.layer_count * ut.n_seq * gm.Hkv);
    if (grid.x > 64) grid.x = 64;
#define TB_SCORE(T, DP) score_kernel<T, DP><<<grid, 256, 0, s>>>(gm, ut, q_imp, scale, (const T*)c->kimp, scores)
    if (gm.dtype == TB_BF16) {
        if (gm.dp == 32) TB_SCORE(__nv_bfloat16, 32); else TB_SCORE(__nv_bfloat16, 16);
    } else {
        if (gm.dp == 32) TB_SCORE(float, 32); else TB_SCORE(float, 16);
    }
#undef TB_SCORE
    return cudaGetLastError();
}

// ---- fused score + exact top-B -------------------------------------------------------------------

struct SelSmem {
    uint64_t full[kStages];
    int warp_a[kSelThreads / 32];
    int warp_b[kSelThreads / 32];
    int tot[kMaxCluster][2];
    int bc_bin, bc_krem, bc_count;
};

// Finds, over `nbins` counters ordered by digit value, the digit b with
//   count(digits > b) < k <= count(digits >= b)
// and returns it with k' = k - count(digits > b) and the population of b.  All threads call it and
// all receive the same answer.  k >= 1 and k <= total count are preconditions.
__device__ __forceinline__ void find_digit(const int* __restrict__ hist, int nbins, int k, SelSmem* sm, int& bin, int& krem,
                                           int& bcount) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int per = nbins / kSelThreads;             // 8 or 4 digits per thread, highest digits first
    const int top = nbins - 1 - tid * per;
    int mine = 0;
    for (int i = 0; i < per; ++i) mine += hist[top - i];
    int incl = warp_incl_scan(mine, lane);
    if (lane == 31) sm->warp_a[warp] = incl;
    __syncthreads();
    int before = 0;
    for (int w = 0; w < warp; ++w) before += sm->warp_a[w];
    incl += before;
    int excl = incl - mine;
    if (excl < k && k <= incl) {                     // exactly one thread
        int run = excl;
        for (int i = 0; i < per; ++i) {
            int cnt = hist[top - i];
            if (run + cnt >= k) {
                sm->bc_bin = top - i;
                sm->bc_krem = k - run;
                sm->bc_count = cnt;
                break;
            }
            run += cnt;
        }
    }
    __syncthreads();
    bin = sm->bc_bin, krem = sm->bc_krem, bcount = sm->bc_count;
    __syncthreads();                                  // bc_* and warp_a may be reused right away
}

template <typename T, int DP>
__global__ void __launch_bounds__(kSelThreads) select_kernel(const __grid_constant__ CUtensorMap tmap, Geom gm, UnitTable ut,
                                                             SelectArgs a, int tiles_per_cta, int32_t* __restrict__ state_idx,
                                                             int32_t* __restrict__ state_cnt, int32_t* __restrict__ status) {
    constexpr int RB = DP * Elem<T>::kBytes;          // bytes per projected-key row: 32, 64 or 128
    constexpr int NCH = RB / 16;
    constexpr uint32_t kTileBytes = kTileRows * RB;

    extern __shared__ unsigned char smem_raw[];
    // swizzled TMA boxes need their shared-memory base on the swizzle period (up to 1024 bytes)
    unsigned char* stage_base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // kStages * kTileBytes
    int* hist = reinterpret_cast<int*>(stage_base + kStages * kTileBytes);        // local histogram
    int* merged = hist + kBins;                                                   // 3 cluster-merged histograms
    SelSmem* sm = reinterpret_cast<SelSmem*>(merged + 3 * kBins);
    uint32_t* keys = reinterpret_cast<uint32_t*>(sm + 1);                         // tiles_per_cta * kTileRows

    cg::cluster_group cluster = cg::this_cluster();
    const int C = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    int ll, s, h;
    decode_unit(gm, ut, blockIdx.y, ll, s, h);
    const int L = ut.len[ll * ut.n_seq + s];
    const int lo = min(a.sinks, L);
    const int hi = max(lo, L - a.recent);
    const int ncand = hi - lo;
    const int k = min(a.budget, ncand);
    const size_t cu = cache_unit(gm, ut, ll, s, h);
    const size_t dst_row = a.dst_is_state ? cu : (size_t)blockIdx.y;
    int32_t* idx_dst = (a.dst_is_state ? state_idx : a.idx_dst) + dst_row * a.idx_stride;
    int32_t* cnt_dst = (a.dst_is_state ? state_cnt : a.cnt_dst) + dst_row;

    // Everything above is uniform over the cluster, so these early exits are taken by all of its
    // blocks together and no block waits for one that left.
    if (k <= 0) {
        if (rank == 0 && tid == 0) *cnt_dst = 0;
        return;
    }
    if (k == ncand) {                                  // budget covers every candidate: no ranking needed
        for (int i = rank * kSelThreads + tid; i < ncand; i += C * kSelThreads) idx_dst[i] = lo + i;
        if (rank == 0 && tid == 0) *cnt_dst = k;
        return;
    }

    // ---- set-up -------------------------------------------------------------------------------
    phase_stamp(0);
    for (int i = tid; i < 4 * kBins; i += kSelThreads) hist[i] = 0;               // local + 3 merged
    if (tid == 0) {
        prefetch_tmap(&tmap);
        for (int i = 0; i < kStages; ++i) mbar_init(&sm->full[i], 1);
        fence_mbar_init();
    }
    __syncthreads();
    if (C > 1) cluster.sync();                         // every block's merged histograms are zero before any push

    phase_stamp(1);
    const int n_tiles = (ncand + kTileRows - 1) / kTileRows;
    const int tile0 = rank * tiles_per_cta;
    const int my_tiles = max(0, min(tiles_per_cta, n_tiles - tile0));
    const int tok0 = lo + tile0 * kTileRows;           // token of local slot 0
    const int n_local = max(0, min(my_tiles * kTileRows, hi - tok0));
    const long long row_base = (long long)cu * gm.max_seq_len + tok0;   // row of the 2-D view of the cache

    float qr[DP];
    load_group_query<DP>(a.q_imp + ((size_t)(ll * ut.n_seq + s) * gm.Hq + h * gm.g) * DP, gm.g, qr);

    if (tid == 0) {
        for (int i = 0; i < kStages && i < my_tiles; ++i) {
            mbar_arrive_expect_tx(&sm->full[i], kTileBytes);
            tma_load_2d(stage_base + i * kTileBytes, &tmap, 0, (int)(row_base + (long long)i * kTileRows), &sm->full[i]);
        }
    }

    // ---- stream + score + first digit histogram -------------------------------------------------
    bool timed_out = false;
    for (int i = 0; i < my_tiles; ++i) {
        const int st = i % kStages;
        if (!mbar_wait(&sm->full[st], (i / kStages) & 1)) timed_out = true;   // keep going: control flow stays uniform
        const unsigned char* tile = stage_base + st * kTileBytes;
        const int slot = i * kTileRows + tid;
        if (slot < n_local) {
            const uint32_t off = tid * RB;
            float sc = row_score<T, DP>(qr, [&](int c) {
                uint32_t o = off + c * 16;
                o ^= ((o >> 7) & (NCH - 1)) << 4;      // TMA swizzle of 16-byte chunks (mode = row size)
                return *reinterpret_cast<const uint4*>(tile + o);
            });
            uint32_t key = order_key(sc);
            keys[slot] = key;
            atomicAdd(&hist[key >> 21], 1);
        }
        __syncthreads();                               // all reads of this stage are done
        if (tid == 0 && i + kStages < my_tiles) {
            fence_proxy_async();
            mbar_arrive_expect_tx(&sm->full[st], kTileBytes);
            tma_load_2d(stage_base + st * kTileBytes, &tmap, 0, (int)(row_base + (long long)(i + kStages) * kTileRows),
                        &sm->full[st]);
        }
    }
    if (timed_out && lane == 0) atomicExch(status, kStatusTimeout);
    phase_stamp(2);

    // ---- radix select: three digits (11, 11, 10 bits), histograms merged over the cluster --------
    uint32_t prefix = 0;          // digits fixed so far (value of key >> low_bits)
    int low_bits = 32;            // bits of the key not yet fixed
    int krem = k;
    bool exact = false;           // the class {key >> low_bits == prefix} is taken whole
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
        const int bits = pass == 2 ? 10 : 11;
        const int nbins = 1 << bits;
        const int shift = low_bits - bits;
        if (pass > 0) {
            if (!exact) {
                for (int i = tid; i < n_local; i += kSelThreads) {
                    uint32_t key = keys[i];
                    if ((key >> low_bits) == prefix) atomicAdd(&hist[(key >> shift) & (nbins - 1)], 1);
                }
            }
            __syncthreads();
        }
        const int* src = hist;
        if (C > 1) {
            if (!exact) {
                for (int b = tid; b < nbins; b += kSelThreads) {
                    int v = hist[b];
                    if (v)
                        for (int r = 0; r < C; ++r) atomicAdd(cluster.map_shared_rank(&merged[pass * kBins + b], r), v);
                }
            }
            cluster.sync();
            src = merged + pass * kBins;
        }
        if (!exact) {
            int bin, kr, bc;
            find_digit(src, nbins, krem, sm, bin, kr, bc);
            prefix = (prefix << bits) | (uint32_t)bin;
            low_bits = shift;
            krem = kr;
            if (bc == kr) exact = true;                // whole class fits: later digits cannot matter
            for (int i = tid; i < kBins; i += kSelThreads) hist[i] = 0;
        }
        __syncthreads();
        phase_stamp(3 + pass);
    }

    // ---- ordered compaction ------------------------------------------------------------------------
    // A slot is taken if its key is above the class, or inside the class and among the class's first
    // `krem` members in position order (the lower-position tie rule).
    const int seg = ((n_local + kSelThreads - 1) / kSelThreads) * 32;   // slots per warp, multiple of 32
    const int seg_begin = min(n_local, warp * seg), seg_end = min(n_local, (warp + 1) * seg);
    int n_gt = 0, n_eq = 0;
    for (int i = seg_begin + lane; i < seg_end; i += 32) {
        uint32_t kk = keys[i] >> low_bits;
        n_gt += kk > prefix;
        n_eq += kk == prefix;
    }
    n_gt = warp_sum_int(n_gt);
    n_eq = warp_sum_int(n_eq);
    if (lane == 0) sm->warp_a[warp] = n_gt, sm->warp_b[warp] = n_eq;
    __syncthreads();
    int gt_before = 0, eq_before = 0, gt_cta = 0, eq_cta = 0;
    for (int w = 0; w < kSelThreads / 32; ++w) {
        if (w < warp) gt_before += sm->warp_a[w], eq_before += sm->warp_b[w];
        gt_cta += sm->warp_a[w], eq_cta += sm->warp_b[w];
    }
    if (C > 1) {
        if (tid < C) {
            int* dst = cluster.map_shared_rank(&sm->tot[rank][0], tid);
            dst[0] = gt_cta, dst[1] = eq_cta;
        }
        cluster.sync();
        for (int r = 0; r < rank; ++r) gt_before += sm->tot[r][0], eq_before += sm->tot[r][1];
    }
    phase_stamp(6);
    int out_pos = gt_before + min(eq_before, krem);
    const unsigned lt_mask = (1u << lane) - 1u;
    for (int i0 = seg_begin; i0 < seg_end; i0 += 32) {
        const int i = i0 + lane;
        uint32_t kk = 0;
        bool in = i < seg_end;
        if (in) kk = keys[i] >> low_bits;
        const bool is_gt = in && kk > prefix, is_eq = in && kk == prefix;
        const unsigned eq_ballot = __ballot_sync(0xffffffffu, is_eq);
        const bool take = is_gt || (is_eq && eq_before + __popc(eq_ballot & lt_mask) < krem);
        const unsigned take_ballot = __ballot_sync(0xffffffffu, take);
        if (take) idx_dst[out_pos + __popc(take_ballot & lt_mask)] = tok0 + i;
        out_pos += __popc(take_ballot);
        eq_before += __popc(eq_ballot);
    }
    if (rank == 0 && tid == 0) *cnt_dst = k;
    phase_stamp(7);
}

size_t select_smem_bytes(const tb_ctx* c, int tiles_per_cta) {
    int rb = c->geom.dp * (c->geom.dtype == TB_BF16 ? 2 : 4);
    return 1024 + (size_t)kStages * kTileRows * rb + 4 * kBins * sizeof(int) + sizeof(SelSmem) + (size_t)tiles_per_cta * kTileRows * 4;
}

cudaError_t launch_select(const tb_ctx* c, const UnitTable& ut, const SelectArgs& a, cudaStream_t s) {
    const Geom& gm = c->geom;
    const int n_units = ut.layer_count * ut.n_seq * gm.Hkv;
    int max_cand = 0;
    for (int i = 0; i < ut.layer_count * ut.n_seq; ++i) {
        int L = ut.len[i], lo = a.sinks < L ? a.sinks : L, hi = L - a.recent > lo ? L - a.recent : lo;
        if (hi - lo > max_cand) max_cand = hi - lo;
    }
    const int n_tiles = (max_cand + kTileRows - 1) / kTileRows;
    // Cluster size: enough blocks to cover the GPU about twice, at least 4 tiles per block, and a
    // key array per block of at most 64 KB.
    int C = 1;
    while (C < kMaxCluster && (n_units * C < 2 * c->sm_count && n_tiles / (2 * C) >= 4)) C *= 2;
    while (C < kMaxCluster && (n_tiles + C - 1) / C * kTileRows > 8192) C *= 2;
    int tiles_per_cta = (n_tiles + C - 1) / C;
    if (tiles_per_cta < 1) tiles_per_cta = 1;
    if (tiles_per_cta * kTileRows > 16384) return cudaErrorInvalidConfiguration;
    size_t smem = select_smem_bytes(c, tiles_per_cta);

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(C, n_units, 1);
    cfg.blockDim = dim3(kSelThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = C;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;

#define TB_SEL(T, DP)                                                                                              \
    do {                                                                                                           \
        static bool configured = false;                                                                            \
        if (!configured) {                                                                                         \
            cudaError_t e = cudaFuncSetAttribute(select_kernel<T, DP>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                                 200 * 1024);                                                      \
            if (e != cudaSuccess) return e;                                                                        \
            configured = true;                                                                                     \
        }                                                                                                          \
        return cudaLaunchKernelEx(&cfg, select_kernel<T, DP>, c->kimp_map, gm, ut, a, tiles_per_cta, c->st.idx,    \
                                  c->st.cnt, c->st.status);                                                        \
    } while (0)
    if (gm.dtype == TB_BF16) {
        if (gm.dp == 32) TB_SEL(__nv_bfloat16, 32); else TB_SEL(__nv_bfloat16, 16);
    } else {
        if (gm.dp == 32) TB_SEL(float, 32); else TB_SEL(float, 16);
    }
#undef TB_SEL
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
    const int L = ut.len[ll * ut.n_seq + s];
    const int lo = min(a.sinks, L), hi = max(lo, L - a.recent);
    const int span = hi - lo;
    const int n_words = (span + 31) / 32;
    const int32_t* src = a.idx_src + (size_t)blockIdx.x * a.src_stride;
    const int cnt = a.cnt_src[blockIdx.x];
    const size_t cu = cache_unit(gm, ut, ll, s, h);
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

cudaError_t launch_neighbors(const tb_ctx* c, const UnitTable& ut, const NeighborArgs& a, cudaStream_t s) {
    const Geom& gm = c->geom;
    int max_span = 0;
    for (int i = 0; i < ut.layer_count * ut.n_seq; ++i) {
        int L = ut.len[i], lo = a.sinks < L ? a.sinks : L, hi = L - a.recent > lo ? L - a.recent : lo;
        if (hi - lo > max_span) max_span = hi - lo;
    }
    size_t smem = (size_t)((max_span + 31) / 32) * 4 + 16;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(neighbor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    if (smem > 200 * 1024) return cudaErrorInvalidConfiguration;
    neighbor_kernel<<<ut.layer_count * ut.n_seq * gm.Hkv, kNbThreads, smem, s>>>(gm, ut, a, c->st.idx, c->st.cnt);
    return cudaGetLastError();
}

// ---- copy stored lists out --------------------------------------------------------------------------

__global__ void copy_lists_kernel(Geom gm, UnitTable ut, const int32_t* __restrict__ state_idx, const int32_t* __restrict__ state_cnt,
                                  int32_t* __restrict__ idx_out, int32_t* __restrict__ cnt_out) {
    int ll, s, h;
    decode_unit(gm, ut, blockIdx.x, ll, s, h);
    const size_t cu = cache_unit(gm, ut, ll, s, h);
    const int n = state_cnt[cu];
    if (idx_out)
        for (int i = threadIdx.x; i < n; i += blockDim.x) idx_out[(size_t)blockIdx.x * gm.idx_cap + i] = state_idx[cu * gm.idx_cap + i];
    if (cnt_out && threadIdx.x == 0) cnt_out[blockIdx.x] = n;
}

cudaError_t launch_copy_lists(const tb_ctx* c, const UnitTable& ut, int32_t* idx_out, int32_t* cnt_out, cudaStream_t s) {
    copy_lists_kernel<<<ut.layer_count * ut.n_seq * c->geom.Hkv, 256, 0, s>>>(c->geom, ut, c->st.idx, c->st.cnt, idx_out, cnt_out);
    return cudaGetLastError();
}

}  // namespace tb
