// Fused importance scoring + exact top-B selection (paper Sec. 3.4 "score computation against all
// projected keys ... top-B selection", Sec. 4 "Token Selection Policy").
//
// One thread-block cluster (1..8 blocks) per (layer, sequence, KV head).  Each block streams its share
// of the candidate rows of the projected-key cache through shared memory with 2-D TMA tiles, scores
// every row, and keeps the scores on chip as order-preserving 32-bit keys (scores never go to HBM).
// The exact top-B is a radix select on those keys:
//   digit 1 (top 11 bits)  histogrammed while streaming; the blocks publish their non-empty bins to
//                          each other through distributed shared memory, one cluster barrier, and
//                          every block finds the threshold bin itself;
//   digits 2, 3            only the keys of the threshold bin matter (a few per cent): they are
//                          gathered at rank 0, which finishes alone and hands every rank the
//                          threshold and its output offsets;
//   compaction             ordered (warp ballots), ties taken in position order, ascending list
//                          written straight to its destination.
// Unusual inputs (more non-empty bins than a list holds, a crowded threshold bin) and single-block
// launches take the general path: every digit through cluster-merged histograms.
#include <cooperative_groups.h>

#include <cstddef>

#include "tb_select.cuh"

namespace cg = cooperative_groups;

namespace tb {

constexpr int kSelThreads = 256;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kTileRows = 256;      // rows per TMA box = one row per thread
constexpr int kMaxStages = 12;      // depth of the TMA ring is chosen per launch (bytes in flight vs. blocks per SM)
constexpr int kBins = 2048;         // 11-bit digits (the last digit has 10 bits)
constexpr int kMaxCluster = 8;
constexpr int kMaxKeysPerBlock = 32768;   // 128 KB of on-chip keys per block at most
constexpr int kListCap = 256;       // non-empty first-digit bins a block may publish on the fast path
#ifndef TB_CW_FROM
#define TB_CW_FROM (48 * 1024)
#endif
constexpr int kCwFrom = TB_CW_FROM;   // candidates from which the parked-key cluster kernel takes over (macro: tuning builds)
constexpr int kCwLimit = 8 * 262144; // ... and up to which it can (8 blocks x 32 KB of bitmask; the rows' first digits move to the workspace when
                                     // they no longer fit on chip)
constexpr int kCandCap = 4096;      // keys of the threshold bin gathered at rank 0 (aliases merged[1..2])

// Optional per-phase timestamps of the first and last block of unit 0, for tuning builds only
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

struct __align__(16) SelSmem {
    int res[8];                         // rank 0's verdict: prefix, low_bits, krem, gt_base, eq_base (16-byte stores)
    uint64_t full[kMaxStages];
    int warp_a[kSelWarps];
    int warp_b[kSelWarps];
    int tot[kMaxCluster][2];
    int bc_bin, bc_krem, bc_count, pad0;
    int list_len[kMaxCluster];          // per rank: entries in lists[rank]
    int above[kMaxCluster];             // per rank: keys in bins above the threshold bin
    int inbin[kMaxCluster];             // per rank: keys in the threshold bin
    uint32_t lists[kMaxCluster][kListCap];   // (bin << 16 | count) of every rank's non-empty bins
    alignas(16) float qs[kMaxGroup * 32];           // TB_GROUP_MAX: the group's importance queries
};

static_assert(offsetof(SelSmem, qs) % 16 == 0, "qs is read with 16-byte loads");

__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ void smem_add(int* p, int v) {
    asm volatile("red.shared.add.s32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
}

// PER consecutive counters of thread `tid` (16-byte loads, at most 2-way bank conflicts).
template <int PER>
__device__ __forceinline__ void load_bins(const int* hist, int tid, int (&b)[PER]) {
    const int4* p = reinterpret_cast<const int4*>(hist + tid * PER);
#pragma unroll
    for (int v = 0; v < PER / 4; ++v) {
        const int4 x = p[v];
        b[4 * v] = x.x, b[4 * v + 1] = x.y, b[4 * v + 2] = x.z, b[4 * v + 3] = x.w;
    }
}

// Exclusive prefix of `v` over the block in thread order, and the block total.  One barrier; uses
// `slots` (kSelWarps ints), which must not be reused before the next barrier.
__device__ __forceinline__ int block_excl_scan(int v, int* slots, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int incl = warp_incl_scan(v, lane);
    if (lane == 31) slots[warp] = incl;
    __syncthreads();
    int before = 0;
    total = 0;
#pragma unroll
    for (int w = 0; w < kSelWarps; ++w) {
        const int x = slots[w];
        total += x;
        before += w < warp ? x : 0;
    }
    return before + incl - v;
}

// Finds, over PER*256 counters ordered by digit value, the digit b with
//   count(digits > b) < k <= count(digits >= b)
// and returns it with k' = k - count(digits > b) and the population of b.  All threads call it and
// all receive the same answer.  Preconditions: 1 <= k <= total count.
template <int PER>
__device__ __forceinline__ void find_digit(const int* hist, int k, SelSmem* sm, int& bin, int& krem, int& bcount) {
    const int tid = threadIdx.x;
    int b[PER];
    load_bins<PER>(hist, tid, b);
    int mine = 0;
#pragma unroll
    for (int i = 0; i < PER; ++i) mine += b[i];
    int total;
    const int excl = block_excl_scan(mine, sm->warp_a, total);
    const int above = total - excl - mine;           // keys in digits above this thread's digits
    if (above < k && k <= above + mine) {            // exactly one thread
        int run = above;
        bool done = false;
#pragma unroll
        for (int i = PER - 1; i >= 0; --i) {
            if (!done && run + b[i] >= k) {
                sm->bc_bin = tid * PER + i, sm->bc_krem = k - run, sm->bc_count = b[i];
                done = true;
            }
            run += b[i];
        }
    }
    __syncthreads();
    bin = sm->bc_bin, krem = sm->bc_krem, bcount = sm->bc_count;
    __syncthreads();                                  // bc_* and warp_a may be reused right away
}

template <typename T, int DP, int RED>
__global__ void __launch_bounds__(kSelThreads) select_kernel(const __grid_constant__ CUtensorMap tmap, Geom gm, UnitTable ut,
                                                             SelectArgs a, int tiles_per_cta, int n_stages,
                                                             int32_t* __restrict__ state_idx, int32_t* __restrict__ state_cnt,
                                                             int32_t* __restrict__ status) {
    constexpr int RB = DP * Elem<T>::kBytes;          // bytes per projected-key row: 32, 64 or 128
    constexpr int NCH = RB / 16;
    constexpr uint32_t kTileBytes = kTileRows * RB;

    extern __shared__ unsigned char smem_raw[];
    // swizzled TMA boxes need their shared-memory base on the swizzle period (up to 1024 bytes)
    unsigned char* stage_base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // n_stages * kTileBytes
    int* hist = reinterpret_cast<int*>(stage_base + n_stages * kTileBytes);       // local histogram
    int* merged = hist + kBins;                                                   // cluster-merged first-digit histogram
    SelSmem* sm = reinterpret_cast<SelSmem*>(merged + kBins);
    uint32_t* keys = reinterpret_cast<uint32_t*>(sm + 1);                         // tiles_per_cta * kTileRows
    // The ring is idle once the block has streamed its rows; its first 16 KB then serve as the merged
    // histograms of digits 2 and 3 (general path) or as rank 0's candidate buffer (fast path).  Peers
    // write there only after a cluster barrier that every block reaches after its streaming loop.
    int* merged_late = reinterpret_cast<int*>(stage_base);                        // 2 * kBins ints

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
    const size_t cu = list_unit(gm, ut, ll, s, h);
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
    for (int i = tid; i < 2 * kBins; i += kSelThreads) hist[i] = 0;               // local + merged first digit
    if (tid == 0) {
        prefetch_tmap(&tmap);
        for (int i = 0; i < n_stages; ++i) mbar_init(&sm->full[i], 1);
        fence_mbar_init();
    }
    __syncthreads();
    // Split cluster barrier: arrive now, wait only before the first access to a peer's shared memory
    // (after the streaming phase), so its latency hides behind the loads.
    if (C > 1) cluster_arrive();

    phase_stamp(1);
    const int n_tiles = (ncand + kTileRows - 1) / kTileRows;
    const int tile0 = rank * tiles_per_cta;
    const int my_tiles = max(0, min(tiles_per_cta, n_tiles - tile0));
    const int tok0 = lo + tile0 * kTileRows;           // token of local slot 0
    const int n_local = max(0, min(my_tiles * kTileRows, hi - tok0));
    const long long row_base = (long long)key_unit(gm, ut, ll, s, h) * gm.max_seq_len + tok0;   // row of the 2-D view of the cache

    if (tid == 0) {
        for (int i = 0; i < n_stages && i < my_tiles; ++i) {
            mbar_arrive_expect_tx(&sm->full[i], kTileBytes);
            tma_load_2d(stage_base + i * kTileBytes, &tmap, 0, (int)(row_base + (long long)i * kTileRows), &sm->full[i]);
        }
    }
    GroupScorer<T, DP, RED> scorer;
    scorer.load(a.q_imp + query_row(gm, ut, ll, s, h) * DP, gm.gl, sm->qs);
    if (RED != TB_GROUP_SUM) __syncthreads();

    // ---- stream + score + first digit histogram -------------------------------------------------
    bool timed_out = false;
    int st = 0;
    uint32_t phase = 0;
    for (int i = 0; i < my_tiles; ++i) {
        if (!mbar_wait(&sm->full[st], phase)) timed_out = true;   // keep going: control flow stays uniform
        const unsigned char* tile = stage_base + st * kTileBytes;
        const int slot = i * kTileRows + tid;
        if (slot < n_local) {
            const uint32_t off = tid * RB;
            float sc = scorer.score([&](int c) {
                uint32_t o = off + c * 16;
                o ^= ((o >> 7) & (NCH - 1)) << 4;      // TMA swizzle of 16-byte chunks (mode = row size)
                return *reinterpret_cast<const uint4*>(tile + o);
            });
            uint32_t key = order_key(sc);
            keys[slot] = key;
            smem_add(&hist[key >> 21], 1);
        }
        __syncthreads();                               // all reads of this stage are done
        if (tid == 0 && i + n_stages < my_tiles) {
            fence_proxy_async();
            mbar_arrive_expect_tx(&sm->full[st], kTileBytes);
            tma_load_2d(stage_base + st * kTileBytes, &tmap, 0, (int)(row_base + (long long)(i + n_stages) * kTileRows),
                        &sm->full[st]);
        }
        if (++st == n_stages) st = 0, phase ^= 1u;
    }
    if (timed_out && lane == 0) atomicExch(status, kStatusTimeout);
    // the ring is idle now: clear the part that later serves as merged histograms (see merged_late)
    for (int i = tid; i < 2 * kBins; i += kSelThreads) merged_late[i] = 0;
    __syncthreads();
    phase_stamp(2);

    uint32_t prefix = 0;          // digits fixed so far (value of key >> low_bits)
    int low_bits = 32;            // bits of the key not yet fixed
    int krem = k;
    bool exact = false;           // the class {key >> low_bits == prefix} is taken whole
    int start_pass = 0;
    bool have_bases = false;      // fast path: taken / class counts of the lower ranks are already known
    int gt_base = 0, eq_base = 0;

    // ---- fast path over a cluster ----------------------------------------------------------------
    if (C > 1) {
        // my non-empty first-digit bins -> lists[rank] (own copy), then the same entries to every peer
        int b[8];
        load_bins<8>(hist, tid, b);
        int nz = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) nz += b[i] != 0;
        int total;
        int off = block_excl_scan(nz, sm->warp_b, total);
        if (total <= kListCap) {
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if (b[i]) sm->lists[rank][off++] = ((uint32_t)(tid * 8 + i) << 16) | (uint32_t)b[i];
        }
        if (tid == 0) sm->list_len[rank] = total;
        __syncthreads();
        cluster_wait();                                // all peers run and have zeroed their histograms
        if (total <= kListCap) {
            for (int r = 1; r < C; ++r) {              // one remote store per thread and peer
                const int peer = (rank + r) % C;
                if (tid < total) *cluster.map_shared_rank(&sm->lists[rank][tid], peer) = sm->lists[rank][tid];
            }
        }
        if (tid < C && tid != rank) *cluster.map_shared_rank(&sm->list_len[rank], tid) = total;
        phase_stamp(8);
        cluster.sync();                                // barrier 1
        phase_stamp(9);
        bool fast = true;
        for (int r = 0; r < C; ++r) fast = fast && sm->list_len[r] <= kListCap;
        if (fast) {
            // warp w merges rank w's list into merged[0] (still zero)
            if (warp < C)
                for (int i = lane; i < sm->list_len[warp]; i += 32) {
                    const uint32_t e = sm->lists[warp][i];
                    smem_add(&merged[e >> 16], (int)(e & 0xFFFFu));
                }
            __syncthreads();
            int bin, kr, bc;
            find_digit<8>(merged, k, sm, bin, kr, bc);
            prefix = (uint32_t)bin, low_bits = 21, krem = kr, start_pass = 1;
            if (warp < C) {                            // warp w sums rank w's list around the threshold bin
                int ab = 0, ib = 0;
                for (int i = lane; i < sm->list_len[warp]; i += 32) {
                    const uint32_t e = sm->lists[warp][i];
                    const int eb = (int)(e >> 16), ec = (int)(e & 0xFFFFu);
                    ab += eb > bin ? ec : 0;
                    ib += eb == bin ? ec : 0;
                }
                ab = warp_sum_int(ab), ib = warp_sum_int(ib);
                if (lane == 0) sm->above[warp] = ab, sm->inbin[warp] = ib;
            }
            for (int i = tid; i < kBins; i += kSelThreads) hist[i] = 0;
            __syncthreads();
            phase_stamp(10);
            if (bc == kr) {                            // the whole threshold bin is taken: nothing to refine
                exact = true, have_bases = true, start_pass = 3;
                for (int r = 0; r < rank; ++r) gt_base += sm->above[r], eq_base += sm->inbin[r];
            } else if (bc <= kCandCap) {
                // my keys of the threshold bin -> rank 0 (any order inside my region)
                const uint4* keys4 = reinterpret_cast<const uint4*>(keys);
                const int n_vec = (n_local + 3) / 4;
                int mine = 0;
                for (int v = tid; v < n_vec; v += kSelThreads) {
                    const uint4 x = keys4[v];
                    const int base = v * 4;
                    mine += (base < n_local && (x.x >> 21) == (uint32_t)bin) + (base + 1 < n_local && (x.y >> 21) == (uint32_t)bin) +
                            (base + 2 < n_local && (x.z >> 21) == (uint32_t)bin) + (base + 3 < n_local && (x.w >> 21) == (uint32_t)bin);
                }
                int tot_mine;
                int pos = block_excl_scan(mine, sm->warp_b, tot_mine);
                for (int r = 0; r < rank; ++r) pos += sm->inbin[r];
                uint32_t* cand_local = reinterpret_cast<uint32_t*>(merged_late);
                uint32_t* cand0 = cluster.map_shared_rank(cand_local, 0);
                if (mine) {
                    for (int v = tid; v < n_vec; v += kSelThreads) {
                        const uint4 x = keys4[v];
                        const int base = v * 4;
                        if (base < n_local && (x.x >> 21) == (uint32_t)bin) cand0[pos++] = x.x;
                        if (base + 1 < n_local && (x.y >> 21) == (uint32_t)bin) cand0[pos++] = x.y;
                        if (base + 2 < n_local && (x.z >> 21) == (uint32_t)bin) cand0[pos++] = x.z;
                        if (base + 3 < n_local && (x.w >> 21) == (uint32_t)bin) cand0[pos++] = x.w;
                    }
                }
                phase_stamp(11);
                cluster.sync();                        // barrier 2
                phase_stamp(12);
                if (rank == 0) {
                    uint32_t pf = (uint32_t)bin;
                    int lb = 21, kk = kr;
                    bool ex = false;
#pragma unroll 1
                    for (int pass = 1; pass < 3 && !ex; ++pass) {
                        const int bits = pass == 2 ? 10 : 11, nb = 1 << bits, shift = lb - bits;
#pragma unroll 4
                        for (int i = tid; i < bc; i += kSelThreads) {
                            const uint32_t key = cand_local[i];
                            if ((key >> lb) == pf) smem_add(&hist[(key >> shift) & (nb - 1)], 1);
                        }
                        __syncthreads();
                        int d, kr2, c2;
                        if (pass == 1) find_digit<8>(hist, kk, sm, d, kr2, c2);
                        else find_digit<4>(hist, kk, sm, d, kr2, c2);
                        pf = (pf << bits) | (uint32_t)d, lb = shift, kk = kr2;
                        ex = c2 == kr2;
                        if (!ex) {
                            for (int i = tid; i < kBins; i += kSelThreads) hist[i] = 0;
                            __syncthreads();
                        }
                    }
                    if (warp < C) {                    // warp w counts rank w's candidates against the threshold
                        int base_w = 0;
                        for (int r = 0; r < warp; ++r) base_w += sm->inbin[r];
                        const int n_w = sm->inbin[warp];
                        int gt = 0, eq = 0;
#pragma unroll 4
                        for (int i = lane; i < n_w; i += 32) {
                            const uint32_t kk2 = cand_local[base_w + i] >> lb;
                            gt += kk2 > pf, eq += kk2 == pf;
                        }
                        gt = warp_sum_int(gt), eq = warp_sum_int(eq);
                        if (lane == 0) sm->warp_a[warp] = gt, sm->warp_b[warp] = eq;
                    }
                    __syncthreads();
                    if (tid < C) {
                        int gb = 0, eb = 0;
                        for (int r = 0; r < tid; ++r) gb += sm->above[r] + sm->warp_a[r], eb += sm->warp_b[r];
                        int4* dst = reinterpret_cast<int4*>(cluster.map_shared_rank(&sm->res[0], tid));
                        dst[0] = make_int4((int)pf, lb, kk, gb);
                        dst[1] = make_int4(eb, 0, 0, 0);
                    }
                }
                phase_stamp(13);
                cluster.sync();                        // barrier 3
                phase_stamp(14);
                prefix = (uint32_t)sm->res[0], low_bits = sm->res[1], krem = sm->res[2];
                gt_base = sm->res[3], eq_base = sm->res[4];
                exact = true, have_bases = true, start_pass = 3;   // nothing left for the general passes
            }
        }
    }
    phase_stamp(3);

    // ---- general path: digits not yet fixed are found with cluster-merged histograms ----------------
#pragma unroll 1
    for (int pass = start_pass; pass < 3; ++pass) {
        const int bits = pass == 2 ? 10 : 11;
        const int nbins = 1 << bits;
        const int shift = low_bits - bits;
        if (pass > 0) {
            if (!exact) {
                for (int i = tid; i < n_local; i += kSelThreads) {
                    uint32_t key = keys[i];
                    if ((key >> low_bits) == prefix) smem_add(&hist[(key >> shift) & (nbins - 1)], 1);
                }
            }
            __syncthreads();
        }
        const int* src = hist;
        if (C > 1) {
            int* mrg = pass == 0 ? merged : merged_late + (pass - 1) * kBins;
            if (!exact) {
                for (int b = tid; b < nbins; b += kSelThreads) {
                    int v = hist[b];
                    if (v)
                        for (int r = 0; r < C; ++r) atomicAdd(cluster.map_shared_rank(&mrg[b], r), v);
                }
            }
            cluster.sync();
            src = mrg;
        }
        if (!exact) {
            int bin, kr, bc;
            if (pass == 2) find_digit<4>(src, krem, sm, bin, kr, bc);
            else find_digit<8>(src, krem, sm, bin, kr, bc);
            prefix = (prefix << bits) | (uint32_t)bin;
            low_bits = shift;
            krem = kr;
            if (bc == kr) exact = true;                // whole class fits: later digits cannot matter
            for (int i = tid; i < kBins; i += kSelThreads) hist[i] = 0;
        }
        __syncthreads();
    }

    // ---- ordered compaction ------------------------------------------------------------------------
    // A slot is taken if its key is above the class, or inside the class and among the class's first
    // `krem` members in position order (the lower-position tie rule).  Warp w owns a contiguous range.
    // Within a group of 128 slots lane l holds slots 4l..4l+3 (one 16-byte load), so lane order is
    // position order.
    const uint4* keys4 = reinterpret_cast<const uint4*>(keys);
    const int seg = ((n_local + kSelWarps * 128 - 1) / (kSelWarps * 128)) * 128;   // slots per warp, multiple of 128
    const int seg_begin = min(n_local, warp * seg), seg_end = min(n_local, (warp + 1) * seg);
    auto classify = [&](int base, int& gt_bits, int& eq_bits) {   // bit e set: slot base+e is above / in the class
        gt_bits = eq_bits = 0;
        if (base < seg_end) {
            const uint4 x = keys4[base >> 2];
            const uint32_t v[4] = {x.x >> low_bits, x.y >> low_bits, x.z >> low_bits, x.w >> low_bits};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const bool in = base + e < seg_end;
                gt_bits |= (in && v[e] > prefix) << e;
                eq_bits |= (in && v[e] == prefix) << e;
            }
        }
    };
    int n_gt = 0, n_eq = 0;
#pragma unroll 2
    for (int i0 = seg_begin; i0 < seg_end; i0 += 128) {
        int gb, eb;
        classify(i0 + 4 * lane, gb, eb);
        n_gt += __popc(gb), n_eq += __popc(eb);
    }
    n_gt = warp_sum_int(n_gt);
    n_eq = warp_sum_int(n_eq);
    if (lane == 0) sm->warp_a[warp] = n_gt, sm->warp_b[warp] = n_eq;
    __syncthreads();
    int gt_before = 0, eq_before = 0, gt_cta = 0, eq_cta = 0;
#pragma unroll
    for (int w = 0; w < kSelWarps; ++w) {
        const int x = sm->warp_a[w], y = sm->warp_b[w];
        gt_before += w < warp ? x : 0, eq_before += w < warp ? y : 0;
        gt_cta += x, eq_cta += y;
    }
    if (have_bases) {
        gt_before += gt_base, eq_before += eq_base;
    } else if (C > 1) {
        if (tid < C) {
            int* dst = cluster.map_shared_rank(&sm->tot[rank][0], tid);
            dst[0] = gt_cta, dst[1] = eq_cta;
        }
        cluster.sync();
        for (int r = 0; r < rank; ++r) gt_before += sm->tot[r][0], eq_before += sm->tot[r][1];
    }
    phase_stamp(6);
    int out_pos = gt_before + min(eq_before, krem);
    const uint32_t lt = (1u << lane) - 1u;
    // Exclusive prefix over the warp of a per-lane count 0..4, and the warp total, from three ballots
    // (one per bit of the count) instead of a five-step chain of dependent shuffles.
    auto warp_prefix_small = [&](int n, int& total) {
        const uint32_t b0 = __ballot_sync(0xffffffffu, n & 1), b1 = __ballot_sync(0xffffffffu, n & 2),
                       b2 = __ballot_sync(0xffffffffu, n & 4);
        total = __popc(b0) + 2 * __popc(b1) + 4 * __popc(b2);
        return __popc(b0 & lt) + 2 * __popc(b1 & lt) + 4 * __popc(b2 & lt);
    };
#pragma unroll 2
    for (int i0 = seg_begin; i0 < seg_end; i0 += 128) {
        const int base = i0 + 4 * lane;
        int gb, eb;
        classify(base, gb, eb);
        int take = gb;
        if (__any_sync(0xffffffffu, eb != 0)) {        // class members here: hand out what is left of the quota in order
            int ne_warp;
            int before = eq_before + warp_prefix_small(__popc(eb), ne_warp);
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if ((eb >> e) & 1) {
                    if (before < krem) take |= 1 << e;
                    ++before;
                }
            eq_before += ne_warp;
        }
        if (__any_sync(0xffffffffu, take != 0)) {
            int nt_warp;
            int o = out_pos + warp_prefix_small(__popc(take), nt_warp);
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if ((take >> e) & 1) idx_dst[o++] = tok0 + base + e;
            out_pos += nt_warp;
        }
    }
    if (rank == 0 && tid == 0) *cnt_dst = k;
    phase_stamp(7);
}

// Shared memory of one block without its TMA ring: alignment slack, two histograms, control block, keys.
static size_t select_fixed_smem(int tiles_per_cta) {
    return 1024 + 2 * kBins * sizeof(int) + sizeof(SelSmem) + (size_t)tiles_per_cta * kTileRows * 4;
}

// Ring depth: the score pass is bound by bytes in flight (bandwidth x loaded latency is about 90 KB
// per SM), so take as many stages as fit while keeping two blocks per SM when the keys leave room
// for that, one block per SM otherwise.  At least 16 KB of ring (reused after streaming).
static int select_stage_count(int tiles_per_cta, int tile_bytes) {
    const size_t fixed = select_fixed_smem(tiles_per_cta);
    const size_t two_per_sm = 113 * 1024, one_per_sm = 226 * 1024;
    const int min_stages = tile_bytes >= 16384 ? 2 : 16384 / tile_bytes + 1;
    int n = fixed + (size_t)3 * tile_bytes <= two_per_sm ? (int)((two_per_sm - fixed) / tile_bytes)
                                                          : (int)((one_per_sm - fixed) / tile_bytes);
    if (n > kMaxStages) n = kMaxStages;
    if (n > tiles_per_cta && tiles_per_cta >= min_stages) n = tiles_per_cta;
    if (n < min_stages) n = min_stages;
    return n;
}

cudaError_t launch_select(const tb_ctx* c, const UnitTable& ut, const SelectArgs& a, cudaStream_t s) {
    const Geom& gm = c->geom;
    const int n_units = ut.layer_count * ut.n_seq * gm.Hl;
    int max_cand = 0;
    for (int i = 0; i < ut.layer_count * ut.n_seq; ++i) {
        int L = ut.len[i], lo = a.sinks < L ? a.sinks : L, hi = L - a.recent > lo ? L - a.recent : lo;
        if (hi - lo > max_cand) max_cand = hi - lo;
    }
    // Many problems (one and a half per SM or more; measured crossover between 32 and 256 on 148 SMs)
    // fill the GPU by themselves: one block each, no clusters.  So do problems beyond what the parked-key
    // cluster kernel takes.
    if (2 * n_units >= 3 * c->sm_count || max_cand > kCwLimit) return launch_select_wave(c, ut, a, s);
    // Long problems (beyond ~48K candidates) go to the cluster kernel that parks the keys in memory and
    // keeps 2 bytes per row on chip: two blocks per SM where this one, with 4 bytes per row, has room for
    // one (128K tokens: 70.1 -> 59.1 us per launch; at 32K the two are level, below that this one wins).
    if (max_cand > kCwFrom && max_cand <= kCwLimit) return launch_select_cw(c, ut, a, s);
    const int n_tiles = (max_cand + kTileRows - 1) / kTileRows;
    // Cluster size: enough blocks to cover the GPU about twice, at least 4 tiles per block, and a
    // key array per block of at most 32 KB where the cluster limit allows (64 KB otherwise).
    int C = 1;
    if (2 * n_units > c->sm_count) {
        // several waves of blocks: keep the key array small enough for two blocks per SM, so one
        // block's selection phase overlaps the other's streaming
        while (C < kMaxCluster && (n_tiles + C - 1) / C * kTileRows > 8192) C *= 2;
    } else {
        // few problems: one wave.  Two blocks per SM when their key arrays leave room for two rings
        // (more bytes in flight), otherwise one block per SM.
        const int tile_b = kTileRows * gm.dp * (gm.dtype == TB_BF16 ? 2 : 4);
        C = 2 * c->sm_count / n_units;
        if (C > kMaxCluster) C = kMaxCluster;
        while (C > 1 && n_tiles / C < 4) --C;
        const int tpc = (n_tiles + C - 1) / C;
        if (1024 + 2 * kBins * 4 + sizeof(SelSmem) + (size_t)tpc * kTileRows * 4 + 3 * (size_t)tile_b > 113 * 1024) {
            C = c->sm_count / n_units;
            if (C > kMaxCluster) C = kMaxCluster;
            while (C > 1 && n_tiles / C < 4) --C;
        }
    }
    while (C < kMaxCluster && (n_tiles + C - 1) / C * kTileRows > kMaxKeysPerBlock) ++C;
    int tiles_per_cta = (n_tiles + C - 1) / C;
    if (tiles_per_cta < 1) tiles_per_cta = 1;
    if (tiles_per_cta * kTileRows > kMaxKeysPerBlock) return cudaErrorInvalidConfiguration;
    const int tile_bytes = kTileRows * gm.dp * (gm.dtype == TB_BF16 ? 2 : 4);
    const int n_stages = select_stage_count(tiles_per_cta, tile_bytes);
    size_t smem = select_fixed_smem(tiles_per_cta) + (size_t)n_stages * tile_bytes;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(C, n_units, 1);
    cfg.blockDim = dim3(kSelThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    // No programmatic dependent launch here: a selection that starts while the previous kernel still
    // holds SMs gets its clusters placed in two batches (measured: +13 us per launch).
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = C;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;

#define TB_SEL_R(T, DP, RED)                                                                                       \
    do {                                                                                                           \
        static unsigned char seen[64];                                                                            \
        if (first_use_on_this_device(seen)) {                                                                                         \
            cudaError_t e = cudaFuncSetAttribute(select_kernel<T, DP, RED>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                                 227 * 1024);                                                      \
            if (e != cudaSuccess) return e;                                                                        \
        }                                                                                                          \
        return cudaLaunchKernelEx(&cfg, select_kernel<T, DP, RED>, c->kimp_map, gm, ut, a, tiles_per_cta, n_stages, c->st.idx, \
                                  c->st.cnt, c->st.status);                                                        \
    } while (0)
#define TB_SEL(T, DP)                                            \
    do {                                                         \
        if (a.reduce == TB_GROUP_MAX) TB_SEL_R(T, DP, TB_GROUP_MAX); \
        else TB_SEL_R(T, DP, TB_GROUP_SUM);                      \
    } while (0)
    if (gm.dtype == TB_BF16) {
        if (gm.dp == 32) TB_SEL(__nv_bfloat16, 32); else TB_SEL(__nv_bfloat16, 16);
    } else {
        if (gm.dp == 32) TB_SEL(float, 32); else TB_SEL(float, 16);
    }
#undef TB_SEL
#undef TB_SEL_R
}

}  // namespace tb
