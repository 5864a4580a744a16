// Fused importance scoring + exact top-B selection (paper Sec. 3.4 "score computation against all
// projected keys ... top-B selection", Sec. 4 "Token Selection Policy").
//
// One thread-block cluster (1..8 blocks) per (layer, sequence, KV head).  Each block streams its share
// of the candidate rows of the projected-key cache through shared memory with 2-D TMA tiles, scores
// every row, and keeps the scores on chip as order-preserving 32-bit keys (scores never go to HBM).
// The exact top-B is a radix select on those keys whose first digit is placed by a look at the data:
//   sample      every block of the cluster scores the same 64 rows spread over the problem and
//               brackets, generously, where the B-th largest score will fall.  The first digit has
//               1024 bins: 1022 equal slices of key space across the bracket, one open bin below, one
//               above.  It is monotone in the key whatever the sample says, so the result never
//               depends on the sample; only how few keys share the threshold's bin does (a handful).
//   stream      score, key, first-digit histogram.
//   exchange    every block sends its histogram (16-bit counts) to every peer through distributed shared
//               memory, one cluster barrier; every block then finds the threshold bin and every rank's
//               counts above and inside it from its own copy -- no remote read, no serial section.
//   candidates  one pass over the block's keys turns "above the threshold bin" into a bitmask and sends
//               the few keys inside the bin, with their positions, to every peer; second barrier; every
//               block ranks that short list itself (equal keys by position), sets its winners' bits and
//               writes its part of the ascending list.
// A distributed-memory round trip costs 0.3-0.7 us on this part and a cluster barrier 0.2 us, so the
// finish is built from two one-way exchanges instead of request/response steps.
// Unusual inputs (a crowded threshold bin: massive ties, a threshold outside the bracket) and problems
// too small to sample take the general path: the key's own digits (11 + 11 + 10 bits) through
// cluster-merged histograms, then an ordered compaction.
#include <cooperative_groups.h>

#include <cstddef>

#include "tb_select.cuh"

namespace cg = cooperative_groups;

namespace tb {

constexpr int kSelThreads = 256;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kTileRows = 256;      // rows per TMA box = one row per thread
constexpr int kMaxStages = 12;      // depth of the TMA ring is chosen per launch (bytes in flight vs. blocks per SM)
constexpr int kBins = 2048;         // 11-bit digits of the general path (the last digit has 10 bits)
constexpr int kMaxCluster = 8;
constexpr int kMaxKeysPerBlock = 32768;   // 128 KB of on-chip keys per block at most (and 16-bit histogram counts)
constexpr int kFastBins = 1024;     // bins of the sampled first digit
constexpr int kFastCand = 256;      // keys of the threshold bin that every block ranks itself
constexpr int kSampleRows = 64;     // rows scored up front to place the first digit's bins
constexpr int kMinSampled = 2048;   // smaller problems use the key's top bits as first digit
#ifndef TB_CW_FROM
#define TB_CW_FROM (48 * 1024)
#endif
constexpr int kCwFrom = TB_CW_FROM;   // candidates from which the parked-key cluster kernel takes over (macro: tuning builds)
constexpr int kCwLimit = 8 * 262144; // ... and up to which it can (8 blocks x 32 KB of bitmask; the rows' first digits move to the workspace when
                                     // they no longer fit on chip)

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
__device__ unsigned int g_sel_fallbacks[2];
extern "C" int tb_debug_sel_fallbacks(unsigned int* out) { return (int)cudaMemcpyFromSymbol(out, g_sel_fallbacks, sizeof(g_sel_fallbacks)); }
__device__ __forceinline__ void phase_value(int i, unsigned long long v) {
    if (threadIdx.x == 0 && blockIdx.y == 0 && (blockIdx.x == 0 || blockIdx.x == gridDim.x - 1)) g_phase_ns[blockIdx.x == 0 ? 0 : 1][i] = v;
}
#else
__device__ __forceinline__ void phase_stamp(int) {}
__device__ __forceinline__ void phase_value(int, unsigned long long) {}
#endif

struct __align__(16) SelSmem {
    uint32_t peer_hi[kBins];            // directly behind `merged`: together the peers' 16-bit histograms, [8][1024]
    uint32_t sample[kSampleRows];       // read with 16-byte loads
    uint64_t full[kMaxStages];
    int warp_a[kSelWarps];
    int warp_b[kSelWarps];
    int tot[kMaxCluster][2];
    int bc_bin, bc_krem, bc_count, n_cand;
    uint32_t s_lo, s_hi;                // sample keys bracketing the expected threshold
    int pad1[2];
    int inbin[kMaxCluster];             // per rank: keys in the threshold bin
    int winners[kMaxCluster];           // per rank: keys of the threshold bin that made it
    alignas(16) float qs[kMaxGroup * 32];           // TB_GROUP_MAX: the group's importance queries
};

static_assert(offsetof(SelSmem, peer_hi) == 0, "the peers' histograms continue from `merged` into peer_hi");
static_assert(offsetof(SelSmem, qs) % 16 == 0 && offsetof(SelSmem, sample) % 16 == 0, "read with 16-byte loads");
static_assert(kMaxCluster * kFastBins * 2 <= 2 * kBins * 4, "peers' histograms fit merged + peer_hi");

__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ void smem_add(int* p, int v) {
    asm volatile("red.shared.add.s32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
}

// First digit of the fast path: 1024 bins, monotone in the key.  Bin 0 = below `base`, bins 1..1022 =
// equal slices of 2^shift keys from `base` up, bin 1023 = everything above.
struct SampledDigit {
    uint32_t base;
    int shift;
    __device__ __forceinline__ int bin(uint32_t key) const {
        return key < base ? 0 : (int)min((key - base) >> shift, (uint32_t)(kFastBins - 2)) + 1;
    }
};

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

// Finds, over PER*256 counters ordered by digit value (thread `tid` holds counters tid*PER .. +PER-1 in
// `b`), the digit d with
//   count(digits > d) < k <= count(digits >= d)
// and returns it with k' = k - count(digits > d) and the population of d.  All threads call it and
// all receive the same answer.  Preconditions: 1 <= k <= total count.
template <int PER>
__device__ __forceinline__ void find_digit_regs(const int (&b)[PER], int k, SelSmem* sm, int& bin, int& krem, int& bcount) {
    const int tid = threadIdx.x;
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
template <int PER>
__device__ __forceinline__ void find_digit(const int* hist, int k, SelSmem* sm, int& bin, int& krem, int& bcount) {
    int b[PER];
    load_bins<PER>(hist, threadIdx.x, b);
    find_digit_regs<PER>(b, k, sm, bin, krem, bcount);
}

template <typename T, int DP, int RED>
__global__ void __launch_bounds__(kSelThreads) select_kernel(const __grid_constant__ CUtensorMap tmap, const unsigned char* __restrict__ kimp,
                                                             Geom gm, UnitTable ut, SelectArgs a, int tiles_per_cta, int n_stages,
                                                             uint32_t wait_limit, int drop_tile,
                                                             int32_t* __restrict__ state_idx, int32_t* __restrict__ state_cnt,
                                                             int32_t* __restrict__ status) {
    constexpr int RB = DP * Elem<T>::kBytes;          // bytes per projected-key row: 32, 64 or 128
    constexpr int NCH = RB / 16;
    constexpr uint32_t kTileBytes = kTileRows * RB;

    extern __shared__ unsigned char smem_raw[];
    // swizzled TMA boxes need their shared-memory base on the swizzle period (up to 1024 bytes)
    unsigned char* stage_base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // n_stages * kTileBytes
    int* hist = reinterpret_cast<int*>(stage_base + n_stages * kTileBytes);       // local histogram
    int* merged = hist + kBins;                                                   // general path: cluster-merged first-digit histogram
    SelSmem* sm = reinterpret_cast<SelSmem*>(merged + kBins);
    uint32_t* keys = reinterpret_cast<uint32_t*>(sm + 1);                         // tiles_per_cta * kTileRows
    unsigned char* sample_rows = reinterpret_cast<unsigned char*>(keys + tiles_per_cta * kTileRows);   // kSampleRows * RB
    // fast path: every rank's first-digit histogram, 16-bit counts, written by the peers (merged + sm->peer_hi)
    uint16_t* peer_hist = reinterpret_cast<uint16_t*>(merged);                    // [kMaxCluster][kFastBins]
    // The ring is idle once the block has streamed its rows.  Its first 16 KB then serve as the merged
    // histograms of digits 2 and 3 (general path) or as bitmask and candidate list (fast path).  Peers
    // write there only after a cluster barrier that every block reaches after its streaming loop.
    int* merged_late = reinterpret_cast<int*>(stage_base);                        // 2 * kBins ints
    uint32_t* mask = reinterpret_cast<uint32_t*>(stage_base);                     // one bit per local slot: up to 4 KB
    uint2* cand = reinterpret_cast<uint2*>(stage_base + kMaxKeysPerBlock / 8);    // kFastCand (key, candidate index) pairs
    uint2* cand_mine = cand + kFastCand;                                          // this block's own, before they are sent

    cg::cluster_group cluster = cg::this_cluster();
    const int C = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    int ll, s, h;
    decode_unit(gm, ut, blockIdx.y, ll, s, h);
    const int L = unit_len(gm, ut, ll, s);
    const int lo = min(a.sinks, L);
    const int hi = max(lo, L - a.recent);
    const int ncand = hi - lo;
    const int k = min(a.budget, ncand);
    check_candidates_projected(gm, ut, ll, s, hi, status);
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
    const int n_tiles = (ncand + kTileRows - 1) / kTileRows;
    const int tile0 = rank * tiles_per_cta;
    const int my_tiles = max(0, min(tiles_per_cta, n_tiles - tile0));
    const int slot0 = tile0 * kTileRows;               // candidate index of local slot 0
    const int tok0 = lo + slot0;                       // its token
    const int n_local = max(0, min(my_tiles * kTileRows, ncand - slot0));
    const long long unit_row = (long long)key_unit(gm, ut, ll, s, h) * gm.max_seq_len;   // row of token 0 in the 2-D view of the cache
    const long long row_base = unit_row + tok0;

    const bool sampled = ncand >= kMinSampled;
    // What everything else waits for is requested first, straight into shared memory with asynchronous
    // copies: the unit's importance queries, then the sample rows.  Requested behind the grid's opening
    // burst of bulk copies they would queue for microseconds (measured: 5 us for the queries, with the
    // ring full and idle meanwhile).  Every block of the cluster reads the same sample rows (L2 hits for
    // all but one); nothing waits for them here: the digit is placed a few tiles into the stream (below).
    {
        const float* q_unit = a.q_imp + query_row(gm, ut, ll, s, h) * DP;
        if (tid < gm.gl * DP)
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(sm->qs + tid)), "l"(q_unit + tid) : "memory");
        asm volatile("cp.async.commit_group;" ::: "memory");
        if (sampled) {
            for (int c = tid; c < kSampleRows * NCH; c += kSelThreads) {
                const int row = c / NCH, ch = c % NCH;
                const int slot = (int)(((long long)row * ncand) / kSampleRows);
                const unsigned char* src = kimp + (size_t)(unit_row + lo + slot) * RB + ch * 16;
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(sample_rows + c * 16)), "l"(src) : "memory");
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    // `issued`: tiles whose copy has been requested.  A wait that runs out (wait_limit polls; a correct
    // run never gets there) makes the block give up streaming: it requests nothing further, still
    // waits -- bounded -- for what it had in flight, scores the rows it never received as the lowest key
    // and goes through every later phase and barrier, so the cluster stays in step and nothing is left
    // in flight at exit.  The caller learns of it from the status word; that call's lists are then
    // unspecified (valid positions, wrong choice).
    int issued = min(n_stages, my_tiles);
    if (tid == 0) {
        prefetch_tmap(&tmap);
        for (int i = 0; i < n_stages; ++i) mbar_init(&sm->full[i], 1);
        fence_mbar_init();
        for (int i = 0; i < issued; ++i) {
            mbar_arrive_expect_tx(&sm->full[i], kTileBytes);
            // drop_tile: diagnostics only (see tb_set_wait_diagnostics): the barrier is armed and the copy left out
            if (i != drop_tile) tma_load_2d(stage_base + i * kTileBytes, &tmap, 0, (int)(row_base + (long long)i * kTileRows), &sm->full[i]);
        }
    }
    phase_stamp(3);
    // local first-digit histogram; the general path's merged one too when the problem starts there (the
    // fast path never reads `merged` as such: the peers overwrite their slots of it, and a fall-back zeroes it)
    for (int i = tid; i < (sampled ? kBins : 2 * kBins); i += kSelThreads) hist[i] = 0;
    if (tid < kMaxCluster) sm->winners[tid] = 0;
    if (tid == 0) sm->n_cand = 0;
    asm volatile("cp.async.wait_group 1;" ::: "memory");                          // this thread's part of the queries
    __syncthreads();
    GroupScorer<T, DP, RED> scorer;
    scorer.load_staged(sm->qs, gm.gl);
    phase_stamp(6);
    // Split cluster barrier: arrive now, wait only before the first access to a peer's shared memory
    // (after the streaming phase), so its latency hides behind the loads.
    // (Sampled problems have written nothing yet that a peer will touch, so their arrival carries no
    // release: a releasing arrival would first wait for the sample rows still in flight.)
    if (C > 1) {
        if (sampled) asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
        else cluster_arrive();
    }

    // ---- where to put the first digit's bins ---------------------------------------------------------
    // Identical in every block of the cluster: same rows, same arithmetic.  Only the bins' resolution
    // depends on the sample, never the result.  Called by all threads, once, when the sample rows have
    // had time to arrive: the keys scored before that are counted then (`done_tiles` of them per thread).
    SampledDigit dg = {0u, 22};
    auto place_digit = [&](int done_tiles) {
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();
        if (tid < kSampleRows) {
            const unsigned char* row = sample_rows + tid * RB;
            sm->sample[tid] = order_key(scorer.score([&](int c) { return *reinterpret_cast<const uint4*>(row + c * 16); }));
        }
        __syncthreads();
        if (tid < kSampleRows) {   // descending rank of this thread's sample key (equal keys by index)
            const uint32_t mine = sm->sample[tid];
            const uint4* s4 = reinterpret_cast<const uint4*>(sm->sample);
            int r = 0;
#pragma unroll 8
            for (int j4 = 0; j4 < kSampleRows / 4; ++j4) {
                const uint4 x = s4[j4];
                const int j = j4 * 4;
                r += (x.x > mine) | ((x.x == mine) & (j < tid));
                r += (x.y > mine) | ((x.y == mine) & (j + 1 < tid));
                r += (x.z > mine) | ((x.z == mine) & (j + 2 < tid));
                r += (x.w > mine) | ((x.w == mine) & (j + 3 < tid));
            }
            // about p * kSampleRows sample keys lie above the threshold (p = k / candidates); bracket it widely
            const float p = (float)k / (float)ncand, mean = p * kSampleRows, sd = sqrtf(mean * (1.f - p));
            // (+- 4 standard deviations of the sample rank: the threshold falls outside about once in 10^4
            // problems, which then take the general path; a tighter bracket means fewer keys per bin)
            const int r_hi = max(0, (int)floorf(mean - 4.f * sd) - 1), r_lo = min(kSampleRows - 1, (int)ceilf(mean + 4.f * sd) + 1);
            if (r == r_hi) sm->s_hi = mine;
            if (r == r_lo) sm->s_lo = mine;
        }
        __syncthreads();
        const uint32_t s_lo = sm->s_lo, s_hi = sm->s_hi;
        uint32_t range = s_hi - s_lo;
        const uint64_t wide = (uint64_t)range + (range >> 1);   // half as much again above the highest bracketing sample
        range = wide > 0xffffffffull ? 0xffffffffu : (uint32_t)wide;
        dg.base = s_lo, dg.shift = 0;
        while ((range >> dg.shift) >= (uint32_t)(kFastBins - 2)) ++dg.shift;
        for (int i = 0; i < done_tiles; ++i) {
            const int slot = i * kTileRows + tid;
            if (slot < n_local) smem_add(&hist[dg.bin(keys[slot])], 1);   // this thread's own earlier keys
        }
    };
    // the tile before which the digit is placed: late enough for the sample to have landed without a wait
    const int place_at = sampled ? min(my_tiles, 6) : -1;
    phase_stamp(1);

    // ---- stream + score + first digit histogram -------------------------------------------------
    bool dead = false;
    int st = 0;
    uint32_t phase = 0;
    for (int i = 0; i < my_tiles; ++i) {
        if (i == place_at) place_digit(i);
        const bool ok = i < issued && mbar_wait(&sm->full[st], phase, wait_limit);
        const unsigned char* tile = stage_base + st * kTileBytes;
        const int slot = i * kTileRows + tid;
        if (slot < n_local) {
            uint32_t key = 0u;
            if (ok) {
                const uint32_t off = tid * RB;
                const float sc = scorer.score([&](int c) {
                    uint32_t o = off + c * 16;
                    o ^= ((o >> 7) & (NCH - 1)) << 4;  // TMA swizzle of 16-byte chunks (mode = row size)
                    return *reinterpret_cast<const uint4*>(tile + o);
                });
                key = order_key(sc);
            }
            keys[slot] = key;
            if (!sampled) smem_add(&hist[key >> 21], 1);
            else if (i >= place_at) smem_add(&hist[dg.bin(key)], 1);
        }
        if (__syncthreads_or(!ok)) dead = true;        // all reads of this stage are done; uniform verdict on the wait
        if (!dead && i + n_stages < my_tiles) {
            if (tid == 0) {
                fence_proxy_async();
                mbar_arrive_expect_tx(&sm->full[st], kTileBytes);
                if (i + n_stages != drop_tile)
                    tma_load_2d(stage_base + st * kTileBytes, &tmap, 0, (int)(row_base + (long long)(i + n_stages) * kTileRows),
                                &sm->full[st]);
            }
            issued = i + n_stages + 1;
        }
        if (++st == n_stages) st = 0, phase ^= 1u;
    }
    if (dead && tid == 0) atomicExch(status, kStatusTimeout);
    if (place_at == my_tiles) {                        // a short share: the digit is placed after its last tile
        place_digit(my_tiles);
        __syncthreads();                               // the histogram is read next
    }
    phase_stamp(2);

    uint32_t prefix = 0;          // general path: digits fixed so far (value of key >> low_bits)
    int low_bits = 32;            // bits of the key not yet fixed
    int krem = k;
    bool exact = false;           // the class {key >> low_bits == prefix} is taken whole
    bool rebuild_first = false;   // general path after a fast-path attempt: the first digit's histogram comes from the keys

    // ---- fast path --------------------------------------------------------------------------------------
    if (sampled) {
        // my histogram, 16-bit counts, into slot `rank` of every block's copy (4 bins = 8 bytes per thread and peer)
        {
            const int4 x = reinterpret_cast<const int4*>(hist)[tid];
            const uint2 packed = make_uint2((uint32_t)x.x | ((uint32_t)x.y << 16), (uint32_t)x.z | ((uint32_t)x.w << 16));
            uint2* mine = reinterpret_cast<uint2*>(peer_hist + rank * kFastBins) + tid;
            if (C > 1) cluster_wait();                 // every peer runs (its shared memory exists) and is past zeroing it
            for (int r = 0; r < C; ++r) *cluster.map_shared_rank(mine, (rank + r) % C) = packed;
        }
        phase_stamp(8);
        if (C > 1) cluster.sync(); else __syncthreads();   // barrier 1: every block's histogram is everywhere, every ring idle
        phase_stamp(9);
        // threshold bin from the cluster's histogram; with it, the keys that the lower ranks hold above the bin
        // (where this block's part of the list starts) and every rank's keys inside it
        int b[4] = {0, 0, 0, 0}, low[4] = {0, 0, 0, 0};
        for (int r = 0; r < C; ++r) {
            const uint2 x = reinterpret_cast<const uint2*>(peer_hist + r * kFastBins)[tid];
            const int c0 = (int)(x.x & 0xffffu), c1 = (int)(x.x >> 16), c2 = (int)(x.y & 0xffffu), c3 = (int)(x.y >> 16);
            b[0] += c0, b[1] += c1, b[2] += c2, b[3] += c3;
            if (r < rank) low[0] += c0, low[1] += c1, low[2] += c2, low[3] += c3;
        }
        int bin, kr, bc;
        find_digit_regs<4>(b, k, sm, bin, kr, bc);
        {
            int la = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) la += tid * 4 + i > bin ? low[i] : 0;
            la = warp_sum_int(la);
            if (lane == 0) sm->warp_b[warp] = la;
            if (tid < C) sm->inbin[tid] = (int)peer_hist[tid * kFastBins + bin];
        }
        __syncthreads();
        int lower_above = 0;
#pragma unroll
        for (int w = 0; w < kSelWarps; ++w) lower_above += sm->warp_b[w];
        phase_stamp(10);
        phase_value(4, (unsigned long long)bin), phase_value(5, (unsigned long long)bc), phase_value(14, (unsigned long long)kr);
        phase_value(15, ((unsigned long long)dg.base << 8) | (unsigned)dg.shift);
        const bool whole = bc == kr;                   // the whole threshold bin is taken: nothing to rank
#ifdef TB_PHASE_TIMING
        if (rank == 0 && tid == 0) atomicAdd(&g_sel_fallbacks[whole || bc <= kFastCand ? 0 : 1], 1u);
#endif
        if (whole || bc <= kFastCand) {
            // Keys of the threshold bin: [bin_from, above_from); keys of the bins above it: [above_from, 2^32), if any.
            const uint64_t above64 = bin == 0 ? (uint64_t)dg.base : bin == kFastBins - 1 ? (1ull << 32) : (uint64_t)dg.base + ((uint64_t)bin << dg.shift);
            const uint64_t from64 = bin == 0 ? 0ull : (uint64_t)dg.base + ((uint64_t)(bin - 1) << dg.shift);
            const uint32_t above_ok = above64 <= 0xffffffffull ? 0xfu : 0u, above_from = (uint32_t)above64;
            const uint32_t from_ok = from64 <= 0xffffffffull ? 0xfu : 0u, bin_from = (uint32_t)from64;
            int cand_base = 0;
            for (int r = 0; r < rank; ++r) cand_base += sm->inbin[r];
            // own keys -> bitmask (lane l of a warp holds slots 128 g + 4 l .. + 3: its four verdicts are a
            // nibble, eight lanes' nibbles make a mask word); own keys of the threshold bin -> every block's list
            const uint4* keys4 = reinterpret_cast<const uint4*>(keys);
            const int n_grp = (n_local + kTileRows - 1) / kTileRows;
#pragma unroll 4
            for (int v = tid; v < n_grp * (kTileRows / 4); v += kSelThreads) {
                const uint4 x = keys4[v];
                const uint32_t kk[4] = {x.x, x.y, x.z, x.w};
                uint32_t ab = (uint32_t)(kk[0] >= above_from) | (uint32_t)(kk[1] >= above_from) << 1 | (uint32_t)(kk[2] >= above_from) << 2 |
                              (uint32_t)(kk[3] >= above_from) << 3;
                uint32_t ge = (uint32_t)(kk[0] >= bin_from) | (uint32_t)(kk[1] >= bin_from) << 1 | (uint32_t)(kk[2] >= bin_from) << 2 |
                              (uint32_t)(kk[3] >= bin_from) << 3;
                ab &= above_ok, ge &= from_ok;
                const uint32_t vm = v * 4 + 3 < n_local ? 0xfu : v * 4 < n_local ? (1u << (n_local - v * 4)) - 1u : 0u;   // slots past the end hold stale keys
                ab &= vm, ge &= vm;
                uint32_t eqm = whole ? 0u : ge & ~ab;
                uint32_t word = (whole ? ge : ab) << (4 * (lane & 7));
                word |= __shfl_xor_sync(0xffffffffu, word, 1);
                word |= __shfl_xor_sync(0xffffffffu, word, 2);
                word |= __shfl_xor_sync(0xffffffffu, word, 4);
                if ((lane & 7) == 0) mask[v >> 3] = word;
                while (eqm) {                          // rare: a handful of keys per block
                    const int e = __ffs(eqm) - 1;
                    eqm &= eqm - 1;
                    cand_mine[atomicAdd(&sm->n_cand, 1)] = make_uint2(kk[e], (uint32_t)(slot0 + v * 4 + e));
                }
            }
            // ... sent to every block's list one (entry, peer) pair per thread: remote stores issued one after
            // the other by the thread that found the key held its whole warp up
            __syncthreads();
            for (int t = tid; t < sm->n_cand * C; t += kSelThreads)
                *cluster.map_shared_rank(&cand[cand_base + t / C], (rank + t % C) % C) = cand_mine[t / C];
            phase_stamp(11);
            if (C > 1) cluster.sync(); else __syncthreads();   // barrier 2: the list is complete everywhere
            // What is left is short and local.  A successor launched as a programmatic dependent (the first
            // layer's attention) may be set up now; it waits for this grid's completion before it reads a list.
            pdl_launch_dependents();
            phase_stamp(12);
            if (!whole) {
                // every block ranks the list itself: an entry counts the entries ranked before it (larger key, or
                // equal key at a lower position) and knows at once whether it is among the `kr` winners
                if (tid < bc) {
                    const uint2 it = cand[tid];
                    int before = 0;
#pragma unroll 4
                    for (int j = 0; j < bc; ++j) {
                        const uint2 o = cand[j];
                        before += (o.x > it.x) | ((o.x == it.x) & (o.y < it.y));
                    }
                    if (before < kr) {
                        int r_of = 0, i_of = tid;
                        while (i_of >= sm->inbin[r_of]) i_of -= sm->inbin[r_of], ++r_of;
                        atomicAdd(&sm->winners[r_of], 1);
                        if (r_of == rank) {
                            const int ls = (int)it.y - slot0;
                            atomicOr(&mask[ls >> 5], 1u << (ls & 31));
                        }
                    }
                }
                __syncthreads();
            }
            phase_stamp(13);
            // ascending list from the mask: each thread owns a run of 16-bit half words
            int out_base = lower_above;
            for (int r = 0; r < rank; ++r) out_base += whole ? sm->inbin[r] : sm->winners[r];
            const uint16_t* mask16 = reinterpret_cast<const uint16_t*>(mask);
            const int n_half = n_grp * (kTileRows / 16);
            const int per = (n_half + kSelThreads - 1) / kSelThreads;
            const int w0 = min(n_half, tid * per), w1 = min(n_half, w0 + per);
            int cnt = 0;
            for (int w = w0; w < w1; ++w) cnt += __popc((uint32_t)mask16[w]);
            int total;
            int o = out_base + block_excl_scan(cnt, sm->warp_b, total);
            for (int w = w0; w < w1; ++w) {
                uint32_t bits = mask16[w];
                while (bits) {
                    const int bpos = __ffs(bits) - 1;
                    bits &= bits - 1;
                    if (o < k) idx_dst[o] = tok0 + w * 16 + bpos;
                    ++o;
                }
            }
            if (rank == 0 && tid == 0) *cnt_dst = k;
            phase_stamp(7);
            return;
        }
        // A crowded threshold bin (massive ties, a threshold outside the bracket).  The decision is the same
        // in every block.  The general path needs the merged histograms zero before any peer adds to them.
        for (int i = tid; i < 2 * kBins; i += kSelThreads) hist[i] = 0;
        for (int i = tid; i < 2 * kBins; i += kSelThreads) merged_late[i] = 0;
        rebuild_first = true;
        if (C > 1) cluster.sync(); else __syncthreads();
    } else {
        // the ring is idle now: clear the part that later serves as merged histograms (see merged_late)
        for (int i = tid; i < 2 * kBins; i += kSelThreads) merged_late[i] = 0;
        __syncthreads();
        if (C > 1) cluster_wait();                     // every peer runs and has zeroed its histograms
    }
    phase_stamp(3);

    // ---- general path: the key's own digits through cluster-merged histograms -----------------------------
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
        const int bits = pass == 2 ? 10 : 11;
        const int nbins = 1 << bits;
        const int shift = low_bits - bits;
        if (pass > 0 || rebuild_first) {
            if (!exact) {
                for (int i = tid; i < n_local; i += kSelThreads) {
                    uint32_t key = keys[i];
                    if (pass == 0 || (key >> low_bits) == prefix) smem_add(&hist[(key >> shift) & (nbins - 1)], 1);
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

// Shared memory of one block without its TMA ring: alignment slack, two histograms, control block, keys, sample rows.
static size_t select_fixed_smem(int tiles_per_cta, int tile_bytes) {
    return 1024 + 2 * kBins * sizeof(int) + sizeof(SelSmem) + (size_t)tiles_per_cta * kTileRows * 4 + (size_t)kSampleRows * (tile_bytes / kTileRows);
}

// Ring depth: the score pass is bound by bytes in flight (bandwidth x loaded latency is about 90 KB
// per SM), so take as many stages as fit while keeping two blocks per SM when the keys leave room
// for that, one block per SM otherwise.  At least 16 KB of ring (reused after streaming).
static int select_stage_count(int tiles_per_cta, int tile_bytes) {
    const size_t fixed = select_fixed_smem(tiles_per_cta, tile_bytes);
    const size_t two_per_sm = 113 * 1024, one_per_sm = 226 * 1024;
    const int min_stages = tile_bytes >= 16384 ? 2 : 16384 / tile_bytes + 1;
    int n = fixed + (size_t)3 * tile_bytes <= two_per_sm ? (int)((two_per_sm - fixed) / tile_bytes)
                                                          : (int)((one_per_sm - fixed) / tile_bytes);
    if (n > kMaxStages) n = kMaxStages;
    if (n > tiles_per_cta && tiles_per_cta >= min_stages) n = tiles_per_cta;
    if (n < min_stages) n = min_stages;
    return n;
}

cudaError_t launch_select(const tb_ctx* c, const UnitTable& ut, const SelectArgs& a, cudaStream_t s, bool dry) {
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
    const bool to_wave = 2 * n_units >= 3 * c->sm_count || max_cand > kCwLimit, to_cw = max_cand > kCwFrom && max_cand <= kCwLimit;
    if (c->drop_tile >= 0 && (to_wave || to_cw)) return cudaErrorInvalidConfiguration;   // wait diagnostics: single-block launches of this kernel only
    if (to_wave) return launch_select_wave(c, ut, a, s, dry);
    // Long problems (beyond ~48K candidates) go to the cluster kernel that parks the keys in memory and
    // keeps 2 bytes per row on chip: two blocks per SM where this one, with 4 bytes per row, has room for
    // one (128K tokens: 70.1 -> 59.1 us per launch; at 32K the two are level, below that this one wins).
    if (to_cw) return launch_select_cw(c, ut, a, s, dry);
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
        if (select_fixed_smem(tpc, tile_b) + 3 * (size_t)tile_b > 113 * 1024) {
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
    size_t smem = select_fixed_smem(tiles_per_cta, tile_bytes) + (size_t)n_stages * tile_bytes;

    // diagnostics of the bounded waits (tb_set_wait_diagnostics): one-shot, single-block launches only
    const uint32_t wait_limit = c->wait_poll_limit > 0 ? (uint32_t)c->wait_poll_limit : kWaitPollLimit;
    const int drop_tile = C == 1 && n_units == 1 ? c->drop_tile : -1;
    if (c->drop_tile >= 0 && drop_tile < 0) return cudaErrorInvalidConfiguration;
    if (dry) return cudaSuccess;
    const_cast<tb_ctx*>(c)->drop_tile = -1;

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
        return cudaLaunchKernelEx(&cfg, select_kernel<T, DP, RED>, c->kimp_map, (const unsigned char*)c->kimp, gm, ut, a, \
                                  tiles_per_cta, n_stages, wait_limit, drop_tile, c->st.idx, c->st.cnt, c->st.status); \
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
