// Fused importance scoring + exact top-B selection on parked keys: the kernel for launches with many
// problems (below) and, at the end of the file, the cluster kernel for few long problems (paper Sec. 3.4
// "score computation against all projected keys ... top-B selection", Sec. 4 "Token Selection
// Policy"): batched serving, where one launch holds several hundred (layer, sequence, KV head)
// problems and the GPU is filled by problems, not by splitting one.
//
// One block per problem, four blocks per SM, longest problems first.
//   sample   the block scores 64 rows spread over its problem and brackets, generously, where the
//            B-th largest score will fall.  That only places the bins of the first radix digit: 2046
//            equal slices across the bracket, one open bin below, one above.  The digit is monotone in
//            the key whatever the sample says, so the result never depends on it; only how few keys
//            share the threshold's bin does (a handful, against a tenth of the problem for the key's
//            top bits).
//   stream   candidate rows of the projected-key cache through a ring of 2-D TMA tiles (evict-first in
//            L2); every row is scored, its order-preserving 32-bit key parked in a workspace row
//            (4 bytes per token against the 64 just read, evict-last so it is still in L2 later) and
//            its first digit counted in shared memory.
//   finish   threshold bin from the histogram; one pass over the parked keys turns "above the bin"
//            into a bitmask (one word per eight lanes) and sets the few keys inside the bin aside;
//            those are ranked among themselves (equal keys by position), the winners' bits set, and a
//            prefix over the mask's popcounts places the ascending list.
//   general  a threshold in the open bin below the bracket, or a bin too crowded to set aside
//            (massive ties), falls back to a plain three-digit radix select over all parked keys with
//            an ordered compaction.  Slower, never wrong.
// No block waits for another.  The cluster kernel in tb_select.cu serves launches with few, large
// problems, where one problem must be split over many SMs; in this regime it would spend its time in
// cluster barriers.
#include <algorithm>
#include <cstddef>

#include "tb_select.cuh"

namespace tb {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kRows = 256;          // rows per TMA box = one row per thread
constexpr int kStagesMax = 8;
constexpr int kDigitBins = 2048;    // 11-bit digits (the last digit has 10 bits)
constexpr int kSampleRows = 64;     // rows scored up front to place the first digit's bins
constexpr int kMinSampled = 2048;   // smaller problems use the key's top bits as first digit
constexpr int kBatch = 8;           // 16-byte key loads a thread keeps in flight

// Launch order of the (layer, sequence) pairs: longest first, so that the blocks still running when
// the grid drains are the short ones.
struct WaveOrder {
    uint16_t pair[kMaxLaunchUnits];
};

#ifdef TB_PHASE_TIMING
__device__ unsigned long long g_fin_ns[8];
__device__ unsigned long long g_cw_ns[8];
__device__ unsigned int g_wave_smid[1024];
__device__ unsigned long long g_fin_blk[4][1024];
__device__ unsigned long long g_wave_ns[4][1024];       // per block: start, first tile landed, rows streamed, end
__device__ __forceinline__ unsigned long long wave_now() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void wave_stamp(int i) {
    if (threadIdx.x == 0 && blockIdx.x < 1024) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        g_wave_ns[i][blockIdx.x] = t;
        if (i == 0) {
            unsigned smid;
            asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
            g_wave_smid[blockIdx.x] = smid;
        }
    }
}
#else
__device__ __forceinline__ void wave_stamp(int) {}
#endif

struct __align__(16) WaveSmem {
    uint32_t sample[kSampleRows];   // first: read with 16-byte loads
    uint64_t full[kStagesMax];
    int warp_a[kWarps];
    int warp_b[kWarps];
    int bc_bin, bc_krem, bc_count, n_list;
    uint32_t s_lo, s_hi;            // sample keys bracketing the expected threshold
    alignas(16) float qs[kMaxGroup * 32];       // TB_GROUP_MAX: the group's importance queries
};
static_assert(offsetof(WaveSmem, sample) % 16 == 0 && offsetof(WaveSmem, qs) % 16 == 0, "read with 16-byte loads");

// First digit of the radix select: 2048 bins, monotone in the key.  Bin 0 = below `base`, bins
// 1..2046 = equal slices of 2^shift keys from `base` up, bin 2047 = everything above.  With base = 0
// and shift = 21 it is the key's top 11 bits; with base and shift taken from a sample of the problem's
// scores the slices around the expected threshold hold a handful of keys each.
struct Digit {
    uint32_t base;
    int shift;
    __device__ __forceinline__ int bin(uint32_t key) const {
        return key < base ? 0 : (int)min((key - base) >> shift, 2046u) + 1;
    }
};

__device__ __forceinline__ void hist_add(int* p) {
    asm volatile("red.shared.add.s32 [%0], 1;" ::"r"(smem_u32(p)) : "memory");
}

// Exclusive prefix of `v` over the block in thread order, and the block total.  One barrier; uses
// `slots` (kWarps ints), which must not be reused before the next barrier.
__device__ __forceinline__ int wave_excl_scan(int v, int* slots, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int incl = warp_incl_scan(v, lane);
    if (lane == 31) slots[warp] = incl;
    __syncthreads();
    int before = 0;
    total = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
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
__device__ __forceinline__ void wave_find_digit(const int* hist, int k, WaveSmem* sm, int& bin, int& krem, int& bcount) {
    const int tid = threadIdx.x;
    int b[PER];
    const int4* p = reinterpret_cast<const int4*>(hist + tid * PER);
#pragma unroll
    for (int v = 0; v < PER / 4; ++v) {
        const int4 x = p[v];
        b[4 * v] = x.x, b[4 * v + 1] = x.y, b[4 * v + 2] = x.z, b[4 * v + 3] = x.w;
    }
    int mine = 0;
#pragma unroll
    for (int i = 0; i < PER; ++i) mine += b[i];
    int total;
    const int excl = wave_excl_scan(mine, sm->warp_a, total);
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

}  // namespace

// Finish of one problem from its complete first-digit histogram, with ONE pass over the keys.
// The first digit already decides almost every key: above the threshold bin = selected, below = not.
// The pass turns that into a bitmask (one ballot per 32 positions) and sets aside the few keys of the
// threshold bin as (low 21 bits, position) pairs; two more digits are then resolved on that short
// list, equal keys by position, the winners' bits are set, and a prefix over the mask's popcounts
// places the ascending list.  `scratch` (the idle ring) holds mask and list.  Returns false, having
// written nothing, when they do not fit (a crowded threshold bin): the caller then takes the general
// path.  All threads call it and all get the same answer.
__device__ __forceinline__ bool wave_finish_mask(int* hist, WaveSmem* sm, const Digit dg, const uint32_t* __restrict__ keys,
                                                 unsigned char* scratch, int scratch_bytes, int ncand, int k, int lo,
                                                 int32_t* __restrict__ idx_dst, int32_t* __restrict__ cnt_dst) {
    const int tid = threadIdx.x, lane = tid & 31;
#ifdef TB_PHASE_TIMING
    unsigned long long tf0 = wave_now();
#define FIN_MARK(i) do { if (tid == 0) { unsigned long long tn = wave_now(); atomicAdd(&g_fin_ns[i], tn - tf0); if (blockIdx.x < 1024 && (i) < 4) g_fin_blk[i][blockIdx.x] = tn - tf0; tf0 = tn; } } while (0)
#else
#define FIN_MARK(i) do {} while (0)
#endif
    int bin, krem, bc;
    wave_find_digit<8>(hist, k, sm, bin, krem, bc);
    FIN_MARK(0);
    const bool exact = bc == krem;                     // the whole threshold bin is selected
    const int n_grp = (ncand + kRows - 1) / kRows;     // groups of 256 positions = 8 mask words
    const int n_words = n_grp * kWarps;
    const int mask_bytes = (n_words * 4 + 15) & ~15;
    uint32_t* mask = reinterpret_cast<uint32_t*>(scratch);
    uint2* list = reinterpret_cast<uint2*>(scratch + mask_bytes);
    // bin 0 (everything below the sampled range) is too crowded to list
    if (mask_bytes > scratch_bytes || (!exact && (bc > (scratch_bytes - mask_bytes) / 8 || bin == 0))) return false;
    const uint32_t bin_base = dg.base + ((uint32_t)(bin - 1) << dg.shift);       // lowest key of the threshold bin
    const int bin_bits = bin == 2047 ? 32 : dg.shift;  // bits of (key - bin_base) inside the bin; the top bin is open-ended
    // Keys of the threshold bin: [bin_from, above_from); keys of the bins above it: [above_from, 2^32), if any.
    // Bin 0 holds the keys below the digit's base, bin 2047 is open-ended.
    const uint64_t above64 = bin == 0 ? (uint64_t)dg.base : bin == 2047 ? (1ull << 32) : (uint64_t)dg.base + ((uint64_t)bin << dg.shift);
    const uint32_t above_mask = above64 <= 0xffffffffull ? 0xfu : 0u;
    const uint32_t above_from = (uint32_t)above64, bin_from = bin == 0 ? 0u : bin_base;
    if (tid == 0) sm->n_list = 0;
    __syncthreads();
#ifdef TB_PHASE_TIMING
    if (tid == 0) atomicAdd(&g_fin_ns[7], 1ull), atomicAdd(&g_fin_ns[6], (unsigned long long)(exact ? 0 : bc));
#endif

    // Lane l of a warp holds positions 128 g + 4 l .. + 3 (one 16-byte load): its four verdicts are a
    // nibble, eight lanes' nibbles make a mask word.
    const uint4* keys4 = reinterpret_cast<const uint4*>(keys);
    const int n_vec = (ncand + 3) / 4;
    for (int v0 = tid; v0 < n_grp * (kRows / 4); v0 += kThreads * kBatch) {   // kBatch loads in flight, then their verdicts
        uint4 x[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int v = v0 + u * kThreads;
            x[u] = make_uint4(0u, 0u, 0u, 0u);
            if (v < n_vec) x[u] = __ldcg(keys4 + v);
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int v = v0 + u * kThreads;
            if (v - lane >= n_grp * (kRows / 4)) break;    // warp-uniform: whole warps leave together
            const uint32_t kk[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
            // the keys' digits against the threshold bin, as compares with the bin's two bounds (the pass
            // is bound by instruction issue: a digit per key, with a validity test per key, cost 2.5 x as much)
            uint32_t ab = (uint32_t)(kk[0] >= above_from) | (uint32_t)(kk[1] >= above_from) << 1 | (uint32_t)(kk[2] >= above_from) << 2 |
                          (uint32_t)(kk[3] >= above_from) << 3;
            uint32_t ge = (uint32_t)(kk[0] >= bin_from) | (uint32_t)(kk[1] >= bin_from) << 1 | (uint32_t)(kk[2] >= bin_from) << 2 |
                          (uint32_t)(kk[3] >= bin_from) << 3;
            ab &= above_mask;
            if (v * 4 + 3 >= ncand) {                  // the problem's last vector (and the padding after it)
                const uint32_t vm = v * 4 < ncand ? (1u << (ncand - v * 4)) - 1u : 0u;
                ab &= vm, ge &= vm;
            }
            const uint32_t eqm = ge & ~ab;
            const uint32_t take = exact ? ge : ab;
            uint32_t word = take << (4 * (lane & 7));  // three shuffles: a reduction over a part of the warp was far slower
            word |= __shfl_xor_sync(0xffffffffu, word, 1);
            word |= __shfl_xor_sync(0xffffffffu, word, 2);
            word |= __shfl_xor_sync(0xffffffffu, word, 4);
            if ((lane & 7) == 0) mask[v >> 3] = word;  // positions 32 (v / 8) .. + 31
            if (!exact && __any_sync(0xffffffffu, eqm != 0)) {
                const int ne = __popc(eqm);
                const int incl = warp_incl_scan(ne, lane);
                int base = 0;
                if (lane == 31) base = atomicAdd(&sm->n_list, incl);
                base = __shfl_sync(0xffffffffu, base, 31) + incl - ne;
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if ((eqm >> e) & 1) list[base++] = make_uint2(kk[e] - bin_base, (uint32_t)(v * 4 + e));
            }
        }
    }
    __syncthreads();
    FIN_MARK(1);

    if (!exact) {
        const int n_in = sm->n_list;                   // == bc
        uint32_t prefix = 0;
        int low_bits = bin_bits;
        bool ex = false;
        if (n_in <= kThreads) {
            // a short list: every entry counts the entries ranked before it (larger key, or equal key at
            // a lower position) and knows at once whether it is among the `krem` winners
            if (tid < n_in) {
                const uint2 it = list[tid];
                int before = 0;
                for (int j = 0; j < n_in; ++j) {
                    const uint2 o = list[j];
                    before += (o.x > it.x) | ((o.x == it.x) & (o.y < it.y));
                }
                if (before < krem) atomicOr(&mask[it.y >> 5], 1u << (it.y & 31));
            }
            __syncthreads();
            low_bits = -1;                             // done
        }
        // otherwise the remaining bits of the keys in the list, 11 at a time
#pragma unroll 1
        while (!ex && low_bits > 0) {
            const int bits = low_bits < 11 ? low_bits : 11, shift = low_bits - bits;
            const uint32_t dmask = (1u << bits) - 1u;
            for (int i = tid; i < kDigitBins; i += kThreads) hist[i] = 0;
            __syncthreads();
            for (int i = tid; i < n_in; i += kThreads) {
                const uint32_t v = list[i].x;
                if ((uint32_t)((uint64_t)v >> low_bits) == prefix) hist_add(&hist[(v >> shift) & dmask]);
            }
            __syncthreads();
            int d, kr, c;
            wave_find_digit<8>(hist, krem, sm, d, kr, c);
            prefix = (prefix << bits) | (uint32_t)d, low_bits = shift, krem = kr, ex = c == kr;
        }
        // winners: above the class; the whole class when `ex`; else (equal keys, more than places
        // left) the `krem` lowest positions among them
        for (int i = tid; i < n_in && low_bits >= 0; i += kThreads) {
            const uint2 it = list[i];
            const uint32_t c = it.x >> low_bits;
            bool take = c > prefix;
            if (c == prefix) {
                take = ex;
                if (!ex) {
                    int before = 0;                    // equal keys at lower positions
                    for (int j = 0; j < n_in; ++j) {
                        const uint2 o = list[j];
                        before += (o.x == it.x) & (o.y < it.y);
                    }
                    take = before < krem;
                }
            }
            if (take) atomicOr(&mask[it.y >> 5], 1u << (it.y & 31));
        }
        __syncthreads();
    }

    FIN_MARK(2);
    // ascending list from the mask: each thread owns a run of words
    const int per = (n_words + kThreads - 1) / kThreads;
    const int w0 = min(n_words, tid * per), w1 = min(n_words, w0 + per);
    int cnt = 0;
    for (int w = w0; w < w1; ++w) cnt += __popc(mask[w]);
    int total;
    int o = wave_excl_scan(cnt, sm->warp_a, total);
    for (int w = w0; w < w1; ++w) {
        uint32_t bits = mask[w];
        while (bits) {
            const int b = __ffs(bits) - 1;
            bits &= bits - 1;
            if (o < k) idx_dst[o] = lo + w * 32 + b;
            ++o;
        }
    }
    if (tid == 0) *cnt_dst = k;
    FIN_MARK(3);
    return true;
}

// General path: exact radix select (11 + 11 + 10 bits of the key itself) over all of a problem's
// parked keys, then an ordered compaction with the lower-position tie rule.  The first pass over the
// keys leaves them in `key_cache` (shared memory, `cache_vecs` 16-byte vectors; 0 = none).  `hist` is
// scratch.  Called by all threads of the block.
__device__ __forceinline__ void wave_general(int* hist, WaveSmem* sm, const uint32_t* __restrict__ keys_unit, uint4* key_cache,
                                             int cache_vecs, int ncand, int k, int lo, int32_t* __restrict__ idx_dst,
                                             int32_t* __restrict__ cnt_dst) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint4* keys4 = reinterpret_cast<const uint4*>(keys_unit);
    const int n_vec = (ncand + 3) / 4;
    bool cached = false;                               // key_cache holds vectors [0, min(n_vec, cache_vecs))
    // One pass over all key vectors, kBatch loads in flight per thread; the first pass leaves the keys
    // in the ring.  f(v, x): vector index and its four keys (slots 4v .. 4v+3; slots >= ncand are stale).
    auto scan = [&](auto&& f) {
        for (int v0 = tid; v0 < n_vec; v0 += kThreads * kBatch) {
            uint4 x[kBatch];
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const int v = v0 + u * kThreads;
                x[u] = make_uint4(0u, 0u, 0u, 0u);
                if (v < n_vec) x[u] = (cached && v < cache_vecs) ? key_cache[v] : __ldcg(keys4 + v);
            }
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const int v = v0 + u * kThreads;
                if (v < n_vec) {
                    if (!cached && v < cache_vecs) key_cache[v] = x[u];
                    f(v, x[u]);
                }
            }
        }
        __syncthreads();
        cached = true;
    };

    uint32_t prefix = 0;                               // digits fixed so far (value of key >> low_bits)
    int low_bits = 32, krem = k;
    bool exact = false;                                // the class {key >> low_bits == prefix} is taken whole
#pragma unroll 1
    for (int pass = 0; pass < 3 && !exact; ++pass) {   // 11 + 11 + 10 bits of the key itself
        const int bits = pass == 2 ? 10 : 11, shift = low_bits - bits;
        const uint32_t dmask = (1u << bits) - 1u;
        for (int i = tid; i < kDigitBins; i += kThreads) hist[i] = 0;
        __syncthreads();
        scan([&](int v, const uint4& x) {
            const uint32_t kk[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (v * 4 + e < ncand && (pass == 0 || (kk[e] >> low_bits) == prefix)) hist_add(&hist[(kk[e] >> shift) & dmask]);
        });
        int d, kr, c;
        if (pass < 2) wave_find_digit<8>(hist, krem, sm, d, kr, c);
        else wave_find_digit<4>(hist, krem, sm, d, kr, c);
        prefix = (prefix << bits) | (uint32_t)d, low_bits = shift, krem = kr, exact = c == kr;
    }

    // ---- ordered compaction ------------------------------------------------------------------------
    // A slot is taken if its key is above the class, or inside the class and among the class's first
    // `krem` members in position order (the lower-position tie rule).  Warp w owns a contiguous range;
    // within a group of 128 slots lane l holds slots 4l..4l+3 (one 16-byte load), so lane order is
    // position order.
    const int seg = ((ncand + kWarps * 128 - 1) / (kWarps * 128)) * 128;          // slots per warp, multiple of 128
    const int seg_begin = min(ncand, warp * seg), seg_end = min(ncand, (warp + 1) * seg);
    auto classify = [&](int base, int& gt_bits, int& eq_bits) {   // bit e: slot base+e above / in the class
        gt_bits = eq_bits = 0;
        if (base < seg_end) {
            const int v = base >> 2;
            const uint4 x = v < cache_vecs ? key_cache[v] : __ldcg(keys4 + v);
            const uint32_t c[4] = {x.x >> low_bits, x.y >> low_bits, x.z >> low_bits, x.w >> low_bits};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const bool in = base + e < seg_end;
                gt_bits |= (in && c[e] > prefix) << e;
                eq_bits |= (in && c[e] == prefix) << e;
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
    int gt_before = 0, eq_before = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        const int x = sm->warp_a[w], y = sm->warp_b[w];
        gt_before += w < warp ? x : 0, eq_before += w < warp ? y : 0;
    }
    int out_pos = gt_before + min(eq_before, krem);
#pragma unroll 2
    for (int i0 = seg_begin; i0 < seg_end; i0 += 128) {
        const int base = i0 + 4 * lane;
        int gb, eb;
        classify(base, gb, eb);
        int take = gb;
        if (__any_sync(0xffffffffu, eb != 0)) {        // class members here: hand out what is left of the quota in order
            const int ne = __popc(eb);
            int before = eq_before + warp_incl_scan(ne, lane) - ne;
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if ((eb >> e) & 1) {
                    if (before < krem) take |= 1 << e;
                    ++before;
                }
            eq_before += warp_sum_int(ne);
        }
        const int nt = __popc(take);
        if (__any_sync(0xffffffffu, nt != 0)) {
            const int incl = warp_incl_scan(nt, lane);
            int o = out_pos + incl - nt;
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if ((take >> e) & 1) idx_dst[o++] = lo + base + e;
            out_pos += __shfl_sync(0xffffffffu, incl, 31);
        }
    }
    if (tid == 0) *cnt_dst = k;

}

template <typename T, int DP, int RED>
__global__ void __launch_bounds__(kThreads, 4)
    select_wave_kernel(const __grid_constant__ CUtensorMap tmap, const unsigned char* __restrict__ kimp, Geom gm, UnitTable ut,
                       WaveOrder order, SelectArgs a, int n_stages, int keep_in_l2,
                       int32_t* __restrict__ state_idx, int32_t* __restrict__ state_cnt, int32_t* __restrict__ status,
                       uint32_t* __restrict__ keys_g) {
    constexpr int RB = DP * Elem<T>::kBytes;          // bytes per projected-key row: 32, 64 or 128
    constexpr int NCH = RB / 16;
    constexpr uint32_t kTileBytes = kRows * RB;

    extern __shared__ unsigned char smem_raw[];
    // swizzled TMA boxes need their shared-memory base on the swizzle period (up to 1024 bytes)
    unsigned char* stage_base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    int* hist = reinterpret_cast<int*>(stage_base + n_stages * kTileBytes);       // one digit at a time
    WaveSmem* sm = reinterpret_cast<WaveSmem*>(hist + kDigitBins);
    // The ring is idle once the rows are streamed; it then caches the problem's keys (as many as fit).
    uint4* key_cache = reinterpret_cast<uint4*>(stage_base);
    const int cache_vecs = n_stages * (int)kTileBytes / 16;                      // 16-byte vectors of 4 keys

    const int tid = threadIdx.x, lane = tid & 31;
    const int pair = order.pair[blockIdx.x / gm.Hl], h = blockIdx.x % gm.Hl;
    const int ll = pair / ut.n_seq, s = pair % ut.n_seq;
    const int L = unit_len(gm, ut, ll, s);
    const int lo = min(a.sinks, L);
    const int hi = max(lo, L - a.recent);
    const int ncand = hi - lo;
    const int k = min(a.budget, ncand);
    check_candidates_projected(gm, ut, ll, s, hi, status);
    const size_t cu = list_unit(gm, ut, ll, s, h);
    const size_t dst_row = a.dst_is_state ? cu : (size_t)pair * gm.Hl + h;
    int32_t* idx_dst = (a.dst_is_state ? state_idx : a.idx_dst) + dst_row * a.idx_stride;
    int32_t* cnt_dst = (a.dst_is_state ? state_cnt : a.cnt_dst) + dst_row;

    if (k <= 0) {
        if (tid == 0) *cnt_dst = 0;
        return;
    }
    if (k == ncand) {                                  // budget covers every candidate: no ranking needed
        for (int i = tid; i < ncand; i += kThreads) idx_dst[i] = lo + i;
        if (tid == 0) *cnt_dst = k;
        return;
    }

    // ---- set-up -------------------------------------------------------------------------------
    wave_stamp(0);
    for (int i = tid; i < kDigitBins; i += kThreads) hist[i] = 0;
    if (tid == 0) {
        prefetch_tmap(&tmap);
        for (int i = 0; i < n_stages; ++i) mbar_init(&sm->full[i], 1);
        fence_mbar_init();
    }
    __syncthreads();

    const int n_tiles = (ncand + kRows - 1) / kRows;
    const long long row_base = (long long)key_unit(gm, ut, ll, s, h) * gm.max_seq_len + lo;              // row of candidate 0 in the 2-D view
    uint32_t* keys_unit = keys_g + cu * (size_t)((gm.max_seq_len + 255) & ~255); // by candidate index, 16-byte aligned
    // The projected keys stream through L2 once; the score keys parked there must still be there when
    // the block comes back for them.
    const uint64_t stream_policy = l2_policy_evict_first(), keep_policy = keep_in_l2 ? l2_policy_evict_last() : stream_policy;
    // The sample row and the query are requested before the ring's first tiles: behind the whole
    // grid's opening burst of bulk copies they would wait for microseconds.
    const bool sampled = ncand >= kMinSampled;
    uint4 srow[NCH];
#pragma unroll
    for (int c = 0; c < NCH; ++c) srow[c] = make_uint4(0u, 0u, 0u, 0u);
    if (sampled && tid < kSampleRows) {
        const int slot = (int)(((long long)tid * ncand) / kSampleRows);
        const uint4* rowp = reinterpret_cast<const uint4*>(kimp + (size_t)(row_base + slot) * RB);
#pragma unroll
        for (int c = 0; c < NCH; ++c) srow[c] = __ldg(rowp + c);
    }
    GroupScorer<T, DP, RED> scorer;
    scorer.load(a.q_imp + query_row(gm, ut, ll, s, h) * DP, gm.gl, sm->qs);
    if (RED != TB_GROUP_SUM) __syncthreads();
    if (tid == 0)
        for (int i = 0; i < n_stages && i < n_tiles; ++i) {
            mbar_arrive_expect_tx(&sm->full[i], kTileBytes);
            tma_load_2d_hint(stage_base + i * kTileBytes, &tmap, 0, (int)(row_base + (long long)i * kRows), &sm->full[i], stream_policy);
        }

    // ---- where to put the first digit's bins: a look at 256 rows spread over the problem ----------------
    // Only the bins' resolution depends on the sample, never the result: the digit is monotone in the
    // key whatever base and shift are, and a threshold that falls outside the sampled range lands in an
    // open-ended bin, which sends the problem down the general path.
    Digit dg = {0u, 21};
    if (sampled) {
        if (tid < kSampleRows) sm->sample[tid] = order_key(scorer.score([&](int c) { return srow[c]; }));
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
            const int r_hi = max(0, (int)floorf(mean - 6.f * sd) - 3), r_lo = min(kSampleRows - 1, (int)ceilf(mean + 6.f * sd) + 3);
            if (r == r_hi) sm->s_hi = mine;
            if (r == r_lo) sm->s_lo = mine;
        }
        __syncthreads();
        const uint32_t s_lo = sm->s_lo, s_hi = sm->s_hi;
        uint32_t range = s_hi - s_lo;
        range += range >> 1;                           // room above the highest bracketing sample
        if (range < s_hi - s_lo) range = 0xffffffffu;
        dg.base = s_lo, dg.shift = 0;
        while ((range >> dg.shift) >= 2046u) ++dg.shift;
    }

    // ---- stream + score + first digit histogram -------------------------------------------------
    // A wait that runs out (never in a correct run) makes the block give up streaming: it requests no
    // further tile, still waits -- bounded -- for those in flight, gives the rows it never received the
    // lowest key and finishes normally; the status word tells the caller that this call's lists are void.
    bool dead = false;
    int issued = min(n_stages, n_tiles);               // tiles whose copy has been requested
    int st = 0;
    uint32_t phase = 0;
    for (int i = 0; i < n_tiles; ++i) {
        const bool ok = i < issued && mbar_wait(&sm->full[st], phase);
        const unsigned char* tile = stage_base + st * kTileBytes;
        const int slot = i * kRows + tid;
        if (i == 0) wave_stamp(1);
        if (slot < ncand) {
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
            st_global_hint(keys_unit + slot, key, keep_policy);
            hist_add(&hist[dg.bin(key)]);
        }
        if (__syncthreads_or(!ok)) dead = true;        // all reads of this stage are done; uniform verdict on the wait
        if (!dead && i + n_stages < n_tiles) {
            if (tid == 0) {
                fence_proxy_async();
                mbar_arrive_expect_tx(&sm->full[st], kTileBytes);
                tma_load_2d_hint(stage_base + st * kTileBytes, &tmap, 0, (int)(row_base + (long long)(i + n_stages) * kRows), &sm->full[st],
                                 stream_policy);
            }
            issued = i + n_stages + 1;
        }
        if (++st == n_stages) st = 0, phase ^= 1u;
    }
    if (dead && tid == 0) atomicExch(status, kStatusTimeout);
    __syncthreads();                                   // histogram complete, own keys visible to the block
    wave_stamp(2);

    // ---- finish -----------------------------------------------------------------------------------
    if (wave_finish_mask(hist, sm, dg, keys_unit, stage_base, n_stages * (int)kTileBytes, ncand, k, lo, idx_dst, cnt_dst)) {
        wave_stamp(3);
        return;
    }
    wave_general(hist, sm, keys_unit, key_cache, cache_vecs, ncand, k, lo, idx_dst, cnt_dst);
    wave_stamp(3);
}

#ifdef TB_PHASE_TIMING
extern "C" int tb_debug_cw_ns(unsigned long long* out) { return (int)cudaMemcpyFromSymbol(out, g_cw_ns, sizeof(g_cw_ns)); }
extern "C" int tb_debug_fin_ns(unsigned long long* out) { return (int)cudaMemcpyFromSymbol(out, g_fin_ns, sizeof(g_fin_ns)); }
extern "C" int tb_debug_wave_smid(unsigned int* out) { return (int)cudaMemcpyFromSymbol(out, g_wave_smid, sizeof(g_wave_smid)); }
extern "C" int tb_debug_fin_blk(unsigned long long* out) { return (int)cudaMemcpyFromSymbol(out, g_fin_blk, sizeof(g_fin_blk)); }
extern "C" int tb_debug_wave_ns(unsigned long long* out) { return (int)cudaMemcpyFromSymbol(out, g_wave_ns, sizeof(g_wave_ns)); }
#endif

cudaError_t launch_select_wave(const tb_ctx* c, const UnitTable& ut, const SelectArgs& a, cudaStream_t s, bool dry) {
    const Geom& gm = c->geom;
    const int n_pairs = ut.layer_count * ut.n_seq, n_units = n_pairs * gm.Hl;
    WaveOrder order;
    int cand[kMaxLaunchUnits];
    for (int i = 0; i < n_pairs; ++i) {
        const int L = ut.len[i], lo = a.sinks < L ? a.sinks : L, hi = L - a.recent > lo ? L - a.recent : lo;
        cand[i] = hi - lo, order.pair[i] = (uint16_t)i;
    }
    std::stable_sort(order.pair, order.pair + n_pairs, [&](uint16_t x, uint16_t y) { return cand[x] > cand[y]; });
    const int tile_bytes = kRows * gm.dp * (gm.dtype == TB_BF16 ? 2 : 4);
    // Ring depth: the SM's shared memory split among the blocks it will hold (four when the launch has
    // that many per SM: 32 KB rings, 128 KB in flight; fewer blocks get deeper rings).
    const size_t fixed = 1024 + kDigitBins * sizeof(int) + sizeof(WaveSmem);
    int per_sm = (n_units + c->sm_count - 1) / c->sm_count;
    per_sm = per_sm < 1 ? 1 : per_sm > 4 ? 4 : per_sm;
    int n_stages = (int)(((size_t)224 * 1024 / per_sm - 1024 - fixed) / tile_bytes);
    if (n_stages > kStagesMax) n_stages = kStagesMax;
    if (n_stages < 2) n_stages = 2;
    const size_t smem = fixed + (size_t)n_stages * tile_bytes;
    // 4 bytes of key per candidate: ask L2 to keep them only while a launch's worth fits comfortably
    double parked = 0;
    for (int i = 0; i < n_pairs; ++i) parked += 4.0 * cand[i] * gm.Hl;
#ifndef TB_KEEP_BYTES
#define TB_KEEP_BYTES 96e6
#endif
    const int keep_in_l2 = parked <= TB_KEEP_BYTES;
    if (dry) return cudaSuccess;

#define TB_SEL_R(T, DP, RED)                                                                                                   \
    do {                                                                                                                \
        static unsigned char seen[64];                                                                                  \
        if (first_use_on_this_device(seen)) {                                                                           \
            cudaError_t e = cudaFuncSetAttribute(select_wave_kernel<T, DP, RED>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                                 226 * 1024);                                                            \
            if (e != cudaSuccess) return e;                                                                             \
        }                                                                                                               \
        select_wave_kernel<T, DP, RED><<<n_units, kThreads, smem, s>>>(c->kimp_map, (const unsigned char*)c->kimp, gm, ut, order, a, n_stages, keep_in_l2, c->st.idx, c->st.cnt, \
                                                                  c->st.status, c->wk.sel_keys);                        \
        return cudaGetLastError();                                                                                      \
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

// ===================================================================================================
// Few, long problems (one sequence, or a small batch, at 32K tokens and beyond): a thread-block cluster
// per problem, built from the same pieces as the kernel above.  Every block of the cluster places the
// first digit from the same 64-row sample, streams its share of the rows, parks the keys in the
// workspace row and keeps, on chip, only each row's first digit (2 bytes) and the digit histogram.
// Barrier 1.  Every block sums the cluster's histograms through distributed shared memory, finds the
// threshold bin itself, turns its own digits into a bitmask, fetches the full keys of its few rows
// in the threshold bin and sends them, with its count of selected rows, to every peer.  Barrier 2.
// Every block ranks the (tiny) list itself, knows every rank's count, and writes its part of the
// ascending list.  Two cluster barriers after the stream, no serial section, 2 bytes of shared memory
// per row (so two blocks per SM at 128K tokens).  A crowded or open-below threshold bin sends the
// problem to the general path, run by rank 0 on the parked keys.
constexpr int kCwListCap = 256;      // keys of the threshold bin set aside per problem (more: the bin is cut again)
constexpr int kCwMaxCluster = 8;

struct __align__(16) CwSmem {
    WaveSmem w;
    int take[kCwMaxCluster];         // per rank: rows its bitmask selects by the first digit alone
    int n_in[kCwMaxCluster];         // per rank: entries in its region of the list
    int winners[kCwMaxCluster];      // per rank: list entries that made it
    int my_n;
    int fine8[8];
    int coarse[kThreads];            // this block's histogram, 8 first-digit bins per entry
};

__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
template <typename P>
__device__ __forceinline__ P* peer_ptr(P* p, int rank) {       // the same shared-memory object in block `rank` of the cluster
    uint64_t out;
    asm volatile("mapa.u64 %0, %1, %2;" : "=l"(out) : "l"(reinterpret_cast<uint64_t>(p)), "r"(rank));
    return reinterpret_cast<P*>(out);
}

template <typename T, int DP, int RED>
__global__ void __launch_bounds__(kThreads, 2)
    select_cw_kernel(const __grid_constant__ CUtensorMap tmap, const unsigned char* __restrict__ kimp, Geom gm, UnitTable ut, SelectArgs a,
                     int tiles_per_cta, int n_stages, int32_t* __restrict__ state_idx, int32_t* __restrict__ state_cnt,
                     int32_t* __restrict__ status, uint32_t* __restrict__ keys_g, uint16_t* bins_g, int keep_in_l2) {
    constexpr int RB = DP * Elem<T>::kBytes;
    constexpr int NCH = RB / 16;
    constexpr uint32_t kTileBytes = kRows * RB;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* stage_base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int ring_bytes = n_stages * (int)kTileBytes;
    int* hist = reinterpret_cast<int*>(stage_base + ring_bytes);                 // this block's first-digit histogram
    // first digit of every row of this block: on chip, or (bins_g: problems of several hundred thousand
    // rows per block) in the workspace row, through the same pointer
    uint16_t* bins_sm = reinterpret_cast<uint16_t*>(hist + kDigitBins);
    uint32_t* mask = reinterpret_cast<uint32_t*>(bins_sm + (bins_g ? 0 : (size_t)tiles_per_cta * kRows));   // tiles_per_cta * 8 words
    CwSmem* cs = reinterpret_cast<CwSmem*>(mask + tiles_per_cta * (kRows / 32));
    WaveSmem* sm = &cs->w;
    // after the stream the ring holds the list (one region per rank)
    uint2* list = reinterpret_cast<uint2*>(stage_base);

    unsigned C, rank;
    asm volatile("mov.u32 %0, %%cluster_nctaid.x;" : "=r"(C));
    asm volatile("mov.u32 %0, %%cluster_ctaid.x;" : "=r"(rank));
    const int tid = threadIdx.x, lane = tid & 31;
    int ll, s, h;
    decode_unit(gm, ut, blockIdx.y, ll, s, h);
    const int L = unit_len(gm, ut, ll, s);
    const int lo = min(a.sinks, L), ncand = max(lo, L - a.recent) - lo, k = min(a.budget, ncand);
    check_candidates_projected(gm, ut, ll, s, lo + ncand, status);
    const size_t cu = list_unit(gm, ut, ll, s, h);
    const size_t dst_row = a.dst_is_state ? cu : (size_t)blockIdx.y;
    int32_t* idx_dst = (a.dst_is_state ? state_idx : a.idx_dst) + dst_row * a.idx_stride;
    int32_t* cnt_dst = (a.dst_is_state ? state_cnt : a.cnt_dst) + dst_row;
    // uniform over the cluster: all of its blocks leave together
    if (k <= 0) {
        if (rank == 0 && tid == 0) *cnt_dst = 0;
        return;
    }
    if (k == ncand) {
        for (int i = rank * kThreads + tid; i < ncand; i += C * kThreads) idx_dst[i] = lo + i;
        if (rank == 0 && tid == 0) *cnt_dst = k;
        return;
    }

#ifdef TB_PHASE_TIMING
    const unsigned long long tc0 = wave_now();
#define CW_MARK(i) do { if (tid == 0) { const int bb = blockIdx.y * gridDim.x + blockIdx.x; if (bb < 1024) { g_wave_ns[(i) & 3][bb] = wave_now() - ((i) == 0 ? 0 : tc0); if ((i) == 0) { unsigned smid_; asm volatile("mov.u32 %0, %%smid;" : "=r"(smid_)); g_wave_smid[bb] = smid_; } } } } while (0)
#else
#define CW_MARK(i) do {} while (0)
#endif
    CW_MARK(0);
    for (int i = tid; i < kDigitBins; i += kThreads) hist[i] = 0;
    if (tid == 0) {
        prefetch_tmap(&tmap);
        for (int i = 0; i < n_stages; ++i) mbar_init(&sm->full[i], 1);
        fence_mbar_init();
        cs->my_n = 0;
    }
    if (tid < kCwMaxCluster) cs->winners[tid] = 0;
    __syncthreads();

    const int n_tiles = (ncand + kRows - 1) / kRows;
    const int tile0 = rank * tiles_per_cta, my_tiles = max(0, min(tiles_per_cta, n_tiles - tile0));
    const int slot0 = tile0 * kRows;                   // candidate index of this block's first row
    const int n_local = max(0, min(my_tiles * kRows, ncand - slot0));
    const long long row_base = (long long)key_unit(gm, ut, ll, s, h) * gm.max_seq_len + lo;              // row of candidate 0
    uint32_t* keys_unit = keys_g + cu * (size_t)((gm.max_seq_len + 255) & ~255);
    uint16_t* bins = bins_g ? bins_g + cu * (size_t)((gm.max_seq_len + 255) & ~255) + slot0 : bins_sm;
    // parked keys are kept in L2 for the block's return to them, unless the launch parks more than L2 can hold
    const uint64_t stream_policy = l2_policy_evict_first(), keep_policy = keep_in_l2 ? l2_policy_evict_last() : stream_policy;

    // The sample rows and the queries are requested first, then the ring's opening tiles; nothing waits for
    // the sample here.  Behind the whole grid's opening burst of bulk copies the sample rows take several
    // microseconds, during which the ring would fill up and stall: the rows stay in registers and the digit
    // is placed a few tiles into the stream; what was scored before that is digitised then from its parked keys.
    const bool sampled = ncand >= kMinSampled;
    uint4 srow[NCH];
#pragma unroll
    for (int c = 0; c < NCH; ++c) srow[c] = make_uint4(0u, 0u, 0u, 0u);
    if (sampled && tid < kSampleRows) {
        const int slot = (int)(((long long)tid * ncand) / kSampleRows);
        const uint4* rowp = reinterpret_cast<const uint4*>(kimp + (size_t)(row_base + slot) * RB);
#pragma unroll
        for (int c = 0; c < NCH; ++c) srow[c] = __ldg(rowp + c);
    }
    {
        const float* q_unit = a.q_imp + query_row(gm, ut, ll, s, h) * DP;
        if (tid < gm.gl * DP)
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(sm->qs + tid)), "l"(q_unit + tid) : "memory");
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    if (tid == 0)
        for (int i = 0; i < n_stages && i < my_tiles; ++i) {
            mbar_arrive_expect_tx(&sm->full[i], kTileBytes);
            tma_load_2d_hint(stage_base + i * kTileBytes, &tmap, 0, (int)(row_base + slot0 + (long long)i * kRows), &sm->full[i], stream_policy);
        }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    GroupScorer<T, DP, RED> scorer;
    scorer.load_staged(sm->qs, gm.gl);
    Digit dg = {0u, 21};
    // identical in every block of the cluster: same rows, same arithmetic.  Called by all threads, once.
    auto place_digit = [&](int done_tiles) {
        if (tid < kSampleRows) sm->sample[tid] = order_key(scorer.score([&](int c) { return srow[c]; }));
        __syncthreads();
        if (tid < kSampleRows) {
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
            const float p = (float)k / (float)ncand, mean = p * kSampleRows, sd = sqrtf(mean * (1.f - p));
            const int r_hi = max(0, (int)floorf(mean - 6.f * sd) - 3), r_lo = min(kSampleRows - 1, (int)ceilf(mean + 6.f * sd) + 3);
            if (r == r_hi) sm->s_hi = mine;
            if (r == r_lo) sm->s_lo = mine;
        }
        __syncthreads();
        const uint32_t s_lo = sm->s_lo, s_hi = sm->s_hi;
        uint32_t range = s_hi - s_lo;
        // room above the highest bracketing sample; twice as much when that is the sample's largest key
        // (few sample keys above the threshold: it may well lie beyond them)
        const float pm = (float)k / (float)ncand * kSampleRows;
        const bool clipped = (int)floorf(pm - 6.f * sqrtf(pm * (1.f - (float)k / (float)ncand))) - 3 <= 0;
        const uint64_t wide = (uint64_t)range * (clipped ? 3u : 1u) + (range >> 1);
        range = wide > 0xffffffffull ? 0xffffffffu : (uint32_t)wide;
        dg.base = s_lo, dg.shift = 0;
        while ((range >> dg.shift) >= 2046u) ++dg.shift;
        uint32_t kk[8];                                // this thread's own earlier keys, back from L2 together
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int slot = i * kRows + tid;
            kk[i] = (i < done_tiles && slot < n_local) ? __ldcg(keys_unit + slot0 + slot) : 0u;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int slot = i * kRows + tid;
            if (i < done_tiles && slot < n_local) {
                const uint16_t b = (uint16_t)dg.bin(kk[i]);
                hist_add(&hist[b]);
                bins[slot] = b;
            }
        }
    };
    const int place_at = sampled ? min(my_tiles, 6) : -1;   // at most 8 (the catch-up's register array)

    CW_MARK(1);
    // ---- stream: score, park the key, keep the first digit ---------------------------------------------
    bool dead = false;                                 // a wait ran out: see the kernel above
    int issued = min(n_stages, my_tiles);
    int st = 0;
    uint32_t phase = 0;
    for (int i = 0; i < my_tiles; ++i) {
        if (i == place_at) place_digit(i);
        const bool placed = !sampled || i >= place_at;
        const bool ok = i < issued && mbar_wait(&sm->full[st], phase);
        const unsigned char* tile = stage_base + st * kTileBytes;
        const int slot = i * kRows + tid;
        uint16_t b = 0;                                // rows past the end: below everything
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
#ifdef TB_NOHINT
            keys_unit[slot0 + slot] = key;
#else
            st_global_hint(keys_unit + slot0 + slot, key, keep_policy);
#endif
            if (placed) {
                b = (uint16_t)dg.bin(key);
                hist_add(&hist[b]);
            }
        }
        bins[slot] = b;
        if (__syncthreads_or(!ok)) dead = true;
        if (!dead && i + n_stages < my_tiles) {
            if (tid == 0) {
                fence_proxy_async();
                mbar_arrive_expect_tx(&sm->full[st], kTileBytes);
                tma_load_2d_hint(stage_base + st * kTileBytes, &tmap, 0, (int)(row_base + slot0 + (long long)(i + n_stages) * kRows),
                                 &sm->full[st], stream_policy);
            }
            issued = i + n_stages + 1;
        }
        if (++st == n_stages) st = 0, phase ^= 1u;
    }
    if (dead && tid == 0) atomicExch(status, kStatusTimeout);
    if (place_at == my_tiles) place_digit(my_tiles);   // a short share: the digit is placed after its last tile
    __syncthreads();
    CW_MARK(2);
#ifdef TB_PHASE_TIMING
    unsigned long long tp = wave_now();
#define CW_PH(i) do { if (tid == 0) { unsigned long long tn = wave_now(); atomicAdd(&g_cw_ns[i], tn - tp); tp = tn; } } while (0)
#else
#define CW_PH(i) do {} while (0)
#endif
    // ---- threshold bin: the cluster's histogram in two levels ---------------------------------------------
    // Every block sums, through distributed shared memory, first a coarse histogram (256 bins of 8
    // first-digit bins each: one remote word per thread and peer), finds the coarse bin of the threshold,
    // then the 8 fine bins inside it.  If the threshold's bin holds more keys than the list takes (a
    // bracket stretched by an outlier in the sample, the open bin above it, many near-equal scores), the
    // bin itself is cut into 2046 slices and the rows inside it are re-digitised from their parked keys:
    // another round, two more barriers, only for the cluster that needs it.
    int bin = 0, krem = k, bc = 0;
    bool exact = false;
    uint32_t bin_base = 0;
    Digit cur = dg;
#pragma unroll 1
    for (int level = 0;; ++level) {
        cs->coarse[tid] = [&] {
            const int4* hp = reinterpret_cast<const int4*>(hist + tid * 8);
            const int4 x0 = hp[0], x1 = hp[1];
            return x0.x + x0.y + x0.z + x0.w + x1.x + x1.y + x1.z + x1.w;
        }();
        __syncthreads();
        cluster_sync_all();                            // every block's histograms are complete (level 0: every ring idle)
        if (level == 0) CW_PH(0);
        int mine = 0;
        for (unsigned r = 0; r < C; ++r) mine += peer_ptr(cs, (int)r)->coarse[tid];
        int total;
        const int excl = wave_excl_scan(mine, sm->warp_a, total);
        const int above = total - excl - mine;         // keys in coarse bins above this thread's
        if (above < krem && krem <= above + mine) sm->bc_bin = tid, sm->bc_krem = krem - above;   // exactly one thread
        __syncthreads();
        const int cb = sm->bc_bin, kc = sm->bc_krem;
        if (tid < 8) {
            int f = 0;
            for (unsigned r = 0; r < C; ++r) f += peer_ptr(hist, (int)r)[cb * 8 + tid];
            cs->fine8[tid] = f;
        }
        __syncthreads();
        {
            int run = 0, e = 7;
            while (e > 0 && run + cs->fine8[e] < kc) run += cs->fine8[e], --e;
            bin = cb * 8 + e, bc = cs->fine8[e], krem = kc - run;
        }
        exact = bc == krem;
        bin_base = cur.base + ((uint32_t)(bin - 1) << cur.shift);
        __syncthreads();                               // bc_*, fine8 and warp_a may be reused
        if (exact || bc <= kCwListCap) break;
        const bool open_top = bin == 2047;
        if (bin == 0 || level == 3 || (cur.shift == 0 && !open_top)) {
            // below the bracket, or more equal keys than the list takes: general path on the parked keys, rank 0 alone
            cluster_sync_all();                        // nobody reads a peer's histogram any more
            if (rank == 0)
                wave_general(hist, sm, keys_unit, reinterpret_cast<uint4*>(stage_base), ring_bytes / 16, ncand, k, lo, idx_dst, cnt_dst);
            return;
        }
        cluster_sync_all();                            // every block has read what it needs of the old histograms
        // the open bin above the bracket: first try twice the bracket's width again (what lies beyond
        // lands in the new digit's own open bin), then everything up to the largest key
        const uint64_t twice = (uint64_t)2 * (2046ull << cur.shift);
        const uint32_t rest = 0xffffffffu - bin_base;
        const uint32_t range = open_top ? (level == 0 && twice < rest ? (uint32_t)twice : rest) : (1u << cur.shift) - 1u;
        Digit nxt = {bin_base, 0};
        while ((range >> nxt.shift) >= 2046u) ++nxt.shift;
        for (int i = tid; i < kDigitBins; i += kThreads) hist[i] = 0;
        __syncthreads();
        for (int sl = tid; sl < my_tiles * kRows; sl += kThreads) {   // rows above the bin: 0xffff from now on; below: 0
            const int d = bins[sl];
            uint16_t nb = d > bin ? (uint16_t)0xffff : (uint16_t)0;
            if (d == bin) {
                nb = (uint16_t)nxt.bin(__ldcg(keys_unit + slot0 + sl));   // >= 1: the key is not below the bin's base
                hist_add(&hist[nb]);
            }
            bins[sl] = nb;
        }
        cur = nxt;
        __syncthreads();
    }
    CW_PH(1);

    // ---- own digits -> bitmask; own rows of the threshold bin -> every peer's list ------------------------
    int my_take = 0;
    int* my_slots = reinterpret_cast<int*>(list + (C + 1) * kCwListCap);       // own rows of the threshold bin (local row numbers)
    {
        const uint4* bins4 = reinterpret_cast<const uint4*>(bins);
        for (int v = tid; v < my_tiles * (kRows / 8); v += kThreads) {          // 8 digits per 16-byte load
            const uint4 x = bins4[v];
            const uint32_t w4[4] = {x.x, x.y, x.z, x.w};
            uint32_t take = 0, eq = 0;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int d = (int)((w4[e >> 1] >> (16 * (e & 1))) & 0xffffu);
                take |= (uint32_t)(d > bin || (d == bin && exact)) << e;
                eq |= (uint32_t)(d == bin && !exact) << e;
            }
            my_take += __popc(take);
            uint32_t word = take << (8 * (lane & 3));  // four lanes' bytes make a mask word
            word |= __shfl_xor_sync(0xffffffffu, word, 1);
            word |= __shfl_xor_sync(0xffffffffu, word, 2);
            if ((lane & 3) == 0) mask[v >> 2] = word;
            while (eq) {                               // a handful of rows per block: only their places are noted here
                const int e = __ffs(eq) - 1;
                eq &= eq - 1;
                my_slots[atomicAdd(&cs->my_n, 1)] = v * 8 + e;
            }
        }
    }
    {
        int total;
        wave_excl_scan(my_take, sm->warp_a, total);
        __syncthreads();
        // The noted rows' parked keys come back from L2 in one round trip, a row per thread (fetched inside the
        // loop above, every such row stalled its warp for that round trip: 2.5 us for the pass instead of 1.3),
        // and go to every peer's list.
        const int n_mine = cs->my_n;
        if (tid < n_mine) {
            const int ls = my_slots[tid];
            const uint2 ent = make_uint2(__ldcg(keys_unit + slot0 + ls) - bin_base, (uint32_t)(slot0 + ls));
            for (unsigned r = 0; r < C; ++r) peer_ptr(list, (int)r)[rank * kCwListCap + tid] = ent;
        }
        if (tid < (int)C) peer_ptr(cs, tid)->take[rank] = total, peer_ptr(cs, tid)->n_in[rank] = n_mine;
    }
    CW_PH(2);
    cluster_sync_all();                                // barrier 2: lists and counts are everywhere
    CW_PH(3);

    // ---- every block ranks the list itself ------------------------------------------------------------
    if (!exact) {
        // the regions' entries side by side first (one entry per thread), so that the ranking loop runs
        // over one short array with a single bound
        uint2* all = list + C * kCwListCap;
        int r_of = 0, i_of = tid, n_all = 0;
        for (unsigned r = 0; r < C; ++r) n_all += cs->n_in[r];
        while (r_of < (int)C && i_of >= cs->n_in[r_of]) i_of -= cs->n_in[r_of], ++r_of;
        uint2 it = make_uint2(0u, 0u);
        if (r_of < (int)C) it = list[r_of * kCwListCap + i_of], all[tid] = it;
        __syncthreads();
        if (r_of < (int)C) {
            int before = 0;                            // larger key, or equal key at a lower position
#pragma unroll 4
            for (int j = 0; j < n_all; ++j) {
                const uint2 o = all[j];
                before += (o.x > it.x) | ((o.x == it.x) & (o.y < it.y));
            }
            if (before < krem) {
                atomicAdd(&cs->winners[r_of], 1);
                if (r_of == (int)rank) {
                    const int ls = (int)it.y - slot0;
                    atomicOr(&mask[ls >> 5], 1u << (ls & 31));
                }
            }
        }
        __syncthreads();
    }
    CW_PH(4);
    int out_base = 0;
    for (unsigned r = 0; r < rank; ++r) out_base += cs->take[r] + cs->winners[r];
    {
        const int n_words = my_tiles * (kRows / 32);
        const int per = (n_words + kThreads - 1) / kThreads;
        const int w0 = min(n_words, tid * per), w1 = min(n_words, w0 + per);
        int cnt = 0;
        for (int w = w0; w < w1; ++w) cnt += __popc(mask[w]);
        int total;
        int o = out_base + wave_excl_scan(cnt, sm->warp_a, total);
        for (int w = w0; w < w1; ++w) {
            uint32_t bits = mask[w];
            while (bits) {
                const int b = __ffs(bits) - 1;
                bits &= bits - 1;
                if (o < k) idx_dst[o] = lo + slot0 + w * 32 + b;
                ++o;
            }
        }
    }
    if (rank == 0 && tid == 0) *cnt_dst = k;
    CW_PH(5);
#ifdef TB_PHASE_TIMING
    if (tid == 0) atomicAdd(&g_cw_ns[7], 1ull);
#endif
    CW_MARK(3);
}

cudaError_t launch_select_cw(const tb_ctx* c, const UnitTable& ut, const SelectArgs& a, cudaStream_t s, bool dry) {
    const Geom& gm = c->geom;
    const int n_units = ut.layer_count * ut.n_seq * gm.Hl;
    int max_cand = 0;
    for (int i = 0; i < ut.layer_count * ut.n_seq; ++i) {
        const int L = ut.len[i], lo = a.sinks < L ? a.sinks : L, hi = L - a.recent > lo ? L - a.recent : lo;
        if (hi - lo > max_cand) max_cand = hi - lo;
    }
    const int n_tiles = (max_cand + kRows - 1) / kRows;
    // cluster size: two resident blocks per SM over the whole GPU, at least 8 tiles per block
    int C = 2 * c->sm_count / n_units;
    if (C > kCwMaxCluster) C = kCwMaxCluster;
    while (C > 1 && n_tiles / C < 8) --C;
    if (C < 1) C = 1;
    const int tiles_per_cta = (n_tiles + C - 1) / C > 0 ? (n_tiles + C - 1) / C : 1;
    const int tile_bytes = kRows * gm.dp * (gm.dtype == TB_BF16 ? 2 : 4);
    const size_t ring_min = (size_t)(C + 1) * kCwListCap * sizeof(uint2) + kCwListCap * sizeof(int);   // list regions + the entries side by side + own rows' places
    const size_t budget = (size_t)(C * n_units > c->sm_count ? 113 : 224) * 1024;
    const size_t fixed_off = 1024 + kDigitBins * sizeof(int) + (size_t)tiles_per_cta * (kRows / 32) * 4 + sizeof(CwSmem);
    const size_t bins_bytes = (size_t)tiles_per_cta * kRows * 2;
    const size_t ring_least = ring_min > 2 * (size_t)tile_bytes ? ring_min : 2 * (size_t)tile_bytes;
    // the rows' first digits stay on chip while they leave the block's share of the SM room for a ring; beyond that they
    // live in the workspace
    const bool digits_on_chip = fixed_off + bins_bytes + ring_least <= budget;
    const size_t fixed = fixed_off + (digits_on_chip ? bins_bytes : 0);
    if (fixed + ring_least > 224 * 1024) return cudaErrorInvalidConfiguration;
    // 4 bytes of key (+ 2 of digit) per candidate: ask L2 to keep them only while a launch's worth fits comfortably
    const int keep_in_l2 = (double)n_units * max_cand * (digits_on_chip ? 4 : 6) <= 64e6;
    int n_stages = fixed < budget ? (int)((budget - fixed) / tile_bytes) : 0;
    if (n_stages > kStagesMax) n_stages = kStagesMax;
    if (n_stages < 2) n_stages = 2;
    while ((size_t)n_stages * tile_bytes < ring_min) ++n_stages;
    const size_t smem = fixed + (size_t)n_stages * tile_bytes;
    if (smem > 226 * 1024 || n_stages > kStagesMax) return cudaErrorInvalidConfiguration;
    if (dry) return cudaSuccess;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(C, n_units, 1), cfg.blockDim = dim3(kThreads, 1, 1), cfg.dynamicSmemBytes = smem, cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = C, attr[0].val.clusterDim.y = 1, attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr, cfg.numAttrs = 1;
#define TB_CW_R(T, DP, RED)                                                                                              \
    do {                                                                                                                 \
        static unsigned char seen[64];                                                                                   \
        if (first_use_on_this_device(seen)) {                                                                            \
            cudaError_t e = cudaFuncSetAttribute(select_cw_kernel<T, DP, RED>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                                 226 * 1024);                                                            \
            if (e != cudaSuccess) return e;                                                                              \
        }                                                                                                                \
        return cudaLaunchKernelEx(&cfg, select_cw_kernel<T, DP, RED>, c->kimp_map, (const unsigned char*)c->kimp, gm, ut, a, \
                                  tiles_per_cta, n_stages, c->st.idx, c->st.cnt, c->st.status, c->wk.sel_keys,           \
                                  digits_on_chip ? (uint16_t*)nullptr : c->wk.sel_bins, keep_in_l2);                    \
    } while (0)
#define TB_CW(T, DP)                                                \
    do {                                                            \
        if (a.reduce == TB_GROUP_MAX) TB_CW_R(T, DP, TB_GROUP_MAX); \
        else TB_CW_R(T, DP, TB_GROUP_SUM);                          \
    } while (0)
    if (gm.dtype == TB_BF16) {
        if (gm.dp == 32) TB_CW(__nv_bfloat16, 32); else TB_CW(__nv_bfloat16, 16);
    } else {
        if (gm.dp == 32) TB_CW(float, 32); else TB_CW(float, 16);
    }
#undef TB_CW
#undef TB_CW_R
}

}  // namespace tb
