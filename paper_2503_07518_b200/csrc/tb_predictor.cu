// Importance-query predictor forward (paper Sec. 3.1 "Query prediction", App. A "two-layer MLP with
// hidden size 512"; Table 6 fixes the shapes: bias-free linears, layer norm with weight and bias):
//     q = W2 . act(W1 . LN(h))          per decoded token h, once per producer layer,
// the step right before the selection path: its output is the q_imp of the producer's consumer layers.
//
// At decode batch sizes both linears are matrix-vector products bound by reading their weights once
// (8 MB per producer for an 8B-shaped model), so there is no tensor-core tile here: one warp per
// output row, 16-byte loads, fp32 accumulation, every token of the call against the row while it is
// in registers.  Two launches: hidden units (layer norm folded in; each block recomputes the few
// tokens' statistics rather than exchanging them), then outputs written in the layout
// tb_select_topk reads.  No context: weights and scratch belong to the caller.
#include <cooperative_groups.h>

#include "tb_common.cuh"
#include "tb_internal.h"

namespace tb {

namespace {

constexpr int kPredThreads = 256;
constexpr int kPredWarps = kPredThreads / 32;
constexpr int kPredMaxTokens = 64;
constexpr int kTokChunk = 8;        // tokens whose accumulators a warp keeps while it walks a weight row
constexpr int kStageTok = 16;       // tokens whose hidden units the output kernel stages in shared memory at once

__device__ __forceinline__ float activate(float a, int act) {
    if (act == TB_ACT_GELU) return 0.5f * a * (1.f + erff(a * 0.70710678118654752f));
    if (act == TB_ACT_SILU) return a / (1.f + __expf(-a));
    return fmaxf(a, 0.f);
}

// hidden[t][j] = act( sum_c W1[j][c] * ((h[t][c] - mean_t) * rstd_t * ln_w[c] + ln_b[c]) )
// A block owns kPredWarps / 2 hidden units, two warps per unit (half of the channels each), so that an
// 8B-shaped layer (512 units x 4096 channels) spreads over 128 blocks and a warp's share of a row is
// eight 16-byte loads, issued four at a time.
template <typename T>
__global__ void __launch_bounds__(kPredThreads) predictor_hidden_kernel(const T* __restrict__ H, const T* __restrict__ ln_w,
                                                                        const T* __restrict__ ln_b, const T* __restrict__ W1,
                                                                        float* __restrict__ hidden, int n_tok, int E, int hid,
                                                                        float eps, int act) {
    constexpr int P = Elem<T>::kPer16;
    constexpr int kUnits = kPredWarps / 2;
    pdl_launch_dependents();                           // the output kernel may start fetching its weights
    __shared__ float s_mean[kPredMaxTokens], s_rstd[kPredMaxTokens];
    __shared__ float s_half[kUnits][kTokChunk];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_vec = E / P;

    // Layer-norm statistics: sums of (h - h[0]) and of its square in one pass (the shift keeps the
    // variance accurate when the token's mean is large against its spread).  Few tokens: the whole
    // block per token; many: one warp per token.
    __shared__ float s_part[kPredWarps][2];
    auto token_sums = [&](int t, int first, int stride, float& s1, float& s2) {
        const uint4* h4 = reinterpret_cast<const uint4*>(H + (size_t)t * E);
        const float shift = Elem<T>::to_f32(H[(size_t)t * E]);
        float f[P];
        s1 = s2 = 0.f;
        for (int v = first; v < n_vec; v += stride) {
            Elem<T>::unpack16(__ldg(h4 + v), f);
#pragma unroll
            for (int e = 0; e < P; ++e) {
                const float d = f[e] - shift;
                s1 += d, s2 = fmaf(d, d, s2);
            }
        }
        s1 = warp_sum(s1), s2 = warp_sum(s2);
        return shift;
    };
    auto publish = [&](int t, float shift, float s1, float s2) {
        const float m = s1 / (float)E;
        s_mean[t] = shift + m, s_rstd[t] = rsqrtf(fmaxf(s2 / (float)E - m * m, 0.f) + eps);
    };
    if (n_tok < kPredWarps) {
        for (int t = 0; t < n_tok; ++t) {
            float s1, s2;
            const float shift = token_sums(t, tid, kPredThreads, s1, s2);
            if (lane == 0) s_part[warp][0] = s1, s_part[warp][1] = s2;
            __syncthreads();
            if (tid == 0) {
                float a = 0.f, b = 0.f;
                for (int w = 0; w < kPredWarps; ++w) a += s_part[w][0], b += s_part[w][1];
                publish(t, shift, a, b);
            }
            __syncthreads();
        }
    } else {
        for (int t = warp; t < n_tok; t += kPredWarps) {
            float s1, s2;
            const float shift = token_sums(t, lane, 32, s1, s2);
            if (lane == 0) publish(t, shift, s1, s2);
        }
        __syncthreads();
    }

    const int unit = warp >> 1, half = warp & 1;
    const int j = blockIdx.x * kUnits + unit;          // this warp pair's hidden unit
    const bool live = j < hid;
    const int v_begin = half * (n_vec / 2), v_end = half ? n_vec : n_vec / 2;
    const uint4* w4 = reinterpret_cast<const uint4*>(W1 + (size_t)(live ? j : 0) * E);
    const uint4* g4 = reinterpret_cast<const uint4*>(ln_w);
    const uint4* b4 = reinterpret_cast<const uint4*>(ln_b);
    for (int t0 = 0; t0 < n_tok; t0 += kTokChunk) {
        float acc[kTokChunk], mean[kTokChunk], rstd[kTokChunk];
#pragma unroll
        for (int u = 0; u < kTokChunk; ++u) {
            acc[u] = 0.f;
            const int t = min(t0 + u, n_tok - 1);
            mean[u] = s_mean[t], rstd[u] = s_rstd[t];
        }
        for (int v0 = v_begin + lane; v0 < v_end; v0 += 4 * 32) {   // four rounds of loads in flight
            uint4 wv[4], gv[4], bv[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const int v = min(v0 + r * 32, v_end - 1);
                wv[r] = __ldg(w4 + v), gv[r] = __ldg(g4 + v), bv[r] = __ldg(b4 + v);
            }
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const int v = v0 + r * 32;
                if (v >= v_end) break;
                float w[P], g[P], b[P];
                Elem<T>::unpack16(wv[r], w);
                Elem<T>::unpack16(gv[r], g);
                Elem<T>::unpack16(bv[r], b);
#pragma unroll
                for (int u = 0; u < kTokChunk; ++u) {
                    const int t = t0 + u;
                    if (t >= n_tok) break;             // uniform
                    float h[P];
                    Elem<T>::unpack16(__ldg(reinterpret_cast<const uint4*>(H + (size_t)t * E) + v), h);
#pragma unroll
                    for (int e = 0; e < P; ++e) acc[u] = fmaf(w[e], fmaf((h[e] - mean[u]) * rstd[u], g[e], b[e]), acc[u]);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kTokChunk; ++u) acc[u] = warp_sum(acc[u]);
        if (half == 1 && lane == 0)
#pragma unroll
            for (int u = 0; u < kTokChunk; ++u) s_half[unit][u] = acc[u];
        __syncthreads();
        if (half == 0 && lane == 0 && live)
#pragma unroll
            for (int u = 0; u < kTokChunk; ++u)
                if (t0 + u < n_tok) hidden[(size_t)(t0 + u) * hid + j] = activate(acc[u] + s_half[unit][u], act);
        __syncthreads();
    }
}

// q_imp[slot][t][head][i] = sum_j W2[(slot, head, i)][j] * hidden[t][j]
template <typename T>
__global__ void __launch_bounds__(kPredThreads) predictor_out_kernel(const T* __restrict__ W2, const float* __restrict__ hidden,
                                                                     float* __restrict__ q_imp, int n_tok, int hid, int n_out,
                                                                     int per_slot, int stage_tok) {
    constexpr int P = Elem<T>::kPer16;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int o_raw = blockIdx.x * kPredWarps + warp;  // this warp's output row
    const bool live = o_raw < n_out;                   // idle warps still take part in the barriers
    const int o = live ? o_raw : 0;
    const uint4* w4 = reinterpret_cast<const uint4*>(W2 + (size_t)o * hid);
    const int n_vec = hid / P;
    const int slot = o / per_slot, within = o % per_slot;   // per_slot = heads * d'
    // The row's first vectors do not depend on the hidden units: fetch them while the kernel that
    // computes those is still running (programmatic dependent launch), then wait for it.
    constexpr int kPre = 2;                            // covers a 512-wide bf16 row
    uint4 pre[kPre];
#pragma unroll
    for (int r = 0; r < kPre; ++r) pre[r] = lane + 32 * r < n_vec ? __ldg(w4 + lane + 32 * r) : make_uint4(0u, 0u, 0u, 0u);
    pdl_wait();
    extern __shared__ float s_hidden[];                // stage_tok rows of `hid` floats
    for (int t0 = 0; t0 < n_tok; t0 += kTokChunk) {
        const int nt = min(kTokChunk, n_tok - t0);
        if (t0 % stage_tok == 0) {                     // (stage_tok is a multiple of kTokChunk)
            const int ns = min(stage_tok, n_tok - t0);
            __syncthreads();                           // the previous tokens are no longer read
            for (int i = threadIdx.x * 4; i < ns * hid; i += kPredThreads * 4)
                *reinterpret_cast<float4*>(s_hidden + i) = __ldcg(reinterpret_cast<const float4*>(hidden + (size_t)t0 * hid + i));
            __syncthreads();
        }
        const float* s_tok = s_hidden + (size_t)(t0 % stage_tok) * hid;
        float acc[kTokChunk];
#pragma unroll
        for (int u = 0; u < kTokChunk; ++u) acc[u] = 0.f;
        auto use = [&](int v, const uint4& wv) {
            float w[P];
            Elem<T>::unpack16(wv, w);
#pragma unroll
            for (int u = 0; u < kTokChunk; ++u) {
                if (u >= nt) break;                    // uniform
                const float* hp = s_tok + u * hid + v * P;
#pragma unroll
                for (int e = 0; e < P; e += 4) {
                    const float4 x = *reinterpret_cast<const float4*>(hp + e);
                    acc[u] = fmaf(w[e], x.x, acc[u]), acc[u] = fmaf(w[e + 1], x.y, acc[u]);
                    acc[u] = fmaf(w[e + 2], x.z, acc[u]), acc[u] = fmaf(w[e + 3], x.w, acc[u]);
                }
            }
        };
#pragma unroll
        for (int r = 0; r < kPre; ++r)
            if (lane + 32 * r < n_vec) use(lane + 32 * r, pre[r]);
        for (int v = lane + 32 * kPre; v < n_vec; v += 32) use(v, __ldg(w4 + v));
#pragma unroll
        for (int u = 0; u < kTokChunk; ++u) {
            const float a = warp_sum(acc[u]);
            if (lane == 0 && live && t0 + u < n_tok) q_imp[((size_t)slot * n_tok + (t0 + u)) * per_slot + within] = a;
        }
    }
}

// ---- several tokens at once (bf16): both linears on the tensor cores ---------------------------------
// With 5 or more tokens the products above re-walk a weight row once per token chunk; a tile of 16
// tokens x 8 outputs per mma.sync.m16n8k16 reads each weight once for all of them.  The left operand
// (normalised hidden states, resp. hidden units) is fp32: it is split into a bf16 high and low part
// and multiplied twice, so the products keep ~16 bits of it and accumulate in fp32.
// The 16 k-indices of an MMA step are mapped to channels so that every thread's operands are 16
// contiguous bytes: over a run of 32 channels, thread (row gid, column pair tig) takes channels
// 8 tig .. 8 tig + 7; the first four feed the first MMA step (k = 2 tig, 2 tig + 1, 2 tig + 8, 2 tig + 9),
// the last four the second.  Both operands use the same mapping, so the sum over channels is unchanged.
__device__ __forceinline__ void mma_bf16_16x8x16(float* d, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// fp32 pair -> bf16x2 high parts and bf16x2 of what they leave
__device__ __forceinline__ void split_bf16x2(float x, float y, uint32_t& hi, uint32_t& lo) {
    const __nv_bfloat16 xh = __float2bfloat16_rn(x), yh = __float2bfloat16_rn(y);
    const __nv_bfloat16 xl = __float2bfloat16_rn(x - __bfloat162float(xh)), yl = __float2bfloat16_rn(y - __bfloat162float(yh));
    hi = (uint32_t)__bfloat16_as_ushort(xh) | ((uint32_t)__bfloat16_as_ushort(yh) << 16);
    lo = (uint32_t)__bfloat16_as_ushort(xl) | ((uint32_t)__bfloat16_as_ushort(yl) << 16);
}
// One run of 32 channels: x0 / x1 = this thread's 8 left-operand values of rows gid / gid + 8 (zeros for
// rows past the tokens), w = its 8 right-operand values (16 bytes of the weight row of output gid).
__device__ __forceinline__ void mma_run32(float* acc, const float* x0, const float* x1, const uint4& w) {
    const uint32_t wb[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int st = 0; st < 2; ++st) {
        uint32_t h0, l0, h1, l1, h2, l2, h3, l3;
        split_bf16x2(x0[4 * st], x0[4 * st + 1], h0, l0);          // row gid,     k = 2 tig, 2 tig + 1
        split_bf16x2(x1[4 * st], x1[4 * st + 1], h1, l1);          // row gid + 8
        split_bf16x2(x0[4 * st + 2], x0[4 * st + 3], h2, l2);      // row gid,     k = 2 tig + 8, 2 tig + 9
        split_bf16x2(x1[4 * st + 2], x1[4 * st + 3], h3, l3);
        mma_bf16_16x8x16(acc, h0, h1, h2, h3, wb[2 * st], wb[2 * st + 1]);
        mma_bf16_16x8x16(acc, l0, l1, l2, l3, wb[2 * st], wb[2 * st + 1]);
    }
}

constexpr int kSplitK = 4;           // thread blocks (one cluster) that share the channels of a hidden-unit tile

// hidden[t][j] for 8 hidden units per cluster of kSplitK blocks: block r takes a quarter of the channels,
// its 8 warps a run of 32 channels at a time; partial tiles are summed in rank 0's shared memory
// (distributed shared memory, fixed order).  The layer-norm statistics of the tokens are split over
// the cluster the same way.
__global__ void __launch_bounds__(kPredThreads) predictor_hidden_mma_kernel(const __nv_bfloat16* __restrict__ H,
                                                                            const __nv_bfloat16* __restrict__ ln_w,
                                                                            const __nv_bfloat16* __restrict__ ln_b,
                                                                            const __nv_bfloat16* __restrict__ W1,
                                                                            float* __restrict__ hidden, int n_tok, int E, int hid,
                                                                            float eps, int act) {
    using EB = Elem<__nv_bfloat16>;
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();        // == blockIdx.x
    pdl_launch_dependents();
    __shared__ float s_mean[kPredMaxTokens], s_rstd[kPredMaxTokens];
    __shared__ float s_acc[kSplitK][kPredWarps][16][8];   // rank 0 receives every block's per-warp tiles
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, gid = lane >> 2, tig = lane & 3;
    // statistics of tokens rank*8+warp, +32, ...: shifted one-pass sums, sixteen 16-byte loads in flight
    for (int t = rank * kPredWarps + warp; t < n_tok; t += kSplitK * kPredWarps) {
        const uint4* h4 = reinterpret_cast<const uint4*>(H + (size_t)t * E);
        const float shift = __bfloat162float(H[(size_t)t * E]);
        float f[8], s1 = 0.f, s2 = 0.f;
#pragma unroll 4
        for (int v = lane; v < E / 8; v += 32) {
            EB::unpack16(__ldg(h4 + v), f);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float d = f[e] - shift;
                s1 += d, s2 = fmaf(d, d, s2);
            }
        }
        s1 = warp_sum(s1), s2 = warp_sum(s2);
        if (lane < kSplitK) {                          // lane r tells block r
            const float m = s1 / (float)E;
            *cluster.map_shared_rank(&s_mean[t], lane) = shift + m;
            *cluster.map_shared_rank(&s_rstd[t], lane) = rsqrtf(fmaxf(s2 / (float)E - m * m, 0.f) + eps);
        }
    }
    cluster.sync();
    const int j0 = blockIdx.y * 8;                     // the cluster's hidden units; hid is a multiple of 8
    const __nv_bfloat16* wrow = W1 + (size_t)(j0 + gid) * E;
    const int n_runs = E / 32, runs_per_block = (n_runs + kSplitK - 1) / kSplitK;
    const int r_begin = rank * runs_per_block, r_end = min(n_runs, r_begin + runs_per_block);
    float(*acc0)[kPredWarps][16][8] = cluster.map_shared_rank(s_acc, 0);
    for (int t0 = 0; t0 < n_tok; t0 += 16) {
        const int ta = t0 + gid, tb_ = t0 + gid + 8;
        const bool va = ta < n_tok, vb = tb_ < n_tok;
        const float ma = va ? s_mean[ta] : 0.f, ra = va ? s_rstd[ta] : 0.f, mb = vb ? s_mean[tb_] : 0.f, rb = vb ? s_rstd[tb_] : 0.f;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int r0 = r_begin + warp; r0 < r_end; r0 += 2 * kPredWarps) {       // two runs' loads in flight
            uint4 wv[2], gv[2], bv[2], hav[2], hbv[2];
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int r = r0 + i * kPredWarps;
                const int c = min(r, r_end - 1) * 32 + 8 * tig;
                wv[i] = __ldg(reinterpret_cast<const uint4*>(wrow + c));
                gv[i] = __ldg(reinterpret_cast<const uint4*>(ln_w + c));
                bv[i] = __ldg(reinterpret_cast<const uint4*>(ln_b + c));
                hav[i] = va ? __ldg(reinterpret_cast<const uint4*>(H + (size_t)ta * E + c)) : make_uint4(0u, 0u, 0u, 0u);
                hbv[i] = vb ? __ldg(reinterpret_cast<const uint4*>(H + (size_t)tb_ * E + c)) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                if (r0 + i * kPredWarps >= r_end) break;   // warp-uniform
                float g[8], b[8], ha[8], hb[8];
                EB::unpack16(gv[i], g), EB::unpack16(bv[i], b), EB::unpack16(hav[i], ha), EB::unpack16(hbv[i], hb);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    ha[e] = va ? fmaf((ha[e] - ma) * ra, g[e], b[e]) : 0.f;
                    hb[e] = vb ? fmaf((hb[e] - mb) * rb, g[e], b[e]) : 0.f;
                }
                mma_run32(acc, ha, hb, wv[i]);
            }
        }
        // acc: rows gid (acc[0..1]) and gid + 8 (acc[2..3]), units 2 tig, 2 tig + 1 -> rank 0
        acc0[rank][warp][gid][2 * tig] = acc[0], acc0[rank][warp][gid][2 * tig + 1] = acc[1];
        acc0[rank][warp][gid + 8][2 * tig] = acc[2], acc0[rank][warp][gid + 8][2 * tig + 1] = acc[3];
        cluster.sync();
        if (rank == 0 && tid < 128) {
            const int row = tid >> 3, col = tid & 7;
            float a = 0.f;
#pragma unroll
            for (int r = 0; r < kSplitK; ++r)
#pragma unroll
                for (int w = 0; w < kPredWarps; ++w) a += s_acc[r][w][row][col];
            if (t0 + row < n_tok) hidden[(size_t)(t0 + row) * hid + j0 + col] = activate(a, act);
        }
        cluster.sync();                                // rank 0 has read the tiles before the next round overwrites them
    }
}

// q_imp for 8 output rows per half block: a block's 8 warps are 2 output tiles x 4 quarters of the row.
__global__ void __launch_bounds__(kPredThreads) predictor_out_mma_kernel(const __nv_bfloat16* __restrict__ W2, const float* __restrict__ hidden,
                                                                         float* __restrict__ q_imp, int n_tok, int hid, int n_out,
                                                                         int per_slot) {
    __shared__ float s_acc[2][4][16][8];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, gid = lane >> 2, tig = lane & 3;
    const int tile = warp >> 2, quarter = warp & 3;
    const int o0 = (blockIdx.x * 2 + tile) * 8;        // n_out is a multiple of 8
    const bool live = o0 < n_out;
    const __nv_bfloat16* wrow = W2 + (size_t)(live ? o0 + gid : 0) * hid;
    const int n_runs = hid / 32, runs_per_q = (n_runs + 3) / 4;
    const int r_begin = quarter * runs_per_q, r_end = min(n_runs, r_begin + runs_per_q);
    // the weights of this warp's first two runs do not depend on the hidden units: fetch them, then wait
    uint4 wpre[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) wpre[i] = __ldg(reinterpret_cast<const uint4*>(wrow + min(r_begin + i, max(n_runs - 1, 0)) * 32 + 8 * tig));
    pdl_wait();                                        // the hidden units come from the previous kernel
    for (int t0 = 0; t0 < n_tok; t0 += 16) {
        const int ta = t0 + gid, tb_ = t0 + gid + 8;
        const bool va = ta < n_tok, vb = tb_ < n_tok;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int r = r_begin; r < r_end; ++r) {
            const int c = r * 32 + 8 * tig;
            const uint4 wv = r - r_begin < 2 ? wpre[r - r_begin] : __ldg(reinterpret_cast<const uint4*>(wrow + c));
            float ha[8], hb[8];
#pragma unroll
            for (int e = 0; e < 8; e += 4) {
                const float4 xa = va ? __ldcg(reinterpret_cast<const float4*>(hidden + (size_t)ta * hid + c + e)) : make_float4(0.f, 0.f, 0.f, 0.f);
                const float4 xb = vb ? __ldcg(reinterpret_cast<const float4*>(hidden + (size_t)tb_ * hid + c + e)) : make_float4(0.f, 0.f, 0.f, 0.f);
                ha[e] = xa.x, ha[e + 1] = xa.y, ha[e + 2] = xa.z, ha[e + 3] = xa.w;
                hb[e] = xb.x, hb[e + 1] = xb.y, hb[e + 2] = xb.z, hb[e + 3] = xb.w;
            }
            mma_run32(acc, ha, hb, wv);
        }
        s_acc[tile][quarter][gid][2 * tig] = acc[0], s_acc[tile][quarter][gid][2 * tig + 1] = acc[1];
        s_acc[tile][quarter][gid + 8][2 * tig] = acc[2], s_acc[tile][quarter][gid + 8][2 * tig + 1] = acc[3];
        __syncthreads();
        {
            const int tl = tid >> 7, row = (tid >> 3) & 15, col = tid & 7;   // 256 threads = 2 tiles x 16 rows x 8 columns
            const int t = t0 + row, o = (blockIdx.x * 2 + tl) * 8 + col;
            const float a = s_acc[tl][0][row][col] + s_acc[tl][1][row][col] + s_acc[tl][2][row][col] + s_acc[tl][3][row][col];
            if (t < n_tok && o < n_out) q_imp[((size_t)(o / per_slot) * n_tok + t) * per_slot + o % per_slot] = a;
        }
        __syncthreads();
    }
}

}  // namespace

}  // namespace tb

extern "C" tb_status tb_predict_importance_queries(const tb_predictor* p, const void* hidden_dev, int32_t n_tokens,
                                                   float* scratch_dev, float* q_imp_dev, void* stream) {
    using namespace tb;
    if (!p || !hidden_dev || !scratch_dev || !q_imp_dev || !p->ln_weight || !p->ln_bias || !p->w1 || !p->w2) return TB_ERR_INVALID_ARG;
    if (p->dtype != TB_F32 && p->dtype != TB_BF16) return TB_ERR_INVALID_ARG;
    if (n_tokens <= 0 || p->model_dim <= 0 || p->hidden_dim <= 0 || p->n_q_heads <= 0 || p->n_slots <= 0 || p->imp_dim <= 0 ||
        !(p->ln_eps >= 0.f))
        return TB_ERR_INVALID_ARG;
    if (p->activation != TB_ACT_GELU && p->activation != TB_ACT_SILU && p->activation != TB_ACT_RELU) return TB_ERR_INVALID_ARG;
    if (n_tokens > kPredMaxTokens) return TB_ERR_CAPACITY;
    const int per16 = p->dtype == TB_BF16 ? 8 : 4;     // rows are read 16 bytes at a time
    if (p->model_dim % per16 || p->hidden_dim % per16 || p->hidden_dim > 1536) return TB_ERR_UNSUPPORTED;
    const uintptr_t align = (uintptr_t)hidden_dev | (uintptr_t)p->ln_weight | (uintptr_t)p->ln_bias | (uintptr_t)p->w1 |
                            (uintptr_t)p->w2 | (uintptr_t)scratch_dev;
    if (align & 15) return TB_ERR_INVALID_ARG;
    const long long n_out = (long long)p->n_slots * p->n_q_heads * p->imp_dim;
    if (n_out > (1ll << 24)) return TB_ERR_UNSUPPORTED;
    cudaStream_t s = (cudaStream_t)stream;
    const int g1 = (p->hidden_dim + kPredWarps / 2 - 1) / (kPredWarps / 2), g2 = (int)((n_out + kPredWarps - 1) / kPredWarps);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(g2, 1, 1), cfg.blockDim = dim3(kPredThreads, 1, 1), cfg.stream = s;
    int stage_tok = (int)(48 * 1024 / (p->hidden_dim * sizeof(float))) / kTokChunk * kTokChunk;   // hidden_dim <= 1536 gives >= 8
    stage_tok = stage_tok > kStageTok ? kStageTok : stage_tok < kTokChunk ? kTokChunk : stage_tok;
    cfg.dynamicSmemBytes = (size_t)stage_tok * p->hidden_dim * sizeof(float);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see pdl_wait()
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr, cfg.numAttrs = 1;
    const int per_slot = p->n_q_heads * p->imp_dim, n_out_i = (int)n_out;
    cudaError_t e;
    if (p->dtype == TB_BF16 && n_tokens >= 5 && p->model_dim % 32 == 0 && p->hidden_dim % 32 == 0 && n_out % 8 == 0) {
        // several tokens: tensor-core tiles of 16 tokens x 8 outputs
        {
            cudaLaunchConfig_t c1 = {};
            c1.gridDim = dim3(kSplitK, p->hidden_dim / 8, 1), c1.blockDim = dim3(kPredThreads, 1, 1), c1.stream = s;
            cudaLaunchAttribute a1[1];
            a1[0].id = cudaLaunchAttributeClusterDimension;
            a1[0].val.clusterDim.x = kSplitK, a1[0].val.clusterDim.y = 1, a1[0].val.clusterDim.z = 1;
            c1.attrs = a1, c1.numAttrs = 1;
            if (cudaLaunchKernelEx(&c1, predictor_hidden_mma_kernel, (const __nv_bfloat16*)hidden_dev, (const __nv_bfloat16*)p->ln_weight,
                                   (const __nv_bfloat16*)p->ln_bias, (const __nv_bfloat16*)p->w1, scratch_dev, (int)n_tokens,
                                   (int)p->model_dim, (int)p->hidden_dim, p->ln_eps, (int)p->activation) != cudaSuccess)
                return TB_ERR_CUDA;
        }
        cfg.gridDim = dim3((unsigned)((n_out / 8 + 1) / 2), 1, 1);
        cfg.dynamicSmemBytes = 0;
        e = cudaLaunchKernelEx(&cfg, predictor_out_mma_kernel, (const __nv_bfloat16*)p->w2, (const float*)scratch_dev, q_imp_dev,
                               (int)n_tokens, (int)p->hidden_dim, n_out_i, per_slot);
    } else if (p->dtype == TB_BF16) {
        predictor_hidden_kernel<__nv_bfloat16><<<g1, kPredThreads, 0, s>>>(
            (const __nv_bfloat16*)hidden_dev, (const __nv_bfloat16*)p->ln_weight, (const __nv_bfloat16*)p->ln_bias,
            (const __nv_bfloat16*)p->w1, scratch_dev, n_tokens, p->model_dim, p->hidden_dim, p->ln_eps, p->activation);
        e = cudaLaunchKernelEx(&cfg, predictor_out_kernel<__nv_bfloat16>, (const __nv_bfloat16*)p->w2, (const float*)scratch_dev,
                               q_imp_dev, (int)n_tokens, (int)p->hidden_dim, n_out_i, per_slot, stage_tok);
    } else {
        predictor_hidden_kernel<float><<<g1, kPredThreads, 0, s>>>((const float*)hidden_dev, (const float*)p->ln_weight,
                                                                   (const float*)p->ln_bias, (const float*)p->w1, scratch_dev, n_tokens,
                                                                   p->model_dim, p->hidden_dim, p->ln_eps, p->activation);
        e = cudaLaunchKernelEx(&cfg, predictor_out_kernel<float>, (const float*)p->w2, (const float*)scratch_dev, q_imp_dev,
                               (int)n_tokens, (int)p->hidden_dim, n_out_i, per_slot, stage_tok);
    }
    if (e != cudaSuccess) return TB_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? TB_OK : TB_ERR_CUDA;
}
