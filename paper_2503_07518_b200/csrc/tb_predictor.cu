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
    if (p->dtype == TB_BF16) {
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
