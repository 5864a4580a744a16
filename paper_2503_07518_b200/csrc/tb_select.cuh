// Pieces shared by the selection kernels: the scoring arithmetic (one definition, so the standalone
// and the fused kernel produce bit-identical scores) and the launch-unit decoding.
#pragma once

#include "tb_common.cuh"
#include "tb_internal.h"

namespace tb {

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

// The same for TB_GROUP_MAX: the row's score is the largest of the g heads' dot products.  `qs` holds
// the g importance queries, [g][DP] floats in shared memory (every lane reads the same words: broadcast).
// Each head's dot product is accumulated exactly as in row_score.
template <typename T, int DP, typename LoadChunk>
__device__ __forceinline__ float row_score_max(const float* qs, int g, LoadChunk ld) {
    constexpr int P = Elem<T>::kPer16;
    constexpr int NCH = DP / P;
    float f[DP];
#pragma unroll
    for (int c = 0; c < NCH; ++c) Elem<T>::unpack16(ld(c), f + c * P);
    float best = -INFINITY;
    for (int u = 0; u < g; ++u) {
        const float4* q4 = reinterpret_cast<const float4*>(qs + u * DP);
        float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
#pragma unroll
            for (int e = 0; e < P; e += 4) {
                const float4 q = q4[(c * P + e) / 4];
                float& acc = (c & 1) ? acc1 : acc0;
                acc = fmaf(q.x, f[c * P + e], acc), acc = fmaf(q.y, f[c * P + e + 1], acc);
                acc = fmaf(q.z, f[c * P + e + 2], acc), acc = fmaf(q.w, f[c * P + e + 3], acc);
            }
        }
        best = fmaxf(best, acc0 + acc1);
    }
    return best;
}

// How a selection kernel scores a row under the reduction RED (TB_GROUP_SUM: one dot product with the
// summed query held in registers; TB_GROUP_MAX: g dot products against the queries in shared memory).
template <typename T, int DP, int RED>
struct GroupScorer {
    float qr[RED == TB_GROUP_SUM ? DP : 1];
    const float* qs;
    int g;
    // q_unit: the group's g queries [g][DP] in global memory; qs_smem: room for kMaxGroup * DP floats.
    // All threads of the block call it; with TB_GROUP_MAX a block barrier must follow before score().
    __device__ __forceinline__ void load(const float* __restrict__ q_unit, int g_, float* qs_smem) {
        g = g_, qs = qs_smem;
        if constexpr (RED == TB_GROUP_SUM) {
            load_group_query<DP>(q_unit, g_, qr);
        } else {
            for (int i = threadIdx.x; i < g_ * DP; i += blockDim.x) qs_smem[i] = q_unit[i];
        }
    }
    // The same from queries that already sit in shared memory ([g][DP] floats, visible to the thread):
    // the summed query is built in the same order, so the scores are the same bits.
    __device__ __forceinline__ void load_staged(const float* qs_smem, int g_) {
        g = g_, qs = qs_smem;
        if constexpr (RED == TB_GROUP_SUM) load_group_query<DP>(qs_smem, g_, qr);
    }
    template <typename LoadChunk>
    __device__ __forceinline__ float score(LoadChunk ld) const {
        if constexpr (RED == TB_GROUP_SUM) return row_score<T, DP>(qr, ld);
        else return row_score_max<T, DP>(qs, g, ld);
    }
};

// A selection unit is one index list: (layer, sequence, list head h < Hl).
__device__ __forceinline__ void decode_unit(const Geom& gm, const UnitTable& ut, int u, int& ll, int& s, int& h) {
    h = u % gm.Hl;
    s = (u / gm.Hl) % ut.n_seq;
    ll = u / (gm.Hl * ut.n_seq);
}
// Row of the unit in the context's lists, counts and parked-key workspace.
__device__ __forceinline__ size_t list_unit(const Geom& gm, const UnitTable& ut, int ll, int s, int h) {
    return ((size_t)(ut.layer_begin + ll) * gm.max_batch + ut.seq_id[s]) * gm.Hl + h;
}
// Key stream of the unit in the projected-key cache: its own (one list per KV head), its KV head's
// (one list per query head) or the layer's only one.
__device__ __forceinline__ size_t key_unit(const Geom& gm, const UnitTable& ut, int ll, int s, int h) {
    return ((size_t)(ut.layer_begin + ll) * gm.max_batch + ut.seq_id[s]) * gm.Hi + (h * gm.Hi) / gm.Hl;
}
// The unit's importance queries: gl consecutive rows of q_imp [layer_count][n_seq][Hl * gl][d'].
__device__ __forceinline__ size_t query_row(const Geom& gm, const UnitTable& ut, int ll, int s, int h) {
    return ((size_t)(ll * ut.n_seq + s) * gm.Hl + h) * gm.gl;
}

// With device-resident lengths the host cannot check, at replay time, that every candidate has a projected
// key: one thread per block does, and reports through the status word (the selection itself goes on).
__device__ __forceinline__ void check_candidates_projected(const Geom& gm, const UnitTable& ut, int ll, int s, int hi, int32_t* status) {
    if (ut.use_dev_len && threadIdx.x == 0) {
        const size_t pair = (size_t)(ut.layer_begin + ll) * gm.max_batch + ut.seq_id[s];
        if (ut.len_proj_dev[pair] < hi) atomicExch(status, kStatusUnprojected);
    }
}

}  // namespace tb
