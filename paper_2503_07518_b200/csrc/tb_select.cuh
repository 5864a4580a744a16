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

__device__ __forceinline__ void decode_unit(const Geom& gm, const UnitTable& ut, int u, int& ll, int& s, int& h) {
    h = u % gm.Hkv;
    s = (u / gm.Hkv) % ut.n_seq;
    ll = u / (gm.Hkv * ut.n_seq);
}
__device__ __forceinline__ size_t cache_unit(const Geom& gm, const UnitTable& ut, int ll, int s, int h) {
    return ((size_t)(ut.layer_begin + ll) * gm.max_batch + ut.seq_id[s]) * gm.Hkv + h;
}

}  // namespace tb
