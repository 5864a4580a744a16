/*
 * TokenButler decode hot path -- CPU ORACLE (test infrastructure, not product code).
 *
 * A plain, slow, obviously-correct restatement of what the path computes, written from the
 * paper's definitions.  Floating point is accumulated in fp64 over the exact stored input
 * values (bf16 inputs are widened exactly).  No blocking, fusion or reordering: every function
 * is the definition written out, in the paper's order of steps.
 *
 * Only tests, the smoke check and the benchmark's cpu_baseline / reference legs may build,
 * load or call this file.  It shares no code, headers, tables or helpers with the CUDA library.
 *
 * Steps (paper section / equation each one follows):
 *   orc_project_keys   K_imp = K . W_K                      Sec. 3.1, "Key-cache projection" equation
 *   orc_reduce_query   importance query of a GQA group      Sec. 3.1 (Q_imp has B*H heads, K_imp has H_kv)
 *   orc_score          q_imp . K_imp over all cached tokens Sec. 3.4 ("score computation against all
 *                                                           projected keys"), App. E
 *   orc_select         candidates minus sinks minus window, Sec. 4 "Token Selection Policy"
 *                      keep top-x by score
 *   orc_neighbors      neighbour fetching                   Sec. 3.4 "Neighbor fetching"
 *   orc_attended_set   Sink | Important | Local-Window      Sec. 3.3 (three buffers)
 *   orc_attention      softmax(q K^T / sqrt(D)) V           Sec. 3.3 ("standard attention kernel")
 *   orc_is_prediction_step  which decode steps re-select    Sec. 3.4 "Prediction interval"
 *   orc_step_units     the steps above chained per unit     Sec. 3.3 / 3.4
 *   orc_predict_queries  Q_imp = f(LN(H)), two-layer MLP    Sec. 3.1 "Query prediction", App. A (hidden
 *                                                           size 512), Table 6 (bias-free linears, LN
 *                                                           with weight and bias)
 *
 * Parity pins live in tests/test_oracle_pins.py.  The placement rule of the CLUSTER neighbour
 * mode (which side of a run the extra positions go to) is a reading of one sentence of Sec. 3.4:
 * "parity unpinned" beyond the invariants tested there (count = 2B, superset, inside candidates).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORC_F32 = 0, ORC_BF16 = 1 };
enum { ORC_GROUP_SUM = 0, ORC_GROUP_MAX = 1 };
enum { ORC_NEIGHBOR_DILATE = 0, ORC_NEIGHBOR_CLUSTER = 1 };

/* ---------- storage formats ------------------------------------------------------------- */

static double bf16_to_double(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* Round a double to the nearest bf16 (8 significant bits, float exponent range), ties to even,
 * in ONE rounding step (no detour through float, which could round twice). */
static uint16_t double_to_bf16_rne(double x) {
    if (isnan(x)) return 0x7FC0;
    uint16_t sign = signbit(x) ? 0x8000 : 0;
    double a = fabs(x);
    if (a == 0.0) return sign;
    if (isinf(a)) return sign | 0x7F80;
    int e;
    (void)frexp(a, &e);              /* a = m * 2^e, m in [0.5, 1)                       */
    int qe = e - 8;                  /* quantum so that m*2^8 has 8 significant bits     */
    if (qe < -133) qe = -133;        /* bf16 subnormals share the quantum 2^-133         */
    double q = rint(ldexp(a, -qe));  /* default rounding mode: nearest, ties to even     */
    double v = ldexp(q, qe);         /* exactly representable in float                   */
    float f = (float)v;
    if (isinf(f)) return sign | 0x7F80;
    uint32_t u;
    memcpy(&u, &f, 4);
    return sign | (uint16_t)(u >> 16);
}

static double load_elem(const void* p, size_t i, int dtype) {
    if (dtype == ORC_BF16) return bf16_to_double(((const uint16_t*)p)[i]);
    return (double)((const float*)p)[i];
}

static void store_elem(void* p, size_t i, int dtype, double x) {
    if (dtype == ORC_BF16) ((uint16_t*)p)[i] = double_to_bf16_rne(x);
    else ((float*)p)[i] = (float)x;  /* double -> float is a single RNE step */
}

void orc_round_to_storage(const double* x, size_t n, int dtype, void* out) {
    for (size_t i = 0; i < n; ++i) store_elem(out, i, dtype, x[i]);
}

void orc_widen(const void* x, size_t n, int dtype, double* out) {
    for (size_t i = 0; i < n; ++i) out[i] = load_elem(x, i, dtype);
}

/* ---------- Sec. 3.1: K_imp = K . W_K ---------------------------------------------------- */
/* K [T][D] (row stride D), W [D][dp], both in `dtype`.  kimp_out [T][dp] in `dtype` (rounded
 * once from the fp64 sum); kimp_f64 (optional) receives the unrounded sums. */
void orc_project_keys(const void* K, const void* W, int T, int D, int dp, int dtype,
                      void* kimp_out, double* kimp_f64) {
    for (int t = 0; t < T; ++t)
        for (int j = 0; j < dp; ++j) {
            double acc = 0.0;
            for (int c = 0; c < D; ++c)
                acc += load_elem(K, (size_t)t * D + c, dtype) * load_elem(W, (size_t)c * dp + j, dtype);
            if (kimp_out) store_elem(kimp_out, (size_t)t * dp + j, dtype, acc);
            if (kimp_f64) kimp_f64[(size_t)t * dp + j] = acc;
        }
}

/* ---------- Sec. 3.1: one importance query per KV head ----------------------------------- */
/* The g query heads that share a KV head contribute g importance queries [g][dp] (fp32).
 * GROUP_SUM adds them (ranking by the group's mean logit). */
void orc_reduce_query(const float* q_imp, int g, int dp, double* q_red) {
    for (int j = 0; j < dp; ++j) {
        double acc = 0.0;
        for (int u = 0; u < g; ++u) acc += (double)q_imp[(size_t)u * dp + j];
        q_red[j] = acc;
    }
}

/* ---------- Sec. 3.4 / App. E: score every cached token ---------------------------------- */
/* s[t] = scale * sum_j q[j] * K_imp[t][j]   (GROUP_SUM: q = reduced query)
 * s[t] = scale * max_u sum_j q_u[j] * K_imp[t][j]   (GROUP_MAX)                              */
void orc_score(const float* q_imp, int g, int reduce, const void* kimp, int L, int dp, int dtype,
               double scale, double* s) {
    double* qr = (double*)malloc(sizeof(double) * (size_t)dp);
    if (reduce == ORC_GROUP_SUM) orc_reduce_query(q_imp, g, dp, qr);
    for (int t = 0; t < L; ++t) {
        if (reduce == ORC_GROUP_SUM) {
            double acc = 0.0;
            for (int j = 0; j < dp; ++j) acc += qr[j] * load_elem(kimp, (size_t)t * dp + j, dtype);
            s[t] = scale * acc;
        } else {
            double best = -INFINITY;
            for (int u = 0; u < g; ++u) {
                double acc = 0.0;
                for (int j = 0; j < dp; ++j)
                    acc += (double)q_imp[(size_t)u * dp + j] * load_elem(kimp, (size_t)t * dp + j, dtype);
                if (acc > best) best = acc;
            }
            s[t] = scale * best;
        }
    }
    free(qr);
}

/* ---------- Sec. 4 "Token Selection Policy" ---------------------------------------------- */
/* Candidate range: everything except the first S tokens and the last W tokens. */
void orc_candidate_range(int L, int S, int W, int* lo, int* hi) {
    int l = S < L ? S : L;
    int h = L - W;
    if (h < l) h = l;
    *lo = l;
    *hi = h;
}

/* Stable merge sort of positions by score, descending.  Equal scores keep their original
 * (ascending position) order, which is the "lower index wins" tie rule. */
static void stable_sort_desc(int32_t* pos, int32_t* tmp, int n, const double* s) {
    for (int width = 1; width < n; width *= 2) {
        for (int a = 0; a < n; a += 2 * width) {
            int m = a + width < n ? a + width : n;
            int b = a + 2 * width < n ? a + 2 * width : n;
            int i = a, j = m, o = a;
            while (i < m && j < b) {
                /* take from the right run only if it is strictly larger */
                if (s[pos[j]] > s[pos[i]]) tmp[o++] = pos[j++];
                else tmp[o++] = pos[i++];
            }
            while (i < m) tmp[o++] = pos[i++];
            while (j < b) tmp[o++] = pos[j++];
        }
        memcpy(pos, tmp, sizeof(int32_t) * (size_t)n);
    }
}

static int cmp_i32(const void* a, const void* b) {
    int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
    return (x > y) - (x < y);
}

/* Keep the top `budget` candidates by score; output ascending positions; return the count. */
int orc_select(const double* s, int L, int S, int W, int budget, int32_t* idx) {
    int lo, hi;
    orc_candidate_range(L, S, W, &lo, &hi);
    int n = hi - lo;
    int k = budget < n ? budget : n;
    if (k <= 0) return 0;
    int32_t* pos = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    int32_t* tmp = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    for (int i = 0; i < n; ++i) pos[i] = lo + i;
    stable_sort_desc(pos, tmp, n, s);
    memcpy(idx, pos, sizeof(int32_t) * (size_t)k);
    qsort(idx, (size_t)k, sizeof(int32_t), cmp_i32);
    free(pos);
    free(tmp);
    return k;
}

/* ---------- Sec. 3.4 "Neighbor fetching" -------------------------------------------------- */
/* idx: ascending selected positions inside the candidate range [lo, hi).  out must hold
 * (2r+1)*cnt entries (DILATE) or (1+r)*cnt (CLUSTER).  Returns the size of the expanded,
 * ascending, duplicate-free list.
 *   DILATE : every position within distance r of a selected one.
 *   CLUSTER: consecutive selected positions form a run [a,b] of c tokens; the run's r*c extra
 *            positions are placed just outside it, ceil(rc/2) after b and floor(rc/2) before a. */
int orc_neighbors(const int32_t* idx, int cnt, int r, int mode, int lo, int hi, int32_t* out) {
    int span = hi - lo;
    if (span <= 0 || cnt <= 0) return 0;
    uint8_t* mark = (uint8_t*)calloc((size_t)span, 1);
    for (int i = 0; i < cnt; ++i) mark[idx[i] - lo] = 1;
    if (r > 0 && mode == ORC_NEIGHBOR_DILATE) {
        for (int i = 0; i < cnt; ++i)
            for (int d = -r; d <= r; ++d) {
                int p = idx[i] + d;
                if (p >= lo && p < hi) mark[p - lo] = 1;
            }
    } else if (r > 0) {
        int i = 0;
        while (i < cnt) {
            int j = i;
            while (j + 1 < cnt && idx[j + 1] == idx[j] + 1) ++j;
            int a = idx[i], b = idx[j];
            int c = b - a + 1;
            int n = r * c;
            int right = (n + 1) / 2, left = n / 2;
            for (int p = b + 1; p <= b + right; ++p)
                if (p >= lo && p < hi) mark[p - lo] = 1;
            for (int p = a - left; p <= a - 1; ++p)
                if (p >= lo && p < hi) mark[p - lo] = 1;
            i = j + 1;
        }
    }
    int m = 0;
    for (int p = 0; p < span; ++p)
        if (mark[p]) out[m++] = lo + p;
    free(mark);
    return m;
}

/* ---------- Sec. 3.3: what is attended ----------------------------------------------------- */
/* A = sinks [0, min(S,L))  U  important list I  U  window [max(min(S,L), L-W), L).
 * I was selected at an earlier (or the same) length and lies inside that length's candidate
 * range, so the three parts never overlap.  A must hold min(S,L)+nI+W entries. */
int orc_attended_set(int L, int S, int W, const int32_t* I, int nI, int32_t* A) {
    int lo, hi;
    orc_candidate_range(L, S, W, &lo, &hi);
    int n = 0;
    for (int t = 0; t < lo; ++t) A[n++] = t;
    for (int i = 0; i < nI; ++i) A[n++] = I[i];
    for (int t = hi; t < L; ++t) A[n++] = t;
    return n;
}

/* ---------- Sec. 3.3: standard softmax attention over the attended rows -------------------- */
/* q [g][D], K [L][D], V [L][D] in `dtype`; A: nA attended positions.
 * out [g][D] fp64, lse [g] (optional): lse = m + log(sum exp(x - m)). */
void orc_attention(const void* q, const void* K, const void* V, const int32_t* A, int nA,
                   int g, int D, int dtype, double sm_scale, double* out, double* lse) {
    double* x = (double*)malloc(sizeof(double) * (size_t)(nA > 0 ? nA : 1));
    for (int u = 0; u < g; ++u) {
        double m = -INFINITY;
        for (int i = 0; i < nA; ++i) {
            double acc = 0.0;
            size_t t = (size_t)A[i];
            for (int c = 0; c < D; ++c)
                acc += load_elem(q, (size_t)u * D + c, dtype) * load_elem(K, t * D + c, dtype);
            x[i] = sm_scale * acc;
            if (x[i] > m) m = x[i];
        }
        double denom = 0.0;
        for (int i = 0; i < nA; ++i) denom += exp(x[i] - m);
        for (int i = 0; i < nA; ++i) x[i] = exp(x[i] - m) / denom;   /* x now holds softmax p */
        for (int c = 0; c < D; ++c) {
            double acc = 0.0;
            for (int i = 0; i < nA; ++i) acc += x[i] * load_elem(V, (size_t)A[i] * D + c, dtype);
            out[(size_t)u * D + c] = acc;
        }
        if (lse) lse[u] = m + log(denom);
    }
    free(x);
}

/* ---------- the whole step for a batch of independent units -------------------------------- */
/* One unit = one (sequence, layer, KV head).  With refresh != 0 the unit scores, selects and
 * expands (result stored to idx/cnt); otherwise idx/cnt are taken as the stale list.  Then it
 * attends.  Units are independent, so OpenMP runs them side by side; nothing else is parallel. */
typedef struct {
    const void* K;       /* [L][D]   */
    const void* V;       /* [L][D]   */
    const void* Kimp;    /* [L][dp]  */
    const float* q_imp;  /* [g][dp]  */
    const void* q;       /* [g][D]   */
    int32_t* idx;        /* [cap]  in/out */
    int32_t* cnt;        /* [1]    in/out */
    double* out;         /* [g][D] */
    double* lse;         /* [g] or NULL */
    int32_t L;
    int32_t refresh;
} orc_unit;

typedef struct {
    int32_t g, D, dp, dtype;
    int32_t budget, sinks, recent, radius, nmode, reduce;
    double score_scale, sm_scale;
} orc_params;

/* Sec. 3.4 "Prediction interval": with interval P the prediction pipeline (scores, top-B, neighbours)
 * runs once every P decode steps and the P-1 steps in between reuse the stored selection; the local
 * window moves every step regardless.  Steps are counted from the first sparse decode step, which
 * predicts (there is no selection to reuse yet): step t predicts iff t is a multiple of P.  Over T
 * steps that is ceil(T / P) predictions -- the paper's "T to about T/N". */
int orc_is_prediction_step(int step, int interval) {
    if (interval < 1 || step < 0) return -1;
    return step % interval == 0 ? 1 : 0;
}

void orc_step_units(orc_unit* units, int n_units, const orc_params* p, int n_threads) {
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) num_threads(n_threads > 0 ? n_threads : 1)
#endif
    for (int i = 0; i < n_units; ++i) {
        orc_unit* un = &units[i];
        int L = un->L;
        if (un->refresh) {
            double* s = (double*)malloc(sizeof(double) * (size_t)(L > 0 ? L : 1));
            orc_score(un->q_imp, p->g, p->reduce, un->Kimp, L, p->dp, p->dtype, p->score_scale, s);
            int32_t* base = (int32_t*)malloc(sizeof(int32_t) * (size_t)(p->budget > 0 ? p->budget : 1));
            int k = orc_select(s, L, p->sinks, p->recent, p->budget, base);
            int lo, hi;
            orc_candidate_range(L, p->sinks, p->recent, &lo, &hi);
            if (p->radius > 0) *un->cnt = orc_neighbors(base, k, p->radius, p->nmode, lo, hi, un->idx);
            else { memcpy(un->idx, base, sizeof(int32_t) * (size_t)k); *un->cnt = k; }
            free(base);
            free(s);
        }
        int cap = p->sinks + *un->cnt + p->recent;
        int32_t* A = (int32_t*)malloc(sizeof(int32_t) * (size_t)(cap > 0 ? cap : 1));
        int nA = orc_attended_set(L, p->sinks, p->recent, un->idx, *un->cnt, A);
        orc_attention(un->q, un->K, un->V, A, nA, p->g, p->D, p->dtype, p->sm_scale, un->out, un->lse);
        free(A);
    }
}

/* ---------- importance-query predictor (Sec. 3.1 "Query prediction", App. A) --------------------
 * For each token: x = LN(h) (mean and biased variance over the E channels, eps inside the root,
 * weight and bias), u = act(W1 x), q = W2 u.  Linears have no bias (the parameter counts of Table 6
 * leave no room for one).  The paper does not name the activation: act 0 = GELU in its exact erf
 * form (this build's reading), 1 = SiLU, 2 = ReLU.  W1 is [hid][E], W2 is [out][hid], both row-major
 * (one row per output), out = slots * heads * d'.  Everything in fp64 on values the caller widened. */
enum { ORC_ACT_GELU = 0, ORC_ACT_SILU = 1, ORC_ACT_RELU = 2 };

void orc_predict_queries(const double* H, int n_tok, int E, const double* ln_w, const double* ln_b, double eps,
                         const double* W1, int hid, const double* W2, int out, int act, double* q) {
    double* x = (double*)malloc(sizeof(double) * (size_t)E);
    double* u = (double*)malloc(sizeof(double) * (size_t)hid);
    for (int t = 0; t < n_tok; ++t) {
        const double* h = H + (size_t)t * E;
        double mean = 0.0, var = 0.0;
        for (int c = 0; c < E; ++c) mean += h[c];
        mean /= E;
        for (int c = 0; c < E; ++c) var += (h[c] - mean) * (h[c] - mean);
        var /= E;
        const double rstd = 1.0 / sqrt(var + eps);
        for (int c = 0; c < E; ++c) x[c] = (h[c] - mean) * rstd * ln_w[c] + ln_b[c];
        for (int j = 0; j < hid; ++j) {
            double a = 0.0;
            for (int c = 0; c < E; ++c) a += W1[(size_t)j * E + c] * x[c];
            if (act == ORC_ACT_GELU) a = 0.5 * a * (1.0 + erf(a / sqrt(2.0)));
            else if (act == ORC_ACT_SILU) a = a / (1.0 + exp(-a));
            else a = a > 0.0 ? a : 0.0;
            u[j] = a;
        }
        for (int o = 0; o < out; ++o) {
            double a = 0.0;
            for (int j = 0; j < hid; ++j) a += W2[(size_t)o * hid + j] * u[j];
            q[(size_t)t * out + o] = a;
        }
    }
    free(x);
    free(u);
}

int orc_max_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
