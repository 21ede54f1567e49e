/*
 * kimad_oracle.c -- plain CPU oracle for the worker-side Kimad+ compression pass.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, by-the-definition reference
 * that the tests, the smoke check and the benchmark's CPU-baseline leg compare
 * the CUDA library against.  It shares no code, header, table or constant with
 * the CUDA library and must never be called from the product path.
 *
 * What it computes, per simulated worker and per step (paper notation: u is the
 * fresh update / gradient, u^ is the EF21 estimator, called g here):
 *
 *   O1  d = u - u^                     (Section 3 footnote; Algorithm 1, upload line;
 *                                       Eq. 6: the compressor is applied to grad - u^)
 *   O2  TopK order                     (Section 2.2: "K largest absolute value" --
 *                                       ties: larger |x| first, then lower index)
 *   O3  k-table from the ratio grid    (Section 3.2: discrete set of ratios per layer;
 *                                       Omega = {TopK : K > 0}, Section 4.2)
 *   O4  err_l(k) = ||d_l - TopK_k(d_l)||^2   (Eq. 4; "Errors" matrix of Algorithm 3)
 *   O5  byte costs, budget c, budget cells   (Eq. 2, Eq. 3; "Costs" matrix of Algorithm 3)
 *   O6  knapsack DP over the budget axis     (Section 3.2, Algorithm 3)
 *   O7  TopK select + sparse pack            (Algorithm 1, upload line)
 *   O8  EF21 estimator update u^ += C(d)     (Algorithm 1 aggregate line, Eq. 6)
 *
 * and, beyond the worker-side pass:
 *
 *   O9  Kimad without layer adaptivity: one ratio of the grid for every layer, the
 *       largest whose total size fits c      (Section 3.1; the baseline of Section 4.3)
 *   O10 receiver side of a message: u^_m += C_m(.) as a scatter-add of the packed
 *       entries                              (Algorithm 1, "Aggregate all update estimators")
 *   O11 model step x <- x - gamma sum_m w_m u^_m   (Algorithm 1, last line)
 *   O12 the other reading of Algorithm 3: the knapsack axis is the discretised ERROR (its header:
 *       "compression budget E_max", "discretization step E_max / D", "discretized L2"), the value the
 *       size; the answer is the lowest error level whose smallest size fits c
 *   O9b Kimad as Section 3.1 states it: ONE ratio for all layers, SIZED TO THE BUDGET (not taken from
 *       a grid): the largest ratio whose total size fits c.  With one layer spanning the model this is
 *       the whole-model TopK of Section 4.3 at K = floor(c / (4 + vb))
 *   O13 sizes with a dense fallback (Eq. 3 calls b_ij "the size of layer i compressed with c^j" and
 *       fixes no encoding): a candidate whose sparse size reaches the layer's dense size is sent
 *       densely -- all n values, no indices -- and then has no compression error
 *
 * Floating point: the element-wise operations (O1, O8, the DP adds) are single
 * IEEE binary32 operations in a fixed order, because the compared results must be
 * bit-identical.  The error curve is accumulated in binary64 from the smallest
 * magnitude upward and rounded to binary32 once.
 *
 * Pins (tests/test_oracle_*.py): numpy float32 re-computation for O1/O8, full
 * stable sort + math.fsum for O2/O4/O7, closed forms for d_i = i+1, exhaustive
 * enumeration of all K^L assignments for O6, the 0/1-knapsack special case, a
 * hand-computed three-layer example (tests/golden/), torch's bfloat16 cast for
 * the bf16 rounding.  The whole-step composition has no value printed in the
 * paper to compare with: it is pinned by the identities g_new - g = C(d),
 * ||d - C(d)||^2 = err and sum(bytes) <= c only.  O9: brute force over the grid;
 * O10: the receiver's estimator equals the sender's after every message; O11:
 * numpy float32 re-computation and the closed form for equal estimators.  O12: exhaustive
 * enumeration of the discretised objective.  O9b: exact rational arithmetic over every breakpoint
 * of the step function r -> sum_l floor(r n_l), hand values.  O13: hand-computed sizes on the
 * three-layer example, exhaustive enumeration of the assignments with the modified tables.
 *
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC (see kimad_oracle.py).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define KO_OK 0
#define KO_STATUS_INFEASIBLE 1 /* no assignment fits the budget: every layer takes j = 0 */
#define KO_STATUS_PLATEAU 2    /* budget covers the largest candidate of every layer      */
#define KO_ERR_ARG (-1)
#define KO_ERR_NOMEM (-2)
#define KO_ERR_CAPACITY (-3)

typedef struct {
    uint32_t key; /* magnitude bit pattern, bits(d) & 0x7fffffff */
    uint32_t idx; /* layer-local index */
} ko_pair;

static uint32_t f2u(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    return u;
}
static float u2f(uint32_t u) {
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* O2: descending magnitude, then ascending index.  +0 and -0 share key 0. */
static int ko_cmp_order(const void* a, const void* b) {
    const ko_pair* x = (const ko_pair*)a;
    const ko_pair* y = (const ko_pair*)b;
    if (x->key != y->key) return x->key > y->key ? -1 : 1;
    if (x->idx != y->idx) return x->idx < y->idx ? -1 : 1;
    return 0;
}
static int ko_cmp_u32(const void* a, const void* b) {
    uint32_t x = *(const uint32_t*)a, y = *(const uint32_t*)b;
    return x < y ? -1 : (x > y ? 1 : 0);
}

/* round-to-nearest-even binary32 -> bfloat16 bit pattern (finite inputs). */
uint16_t ko_bf16_rne(float x) {
    uint32_t u = f2u(x);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}
float ko_bf16_to_f32(uint16_t h) { return u2f(((uint32_t)h) << 16); }

/* O1 */
void ko_diff(const float* grad, const float* g, float* d, uint64_t n) {
    for (uint64_t i = 0; i < n; ++i) d[i] = grad[i] - g[i];
}

/* O3: k_{l,j} = min(n_l, max(1, ceil(r_j * n_l))) with r_j and the product in binary64. */
int ko_k_table(const uint64_t* layer_sizes, uint32_t L, const double* ratios, uint32_t K,
               uint64_t* k_out /* [L][K] */) {
    if (!layer_sizes || !ratios || !k_out || L == 0 || K == 0) return KO_ERR_ARG;
    for (uint32_t j = 0; j < K; ++j) {
        if (!(ratios[j] > 0.0) || ratios[j] > 1.0) return KO_ERR_ARG;
        if (j > 0 && !(ratios[j] > ratios[j - 1])) return KO_ERR_ARG; /* grid strictly ascending */
    }
    for (uint32_t l = 0; l < L; ++l) {
        uint64_t n = layer_sizes[l];
        if (n == 0 || n > 0xffffffffull) return KO_ERR_ARG;
        for (uint32_t j = 0; j < K; ++j) {
            double x = ceil(ratios[j] * (double)n);
            uint64_t k = (uint64_t)x;
            if (k < 1) k = 1;
            if (k > n) k = n;
            k_out[(size_t)l * K + j] = k;
        }
    }
    return KO_OK;
}

/* sorted (key desc, idx asc) copy of a layer */
static ko_pair* ko_sorted_pairs(const float* d, uint64_t n) {
    ko_pair* p = (ko_pair*)malloc((size_t)(n ? n : 1) * sizeof(ko_pair));
    if (!p) return NULL;
    for (uint64_t i = 0; i < n; ++i) {
        p[i].key = f2u(d[i]) & 0x7fffffffu;
        p[i].idx = (uint32_t)i;
    }
    qsort(p, (size_t)n, sizeof(ko_pair), ko_cmp_order);
    return p;
}

/* O4 on an already sorted layer.  k[] must be non-decreasing, 1 <= k <= n.
 * err[j]  = sum of squares of the entries ranked >= k[j], added from the last rank
 *           (smallest magnitude) upward in binary64, rounded to binary32 once
 * tau[j]  = key of the k[j]-th entry (the selection threshold)
 * keep_eq[j] = how many entries whose key equals tau[j] are kept (the lowest indices)
 * n_gt[j], n_eq[j] = entries with key > tau[j], key == tau[j] */
static int ko_curve_sorted(const ko_pair* p, uint64_t n, const uint64_t* k, uint32_t K, float* err,
                           uint32_t* tau, uint32_t* keep_eq, uint32_t* n_gt, uint32_t* n_eq) {
    for (uint32_t j = 0; j < K; ++j) {
        if (k[j] < 1 || k[j] > n) return KO_ERR_ARG;
        if (j > 0 && k[j] < k[j - 1]) return KO_ERR_ARG;
    }
    double acc = 0.0;
    uint64_t rank = n;
    for (uint32_t jj = K; jj-- > 0;) {
        while (rank > k[jj]) {
            --rank;
            double v = (double)u2f(p[rank].key);
            acc += v * v;
        }
        if (err) err[jj] = (float)acc;
    }
    for (uint32_t j = 0; j < K; ++j) {
        uint32_t t = p[k[j] - 1].key;
        uint64_t lo = k[j] - 1, hi = k[j];
        while (lo > 0 && p[lo - 1].key == t) --lo;
        while (hi < n && p[hi].key == t) ++hi;
        if (tau) tau[j] = t;
        if (n_gt) n_gt[j] = (uint32_t)lo;
        if (n_eq) n_eq[j] = (uint32_t)(hi - lo);
        if (keep_eq) keep_eq[j] = (uint32_t)(k[j] - lo);
    }
    return KO_OK;
}

/* O4 for one layer. */
int ko_layer_curve(const float* d, uint64_t n, const uint64_t* k, uint32_t K, float* err,
                   uint32_t* tau, uint32_t* keep_eq, uint32_t* n_gt, uint32_t* n_eq) {
    if (!d || n == 0 || n > 0xffffffffull || !k || K == 0) return KO_ERR_ARG;
    ko_pair* p = ko_sorted_pairs(d, n);
    if (!p) return KO_ERR_NOMEM;
    int rc = ko_curve_sorted(p, n, k, K, err, tau, keep_eq, n_gt, n_eq);
    free(p);
    return rc;
}

/* O7 on a sorted layer: the first k entries of the order, emitted by ascending index.
 * value_dtype 0: val is float[k] holding d_i; 1: val is uint16_t[k] holding bf16_rne(d_i). */
static int ko_pack_sorted(const ko_pair* p, const float* d, uint64_t k, uint32_t value_dtype,
                          uint32_t* idx_out, void* val_out) {
    for (uint64_t i = 0; i < k; ++i) idx_out[i] = p[i].idx;
    qsort(idx_out, (size_t)k, sizeof(uint32_t), ko_cmp_u32);
    for (uint64_t i = 0; i < k; ++i) {
        float v = d[idx_out[i]];
        if (value_dtype == 0)
            ((float*)val_out)[i] = v;
        else
            ((uint16_t*)val_out)[i] = ko_bf16_rne(v);
    }
    return KO_OK;
}

int ko_select_pack(const float* d, uint64_t n, uint64_t k, uint32_t value_dtype, uint32_t* idx_out,
                   void* val_out) {
    if (!d || n == 0 || n > 0xffffffffull || k < 1 || k > n || value_dtype > 1 || !idx_out || !val_out)
        return KO_ERR_ARG;
    ko_pair* p = ko_sorted_pairs(d, n);
    if (!p) return KO_ERR_NOMEM;
    int rc = ko_pack_sorted(p, d, k, value_dtype, idx_out, val_out);
    free(p);
    return rc;
}

/* O8: g_i <- g_i + v_i on the kept entries, v_i the value actually sent. */
void ko_state_update(float* g, const uint32_t* idx, const void* val, uint64_t k, uint32_t value_dtype) {
    for (uint64_t i = 0; i < k; ++i) {
        float v = value_dtype == 0 ? ((const float*)val)[i] : ko_bf16_to_f32(((const uint16_t*)val)[i]);
        g[idx[i]] = g[idx[i]] + v;
    }
}

/* O5: c = floor(B * t) in binary64 (B in bytes/s, t in s). */
uint64_t ko_budget_bytes(double bandwidth_bytes_per_s, double t_target_s) {
    double c = floor(bandwidth_bytes_per_s * t_target_s);
    if (!(c > 0.0)) return 0;
    if (c >= 18446744073709551615.0) return 0xffffffffffffffffull;
    return (uint64_t)c;
}

/* O5: bytes_{l,j} = k_{l,j} * (4 + vb); cells_{l,j} = ceil(bytes * D / c).
 * Returns KO_STATUS_PLATEAU when c covers the largest candidate of every layer,
 * KO_STATUS_INFEASIBLE when c == 0 (cells then undefined), else 0. */
int ko_units(const uint64_t* k_table, uint32_t L, uint32_t K, uint32_t value_dtype, uint64_t c, uint32_t D,
             uint64_t* units_out /* [L][K] */) {
    uint64_t bpe = value_dtype == 0 ? 8 : 6;
    uint64_t full = 0;
    for (uint32_t l = 0; l < L; ++l) full += k_table[(size_t)l * K + (K - 1)] * bpe;
    if (c >= full) return KO_STATUS_PLATEAU;
    if (c == 0) return KO_STATUS_INFEASIBLE;
    for (uint32_t l = 0; l < L; ++l)
        for (uint32_t j = 0; j < K; ++j) {
            uint64_t bytes = k_table[(size_t)l * K + j] * bpe;
            units_out[(size_t)l * K + j] = (bytes * (uint64_t)D + c - 1) / c;
        }
    return KO_OK;
}

/* O6: Algorithm 3 read with the budget as the knapsack axis (D + 1 cells) and the
 * un-discretised binary32 error as the value.  Layer 1 is treated like every other
 * layer, from a virtual row prev = [0, inf, inf, ...].  Candidates in ascending j,
 * strict '<' (the first candidate that reaches a value keeps the cell), final cell =
 * the lowest b attaining the minimum, then the backward walk through PD.
 * Returns 0 or KO_STATUS_INFEASIBLE (then j_out is all zero). */
int ko_dp(const float* err /* [L][K] */, const uint64_t* units /* [L][K] */, uint32_t L, uint32_t K,
          uint32_t D, uint32_t* j_out /* [L] */, float* best_value, uint32_t* best_cell) {
    if (!err || !units || !j_out || L == 0 || K == 0 || D == 0) return KO_ERR_ARG;
    size_t row = (size_t)D + 1;
    float* prev = (float*)malloc(row * sizeof(float));
    float* cur = (float*)malloc(row * sizeof(float));
    uint32_t* PD = (uint32_t*)malloc(row * L * sizeof(uint32_t));
    if (!prev || !cur || !PD) {
        free(prev); free(cur); free(PD);
        return KO_ERR_NOMEM;
    }
    prev[0] = 0.0f;
    for (size_t b = 1; b < row; ++b) prev[b] = INFINITY;
    for (uint32_t l = 0; l < L; ++l) {
        for (size_t b = 0; b < row; ++b) { cur[b] = INFINITY; PD[(size_t)l * row + b] = 0; }
        for (uint32_t j = 0; j < K; ++j) {
            uint64_t u = units[(size_t)l * K + j];
            if (u > D) continue;
            float e = err[(size_t)l * K + j];
            for (size_t b = (size_t)u; b < row; ++b) {
                float t = prev[b - u] + e;
                if (t < cur[b]) { cur[b] = t; PD[(size_t)l * row + b] = j; }
            }
        }
        float* sw = prev; prev = cur; cur = sw;
    }
    size_t bstar = 0;
    for (size_t b = 1; b < row; ++b)
        if (prev[b] < prev[bstar]) bstar = b;
    int status = KO_OK;
    if (!(prev[bstar] < INFINITY)) {
        status = KO_STATUS_INFEASIBLE;
        for (uint32_t l = 0; l < L; ++l) j_out[l] = 0;
    } else {
        size_t b = bstar;
        for (uint32_t l = L; l-- > 0;) {
            uint32_t j = PD[(size_t)l * row + b];
            j_out[l] = j;
            b -= (size_t)units[(size_t)l * K + j];
        }
    }
    if (best_value) *best_value = prev[bstar];
    if (best_cell) *best_cell = (uint32_t)bstar;
    free(prev); free(cur); free(PD);
    return status;
}

/* Per-worker statistics reported by ko_step. */
typedef struct {
    uint64_t budget_bytes; /* c */
    uint64_t used_bytes;   /* sum_l bytes_{l, j_l} */
    uint64_t n_selected;   /* sum_l k_l */
    float total_err;       /* err_{1,j_1} + ... + err_{L,j_L}, added left to right in binary32 */
    int32_t status;        /* 0, KO_STATUS_INFEASIBLE or KO_STATUS_PLATEAU */
} ko_stats;

void ko_set_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}
int ko_get_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* O9: Kimad with one ratio for all layers (Section 3.1): the candidate index j is shared by the
 * layers and is the largest one whose total size sum_l k_{l,j} (4 + vb) fits the budget c.  Same
 * shortcuts and soft statuses as the layer-adaptive search: c >= full size -> PLATEAU (j = K-1),
 * nothing fits (or c == 0) -> INFEASIBLE (j = 0). */
int ko_uniform(const uint64_t* k_table, uint32_t L, uint32_t K, uint32_t value_dtype, uint64_t c, uint32_t* j_out) {
    if (!k_table || !j_out || L == 0 || K == 0 || value_dtype > 1) return KO_ERR_ARG;
    const uint64_t bpe = value_dtype == 0 ? 8 : 6;
    int found = 0;
    uint32_t best = 0;
    for (uint32_t j = 0; j < K; ++j) {
        uint64_t bytes = 0;
        for (uint32_t l = 0; l < L; ++l) bytes += k_table[(size_t)l * K + j] * bpe;
        if (bytes <= c) { found = 1; best = j; }
    }
    *j_out = best;
    if (!found || c == 0) return KO_STATUS_INFEASIBLE;
    if (best == K - 1) return KO_STATUS_PLATEAU;
    return KO_OK;
}

/* O10: the receiver of a packed message adds it to its copy of the sender's estimator
 * (Algorithm 1: u^_m <- u^_m + C_m(u_m - u^_m)).  est: [N] binary32, layers concatenated;
 * idx layer-local, offs [L+1].  One binary32 add per received entry. */
int ko_apply_packed(const uint64_t* layer_sizes, uint32_t L, const uint32_t* idx, const void* val,
                    const uint64_t* offs, uint32_t value_dtype, float* est) {
    if (!layer_sizes || !idx || !val || !offs || !est || value_dtype > 1) return KO_ERR_ARG;
    uint64_t begin = 0;
    for (uint32_t l = 0; l < L; ++l) {
        for (uint64_t p = offs[l]; p < offs[l + 1]; ++p) {
            if (idx[p] >= layer_sizes[l]) return KO_ERR_ARG;
            float v = value_dtype == 0 ? ((const float*)val)[p] : ko_bf16_to_f32(((const uint16_t*)val)[p]);
            est[begin + idx[p]] = est[begin + idx[p]] + v;
        }
        begin += layer_sizes[l];
    }
    return KO_OK;
}

/* O11: x_i <- x_i - gamma * sum_m w_m u^_{m,i} (Algorithm 1, last line).  binary32 throughout:
 * the sum runs over m = 0..W-1 in order, every product and every add rounded once (no FMA). */
int ko_aggregate(float* x, const float* est, uint64_t stride, uint32_t W, uint64_t N, const float* weights,
                 float gamma) {
    if (!x || !est || !weights || stride < N) return KO_ERR_ARG;
    for (uint64_t i = 0; i < N; ++i) {
        float acc = 0.0f;
        for (uint32_t m = 0; m < W; ++m) {
            float prod = weights[m] * est[(size_t)m * stride + i];
            acc = acc + prod;
        }
        float stepv = gamma * acc;
        x[i] = x[i] - stepv;
    }
    return KO_OK;
}

/* O12: Algorithm 3 read with the ERROR as the knapsack axis (the reading its header suggests).
 *   E_max  = sum_l err_{l,0} in binary64, layers in order: the error of the most aggressive candidate
 *            everywhere, i.e. the largest total error any assignment can have;
 *   cells  e_{l,j} = floor(err_{l,j} * D / E_max) (binary64 product, then quotient), 0 when E_max = 0;
 *            rounding DOWN keeps every assignment on the axis: sum_l e_{l,j_l} <= D;
 *   DP     value[l][e] = fewest kept entries sum k_{l,j} over assignments of layers 1..l whose cells add
 *            up to exactly e; virtual row [0, inf, ...]; candidates ascending, strict '<';
 *   answer the lowest e with value[L][e] * (4 + vb) <= c, then the walk back through PD.
 * Same shortcuts and statuses as O6: c >= full size -> PLATEAU; nothing fits -> INFEASIBLE, all j = 0. */
int ko_dp_error_axis(const float* err /* [L][K] */, const uint64_t* k_table /* [L][K] */, uint32_t L, uint32_t K,
                     uint32_t D, uint32_t value_dtype, uint64_t c, uint32_t* j_out /* [L] */, uint32_t* best_cell) {
    if (!err || !k_table || !j_out || L == 0 || K == 0 || D == 0 || value_dtype > 1) return KO_ERR_ARG;
    const uint64_t bpe = value_dtype == 0 ? 8 : 6;
    uint64_t full = 0;
    for (uint32_t l = 0; l < L; ++l) full += k_table[(size_t)l * K + (K - 1)] * bpe;
    if (c >= full) {
        for (uint32_t l = 0; l < L; ++l) j_out[l] = K - 1;
        return KO_STATUS_PLATEAU;
    }
    const uint64_t INF = UINT64_MAX;
    const size_t row = (size_t)D + 1;
    uint64_t* prev = (uint64_t*)malloc(row * sizeof(uint64_t));
    uint64_t* cur = (uint64_t*)malloc(row * sizeof(uint64_t));
    uint32_t* cells = (uint32_t*)malloc((size_t)L * K * sizeof(uint32_t));
    uint8_t* pd = (uint8_t*)malloc((size_t)L * row);
    if (!prev || !cur || !cells || !pd) { free(prev); free(cur); free(cells); free(pd); return KO_ERR_NOMEM; }
    double emax = 0.0;
    for (uint32_t l = 0; l < L; ++l) emax = emax + (double)err[(size_t)l * K];
    for (size_t i = 0; i < (size_t)L * K; ++i) {
        double q = 0.0;
        if (emax > 0.0) {
            double prod = (double)err[i] * (double)D;
            q = floor(prod / emax);
        }
        cells[i] = q > (double)D ? D : (uint32_t)q;
    }
    for (size_t b = 0; b < row; ++b) prev[b] = INF;
    prev[0] = 0;
    for (uint32_t l = 0; l < L; ++l) {
        for (size_t b = 0; b < row; ++b) cur[b] = INF;
        for (uint32_t j = 0; j < K; ++j) {
            const uint32_t u = cells[(size_t)l * K + j];
            const uint64_t k = k_table[(size_t)l * K + j];
            for (size_t b = u; b < row; ++b) {
                if (prev[b - u] == INF) continue;
                uint64_t t = prev[b - u] + k;
                if (t < cur[b]) { cur[b] = t; pd[(size_t)l * row + b] = (uint8_t)j; }
            }
        }
        uint64_t* sw = prev; prev = cur; cur = sw;
    }
    int status = KO_STATUS_INFEASIBLE;
    size_t bstar = 0;
    for (size_t b = 0; b < row; ++b)
        if (prev[b] != INF && prev[b] * bpe <= c) { bstar = b; status = KO_OK; break; }
    if (status == KO_OK) {
        if (best_cell) *best_cell = (uint32_t)bstar;
        size_t b = bstar;
        for (uint32_t l = L; l-- > 0;) {
            uint32_t j = pd[(size_t)l * row + b];
            j_out[l] = j;
            b -= cells[(size_t)l * K + j];
        }
    } else {
        for (uint32_t l = 0; l < L; ++l) j_out[l] = 0;
    }
    free(prev); free(cur); free(cells); free(pd);
    return status;
}

/* O9b: Kimad as Section 3.1 states it: the same ratio on all layers, sized to the budget.  The ratio
 * is a multiple of 2^-32: r = q / 2^32 with q in [0, 2^32], and layer l keeps
 *     k_l(q) = min(n_l, max(1, floor(q * n_l / 2^32)))      (at least one entry: Omega = {TopK : K > 0})
 * entries (exact integer arithmetic: n_l < 2^32, so the product fits 64 bits).  q is the LARGEST value with
 * sum_l k_l(q) <= entries, where entries = floor(c / (4 + vb)) is what the budget pays for.  k_l(q) does not
 * decrease with q, so q is found by bisection.
 *   entries < L  : not even one entry per layer fits -> q = 0, every k_l = 1, KO_STATUS_INFEASIBLE
 *   entries >= N : q = 2^32, every k_l = n_l, KO_STATUS_PLATEAU
 * With L = 1 this gives k = min(N, max(1, entries)): TopK over the whole model at K = floor(c / (4 + vb))
 * ("select K with the whole model information", Section 4.3), because floor(q N / 2^32) takes every value
 * 0..N as q runs over 0..2^32. */
static uint64_t ko_fit_sum(const uint64_t* layer_sizes, uint32_t L, uint64_t q, uint64_t* k_out) {
    uint64_t sum = 0;
    for (uint32_t l = 0; l < L; ++l) {
        uint64_t n = layer_sizes[l];
        uint64_t k = q >= 4294967296ull ? n : (q * n) >> 32;
        if (k < 1) k = 1;
        if (k > n) k = n;
        if (k_out) k_out[l] = k;
        sum += k;
    }
    return sum;
}

int ko_fit_ratio(const uint64_t* layer_sizes, uint32_t L, uint64_t entries, uint64_t* q_out, uint64_t* k_out /* [L] */) {
    if (!layer_sizes || L == 0) return KO_ERR_ARG;
    uint64_t N = 0;
    for (uint32_t l = 0; l < L; ++l) {
        if (layer_sizes[l] == 0 || layer_sizes[l] > 0xffffffffull) return KO_ERR_ARG;
        N += layer_sizes[l];
    }
    uint64_t q;
    int status = KO_OK;
    if (entries < (uint64_t)L) {
        q = 0;
        status = KO_STATUS_INFEASIBLE;
    } else if (entries >= N) {
        q = 4294967296ull;
        status = KO_STATUS_PLATEAU;
    } else {
        uint64_t lo = 0, hi = 4294967296ull; /* sum(lo) <= entries < sum(hi) */
        while (hi - lo > 1) {
            uint64_t mid = lo + (hi - lo) / 2;
            if (ko_fit_sum(layer_sizes, L, mid, NULL) <= entries) lo = mid; else hi = mid;
        }
        q = lo;
    }
    ko_fit_sum(layer_sizes, L, q, k_out);
    if (q_out) *q_out = q;
    return status;
}

/* O13: size and effect of candidate k of a layer of n elements under the two cost models.
 *   cost_model 0: bytes = k (4 + vb): u32 index + value for every kept entry (also at k = n).
 *   cost_model 1: if k (4 + vb) >= vb n the layer is sent DENSELY: all n values in order, no indices,
 *                 bytes = vb n; the candidate then keeps every entry (k_eff = n) and its error is 0.
 *                 Otherwise as cost model 0. */
void ko_candidate(uint64_t n, uint64_t k, uint32_t value_dtype, uint32_t cost_model, uint64_t* bytes, uint64_t* k_eff,
                  int* dense) {
    const uint64_t vb = value_dtype == 0 ? 4 : 2, bpe = 4 + vb;
    const int d = cost_model == 1 && k * bpe >= vb * n;
    if (bytes) *bytes = d ? vb * n : k * bpe;
    if (k_eff) *k_eff = d ? n : k;
    if (dense) *dense = d;
}

/* O5 on a table of sizes: cells_{l,j} = ceil(bytes_{l,j} * D / c); same return values as ko_units. */
int ko_units_from_bytes(const uint64_t* bytes_tab, uint32_t L, uint32_t K, uint64_t c, uint32_t D, uint64_t* units_out) {
    uint64_t full = 0;
    for (uint32_t l = 0; l < L; ++l) full += bytes_tab[(size_t)l * K + (K - 1)];
    if (c >= full) return KO_STATUS_PLATEAU;
    if (c == 0) return KO_STATUS_INFEASIBLE;
    for (size_t i = 0; i < (size_t)L * K; ++i) units_out[i] = (bytes_tab[i] * (uint64_t)D + c - 1) / c;
    return KO_OK;
}

/* The whole pass (O1..O8) for W workers.  Layout:
 *   grads, state : [W][stride] binary32, layers concatenated in list order (stride >= N)
 *   err/tau/keep_eq out : [W][L][K];  j_out/k_out : [W][L]
 *   idx_out : [W][cap] layer-local indices; val_out : [W][cap] float or uint16 (bf16)
 *   offs_out : [W][L+1] running sum of k_l
 * state is updated in place.  When inject_err != NULL the DP consumes that [W][L][K] table
 * instead of the curves computed here (the curves are still computed and returned).
 * policy 0: layer-adaptive search O6 (Kimad+); policy 1: one ratio of the grid for all layers O9;
 * policy 2: layer-adaptive search on the error axis O12; policy 3: one ratio sized to the budget O9b
 * (K must be 1: err/tau/keep_eq then describe the fitted k of every layer).  cost_model: O13 (0 or 1;
 * 1 only with policies 0 and 1); dense_out [W][L]: 1 where the chosen candidate is sent densely. */
int ko_step_ex(uint32_t policy, uint32_t cost_model, const uint64_t* layer_sizes, uint32_t L, uint32_t W, const double* ratios, uint32_t K, uint32_t D,
            uint32_t value_dtype, uint64_t stride, const float* grads, float* state,
            const double* bandwidth_bytes_per_s, double t_target_s, const float* inject_err, float* err_out,
            uint32_t* tau_out, uint32_t* keep_eq_out, uint32_t* j_out, uint32_t* k_out, uint32_t* idx_out,
            void* val_out, uint64_t cap, uint64_t* offs_out, ko_stats* stats_out, uint32_t* dense_out /* [W][L] or NULL */) {
    if (!layer_sizes || !ratios || !grads || !state || !bandwidth_bytes_per_s || L == 0 || W == 0 || K == 0 ||
        value_dtype > 1 || policy > 3 || cost_model > 1)
        return KO_ERR_ARG;
    if (policy == 3 && (K != 1 || cost_model != 0)) return KO_ERR_ARG; /* the fitted ratio is the only candidate */
    if (policy == 2 && cost_model != 0) return KO_ERR_ARG;
    uint64_t N = 0;
    for (uint32_t l = 0; l < L; ++l) N += layer_sizes[l];
    if (stride < N) return KO_ERR_ARG;
    /* the candidate table is per worker: policies 0..2 fill every worker's copy from the ratio grid, policy 3
     * from the ratio fitted to that worker's budget */
    uint64_t* ktab = (uint64_t*)malloc((size_t)W * L * K * sizeof(uint64_t));
    uint64_t* keff = (uint64_t*)malloc((size_t)W * L * sizeof(uint64_t)); /* entries actually kept per layer */
    uint64_t* loff = (uint64_t*)malloc(((size_t)L + 1) * sizeof(uint64_t));
    float* err = (float*)malloc((size_t)W * L * K * sizeof(float));
    uint32_t* jsel = (uint32_t*)malloc((size_t)W * L * sizeof(uint32_t));
    ko_stats* st = (ko_stats*)malloc((size_t)W * sizeof(ko_stats));
    float* d = (float*)malloc((size_t)W * (N ? N : 1) * sizeof(float));
    int* fit_status = (int*)calloc(W, sizeof(int));
    int rc = KO_OK;
    int fail = 0;
    const uint64_t bpe = value_dtype == 0 ? 8 : 6; /* bytes per kept entry: u32 index + value */
    const size_t vsz = value_dtype == 0 ? 4 : 2;
    if (!ktab || !keff || !loff || !err || !jsel || !st || !d || !fit_status) { rc = KO_ERR_NOMEM; goto done; }
    for (uint32_t w = 0; w < W; ++w) {
        if (policy == 3) {
            uint64_t c = ko_budget_bytes(bandwidth_bytes_per_s[w], t_target_s);
            rc = ko_fit_ratio(layer_sizes, L, c / bpe, NULL, ktab + (size_t)w * L);
            if (rc < 0) goto done;
            fit_status[w] = rc;
            rc = KO_OK;
        } else {
            rc = ko_k_table(layer_sizes, L, ratios, K, ktab + (size_t)w * L * K);
            if (rc != KO_OK) goto done;
        }
    }
    loff[0] = 0;
    for (uint32_t l = 0; l < L; ++l) loff[l + 1] = loff[l] + layer_sizes[l];

    /* O1 + O4: difference and error curve of every (worker, layer) */
#pragma omp parallel for schedule(dynamic, 1) collapse(2)
    for (uint32_t w = 0; w < W; ++w)
        for (uint32_t l = 0; l < L; ++l) {
            uint64_t n = layer_sizes[l];
            float* dl = d + (size_t)w * N + loff[l];
            ko_diff(grads + (size_t)w * stride + loff[l], state + (size_t)w * stride + loff[l], dl, n);
            size_t o = ((size_t)w * L + l) * K;
            int r = ko_layer_curve(dl, n, ktab + ((size_t)w * L + l) * K, K, err + o, tau_out ? tau_out + o : NULL,
                                   keep_eq_out ? keep_eq_out + o : NULL, NULL, NULL);
            if (r != KO_OK) {
#pragma omp atomic write
                fail = r;
            }
        }
    if (fail) { rc = fail; goto done; }
    if (err_out) memcpy(err_out, err, (size_t)W * L * K * sizeof(float));

    /* O5 + O6 per worker */
    for (uint32_t w = 0; w < W; ++w) {
        const float* e_in = (inject_err ? inject_err : err) + (size_t)w * L * K;
        const uint64_t* kt = ktab + (size_t)w * L * K;
        uint64_t c = ko_budget_bytes(bandwidth_bytes_per_s[w], t_target_s);
        uint64_t* units = (uint64_t*)malloc((size_t)L * K * sizeof(uint64_t));
        uint64_t* bytes = (uint64_t*)malloc((size_t)L * K * sizeof(uint64_t));
        uint64_t* kk = (uint64_t*)malloc((size_t)L * K * sizeof(uint64_t));
        float* e = (float*)malloc((size_t)L * K * sizeof(float));
        int* dense = (int*)malloc((size_t)L * K * sizeof(int));
        if (!units || !bytes || !kk || !e || !dense) { free(units); free(bytes); free(kk); free(e); free(dense); rc = KO_ERR_NOMEM; goto done; }
        /* O13: what every candidate costs, keeps and loses under the cost model */
        for (uint32_t l = 0; l < L; ++l)
            for (uint32_t j = 0; j < K; ++j) {
                size_t i = (size_t)l * K + j;
                ko_candidate(layer_sizes[l], kt[i], value_dtype, cost_model, &bytes[i], &kk[i], &dense[i]);
                e[i] = dense[i] ? 0.0f : e_in[i];
            }
        uint32_t* js = jsel + (size_t)w * L;
        int s;
        if (policy == 3) {
            s = fit_status[w];
            for (uint32_t l = 0; l < L; ++l) js[l] = 0;
        } else if (policy == 1) {
            /* O9 on the sizes of the cost model: the largest j whose total size fits */
            int found = 0;
            uint32_t best = 0;
            for (uint32_t j = 0; j < K; ++j) {
                uint64_t tot_b = 0;
                for (uint32_t l = 0; l < L; ++l) tot_b += bytes[(size_t)l * K + j];
                if (tot_b <= c) { found = 1; best = j; }
            }
            s = (!found || c == 0) ? KO_STATUS_INFEASIBLE : (best == K - 1 ? KO_STATUS_PLATEAU : KO_OK);
            for (uint32_t l = 0; l < L; ++l) js[l] = best;
        } else if (policy == 2) {
            s = ko_dp_error_axis(e, kt, L, K, D, value_dtype, c, js, NULL);
        } else {
            s = ko_units_from_bytes(bytes, L, K, c, D, units);
            if (s == KO_STATUS_PLATEAU) {
                for (uint32_t l = 0; l < L; ++l) js[l] = K - 1;
            } else if (s == KO_STATUS_INFEASIBLE) {
                for (uint32_t l = 0; l < L; ++l) js[l] = 0;
            } else {
                s = ko_dp(e, units, L, K, D, js, NULL, NULL);
            }
        }
        if (s < 0) { free(units); free(bytes); free(kk); free(e); free(dense); rc = s; goto done; }
        st[w].budget_bytes = c;
        st[w].status = s;
        st[w].used_bytes = 0;
        st[w].n_selected = 0;
        float tot = 0.0f;
        for (uint32_t l = 0; l < L; ++l) {
            size_t i = (size_t)l * K + js[l];
            keff[(size_t)w * L + l] = kk[i];
            if (dense_out) dense_out[(size_t)w * L + l] = (uint32_t)dense[i];
            st[w].used_bytes += bytes[i];
            st[w].n_selected += kk[i];
            tot = tot + e[i];
        }
        st[w].total_err = tot;
        free(units); free(bytes); free(kk); free(e); free(dense);
        if (st[w].n_selected > cap && idx_out) { rc = KO_ERR_CAPACITY; goto done; }
    }

    /* O7 + O8 */
    for (uint32_t w = 0; w < W; ++w) {
        uint64_t run = 0;
        for (uint32_t l = 0; l < L; ++l) {
            if (offs_out) offs_out[(size_t)w * (L + 1) + l] = run;
            run += keff[(size_t)w * L + l];
        }
        if (offs_out) offs_out[(size_t)w * (L + 1) + L] = run;
    }
#pragma omp parallel for schedule(dynamic, 1) collapse(2)
    for (uint32_t w = 0; w < W; ++w)
        for (uint32_t l = 0; l < L; ++l) {
            uint64_t n = layer_sizes[l];
            uint32_t j = jsel[(size_t)w * L + l];
            uint64_t k = keff[(size_t)w * L + l];
            if (j_out) j_out[(size_t)w * L + l] = j;
            if (k_out) k_out[(size_t)w * L + l] = (uint32_t)k;
            uint64_t off = 0;
            for (uint32_t q = 0; q < l; ++q) off += keff[(size_t)w * L + q];
            const float* dl = d + (size_t)w * N + loff[l];
            uint32_t* ib;
            void* vb;
            uint32_t* itmp = NULL;
            void* vtmp = NULL;
            if (idx_out && val_out) {
                ib = idx_out + (size_t)w * cap + off;
                vb = (char*)val_out + ((size_t)w * cap + off) * vsz;
            } else {
                itmp = (uint32_t*)malloc((size_t)k * sizeof(uint32_t));
                vtmp = malloc((size_t)k * vsz);
                ib = itmp;
                vb = vtmp;
            }
            int r = (ib && vb) ? ko_select_pack(dl, n, k, value_dtype, ib, vb) : KO_ERR_NOMEM;
            if (r == KO_OK) ko_state_update(state + (size_t)w * stride + loff[l], ib, vb, k, value_dtype);
            else {
#pragma omp atomic write
                fail = r;
            }
            free(itmp);
            free(vtmp);
        }
    if (fail) { rc = fail; goto done; }
    if (stats_out) memcpy(stats_out, st, (size_t)W * sizeof(ko_stats));
done:
    free(ktab); free(keff); free(loff); free(err); free(jsel); free(st); free(d); free(fit_status);
    return rc;
}

int ko_step_policy(uint32_t policy, const uint64_t* layer_sizes, uint32_t L, uint32_t W, const double* ratios, uint32_t K, uint32_t D,
            uint32_t value_dtype, uint64_t stride, const float* grads, float* state,
            const double* bandwidth_bytes_per_s, double t_target_s, const float* inject_err, float* err_out,
            uint32_t* tau_out, uint32_t* keep_eq_out, uint32_t* j_out, uint32_t* k_out, uint32_t* idx_out,
            void* val_out, uint64_t cap, uint64_t* offs_out, ko_stats* stats_out) {
    return ko_step_ex(policy, 0, layer_sizes, L, W, ratios, K, D, value_dtype, stride, grads, state, bandwidth_bytes_per_s,
                      t_target_s, inject_err, err_out, tau_out, keep_eq_out, j_out, k_out, idx_out, val_out, cap,
                      offs_out, stats_out, NULL);
}

int ko_step(const uint64_t* layer_sizes, uint32_t L, uint32_t W, const double* ratios, uint32_t K, uint32_t D,
            uint32_t value_dtype, uint64_t stride, const float* grads, float* state,
            const double* bandwidth_bytes_per_s, double t_target_s, const float* inject_err, float* err_out,
            uint32_t* tau_out, uint32_t* keep_eq_out, uint32_t* j_out, uint32_t* k_out, uint32_t* idx_out,
            void* val_out, uint64_t cap, uint64_t* offs_out, ko_stats* stats_out) {
    return ko_step_policy(0, layer_sizes, L, W, ratios, K, D, value_dtype, stride, grads, state, bandwidth_bytes_per_s,
                          t_target_s, inject_err, err_out, tau_out, keep_eq_out, j_out, k_out, idx_out, val_out, cap,
                          offs_out, stats_out);
}
