/*
 * CPU oracle of the MoE expert step (TEST INFRASTRUCTURE -- not a product path).
 *
 * Plain, slow, double-precision C written from the paper's description of the per-layer MoE
 * execution: top-k gating (Background, "Mixture-of-Experts Inference": a routing mechanism
 * selects the top-k experts per token), expert-aligned token repacking (Sec. IV-E: group the
 * (token, expert) pairs by expert id, contiguous per expert), batched dense execution of each
 * expert over its contiguous segment (Sec. IV-E), and the merge of expert outputs back to token
 * order (Sec. IV-D, hybrid pipeline, last paragraph).  The paper writes no formula for the gate
 * or the expert network; the readings taken here are: softmax over the k selected logits, SwiGLU
 * experts without biases, fixed summation order j = 0..k-1 in the merge.
 *
 * Only tests, the smoke check and the benchmark's cpu_baseline leg may call this file.  It shares
 * no code, header, table or helper with the CUDA library.
 *
 * Conventions: bf16 tensors are uint16 bit patterns, widened exactly; all arithmetic in double
 * (or, with acc_fp32 != 0, float accumulators, used only to bound the oracle's own rounding);
 * pair id p = t*k + j for token t and slot j; every matrix row-major.
 *
 * Parity pins (tests/test_oracle_*.py): route against a full sort and closed forms; repack against
 * the paper's worked example and a stable library sort; FFN against a float64 library dense
 * SwiGLU and the identity silu(z) - silu(-z) = z; combine against routing-independence with
 * identical experts and a dense softmax mixture at k = E.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_double(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* ---------------------------------------------------------------------------------- router logits
 * Linear router without bias (the paper only names "a routing mechanism"; reading taken):
 * logits[t, e] = sum_i x[t, i] * w_router[e, i], in double, from bf16 bit patterns.
 */
void saem_oracle_router_logits(const uint16_t* x, const uint16_t* w_router, int T, int E, int d, double* logits) {
    for (int t = 0; t < T; ++t)
        for (int e = 0; e < E; ++e) {
            double a = 0.0;
            for (int i = 0; i < d; ++i)
                a += bf16_to_double(x[(size_t)t * d + i]) * bf16_to_double(w_router[(size_t)e * d + i]);
            logits[(size_t)t * E + e] = a;
        }
}

/* ------------------------------------------------------------------------------------------ route
 * Gating.  For each token: k rounds of arg-max over the experts not yet chosen, comparing
 * (value descending, then expert id ascending); NaN logits count as -inf; +0 and -0 are equal.
 * Slot j holds the j-th largest.  Weights (renorm = 1): softmax over the k chosen logits.
 * renorm = 0: the chosen experts' probabilities under the softmax over all E logits.
 * Degenerate rows: if the largest chosen logit is -inf, every weight is 1/k; if it is +inf, the
 * +inf slots share the weight equally and the rest get 0.
 */
void saem_oracle_route(const float* logits, int T, int E, int k, int renorm,
                       int32_t* topk_idx, double* topk_w) {
    double* v = (double*)malloc(sizeof(double) * (size_t)E);
    char* taken = (char*)malloc((size_t)E);
    for (int t = 0; t < T; ++t) {
        for (int e = 0; e < E; ++e) {
            float l = logits[(size_t)t * E + e];
            v[e] = isnan(l) ? -INFINITY : (double)l;
            taken[e] = 0;
        }
        for (int j = 0; j < k; ++j) {
            int best = -1;
            for (int e = 0; e < E; ++e) {
                if (taken[e]) continue;
                if (best < 0 || v[e] > v[best]) best = e;   /* strict: lower id wins ties */
            }
            taken[best] = 1;
            topk_idx[(size_t)t * k + j] = best;
        }
        double m = v[topk_idx[(size_t)t * k]];
        double* w = topk_w + (size_t)t * k;
        if (m == -INFINITY) {
            for (int j = 0; j < k; ++j) w[j] = 1.0 / k;
        } else if (m == INFINITY) {
            int n_inf = 0;
            for (int j = 0; j < k; ++j) n_inf += (v[topk_idx[(size_t)t * k + j]] == INFINITY);
            for (int j = 0; j < k; ++j)
                w[j] = (v[topk_idx[(size_t)t * k + j]] == INFINITY) ? 1.0 / n_inf : 0.0;
        } else {
            double denom = 0.0;
            if (renorm) {
                for (int j = 0; j < k; ++j) denom += exp(v[topk_idx[(size_t)t * k + j]] - m);
            } else {
                for (int e = 0; e < E; ++e) denom += exp(v[e] - m);
            }
            for (int j = 0; j < k; ++j) w[j] = exp(v[topk_idx[(size_t)t * k + j]] - m) / denom;
        }
    }
    free(v);
    free(taken);
}

/* ----------------------------------------------------------------------------------------- repack
 * Expert-aligned token repacking (Sec. IV-E).  counts[e] = number of pairs routed to e; offsets =
 * exclusive prefix sum (offsets[E] = T*k); segments in ascending expert id; inside a segment the
 * pairs keep ascending pair id (so x0 precedes x3 for E0 in the paper's example).  perm[r] = pair
 * stored at packed row r; inv_perm[p] = packed row of pair p; x_packed[r] = x[perm[r] / k].
 */
void saem_oracle_repack(const int32_t* topk_idx, const uint16_t* x, int T, int E, int k, int d,
                        int32_t* counts, int32_t* offsets, int32_t* perm, int32_t* inv_perm,
                        uint16_t* x_packed) {
    int P = T * k;
    for (int e = 0; e < E; ++e) counts[e] = 0;
    for (int p = 0; p < P; ++p) counts[topk_idx[p]] += 1;
    offsets[0] = 0;
    for (int e = 0; e < E; ++e) offsets[e + 1] = offsets[e] + counts[e];
    int32_t* pos = (int32_t*)malloc(sizeof(int32_t) * (size_t)(E > 0 ? E : 1));
    for (int e = 0; e < E; ++e) pos[e] = offsets[e];
    for (int p = 0; p < P; ++p) {
        int e = topk_idx[p];
        int r = pos[e]++;
        perm[r] = p;
        inv_perm[p] = r;
        if (x && x_packed) memcpy(x_packed + (size_t)r * d, x + (size_t)(p / k) * d, sizeof(uint16_t) * (size_t)d);
    }
    free(pos);
}

/* -------------------------------------------------------------------------------------------- ffn
 * Dense per-expert execution over each contiguous segment.  Expert e owns rows
 * [offsets[e], offsets[e+1]).  For a row x_r:  g = Wg_e x_r,  u = Wu_e x_r,
 * h = g / (1 + exp(-g)) * u  (SiLU(g) * u),  y_r = Wd_e h.   gate/up: [f,d]; down: [d,f].
 * Pointer arrays are indexed by expert id; an expert with an empty segment may be NULL.
 */
static void ffn_row(const uint16_t* xr, const uint16_t* Wg, const uint16_t* Wu, const uint16_t* Wd,
                    int d, int f, int acc_fp32, double* xd, double* h, double* y) {
    for (int i = 0; i < d; ++i) xd[i] = bf16_to_double(xr[i]);
    for (int j = 0; j < f; ++j) {
        const uint16_t* wg = Wg + (size_t)j * d;
        const uint16_t* wu = Wu + (size_t)j * d;
        double g, u;
        if (acc_fp32) {
            float gf = 0.f, uf = 0.f;
            for (int i = 0; i < d; ++i) {
                gf += (float)bf16_to_double(wg[i]) * (float)xd[i];
                uf += (float)bf16_to_double(wu[i]) * (float)xd[i];
            }
            g = gf; u = uf;
        } else {
            g = 0.0; u = 0.0;
            for (int i = 0; i < d; ++i) {
                g += bf16_to_double(wg[i]) * xd[i];
                u += bf16_to_double(wu[i]) * xd[i];
            }
        }
        h[j] = g / (1.0 + exp(-g)) * u;
    }
    for (int c = 0; c < d; ++c) {
        const uint16_t* wd = Wd + (size_t)c * f;
        if (acc_fp32) {
            float a = 0.f;
            for (int j = 0; j < f; ++j) a += (float)bf16_to_double(wd[j]) * (float)h[j];
            y[c] = a;
        } else {
            double a = 0.0;
            for (int j = 0; j < f; ++j) a += bf16_to_double(wd[j]) * h[j];
            y[c] = a;
        }
    }
}

void saem_oracle_expert_ffn(const uint16_t* x_packed, const int32_t* offsets, int E, int d, int f,
                            const uint16_t* const* gate, const uint16_t* const* up,
                            const uint16_t* const* down, int acc_fp32, double* y_packed) {
    int P = offsets[E];
#pragma omp parallel
    {
        double* xd = (double*)malloc(sizeof(double) * (size_t)d);
        double* h = (double*)malloc(sizeof(double) * (size_t)f);
#pragma omp for schedule(dynamic, 1)
        for (int r = 0; r < P; ++r) {
            int e = 0;
            while (!(offsets[e] <= r && r < offsets[e + 1])) ++e;
            ffn_row(x_packed + (size_t)r * d, gate[e], up[e], down[e], d, f, acc_fp32, xd, h,
                    y_packed + (size_t)r * d);
        }
        free(xd);
        free(h);
    }
}

/* ---------------------------------------------------------------------------------------- combine
 * Merge back to token order: out[t] = sum_{j = 0..k-1, in that order} w[t,j] * y_packed[inv_perm[t*k+j]]
 * (+ shared_y[t] when the layer has always-on shared experts, added last, weight 1).
 */
void saem_oracle_combine(const double* y_packed, const int32_t* inv_perm, const double* topk_w,
                         int T, int k, int d, const double* shared_y, double* out) {
    for (int t = 0; t < T; ++t) {
        for (int c = 0; c < d; ++c) {
            double a = 0.0;
            for (int j = 0; j < k; ++j)
                a += topk_w[(size_t)t * k + j] * y_packed[(size_t)inv_perm[(size_t)t * k + j] * d + c];
            if (shared_y) a += shared_y[(size_t)t * d + c];
            out[(size_t)t * d + c] = a;
        }
    }
}

/* --------------------------------------------------------------------------------------- full step
 * route -> repack -> expert FFN -> (shared expert over every token) -> combine.
 * Scratch outputs may be NULL except out; shared_* NULL / f_shared = 0 when the layer has none.
 */
void saem_oracle_moe_step(const float* logits, const uint16_t* x, int T, int E, int k, int d, int f,
                          int renorm, const uint16_t* const* gate, const uint16_t* const* up,
                          const uint16_t* const* down, int f_shared, const uint16_t* shared_gate,
                          const uint16_t* shared_up, const uint16_t* shared_down, int acc_fp32,
                          int32_t* topk_idx, double* topk_w, int32_t* counts, int32_t* offsets,
                          int32_t* perm, int32_t* inv_perm, uint16_t* x_packed, double* y_packed,
                          double* shared_y, double* out) {
    int P = T * k;
    saem_oracle_route(logits, T, E, k, renorm, topk_idx, topk_w);
    saem_oracle_repack(topk_idx, x, T, E, k, d, counts, offsets, perm, inv_perm, x_packed);
    saem_oracle_expert_ffn(x_packed, offsets, E, d, f, gate, up, down, acc_fp32, y_packed);
    (void)P;
    if (f_shared > 0) {
        int32_t so[2] = {0, T};
        const uint16_t* g1[1] = {shared_gate};
        const uint16_t* u1[1] = {shared_up};
        const uint16_t* d1[1] = {shared_down};
        saem_oracle_expert_ffn(x, so, 1, d, f_shared, g1, u1, d1, acc_fp32, shared_y);
    }
    saem_oracle_combine(y_packed, inv_perm, topk_w, T, k, d, f_shared > 0 ? shared_y : NULL, out);
}

int saem_oracle_max_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
