/*
 * CPU oracle for the D-cut verify hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, by-the-definition implementation used by the tests, by the smoke check and by
 * the CPU-baseline leg of the benchmark.  Nothing in the product path may call it, and it shares
 * no code, header, table or helper with the CUDA library.
 *
 * What each function follows (paper = "D-cut: Adaptive Verification Depth Pruning for Batched
 * Speculative Decoding"):
 *   oracle_scores       Eq. 3 (prefix-product survival score), Algorithm 1 step 2
 *   oracle_budget       Eq. 4 (ratio bucket capacity)
 *   oracle_select       Eq. 3-5, Algorithm 1 steps 2-12, Appendix A "Retained positions form a
 *                       contiguous prefix", Appendix C "Packing"
 *   oracle_verify_attn  Appendix C "score each retained position against its accepted prefix":
 *                       plain causal softmax attention over the paged cache, in double
 *   oracle_accept       Section 3.1 / 3.2 (sequential greedy acceptance, A_i = 1 + min(L_i, n_i),
 *                       bonus token)
 *   oracle_layer_*      the decoder-layer pieces of the full-layer workload (textbook RMSNorm,
 *                       rotary embedding, SwiGLU, matrix product; not from the paper)
 *   oracle_scores_shifted, oracle_select_causal, oracle_accept_rs
 *                       Appendix B "Causality under Rejection Sampling": Eq. 7 (shifted score), the
 *                       causal early-stopping frontier scan, standard rejection sampling with the
 *                       residual distribution
 *
 * Parity pins: every function here is pinned by tests/test_oracle_*.py against closed forms,
 * brute force, hand-derived examples or numpy float64 formulas, except the comparison of the
 * selector's expected advance with the realised accepted count, which is "parity unpinned"
 * (the synthetic confidences are only loosely calibrated to the planted rejects).
 *
 * Readings of points the paper leaves open are listed next to the code that takes them.
 * Build: gcc -O2 -fopenmp -ffp-contract=off (no fast-math: fp32 products must round once each).
 */
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_EINVAL 1
#define ORACLE_ECOST 4

/* ------------------------------------------------------------------------------------------ */
/* bf16 helpers                                                                                */

static float bf16_to_float(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* round-to-nearest-even fp32 -> bf16 (used only where the layer materialises a bf16 tensor) */
static uint16_t float_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u); /* quiet NaN */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

/* ------------------------------------------------------------------------------------------ */
/* Eq. 3: s_{i,k} = prod_{t<=k} c_{i,t}, s_{i,0} = 1.                                           */
/* Reading: confidences are clamped to [0,1] and NaN counts as 0 (keeps the score non-increasing */
/* for any input); the product is taken directly in fp32, left to right, one rounding per        */
/* multiply (the appendix mentions accumulated log-confidences; Eq. 3 and Eq. 5 need s itself);  */
/* -0 is written as +0.  scores is [B, gamma]: entry (i, k-1) holds s_{i,k}.                     */

static float clamp_conf(float c) {
    if (!(c == c)) return 0.0f;
    if (c < 0.0f) return 0.0f;
    if (c > 1.0f) return 1.0f;
    return c;
}

int oracle_scores(const float* conf, int B, int gamma, float* scores) {
    if (!conf || !scores || B < 0 || gamma < 0) return ORACLE_EINVAL;
    for (int i = 0; i < B; ++i) {
        float s = 1.0f; /* s_{i,0} */
        for (int k = 1; k <= gamma; ++k) {
            float c = clamp_conf(conf[(size_t)i * gamma + (k - 1)]);
            s = s * c;             /* one fp32 rounding per step */
            if (s == 0.0f) s = 0.0f; /* -0 -> +0 */
            scores[(size_t)i * gamma + (k - 1)] = s;
        }
    }
    return ORACLE_OK;
}

/* Eq. 4: K_rho(B) = max(B, ceil(rho * B * (D+1))) with rho = num/den, in exact integers. */
int oracle_budget(int B, int gamma, int num, int den, int* K) {
    if (!K || B < 0 || gamma < 0 || num < 0 || den <= 0) return ORACLE_EINVAL;
    int64_t total = (int64_t)B * (gamma + 1);
    int64_t k = (total * num + den - 1) / den;
    if (k < B) k = B;
    if (k > total) k = total;
    *K = (int)k;
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------ */
/* Selection.                                                                                   */

typedef struct {
    float p;
    int k; /* depth 1..gamma */
    int i; /* request */
} pos_t;

/* Ranking order (Algorithm 1 step 5 "ties toward smaller k"; Appendix B "shallower depth and   */
/* then request index"): score descending, then depth ascending, then request ascending.        */
static int pos_before(const void* a, const void* b) {
    const pos_t* x = (const pos_t*)a;
    const pos_t* y = (const pos_t*)b;
    if (x->p > y->p) return -1;
    if (x->p < y->p) return 1;
    if (x->k != y->k) return x->k < y->k ? -1 : 1;
    if (x->i != y->i) return x->i < y->i ? -1 : 1;
    return 0;
}

typedef struct {
    int32_t n_star;      /* selected draft positions N* (= K* - B)                       */
    int32_t t_total;     /* packed length T = B + N* (= the paper's K)                    */
    int32_t candidate;   /* index of the winning candidate (dense: N*; bucket: bucket id) */
    int32_t closure_ok;  /* 1 if every request's selected set is a contiguous prefix      */
    int64_t sum_fixed;   /* B*2^40 + sum of floor(p*2^40) over the selected positions     */
    double objective;    /* sum_fixed / cost                                              */
    double sum_f64;      /* B + plain sequential double sum of the selected scores        */
} oracle_select_info;

/*
 * mode 0 (dense): candidates N = 0..B*gamma, cost_ms[T] indexed by the packed length T = B + N
 *                 (n_cost entries; needs n_cost > B*(gamma+1)).
 * mode 1 (bucket, the paper's Eq. 4-5): candidates N_r = bucket_K[r] - B, cost_ms[r] per bucket;
 *                 bucket_K ascending, B <= K <= B*(gamma+1).
 *
 * Readings: the paper ranks all B(D+1) positions including the B bonus positions whose score is
 * 1; with the tie rule above those always come first, so top-K of the paper = the B bonus
 * positions plus the top-(K-B) draft positions, and the numerator of Eq. 5 is B + sum of the
 * top-N draft scores.  The sum is taken exactly: each score is truncated to a multiple of 2^-40
 * and summed in int64 (order independent; changes the objective by < 4e-9 relative); the plain
 * double sum is reported beside it.  The objective is one fp64 divide by (double)cost_fp32; among
 * equal objectives the smallest N wins.  n_i is the count of selected positions of request i
 * (Algorithm 1 step 10 takes the max k; both agree because the set is prefix-closed, which is
 * checked and reported in closure_ok).  Packing is request-major, bonus first, positions
 * ascending; tok_pos = L_i + t.
 */
int oracle_select(const float* conf, int B, int gamma, const int32_t* draft_ids,
                  const int32_t* bonus_ids, const int32_t* ctx_lens, int mode, const float* cost_ms,
                  int n_cost, const int32_t* bucket_K, int32_t* depths, int32_t* cu_q,
                  int32_t* tok_req, int32_t* tok_pos, int32_t* tok_id, int32_t* ranks,
                  float* scores_out, oracle_select_info* info) {
    if (!conf || !depths || !cu_q || !info || !cost_ms || B < 0 || gamma < 0) return ORACLE_EINVAL;
    const int n = B * gamma;
    const int64_t ONE = (int64_t)1 << 40;
    float* p = (float*)malloc(sizeof(float) * (size_t)(n > 0 ? n : 1));
    pos_t* order = (pos_t*)malloc(sizeof(pos_t) * (size_t)(n > 0 ? n : 1));
    int64_t* Q = (int64_t*)malloc(sizeof(int64_t) * (size_t)(n + 1));
    double* S = (double*)malloc(sizeof(double) * (size_t)(n + 1));
    int rc = ORACLE_OK;
    oracle_scores(conf, B, gamma, p);
    if (scores_out) memcpy(scores_out, p, sizeof(float) * (size_t)n);
    for (int i = 0; i < B; ++i)
        for (int k = 1; k <= gamma; ++k) {
            pos_t* e = &order[i * gamma + (k - 1)];
            e->p = p[i * gamma + (k - 1)];
            e->k = k;
            e->i = i;
        }
    qsort(order, (size_t)n, sizeof(pos_t), pos_before);
    Q[0] = 0;
    S[0] = 0.0;
    for (int r = 0; r < n; ++r) {
        double scaled = (double)order[r].p * 1099511627776.0; /* exact: power-of-two scaling */
        Q[r + 1] = Q[r] + (int64_t)floor(scaled);
        S[r + 1] = S[r] + (double)order[r].p;
    }
    /* candidates */
    int best = -1, best_N = 0;
    double best_obj = 0.0;
    int n_cand = (mode == 0) ? n + 1 : n_cost;
    if (mode == 0 && n_cost < B + n + 1) rc = ORACLE_ECOST;
    if (mode == 1 && (!bucket_K || n_cost <= 0)) rc = ORACLE_EINVAL;
    for (int c = 0; rc == ORACLE_OK && c < n_cand; ++c) {
        int N;
        float cost;
        if (mode == 0) {
            N = c;
            cost = cost_ms[B + N];
        } else {
            if (bucket_K[c] < B || bucket_K[c] > B + n || (c > 0 && bucket_K[c] <= bucket_K[c - 1])) {
                rc = ORACLE_EINVAL;
                break;
            }
            N = bucket_K[c] - B;
            cost = cost_ms[c];
        }
        if (!(cost > 0.0f) || isinf(cost)) {
            rc = ORACLE_ECOST;
            break;
        }
        double obj = (double)((int64_t)B * ONE + Q[N]) / (double)cost;
        if (best < 0 || obj > best_obj) {
            best = c;
            best_obj = obj;
            best_N = N;
        }
    }
    if (rc == ORACLE_OK) {
        info->n_star = best_N;
        info->t_total = B + best_N;
        info->candidate = best;
        info->sum_fixed = (int64_t)B * ONE + Q[best_N];
        info->objective = best_obj;
        info->sum_f64 = (double)B + S[best_N];
        int closure = 1;
        for (int i = 0; i < B; ++i) depths[i] = 0;
        int* maxk = (int*)calloc((size_t)(B > 0 ? B : 1), sizeof(int));
        for (int r = 0; r < n; ++r) {
            if (ranks) ranks[order[r].i * gamma + (order[r].k - 1)] = r;
            if (r < best_N) {
                depths[order[r].i] += 1;
                if (order[r].k > maxk[order[r].i]) maxk[order[r].i] = order[r].k;
            }
        }
        for (int i = 0; i < B; ++i)
            if (maxk[i] != depths[i]) closure = 0;
        free(maxk);
        info->closure_ok = closure;
        cu_q[0] = 0;
        for (int i = 0; i < B; ++i) cu_q[i + 1] = cu_q[i] + 1 + depths[i];
        for (int i = 0; i < B; ++i)
            for (int t = 0; t <= depths[i]; ++t) {
                int r = cu_q[i] + t;
                if (tok_req) tok_req[r] = i;
                if (tok_pos) tok_pos[r] = (ctx_lens ? ctx_lens[i] : 0) + t;
                if (tok_id) {
                    if (t == 0)
                        tok_id[r] = bonus_ids ? bonus_ids[i] : -1;
                    else
                        tok_id[r] = draft_ids ? draft_ids[i * gamma + (t - 1)] : -1;
                }
            }
    }
    free(p);
    free(order);
    free(Q);
    free(S);
    return rc;
}

/* ------------------------------------------------------------------------------------------ */
/* Verification attention: each retained position (i, t), t = 0..d_i, attends to the cache     */
/* positions j <= L_i + t of its own request (its accepted prefix, the bonus and the shallower  */
/* drafts, all of which already sit in the paged cache).  Grouped-query: q head h reads kv head */
/* h / (Hq/Hkv).  Cache layout [num_pages, Hkv, page_size, Dh]; position j lives in page        */
/* block_table[i][j / page_size], slot j % page_size.  Everything in double.                    */
/* samples: if n_samples > 0, only rows (sample_tok[s], sample_head[s]) are computed and out is */
/* [n_samples, Dh], lse [n_samples]; otherwise out is [T, Hq, Dh], lse [T, Hq].                 */

int oracle_verify_attn(const uint16_t* q, const uint16_t* k_cache, const uint16_t* v_cache,
                       const int32_t* block_table, const int32_t* ctx_lens, const int32_t* cu_q,
                       int B, int n_q_heads, int n_kv_heads, int head_dim, int page_size,
                       int max_pages_per_req, double scale, const int32_t* sample_tok,
                       const int32_t* sample_head, int n_samples, double* out, double* lse) {
    if (!q || !k_cache || !v_cache || !block_table || !ctx_lens || !cu_q || !out) return ORACLE_EINVAL;
    if (n_kv_heads <= 0 || n_q_heads % n_kv_heads) return ORACLE_EINVAL;
    const int T = cu_q[B];
    const int group = n_q_heads / n_kv_heads;
    const long n_rows = n_samples > 0 ? n_samples : (long)T * n_q_heads;
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 4)
    for (long row = 0; row < n_rows; ++row) {
        int tok, h;
        if (n_samples > 0) {
            tok = sample_tok[row];
            h = sample_head[row];
        } else {
            tok = (int)(row / n_q_heads);
            h = (int)(row % n_q_heads);
        }
        if (tok < 0 || tok >= T || h < 0 || h >= n_q_heads) {
            bad = 1;
            continue;
        }
        int i = 0;
        while (!(cu_q[i] <= tok && tok < cu_q[i + 1])) ++i;
        const int t = tok - cu_q[i];
        const int n_keys = ctx_lens[i] + t + 1; /* j = 0 .. L_i + t */
        const int kvh = h / group;
        const uint16_t* qv = q + ((size_t)tok * n_q_heads + h) * head_dim;
        double* s = (double*)malloc(sizeof(double) * (size_t)n_keys);
        double m = -INFINITY;
        for (int j = 0; j < n_keys; ++j) {
            const int page = block_table[(size_t)i * max_pages_per_req + j / page_size];
            const uint16_t* kv =
                k_cache + (((size_t)page * n_kv_heads + kvh) * page_size + j % page_size) * head_dim;
            double acc = 0.0;
            for (int e = 0; e < head_dim; ++e) acc += (double)bf16_to_float(qv[e]) * (double)bf16_to_float(kv[e]);
            s[j] = acc * scale;
            if (s[j] > m) m = s[j];
        }
        double denom = 0.0;
        for (int j = 0; j < n_keys; ++j) {
            s[j] = exp(s[j] - m);
            denom += s[j];
        }
        double* o = out + (size_t)row * head_dim;
        for (int e = 0; e < head_dim; ++e) o[e] = 0.0;
        for (int j = 0; j < n_keys; ++j) {
            const int page = block_table[(size_t)i * max_pages_per_req + j / page_size];
            const uint16_t* vv =
                v_cache + (((size_t)page * n_kv_heads + kvh) * page_size + j % page_size) * head_dim;
            const double w = s[j] / denom;
            for (int e = 0; e < head_dim; ++e) o[e] += w * (double)bf16_to_float(vv[e]);
        }
        if (lse) lse[row] = m + log(denom);
        free(s);
    }
    return bad ? ORACLE_EINVAL : ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------ */
/* Greedy acceptance.  Row (i, t) of the packed logits sits at the token z_{i,t} and predicts    */
/* z_{i,t+1}.  a_{i,t} = argmax_v logits[cu_q[i]+t, v]; ascending scan with strict '>' on the    */
/* bf16 values widened to float, so the lowest index wins ties and NaN never wins (an all-NaN    */
/* row gives 0).  m_i = the longest prefix with a_{i,t} = z_{i,t+1}, t < d_i; the bonus is       */
/* a_{i,m_i}; emitted tokens = z_{i,1..m_i} then the bonus; out_tokens is [B, gamma+1], -1       */
/* padded; n_accepted_total = sum_i (m_i + 1) = sum_i A_i with A_i = 1 + min(L_i, n_i).          */

int oracle_accept(const uint16_t* logits, int V, const int32_t* draft_ids, const int32_t* cu_q, int B,
                  int gamma, int32_t* accept_len, int32_t* bonus, int32_t* out_tokens,
                  int32_t* n_accepted_total, int32_t* argmax_out) {
    if (!logits || !draft_ids || !cu_q || !accept_len || !bonus || V <= 0) return ORACLE_EINVAL;
    const int T = cu_q[B];
    int32_t* am = (int32_t*)malloc(sizeof(int32_t) * (size_t)(T > 0 ? T : 1));
#pragma omp parallel for schedule(static)
    for (int r = 0; r < T; ++r) {
        const uint16_t* row = logits + (size_t)r * V;
        int best = 0;
        float bv = -INFINITY;
        int have = 0;
        for (int v = 0; v < V; ++v) {
            float x = bf16_to_float(row[v]);
            if (!(x == x)) continue;
            if (!have || x > bv) {
                have = 1;
                bv = x;
                best = v;
            }
        }
        am[r] = best;
    }
    long total = 0;
    for (int i = 0; i < B; ++i) {
        const int d = cu_q[i + 1] - cu_q[i] - 1;
        int m = 0;
        while (m < d && am[cu_q[i] + m] == draft_ids[(size_t)i * gamma + m]) ++m;
        accept_len[i] = m;
        bonus[i] = am[cu_q[i] + m];
        if (out_tokens) {
            for (int t = 0; t <= gamma; ++t) out_tokens[(size_t)i * (gamma + 1) + t] = -1;
            for (int t = 0; t < m; ++t) out_tokens[(size_t)i * (gamma + 1) + t] = draft_ids[(size_t)i * gamma + t];
            out_tokens[(size_t)i * (gamma + 1) + m] = bonus[i];
        }
        total += m + 1;
    }
    if (n_accepted_total) *n_accepted_total = (int32_t)total;
    if (argmax_out) memcpy(argmax_out, am, sizeof(int32_t) * (size_t)T);
    free(am);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------ */
/* Decoder-layer pieces (full-layer workload).  Double-precision math on bf16 inputs; each      */
/* function returns doubles and, where asked, the bf16 rounding of them, so the caller can      */
/* round at the tensor boundaries the GPU materialises.                                          */

void oracle_round_bf16(const double* x, long n, uint16_t* out) {
    for (long i = 0; i < n; ++i) out[i] = float_to_bf16((float)x[i]);
}

/* y[r, :] = x[r, :] / sqrt(mean(x[r,:]^2) + eps) * gain */
int oracle_rmsnorm(const uint16_t* x, const uint16_t* gain, int rows, int hidden, double eps, double* y) {
    if (!x || !gain || !y) return ORACLE_EINVAL;
#pragma omp parallel for
    for (int r = 0; r < rows; ++r) {
        double ss = 0.0;
        for (int c = 0; c < hidden; ++c) {
            double v = bf16_to_float(x[(size_t)r * hidden + c]);
            ss += v * v;
        }
        double inv = 1.0 / sqrt(ss / hidden + eps);
        for (int c = 0; c < hidden; ++c)
            y[(size_t)r * hidden + c] =
                (double)bf16_to_float(x[(size_t)r * hidden + c]) * inv * (double)bf16_to_float(gain[c]);
    }
    return ORACLE_OK;
}

/* C[m, n] = sum_k A[m, k] * W[n, k]   (activations times a weight stored [out, in]) */
int oracle_linear(const uint16_t* a, const uint16_t* w, int M, int N, int K, double* c) {
    if (!a || !w || !c) return ORACLE_EINVAL;
#pragma omp parallel for collapse(2) schedule(static)
    for (int m = 0; m < M; ++m)
        for (int n = 0; n < N; ++n) {
            double acc = 0.0;
            const uint16_t* ar = a + (size_t)m * K;
            const uint16_t* wr = w + (size_t)n * K;
            for (int k = 0; k < K; ++k) acc += (double)bf16_to_float(ar[k]) * (double)bf16_to_float(wr[k]);
            c[(size_t)m * N + n] = acc;
        }
    return ORACLE_OK;
}

/* Rotary embedding, rotate-half form on the whole head: for e < Dh/2,                         */
/*   out[e] = x[e] cos(a_e) - x[e+Dh/2] sin(a_e),  out[e+Dh/2] = x[e+Dh/2] cos(a_e) + x[e] sin(a_e), */
/*   a_e = pos * theta^(-2e/Dh).  x is [rows, heads, Dh] bf16; pos is per row.                   */
int oracle_rope(const uint16_t* x, const int32_t* pos, int rows, int heads, int head_dim, double theta,
                double* y) {
    if (!x || !pos || !y || head_dim % 2) return ORACLE_EINVAL;
    const int half = head_dim / 2;
    for (int r = 0; r < rows; ++r)
        for (int h = 0; h < heads; ++h) {
            const uint16_t* xv = x + ((size_t)r * heads + h) * head_dim;
            double* yv = y + ((size_t)r * heads + h) * head_dim;
            for (int e = 0; e < half; ++e) {
                double ang = (double)pos[r] * pow(theta, -2.0 * e / head_dim);
                double c = cos(ang), s = sin(ang);
                double x0 = bf16_to_float(xv[e]), x1 = bf16_to_float(xv[e + half]);
                yv[e] = x0 * c - x1 * s;
                yv[e + half] = x1 * c + x0 * s;
            }
        }
    return ORACLE_OK;
}

/* SwiGLU gate: y = silu(g) * u, silu(g) = g / (1 + exp(-g)) */
int oracle_swiglu(const uint16_t* g, const uint16_t* u, long n, double* y) {
    if (!g || !u || !y) return ORACLE_EINVAL;
    for (long i = 0; i < n; ++i) {
        double gv = bf16_to_float(g[i]), uv = bf16_to_float(u[i]);
        y[i] = gv / (1.0 + exp(-gv)) * uv;
    }
    return ORACLE_OK;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* SwiGLU on double inputs (the product is the only tensor the GPU materialises, so gate and up are
 * not rounded in between): y = g / (1 + exp(-g)) * u */
int oracle_swiglu_f64(const double* g, const double* u, long n, double* y) {
    if (!g || !u || !y) return ORACLE_EINVAL;
    for (long i = 0; i < n; ++i) y[i] = g[i] / (1.0 + exp(-g[i])) * u[i];
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------ */
/* Stochastic variant (Appendix B "Causality under Rejection Sampling").                       */
/*                                                                                              */
/* Shifted score (Eq. 7): s~_{i,1} = 1 and s~_{i,k} = prod_{t=1}^{k-1} c_{i,t}: the admission    */
/* score of depth k uses only the confidences before k, fp32 left to right like Eq. 3.           */
int oracle_scores_shifted(const float* conf, int B, int gamma, float* scores) {
    if (!conf || !scores || B < 0 || gamma < 0) return ORACLE_EINVAL;
    for (int i = 0; i < B; ++i) {
        float s = 1.0f;
        for (int k = 1; k <= gamma; ++k) {
            scores[(size_t)i * gamma + (k - 1)] = s;   /* before the k-th confidence is applied */
            s = s * clamp_conf(conf[(size_t)i * gamma + (k - 1)]);
            if (s == 0.0f) s = 0.0f;
        }
    }
    return ORACLE_OK;
}

/*
 * Causal early-stopping scan ("maintains one frontier position per request and repeatedly considers
 * the frontier with the largest shifted score ... if the objective improves, the position is
 * irrevocably admitted and the next position from that request is exposed, otherwise the scan
 * stops").  Written as that loop, one admission per iteration.
 * Readings: ties between frontiers by shallower depth, then request index (same paragraph); the
 * utility is B + the sum of the admitted SHIFTED scores (the only quantity the scan may consult),
 * summed exactly in units of 2^-40 like oracle_select; "improves" is a strict '>' between two fp64
 * quotients by (double)cost_fp32; the cost table is dense in the packed length T = B + N.
 * Outputs as oracle_select (depths, cu_q, packed metadata, info; candidate = n_star).
 */
int oracle_select_causal(const float* conf, int B, int gamma, const int32_t* draft_ids,
                         const int32_t* bonus_ids, const int32_t* ctx_lens, const float* cost_ms, int n_cost,
                         int32_t* depths, int32_t* cu_q, int32_t* tok_req, int32_t* tok_pos, int32_t* tok_id,
                         float* scores_out, oracle_select_info* info) {
    if (!conf || !depths || !cu_q || !info || !cost_ms || B < 0 || gamma < 0) return ORACLE_EINVAL;
    const int n = B * gamma;
    if (n_cost < B + n + 1) return ORACLE_ECOST;
    for (int t = B; t <= B + n; ++t)
        if (!(cost_ms[t] > 0.0f) || isinf(cost_ms[t])) return ORACLE_ECOST;
    const int64_t ONE = (int64_t)1 << 40;
    float* s = (float*)malloc(sizeof(float) * (size_t)(n > 0 ? n : 1));
    oracle_scores_shifted(conf, B, gamma, s);
    if (scores_out) memcpy(scores_out, s, sizeof(float) * (size_t)n);
    int* frontier = (int*)malloc(sizeof(int) * (size_t)(B > 0 ? B : 1));   /* next depth to expose, 1-based */
    for (int i = 0; i < B; ++i) frontier[i] = 1;
    int N = 0;
    int64_t Q = 0;
    double S = 0.0;
    double cur = (double)((int64_t)B * ONE) / (double)cost_ms[B];
    for (;;) {
        int bi = -1;
        for (int i = 0; i < B; ++i) {
            if (frontier[i] > gamma) continue;
            if (bi < 0) { bi = i; continue; }
            const float a = s[i * gamma + frontier[i] - 1], b = s[bi * gamma + frontier[bi] - 1];
            if (a > b || (a == b && frontier[i] < frontier[bi])) bi = i;   /* equal depth: the lower request stays */
        }
        if (bi < 0) break;
        const float sc = s[bi * gamma + frontier[bi] - 1];
        const int64_t q = (int64_t)floor((double)sc * 1099511627776.0);
        const double obj = (double)((int64_t)B * ONE + Q + q) / (double)cost_ms[B + N + 1];
        if (!(obj > cur)) break;
        cur = obj;
        Q += q;
        S += (double)sc;
        N += 1;
        frontier[bi] += 1;
    }
    info->n_star = N;
    info->t_total = B + N;
    info->candidate = N;
    info->closure_ok = 1;   /* by construction: a request's positions are admitted in depth order */
    info->sum_fixed = (int64_t)B * ONE + Q;
    info->objective = cur;
    info->sum_f64 = (double)B + S;
    cu_q[0] = 0;
    for (int i = 0; i < B; ++i) {
        depths[i] = frontier[i] - 1;
        cu_q[i + 1] = cu_q[i] + 1 + depths[i];
    }
    for (int i = 0; i < B; ++i)
        for (int t = 0; t <= depths[i]; ++t) {
            const int r = cu_q[i] + t;
            if (tok_req) tok_req[r] = i;
            if (tok_pos) tok_pos[r] = (ctx_lens ? ctx_lens[i] : 0) + t;
            if (tok_id) tok_id[r] = t == 0 ? (bonus_ids ? bonus_ids[i] : -1) : (draft_ids ? draft_ids[i * gamma + (t - 1)] : -1);
        }
    free(frontier);
    free(s);
    return ORACLE_OK;
}

/*
 * Rejection-sampling acceptance ("Standard RS then accepts with probability min(1, p(z)/q(z)) and,
 * upon rejection, samples from the residual distribution proportional to (p - q)+; if the retained
 * block is fully accepted, the bonus token is sampled directly from the next target distribution").
 * p = softmax of the target logits row (cu_q[i] + t), q = softmax of the draft logits row (i, t),
 * both at temperature 1, in double.  The random numbers are inputs: u_accept[i, t] decides draft
 * t + 1 of request i (accepted iff u * q(z) < p(z)), u_sample[i] draws the one token that ends the
 * request's step by inversion over ascending token index (the smallest v whose cumulative weight
 * exceeds u * total; all weights zero -> the same draw from p).
 * Outputs as oracle_accept; out_prob (optional) = the probabilities the decisions used:
 * [i][0] = p(z) / q(z) of the first rejected draft (or of the last accepted one), [i][1] = total
 * residual mass (0 when the block was fully accepted).
 */
static void softmax_row(const uint16_t* row, int V, double* out) {
    double m = -INFINITY;
    for (int v = 0; v < V; ++v) {
        const double x = (double)bf16_to_float(row[v]);
        if (x > m) m = x;
    }
    double z = 0.0;
    for (int v = 0; v < V; ++v) {
        out[v] = exp((double)bf16_to_float(row[v]) - m);
        z += out[v];
    }
    for (int v = 0; v < V; ++v) out[v] /= z;
}

static int inverse_cdf(const double* w, int V, double u) {
    double total = 0.0;
    for (int v = 0; v < V; ++v) total += w[v];
    if (!(total > 0.0)) return -1;
    const double target = u * total;
    double run = 0.0;
    int last = 0;
    for (int v = 0; v < V; ++v) {
        if (w[v] > 0.0) last = v;
        run += w[v];
        if (run > target) return v;
    }
    return last;   /* rounding left run == target at the end */
}

int oracle_accept_rs(const uint16_t* target_logits, const uint16_t* draft_logits, int V, const int32_t* draft_ids,
                     const int32_t* cu_q, int B, int gamma, const float* u_accept, const float* u_sample,
                     int32_t* accept_len, int32_t* bonus, int32_t* out_tokens, int32_t* n_accepted_total,
                     double* out_prob) {
    if (!target_logits || !draft_logits || !draft_ids || !cu_q || !u_accept || !u_sample || !accept_len || !bonus || V < 1)
        return ORACLE_EINVAL;
    double* p = (double*)malloc(sizeof(double) * (size_t)V);
    double* q = (double*)malloc(sizeof(double) * (size_t)V);
    int total = 0, rc = ORACLE_OK;
    for (int i = 0; i < B && rc == ORACLE_OK; ++i) {
        const int d = cu_q[i + 1] - cu_q[i] - 1;
        int m = 0, tok = -1;
        double ratio = 0.0, mass = 0.0;
        for (; m < d; ++m) {
            const int z = draft_ids[i * gamma + m];
            if (z < 0 || z >= V) { rc = ORACLE_EINVAL; break; }
            softmax_row(target_logits + (size_t)(cu_q[i] + m) * V, V, p);
            softmax_row(draft_logits + ((size_t)i * gamma + m) * V, V, q);
            ratio = p[z] / q[z];
            if ((double)u_accept[i * gamma + m] * q[z] < p[z]) continue;   /* accepted */
            for (int v = 0; v < V; ++v) {
                q[v] = p[v] > q[v] ? p[v] - q[v] : 0.0;                    /* residual (p - q)+ */
                mass += q[v];
            }
            tok = inverse_cdf(q, V, (double)u_sample[i]);
            if (tok < 0) tok = inverse_cdf(p, V, (double)u_sample[i]);
            break;
        }
        if (rc != ORACLE_OK) break;
        if (tok < 0) {   /* every retained draft accepted: the bonus comes from the next target distribution */
            softmax_row(target_logits + (size_t)(cu_q[i] + d) * V, V, p);
            tok = inverse_cdf(p, V, (double)u_sample[i]);
            m = d;
        }
        accept_len[i] = m;
        bonus[i] = tok;
        total += m + 1;
        if (out_tokens)
            for (int t = 0; t <= gamma; ++t)
                out_tokens[i * (gamma + 1) + t] = t < m ? draft_ids[i * gamma + t] : (t == m ? tok : -1);
        if (out_prob) {
            out_prob[2 * i] = ratio;
            out_prob[2 * i + 1] = mass;
        }
    }
    if (n_accepted_total) *n_accepted_total = total;
    free(p);
    free(q);
    return rc;
}
