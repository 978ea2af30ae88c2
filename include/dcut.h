/*
 * libdcut.so - the verify hot path of D-cut (adaptive verification-depth pruning for batched
 * speculative decoding) as hand-written sm_100a kernels behind a plain C ABI.
 *
 * Vocabulary.  B requests; gamma draft tokens per request (the paper's D); c_{i,k} the drafter's
 * confidence at depth k = 1..gamma; p_{i,k} = prod_{t<=k} c_{i,t} the prefix score (the paper's
 * s_{i,k}, Eq. 3); d_i the kept depth (the paper's n_i); N the number of kept draft positions over
 * the batch; T = B + N the packed verification length (the paper's budget K); L_i the number of
 * tokens request i already has in the KV cache.
 *
 * Conventions.
 *   - Every pointer argument is marked HOST or DEVICE.  Device buffers are owned by the caller
 *     (any allocator); the library never frees or keeps them beyond the call.
 *   - Calls that take a `stream` are asynchronous on that CUDA stream (a cudaStream_t passed as
 *     void*; NULL = the legacy default stream) and never synchronise it.
 *   - The context owns only its scratch memory, allocated once in dcut_create from dcut_limits;
 *     no call on the hot path allocates.  One context serves one stream at a time: calls that
 *     overlap on the GPU share the scratch and race.
 *   - A context belongs to the device it was created on.  Every call that launches work checks that
 *     this device is the current one (cudaGetDevice) and returns DCUT_EINVAL otherwise: a launch on
 *     another device would hand that device this context's scratch pointers.
 *   - Every call returns a dcut_status.  Errors the host can see (null pointer, a size over the
 *     limits, a bad cost table) are returned before anything is launched.  Nothing aborts or traps;
 *     dcut_last_error gives a message for the last failing call on that context.
 *   - bf16 tensors are passed as const void* / void* (2 bytes per element, row-major).
 *   - KV cache layout, for K and for V: [num_pages, n_kv_heads, page_size, head_dim] bf16, so the
 *     (page, kv head) tile is one contiguous block.  The cache base must be 128-byte aligned.
 *     Position j of request i lives in page block_table[i][j / page_size], slot j % page_size.
 *
 * Environment variables read once, in dcut_create (measurement knobs; the defaults are the measured best):
 *   DCUT_ATTN_TC_MIN_ROWS     query rows from which a work item goes to the tcgen05 phase (17; above 128: never)
 *   DCUT_ATTN_MIN_CHUNK_PAGES a work item that a segment boundary cuts is cut at multiples of this many pages (8)
 *   DCUT_ATTN_TAIL_ROWS       0 = a query tile above 128 rows becomes two work items instead of one with tail rows
 *   DCUT_GEMM_2CTA            0 = never run GEMM tiles on pairs of SMs (tcgen05 cta_group::2); default: where it pays
 *   DCUT_GEMM_WIDTHS          bit mask of the GEMM tile widths that may be chosen (bit i: 256 - 32 i columns; default 0x7f)
 *   DCUT_GEMM_FORCE           experiments: 0..6 = that width on one SM per tile, 8..14 = on a pair, 16..22 = a pair splitting K,
 *                             whatever the packed length (a split needs every tile to fit one wave of pairs)
 */
#ifndef DCUT_H_
#define DCUT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dcut_ctx dcut_ctx;

typedef enum {
    DCUT_OK = 0,
    DCUT_EINVAL = 1,    /* null pointer, negative size, unsupported shape                        */
    DCUT_ECAPACITY = 2, /* a size exceeds what dcut_limits reserved                               */
    DCUT_ECUDA = 3,     /* a CUDA runtime / driver call failed (message in dcut_last_error)       */
    DCUT_ECOST = 4,     /* cost table missing, too short, or holding a value <= 0, NaN or inf     */
    DCUT_EDEVICE = 5    /* a kernel reported an error through the device status word             */
} dcut_status;

typedef struct {
    int max_B;             /* requests per step                                  */
    int max_gamma;         /* draft tokens per request; max_B * max_gamma <= 8192 */
    int n_q_heads;         /* query heads (multiple of n_kv_heads, group <= 16)   */
    int n_kv_heads;
    int head_dim;          /* 64 or 128                                          */
    int page_size;         /* 16                                                 */
    int max_pages_per_req; /* columns of the block table that may be used        */
    int vocab;             /* largest vocabulary dcut_accept will see            */
    int hidden;            /* decoder-layer calls only, else 0                   */
    int intermediate;      /* decoder-layer calls only, else 0                   */
} dcut_limits;

/* Result record of dcut_select, written to DEVICE memory (16-byte aligned). */
typedef struct {
    int32_t n_star;    /* kept draft positions N*                                              */
    int32_t t_total;   /* packed length T = B + N*                                             */
    int32_t candidate; /* index of the winning candidate: N* (dense mode) or the bucket index  */
    int32_t reserved;
    int64_t sum_fixed; /* B * 2^40 + sum over the kept positions of floor(p * 2^40)            */
    double objective;  /* sum_fixed / cost of the winning candidate                            */
} dcut_select_info;

/* Context.  `device` is the CUDA device ordinal; the context's scratch lives there.
 * dcut_create allocates; dcut_destroy frees (synchronises the device). */
dcut_status dcut_create(dcut_ctx** ctx, const dcut_limits* limits, int device);
dcut_status dcut_destroy(dcut_ctx* ctx);
const char* dcut_last_error(const dcut_ctx* ctx);

/*
 * Runtime cost table (Section 3.3, Appendix C "Cost-table profiling protocol"): the latency of a
 * speculative step as a function of how many positions are verified.  HOST pointers, copied.
 *
 * Dense form: cost_ms[T] for packed lengths T = 0..n-1.  dcut_select then searches every
 * N = 0..B*gamma and needs n > B*(gamma+1).
 * Bucket form (the paper's Eq. 4-5): n_buckets budgets K[r] (strictly ascending,
 * B <= K[r] <= B*(gamma+1), total positions including the B bonus positions) and their costs;
 * valid for exactly this B and gamma.  n_buckets <= 64.
 * Any cost <= 0, NaN or inf gives DCUT_ECOST.  Setting one form replaces the other.
 * The table lives in one device buffer that the copy overwrites in place (a synchronous copy that is not
 * ordered against work on other streams): no dcut_select of this context may be running or enqueued when the
 * table is replaced.  A captured CUDA graph of a step reads whatever table is in the buffer when it is replayed.
 */
dcut_status dcut_set_cost_dense(dcut_ctx* ctx, const float* cost_ms, int n);
dcut_status dcut_set_cost_buckets(dcut_ctx* ctx, int B, int gamma, const int* K, const float* cost_ms,
                                  int n_buckets);

/* Eq. 4: K = max(B, ceil(num/den * B * (gamma+1))), in exact integer arithmetic.  Host only. */
dcut_status dcut_budget_from_ratio(int B, int gamma, int num, int den, int* K);

/*
 * Cross-request depth selection (Eq. 3-5; Algorithm 1 steps 2-12; Appendix A, contiguous prefix;
 * Appendix C, packing).
 *   p_{i,k} = p_{i,k-1} * clamp(c_{i,k}, 0, 1) in fp32, left to right, p_{i,0} = 1 (NaN counts as 0);
 *   the B*gamma draft positions are ranked by (p descending, depth ascending, request ascending);
 *   for each candidate N the objective is (B*2^40 + sum of floor(p*2^40) over the top N) / cost,
 *   one fp64 divide; the largest objective wins, the smallest N among equals;
 *   d_i = number of kept positions of request i (a contiguous prefix); cu_q = exclusive prefix sum
 *   of 1 + d_i; packed tokens are request-major, bonus first: tok_req = i, tok_pos = L_i + t,
 *   tok_id = z_{i,t}.
 * DEVICE in:  conf fp32 [B,gamma]; draft_ids i32 [B,gamma]; bonus_ids i32 [B]; ctx_lens i32 [B]
 *             (draft_ids / bonus_ids / ctx_lens may be NULL if tok_id / tok_pos are NULL).
 * DEVICE out: depths i32 [B]; cu_q i32 [B+1]; tok_req, tok_pos, tok_id i32 [B*(gamma+1)] (entries
 *             past T are set to -1; each may be NULL); info (may be NULL); scores_out fp32
 *             [B,gamma] and ranks_out i32 [B,gamma] (global rank of every draft position), or NULL.
 * Errors: DCUT_ECOST if no table is set, the dense table is shorter than B*(gamma+1)+1, or the
 * bucket table was set for another (B, gamma); DCUT_ECAPACITY if B*gamma > 8192 or over limits.
 */
dcut_status dcut_select(dcut_ctx* ctx, const float* conf, int B, int gamma, const int* draft_ids,
                        const int* bonus_ids, const int* ctx_lens, int* depths, int* cu_q, int* tok_req,
                        int* tok_pos, int* tok_id, dcut_select_info* info, float* scores_out,
                        int* ranks_out, void* stream);

/*
 * Ragged causal multi-token verification attention over the paged cache (Appendix C: each kept
 * position is scored against its accepted prefix; Section 1: B*(D+1) tokens verified per step).
 * For request i, packed token t = 0..d_i (d_i = cu_q[i+1]-cu_q[i]-1), query head h:
 *   out = softmax_j( q . k_j * scale ) v_j  over cache positions j = 0 .. L_i + t,
 * reading kv head h / (n_q_heads / n_kv_heads).  The K/V of the 1 + d_i new tokens must already
 * be in the cache at positions L_i .. L_i + d_i.  bf16 in, fp32 accumulate, bf16 out.
 * DEVICE in:  q bf16 [T, n_q_heads, head_dim]; k_cache, v_cache (layout above, num_pages pages);
 *             block_table i32 [B, block_table_stride]; ctx_lens i32 [B] (= L_i); cu_q i32 [B+1].
 * DEVICE out: out bf16 [T, n_q_heads, head_dim]; lse fp32 [T, n_q_heads] (natural log of the
 *             softmax denominator, scale applied) or NULL.
 * T is read on the device from cu_q[B]; T_cap is a host-known upper bound used to size launches
 * (T_cap <= max_B*(max_gamma+1)).  Shapes come from dcut_limits.  Split-KV partial results live
 * in the context's scratch.
 */
dcut_status dcut_verify_attn(dcut_ctx* ctx, const void* q, const void* k_cache, const void* v_cache,
                             long long num_pages, const int* block_table, int block_table_stride,
                             const int* ctx_lens, const int* cu_q, int B, int T_cap, float scale,
                             void* out, float* lse, void* stream);

/*
 * Greedy acceptance (Section 3.1-3.2: sequential acceptance, A_i = 1 + min(L_i, n_i), bonus token).
 * Row cu_q[i]+t of the packed logits predicts z_{i,t+1}.  a_{i,t} = argmax over the vocabulary
 * (lowest index among equal maxima; NaN never wins; an all-NaN row gives 0);
 * m_i = longest prefix with a_{i,t} = draft_ids[i][t], t < d_i; bonus_i = a_{i,m_i}.
 * DEVICE in:  logits bf16 [T, V]; draft_ids i32 [B,gamma]; cu_q i32 [B+1].
 * DEVICE out: accept_len i32 [B] (= m_i); bonus i32 [B]; out_tokens i32 [B,gamma+1] (m_i drafts,
 *             the bonus, then -1), may be NULL; n_accepted_total i32 [1] = sum (m_i + 1), may be NULL.
 * Per-row partial maxima live in the context's scratch.
 */
dcut_status dcut_accept(dcut_ctx* ctx, const void* logits, int V, const int* draft_ids, const int* cu_q,
                        int B, int gamma, int T_cap, int* accept_len, int* bonus, int* out_tokens,
                        int* n_accepted_total, void* stream);

/*
 * Dense projection on the tensor cores: out[T, N] = a[T, K] . w[N, K]^T  (bf16 in, fp32 accumulate, bf16 out),
 * over the ragged packed batch (T = cu_q[B] read on the device, T_cap the host-known bound).  This is the
 * building block of dcut_layer_forward, exported for tests and measurements.
 *   mode 0: plain.   mode 1: out = residual + a . w^T (residual bf16 [T, N]).
 *   mode 2: SwiGLU, out[T, N] = silu(a . w^T) * (a . w2^T) with w = gate weight, w2 = up weight, both [N, K].
 * DEVICE pointers; a must have room for T_cap rows (rows past T are read and ignored).  Requirements: K a
 * multiple of 64; N a multiple of 256 (128 in mode 2); all bases 128-byte aligned.
 */
dcut_status dcut_gemm_bf16(dcut_ctx* ctx, const void* a, const void* w, const void* w2, int mode, int N, int K,
                           const int* cu_q, int B, int T_cap, void* out, const void* residual, void* stream);

/*
 * One pre-norm decoder layer of the target model over the packed verification batch (the full-layer workload:
 * the paper's verification forward is this layer repeated; Section 1 and Appendix C):
 *   n  = RMSNorm(x) * g_attn;  [q|k|v] = n . w_qkv^T;  rotate-half RoPE (angle = position * theta^(-2e/Dh)) on q, k;
 *   the new K (after RoPE) and V are written into the paged cache at position tok_pos = L_i + t;
 *   a  = dcut_verify_attn(q, cache);  h1 = x + a . w_o^T;
 *   n2 = RMSNorm(h1) * g_mlp;  y = h1 + (silu(n2 . w_gate^T) * (n2 . w_up^T)) . w_down^T.
 * No biases, no q/k norm.  bf16 tensors, fp32 accumulation; intermediate tensors are rounded to bf16 where they
 * are materialised (n, qkv, q/k after RoPE, a, h1, n2, the SwiGLU product, y).
 * DEVICE in: x bf16 [T, hidden]; weights (w_qkv [(Hq+2Hkv)*Dh, hidden] rows = q heads, k heads, v heads;
 *   w_o [hidden, Hq*Dh]; w_gate, w_up [intermediate, hidden]; w_down [hidden, intermediate]; g_attn, g_mlp
 *   [hidden]); block_table, ctx_lens, cu_q, tok_req, tok_pos as written by dcut_select.
 * DEVICE in/out: k_cache, v_cache (the step's new tokens are appended).   DEVICE out: y bf16 [T, hidden].
 * Shapes come from dcut_limits (hidden, intermediate > 0).  Workspace lives in the context.
 */
typedef struct {
    const void* w_qkv;
    const void* w_o;
    const void* w_gate;
    const void* w_up;
    const void* w_down;
    const void* g_attn;
    const void* g_mlp;
    float rms_eps;
    float rope_theta;
} dcut_layer_weights;
dcut_status dcut_layer_forward(dcut_ctx* ctx, const dcut_layer_weights* weights, const void* x, void* y, void* k_cache,
                               void* v_cache, long long num_pages, const int* block_table, int block_table_stride,
                               const int* ctx_lens, const int* cu_q, const int* tok_req, const int* tok_pos, int B,
                               int T_cap, void* stream);

/*
 * The decoder layer cut where a tensor-parallel deployment exchanges (Appendix D runs the targets at TP 1/4/8).  A
 * rank holds its share of the heads and of the MLP width: w_qkv = the rows of its q heads, then of its k heads, then
 * of its v heads; w_o = the matching columns [hidden, n_q_heads_local * head_dim]; w_gate / w_up = its rows
 * [intermediate_local, hidden]; w_down = the matching columns [hidden, intermediate_local]; its own slice of the paged
 * cache [num_pages, n_kv_heads_local, page, head_dim]; a context created with the LOCAL head counts and intermediate
 * width and the full hidden size.  Every rank runs
 *     dcut_layer_attn_part:  o_part = Attn(RoPE(Wqkv . RMSNorm(x))) . Wo^T      (no residual)
 *     -- all-reduce (sum) of o_part over the ranks: the caller's exchange --
 *     dcut_residual_add:     h1 = x + o_sum
 *     dcut_layer_mlp_part:   d_part = (SiLU(Wg . RMSNorm(h1)) * (Wu . RMSNorm(h1))) . Wd^T   (no residual)
 *     -- all-reduce (sum) of d_part --
 *     dcut_residual_add:     y = h1 + d_sum
 * and gets dcut_layer_forward's y up to the rounding of the bf16 partial sums.  The library makes no collective of its
 * own: the exchange is the caller's (NCCL or its own kernels), so these calls run on one GPU as they stand.  Arguments
 * as dcut_layer_forward (all five weight pointers of `weights` must be set in both halves: the layer's tensor maps are
 * cached together).  dcut_residual_add: out = a + b over the rows < cu_q[B] of bf16 [T, width] tensors, width % 8 == 0.
 */
dcut_status dcut_layer_attn_part(dcut_ctx* ctx, const dcut_layer_weights* weights, const void* x, void* o_part, void* k_cache,
                                 void* v_cache, long long num_pages, const int* block_table, int block_table_stride,
                                 const int* ctx_lens, const int* cu_q, const int* tok_req, const int* tok_pos, int B,
                                 int T_cap, void* stream);
dcut_status dcut_layer_mlp_part(dcut_ctx* ctx, const dcut_layer_weights* weights, const void* h1, void* d_part, const int* cu_q,
                                int B, int T_cap, void* stream);
dcut_status dcut_residual_add(dcut_ctx* ctx, const void* a, const void* b, void* out, int width, const int* cu_q, int B,
                              int T_cap, void* stream);

/*
 * Start-up cost table C(B, rho) (Eq. 4-5; Appendix C, "Cost-table profiling protocol"; Table 3 shows two such
 * tables).  The paper's system builds it once before serving: for every batch size B it captures a graph for and
 * every ratio bucket rho it runs dummy speculative steps with the budget K_rho(B) and records the median step
 * latency; at decode time the selector reads the row of the current batch size, and a batch size between captured
 * points uses the nearest captured row.  dcut_cost_grid is that table as a HOST object: the caller runs and times the
 * steps (they go through this library's own calls; paper_2607_14647_b200/profiler.py does it with CUDA events) and
 * records the samples; the library keeps the medians, finds the nearest row and installs it as the bucket table.
 *   batch_sizes ascending, >= 1; ratios num/den ascending in (0, 1]; all HOST arrays, copied.
 *   dcut_cost_grid_budget   K_rho(B) of Eq. 4 for any live B (ceiling in exact integer arithmetic, clamp to [B, B(gamma+1)]).
 *   dcut_cost_grid_record   cell (b, r) := median of n > 0 positive finite samples (an even n: mean of the two middle
 *                           ones, computed in double); DCUT_ECOST on a bad sample.
 *   dcut_cost_grid_nearest  index of the captured batch size nearest to B; the paper does not say how a tie breaks:
 *                           here the larger captured batch wins (its graph can hold the batch and its cost is not an
 *                           underestimate).
 *   dcut_cost_grid_buckets  the bucket table a live batch of B gets: budgets K_rho(B), costs of the nearest row; ratios
 *                           that give the same budget (small B) are merged and keep the smaller cost.  K_out / cost_out
 *                           hold one entry per ratio at most.  DCUT_ECOST if the row has an unrecorded cell.
 *   dcut_set_cost_from_grid the same table handed to dcut_set_cost_buckets(ctx, B, gamma, ...).
 */
typedef struct dcut_cost_grid dcut_cost_grid;
dcut_status dcut_cost_grid_create(dcut_cost_grid** out, const int* batch_sizes, int n_batch, const int* ratio_num,
                                  const int* ratio_den, int n_ratios, int gamma);
dcut_status dcut_cost_grid_destroy(dcut_cost_grid* grid);
dcut_status dcut_cost_grid_budget(const dcut_cost_grid* grid, int B, int r, int* K);
dcut_status dcut_cost_grid_record(dcut_cost_grid* grid, int b, int r, const float* samples_ms, int n);
dcut_status dcut_cost_grid_get(const dcut_cost_grid* grid, int b, int r, float* cost_ms);
dcut_status dcut_cost_grid_nearest(const dcut_cost_grid* grid, int B, int* b);
dcut_status dcut_cost_grid_buckets(const dcut_cost_grid* grid, int B, int* K_out, float* cost_out, int* n_out);
dcut_status dcut_set_cost_from_grid(dcut_ctx* ctx, const dcut_cost_grid* grid, int B);

/*
 * Selection and the attention work list in one launch (Algorithm 1 hands the packed batch straight to the target
 * forward; Appendix C folds the packing cost into verification).  The work list of dcut_verify_attn (how the requests'
 * page lists are cut into items and in which order they run) depends on ctx_lens, cu_q, B and the context's shapes only.
 * After dcut_enable_plan_in_select(ctx, 1), every dcut_select / dcut_select_causal call that is given ctx_lens also
 * builds that list in the selector kernel's tail, for the batch it has just packed; the attention calls that follow
 * (dcut_verify_attn, dcut_layer_forward, dcut_model_verify, any number of them) and are given the SAME cu_q and
 * ctx_lens pointers and the same B use it and launch no work-list kernel of their own.  Contract: between such a
 * select and those calls the caller changes neither the contents of cu_q nor of ctx_lens, and issues them on the same
 * stream (or one ordered after it).  Any other attention call builds its own list, as before.  Results are identical
 * either way (the list is the same).  Off by default; needs a context with attention shapes.
 */
dcut_status dcut_enable_plan_in_select(dcut_ctx* ctx, int on);

/*
 * Stochastic variant, selection (Appendix B "Causality under Rejection Sampling").  Same arguments and outputs as
 * dcut_select, with two differences.  (1) The ranking score of draft depth k is the SHIFTED score of Eq. 7,
 * s~_{i,1} = 1, s~_{i,k} = prod_{t<k} c_{i,t}: it does not depend on the proposal at depth k itself (scores_out
 * returns these).  (2) With a dense cost table the budget comes from the causal early-stopping scan: positions are
 * admitted in ranked order (the order in which the per-request frontiers would be exposed; ties by shallower depth,
 * then request index) while the objective (B + sum of admitted shifted scores) / cost(B + N) strictly improves, and
 * the scan stops at the first position that does not improve it - it may miss a later optimum of a curve that is not
 * unimodal, as the appendix says.  With exactly one bucket (set through dcut_set_cost_buckets) the budget is that
 * bucket's K, fixed before the block is seen (the appendix's history-determined K); more buckets -> DCUT_ECOST.
 * info.candidate = N*.  Same fixed-point sum and fp64 objective as dcut_select.
 */
dcut_status dcut_select_causal(dcut_ctx* ctx, const float* conf, int B, int gamma, const int* draft_ids,
                               const int* bonus_ids, const int* ctx_lens, int* depths, int* cu_q, int* tok_req,
                               int* tok_pos, int* tok_id, dcut_select_info* info, float* scores_out, int* ranks_out,
                               void* stream);

/*
 * Stochastic variant, acceptance by rejection sampling (Appendix B: accept draft z with probability
 * min(1, p(z)/q(z)); upon the first rejection sample from the residual distribution proportional to (p - q)+; if the
 * retained block is fully accepted, sample the bonus token from the next target distribution).
 *   p = softmax(target_logits[cu_q[i] + t, :]), q = softmax(draft_logits[i, t, :]), temperature 1, fp32.
 *   Draft t + 1 of request i (token draft_ids[i, t]) is accepted iff u_accept[i, t] * q(z) < p(z).
 *   The token that ends the request's step is drawn with u_sample[i] by inversion over ascending token index: the
 *   smallest v whose cumulative weight exceeds u * total (weights (p - q)+ of the rejected position, or p of row
 *   cu_q[i] + d_i when every retained draft was accepted; if (p - q)+ vanishes, p).
 * The random numbers are inputs (uniform in [0, 1)); the library draws none.
 * DEVICE in: target_logits bf16 [T, V]; draft_logits bf16 [B, gamma, V] (rows (i, t) with t >= d_i are not read);
 * draft_ids int32 [B, gamma] in [0, V); cu_q; u_accept fp32 [B, gamma]; u_sample fp32 [B].
 * DEVICE out: accept_len, bonus (the sampled token), out_tokens, n_accepted_total as in dcut_accept; prob fp32
 * [B, 2] (optional, may be null): p(z)/q(z) of the deciding draft and the residual mass.
 * Requirements: context created with vocab >= V; V <= 262 144.  Sums run in a fixed order, so results are reproducible; they are
 * fp32 (double for the inversion), so a draw that falls within rounding of a boundary may differ from an fp64
 * evaluation by one token.
 */
dcut_status dcut_accept_rs(dcut_ctx* ctx, const void* target_logits, const void* draft_logits, int V,
                           const int* draft_ids, const int* cu_q, int B, int gamma, int T_cap, const float* u_accept,
                           const float* u_sample, int* accept_len, int* bonus, int* out_tokens, int* n_accepted_total,
                           float* prob, void* stream);

/*
 * End of a step / start of the next (Section 3.1: a request commits its accepted drafts plus one more token;
 * Appendix A: every request advances by at least one token per step).  For every request i, with m_i = accept_len[i]
 * and the emitted tokens out_tokens[i, 0..m_i] (as written by dcut_accept / dcut_accept_rs / dcut_lm_head_accept):
 *   ctx_lens[i] += m_i + 1   the cache now holds the old bonus token and the m_i accepted drafts; the slots of the
 *                            rejected drafts are simply written over by the next step (that is the whole roll-back);
 *   bonus_ids[i] = out_tokens[i, m_i]   the closing token of this step is z_{i,0} of the next one;
 *   stream_tokens[i, stream_len[i] ..] gets the m_i + 1 emitted tokens and stream_len[i] grows by as much (optional:
 *   pass null for both).
 * DEVICE pointers; ctx_lens and stream_len are read and written.  max_ctx = tokens a request's pages can hold: a
 * request left with less than gamma + 1 free positions, or a stream without room, sets the device status word
 * (dcut_poll_device_status: code 5) - the stream is then left as it was, the context length is still advanced.
 * The paper keeps this bookkeeping in the serving engine; it is here so that consecutive steps can run without a
 * host round trip.
 */
dcut_status dcut_commit(dcut_ctx* ctx, const int* accept_len, const int* out_tokens, int B, int gamma, int max_ctx,
                        int* ctx_lens, int* bonus_ids, int* stream_tokens, int* stream_len, int stream_cap, void* stream);

/*
 * LM head fused with acceptance (the step between the last layer and dcut_accept, Section 3.1: the target's next-token
 * prediction at every retained position): logits[T, V] = x[T, hidden] . w_lm[V, hidden]^T (bf16 in, fp32 accumulate,
 * rounded to bf16 exactly as if the logits were stored), reduced inside the GEMM's epilogue to the row's argmax
 * (largest bf16 value, lowest index among equal values, NaN never selected, a row without any selectable value gives
 * 0), followed by the prefix match of dcut_accept.  The T * V * 2 bytes of logits are never written or read.
 * The outputs equal those of dcut_gemm_bf16 (mode 0, N = V) followed by dcut_accept on the same inputs.
 * DEVICE in: x bf16 [T_cap rows readable, hidden], w_lm bf16 [V, hidden] (both 128-byte aligned), draft_ids, cu_q as
 * in dcut_accept.  DEVICE out: as dcut_accept, plus row_argmax int32 [T] (optional, may be null): the argmax of
 * every packed row.  Requirements: context created with layer shapes (hidden > 0); 1 <= V (any value: the ragged
 * last tile is masked).  Uses the context's per-row words (not concurrently with dcut_accept on the same context).
 */
dcut_status dcut_lm_head_accept(dcut_ctx* ctx, const void* x, const void* w_lm, int V, const int* draft_ids,
                                const int* cu_q, int B, int gamma, int T_cap, int* accept_len, int* bonus,
                                int* out_tokens, int* n_accepted_total, int* row_argmax, void* stream);

/*
 * The whole verification forward of a model on the retained tokens (Section 3.1: the target verifies the first d_i
 * draft tokens of every request in one packed forward; the full-layer workload repeated): token embedding,
 * n_layers decoder layers as in dcut_layer_forward (layer l appends to and reads its own paged cache k_caches[l],
 * v_caches[l]; all layers share block_table, ctx_lens and the packing metadata), the final RMSNorm with gain
 * g_final, then dcut_lm_head_accept.  Every step runs in this library's kernels; the hidden states between layers
 * live in the context.
 * The dcut_model struct and its three arrays (layers, k_caches, v_caches: n_layers entries each) are HOST memory,
 * read during the call only; every pointer inside them is a DEVICE pointer: embed bf16 [vocab, hidden], g_final bf16
 * [hidden], w_lm bf16 [vocab, hidden] (may equal embed: tied weights).  rope_theta must be the same in all layers;
 * layers[0].rms_eps is used for the final norm (1e-6 when n_layers = 0).
 * DEVICE in: tok_id i32 [T] = the packed input tokens (request i contributes its bonus token of the previous step
 * followed by its first d_i draft tokens: the layout dcut_select's packing metadata describes); draft_ids
 * i32 [B, gamma]; the other arguments as in dcut_layer_forward / dcut_lm_head_accept.  A token id outside [0, vocab)
 * is read as id 0 and sets device status 6.
 * DEVICE out: as dcut_lm_head_accept, plus hidden_out bf16 [T_cap, hidden] (optional, may be NULL; 16-byte aligned):
 * the last layer's output before the final norm (what a feature-level drafter takes from the target).
 * Alignment: weights, embedding and caches 128 bytes, gains 16 bytes.
 */
typedef struct {
    int n_layers;
    const dcut_layer_weights* layers;
    void* const* k_caches;
    void* const* v_caches;
    const void* embed;
    const void* g_final;
    const void* w_lm;
    int vocab;
} dcut_model;
dcut_status dcut_model_verify(dcut_ctx* ctx, const dcut_model* model, long long num_pages, const int* block_table,
                              int block_table_stride, const int* ctx_lens, const int* cu_q, const int* tok_req,
                              const int* tok_pos, const int* tok_id, const int* draft_ids, int B, int gamma, int T_cap,
                              int* accept_len, int* bonus, int* out_tokens, int* n_accepted_total, int* row_argmax,
                              void* hidden_out, void* stream);

/*
 * dcut_accept without any allocation.  (The paper has no counterpart: this entry point exists for
 * the way the library gets embedded, not for the method.)
 *
 * Who needs it: code that runs inside a serving process after the engine has handed nearly all of
 * the GPU's memory to its KV-cache pool, where a cudaMalloc (and therefore dcut_create) can simply
 * fail; and code on a latency-critical path that is not allowed to call the allocator at all,
 * because cudaMalloc / cudaFree may synchronise the whole device.  Such callers cannot own a
 * dcut_ctx, so this call takes none: the per-row scratch of dcut_accept (one 64-bit word per packed
 * logits row) lives in a fixed array inside the library image, DCUT_ACCEPT_STATIC_MAX_ROWS words
 * (64 KB) on every GPU that loads the library, held until the process exits.
 *
 * Same arguments, same results and same DEVICE / caller-owned buffers as dcut_accept; the device that
 * holds the buffers must be current.  cu_q[B] <= T_cap is the caller's contract, as for dcut_accept; this
 * call has no status word to report a breach through, but it never touches a row at or past T_cap (such
 * rows are left out of the prefix match, a request with no row left reports accept_len 0 and bonus 0), so
 * nothing outside the first T_cap words of the fixed array is read or written.  T_cap > DCUT_ACCEPT_STATIC_MAX_ROWS returns DCUT_ECAPACITY
 * (use dcut_accept then).  errbuf (HOST, may be NULL) receives a message when the status is not
 * DCUT_OK.  The call never calls cudaMalloc, cudaFree or any allocating routine; it issues one
 * cudaMemsetAsync and two kernels on `stream`.
 *
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress, which can
 * make the runtime load the library's device code); make that first call outside any stream
 * capture.  All calls on a device share the one array, and it keeps what the previous call left, so
 * every call clears the words it is going to use first.  Two calls that overlap on the GPU (different
 * streams, or several threads) race on the array and give wrong results: serialise them.
 */
#define DCUT_ACCEPT_STATIC_MAX_ROWS 8192
dcut_status dcut_accept_static(const void* logits, int V, const int* draft_ids, const int* cu_q, int B,
                               int gamma, int T_cap, int* accept_len, int* bonus, int* out_tokens,
                               int* n_accepted_total, void* stream, char* errbuf, size_t errbuf_len);

/*
 * One whole verify step from HOST buffers: select, packing, verification attention, acceptance
 * (Algorithm 1 followed by the target's accept step), with every host<->device copy inside the call.
 * The packed shape is resolved on the host, as the paper's own system does (Section 5, limitation
 * paragraph): after dcut_select the call reads cu_q back, then copies only the kept prefix of every
 * request's query and logits rows to the device, runs dcut_verify_attn and dcut_accept, copies the
 * results back and synchronises `stream` before returning.
 * HOST in (pinned memory recommended): conf fp32 [B,gamma]; draft_ids i32 [B,gamma]; bonus_ids i32
 *   [B]; ctx_lens i32 [B]; block_table i32 [B, block_table_stride]; q_rows bf16
 *   [B, gamma+1, n_q_heads, head_dim] and logits_rows bf16 [B, gamma+1, vocab]: the row of every block
 *   position (i, t), of which the kept ones t <= d_i are used.
 * DEVICE in: k_cache, v_cache (resident state, layout above), num_pages.
 * HOST out: depths, accept_len, bonus i32 [B]; out_tokens i32 [B, gamma+1]; n_accepted_total i32
 *   [1]; attn_out bf16 [T, n_q_heads, head_dim] or NULL; h2d_bytes / d2h_bytes (bytes copied, or NULL).
 * Uses the cost table set on the context.  The first call (and a call with a larger vocab) allocates
 * device staging buffers; later calls allocate nothing.
 * Hidden-state form: a bf16 logits row is 300 KB at V = 151 936 and the kept rows of a step are what fills the bus.
 * With hidden_rows (HOST bf16 [B, gamma+1, hidden], the last hidden state of every block position) and w_lm (DEVICE
 * bf16 [vocab, hidden], resident like the cache) set, and logits_rows NULL, the call copies the kept rows of
 * hidden_rows instead (8 KB each at hidden 4096) and ends in dcut_lm_head_accept (Section 3.1: the target's
 * prediction at every retained position, here from its LM head), so the logits exist neither on the host nor in HBM.
 * Needs a context with layer shapes (hidden > 0).
 */
typedef struct {
    int B, gamma, vocab, block_table_stride;
    long long num_pages;
    float scale;
    const float* conf;
    const int* draft_ids;
    const int* bonus_ids;
    const int* ctx_lens;
    const int* block_table;
    const void* q_rows;
    const void* logits_rows;
    const void* k_cache;
    const void* v_cache;
    int* depths;
    int* accept_len;
    int* bonus;
    int* out_tokens;
    int* n_accepted_total;
    void* attn_out;
    long long* h2d_bytes;
    long long* d2h_bytes;
    const void* hidden_rows;   /* hidden-state form (else NULL) */
    const void* w_lm;
} dcut_host_step;
dcut_status dcut_verify_step_host(dcut_ctx* ctx, const dcut_host_step* step, void* stream);

/* Reads the device status word (0 = no kernel reported an error) after synchronising `stream`,
 * and clears it.  A non-zero code also makes this call return DCUT_EDEVICE.  Codes: 1 = a bounded
 * wait in the attention kernel gave up, 2 = a block-table entry outside [0, num_pages) (page 0 was
 * read instead), 3 = the attention work list did not fit the scratch, 4 = a bounded wait in the GEMM
 * kernel gave up, 5 = dcut_commit ran out of room, 6 = dcut_model_verify met a token id outside [0, vocab),
 * 7 = an acceptance call met a cu_q that is not a packing of B requests of 1 .. gamma + 1 rows inside T_cap
 * (rows at or past T_cap were left out: nothing outside the caller's T_cap rows is read or written). */
dcut_status dcut_poll_device_status(dcut_ctx* ctx, int* code, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* DCUT_H_ */
