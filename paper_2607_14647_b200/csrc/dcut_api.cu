// C ABI of libdcut.so: context, cost tables, argument checks.  Kernels live in the other files.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "dcut_internal.h"

dcut_status dcut_fail(dcut_ctx* ctx, dcut_status st, const char* fmt, ...) {
    if (ctx) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
        va_end(ap);
    }
    return st;
}

dcut_status dcut_check_cuda(dcut_ctx* ctx, cudaError_t e, const char* what) {
    if (e == cudaSuccess) return DCUT_OK;
    return dcut_fail(ctx, DCUT_ECUDA, "%s: %s", what, cudaGetErrorString(e));
}

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) ok = false;
        if (ok && prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

// a launch with another device current would run there with this context's scratch pointers
dcut_status check_device(dcut_ctx* c) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return dcut_fail(c, DCUT_ECUDA, "cudaGetDevice failed");
    if (dev != c->device)
        return dcut_fail(c, DCUT_EINVAL, "device %d is current, but this context belongs to device %d (cudaSetDevice first)", dev, c->device);
    return DCUT_OK;
}
#define DCUT_ON_DEVICE(c)                                   \
    do {                                                    \
        const dcut_status dev_st_ = check_device(c);        \
        if (dev_st_ != DCUT_OK) return dev_st_;             \
    } while (0)

template <typename T>
dcut_status dmalloc(dcut_ctx* ctx, T** p, size_t count, const char* what) {
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(p), sizeof(T) * (count ? count : 1));
    if (e != cudaSuccess) return dcut_check_cuda(ctx, e, what);
    return dcut_check_cuda(ctx, cudaMemset(*p, 0, sizeof(T) * (count ? count : 1)), what);
}

void free_all(dcut_ctx* c) {
    cudaFree(c->d_cost);
    cudaFree(c->d_bucket_K);
    cudaFree(c->d_entries);
    cudaFree(c->d_segs);
    cudaFree(c->d_cuts);
    cudaFree(c->d_plan);
    cudaFree(c->d_part_o);
    cudaFree(c->d_part_lse);
    cudaFree(c->d_row_key);
    cudaFree(c->d_rs_scratch);
    cudaFree(c->d_status);
    cudaFree(c->ly_norm);
    cudaFree(c->ly_qkv);
    cudaFree(c->ly_q);
    cudaFree(c->ly_attn);
    cudaFree(c->ly_h1);
    cudaFree(c->ly_norm2);
    cudaFree(c->ly_act);
    cudaFree(c->ly_x[0]);
    cudaFree(c->ly_x[1]);
    cudaFree(c->ly_inv_freq);
    dcut_free_layer(c);
    cudaFree(c->hs_conf);
    cudaFree(c->hs_draft);
    cudaFree(c->hs_bonus);
    cudaFree(c->hs_ctx_lens);
    cudaFree(c->hs_block_table);
    cudaFree(c->hs_depths);
    cudaFree(c->hs_cu_q);
    cudaFree(c->hs_accept);
    cudaFree(c->hs_q);
    cudaFree(c->hs_out);
    cudaFree(c->hs_logits);
    cudaFree(c->hs_hidden);
    if (c->hs_host_cu_q) cudaFreeHost(c->hs_host_cu_q);
    if (c->hs_copy_stream) cudaStreamDestroy(c->hs_copy_stream);
    if (c->hs_ev_fork) cudaEventDestroy(c->hs_ev_fork);
    if (c->hs_ev_join) cudaEventDestroy(c->hs_ev_join);
}

}  // namespace

extern "C" {

dcut_status dcut_create(dcut_ctx** out, const dcut_limits* lim, int device) {
    if (!out || !lim) return DCUT_EINVAL;
    *out = nullptr;
    dcut_ctx* c = static_cast<dcut_ctx*>(calloc(1, sizeof(dcut_ctx)));
    if (!c) return DCUT_EINVAL;
    c->lim = *lim;
    c->device = device;
    *out = c;   // returned even on failure so the caller can read the message, then destroy
    if (lim->max_B < 1 || lim->max_gamma < 1) return dcut_fail(c, DCUT_EINVAL, "max_B and max_gamma must be >= 1");
    if ((long long)lim->max_B * lim->max_gamma > DCUT_MAX_KEYS || lim->max_B > 65535 || lim->max_gamma > 65535)
        return dcut_fail(c, DCUT_ECAPACITY, "max_B * max_gamma = %lld exceeds %d", (long long)lim->max_B * lim->max_gamma,
                         DCUT_MAX_KEYS);
    const bool has_attn = lim->n_q_heads > 0;
    if (has_attn) {
        if (lim->n_kv_heads < 1 || lim->n_q_heads % lim->n_kv_heads)
            return dcut_fail(c, DCUT_EINVAL, "n_q_heads must be a multiple of n_kv_heads");
        if (lim->head_dim != 64 && lim->head_dim != 128) return dcut_fail(c, DCUT_EINVAL, "head_dim must be 64 or 128");
        if (lim->page_size != 16) return dcut_fail(c, DCUT_EINVAL, "page_size must be 16");
        const int group = lim->n_q_heads / lim->n_kv_heads;
        if ((lim->max_gamma + 1) * group > 144)
            return dcut_fail(c, DCUT_ECAPACITY, "(max_gamma+1) * (n_q_heads/n_kv_heads) = %d exceeds 144 query rows",
                             (lim->max_gamma + 1) * group);
        if (lim->max_pages_per_req < 1) return dcut_fail(c, DCUT_EINVAL, "max_pages_per_req must be >= 1");
    }
    DeviceGuard guard(device);
    if (!guard.ok) return dcut_fail(c, DCUT_ECUDA, "cannot select CUDA device %d", device);
    cudaDeviceProp prop;
    dcut_status st = dcut_check_cuda(c, cudaGetDeviceProperties(&prop, device), "cudaGetDeviceProperties");
    if (st != DCUT_OK) return st;
    if (prop.major != 10) return dcut_fail(c, DCUT_ECUDA, "device %d is sm_%d%d; this library is built for sm_100a only", device, prop.major, prop.minor);
    c->sm_count = prop.multiProcessorCount;

    const int max_T = lim->max_B * (lim->max_gamma + 1);
    c->cost_cap = max_T + 1 > DCUT_MAX_BUCKETS ? max_T + 1 : DCUT_MAX_BUCKETS;
    if ((st = dmalloc(c, &c->d_cost, c->cost_cap, "cudaMalloc(cost)")) != DCUT_OK) return st;
    if ((st = dmalloc(c, &c->d_bucket_K, DCUT_MAX_BUCKETS, "cudaMalloc(bucket_K)")) != DCUT_OK) return st;
    if ((st = dmalloc(c, &c->d_row_key, max_T, "cudaMalloc(row_key)")) != DCUT_OK) return st;
    if ((st = dmalloc(c, &c->d_status, 4, "cudaMalloc(status)")) != DCUT_OK) return st;
    if (lim->vocab > 0) {   // rejection-sampling acceptance: per-row softmax statistics of vocabulary segments of ~8k tokens
        c->rs_n_seg = (lim->vocab + 8191) / 8192;
        if (c->rs_n_seg > 32) c->rs_n_seg = 32;
        unsigned char* p = nullptr;
        if ((st = dmalloc(c, &p, dcut_accept_rs_scratch_bytes(c, c->rs_n_seg), "cudaMalloc(rs scratch)")) != DCUT_OK) return st;
        c->d_rs_scratch = p;
        if ((st = dcut_init_accept_rs(c)) != DCUT_OK) return st;
    }
    if ((st = dcut_init_select(c)) != DCUT_OK) return st;
    if ((st = dcut_init_accept(c)) != DCUT_OK) return st;
    if (has_attn) {
        // The work of a call is cut into one segment per SM (attn_plan.cuh): a table of at most two entries per request
        // (row blocks of its query tile), the segment boundaries, and two partial-result slots per segment (an item cut
        // by the segment's first boundary, one cut by its last).
        const char* env = getenv("DCUT_ATTN_MIN_CHUNK_PAGES");
        c->attn_min_chunk_pages = env ? atoi(env) : 8;
        if (c->attn_min_chunk_pages < 4) c->attn_min_chunk_pages = 4;
        c->attn_min_chunk_pages = (c->attn_min_chunk_pages + 3) & ~3;      // the tcgen05 phase works in groups of four pages
        if (c->sm_count > 256) return dcut_fail(c, DCUT_ECAPACITY, "the attention work partition handles at most 256 SMs, this device has %d", c->sm_count);
        c->max_entries = 2 * lim->max_B;
        const size_t slots = 2 * (size_t)c->sm_count;
        if ((st = dmalloc(c, &c->d_entries, c->max_entries, "cudaMalloc(attention entries)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->d_segs, (size_t)c->sm_count + 1, "cudaMalloc(attention segments)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->d_cuts, (size_t)c->sm_count + 1, "cudaMalloc(attention cuts)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->d_plan, 16, "cudaMalloc(plan)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->d_part_o, slots * 144 * lim->head_dim, "cudaMalloc(part_o)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->d_part_lse, slots * 144, "cudaMalloc(part_lse)")) != DCUT_OK) return st;
        if ((st = dcut_init_verify_attn(c)) != DCUT_OK) return st;
    }
    if (lim->hidden > 0) {
        if (!has_attn) return dcut_fail(c, DCUT_EINVAL, "the decoder layer needs the attention shapes");
        const int q_w = lim->n_q_heads * lim->head_dim, qkv_w = (lim->n_q_heads + 2 * lim->n_kv_heads) * lim->head_dim;
        if (lim->hidden % 256 || lim->intermediate % 128 || lim->intermediate < 128 || qkv_w % 256 || q_w % 64)
            return dcut_fail(c, DCUT_EINVAL, "layer shapes: hidden %% 256, intermediate %% 128, (Hq+2Hkv)*Dh %% 256 must be 0");
        const size_t mt = (size_t)max_T;
        if ((st = dmalloc(c, &c->ly_norm, mt * lim->hidden, "cudaMalloc(layer norm)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->ly_qkv, mt * qkv_w, "cudaMalloc(layer qkv)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->ly_q, mt * q_w, "cudaMalloc(layer q)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->ly_attn, mt * q_w, "cudaMalloc(layer attn)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->ly_h1, mt * lim->hidden, "cudaMalloc(layer h1)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->ly_norm2, mt * lim->hidden, "cudaMalloc(layer norm2)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->ly_act, mt * lim->intermediate, "cudaMalloc(layer act)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->ly_x[0], mt * lim->hidden, "cudaMalloc(model x0)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->ly_x[1], mt * lim->hidden, "cudaMalloc(model x1)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->ly_inv_freq, (size_t)lim->head_dim / 2, "cudaMalloc(inv_freq)")) != DCUT_OK) return st;
    }
    if (has_attn && (st = dcut_init_layer(c)) != DCUT_OK) return st;
    return dcut_check_cuda(c, cudaDeviceSynchronize(), "cudaDeviceSynchronize(create)");
}

dcut_status dcut_destroy(dcut_ctx* c) {
    if (!c) return DCUT_OK;
    {
        DeviceGuard guard(c->device);
        if (guard.ok) {
            cudaDeviceSynchronize();
            free_all(c);
        }
    }
    free(c);
    return DCUT_OK;
}

const char* dcut_last_error(const dcut_ctx* c) { return c ? c->err : "null context"; }

static bool bad_cost(float v) { return !(v > 0.0f) || isinf(v); }

dcut_status dcut_set_cost_dense(dcut_ctx* c, const float* cost_ms, int n) {
    if (!c) return DCUT_EINVAL;
    if (!cost_ms || n < 1) return dcut_fail(c, DCUT_EINVAL, "cost table pointer is null or n < 1");
    if (n > c->cost_cap) return dcut_fail(c, DCUT_ECAPACITY, "cost table of %d entries exceeds the %d reserved", n, c->cost_cap);
    for (int i = 0; i < n; ++i)
        if (bad_cost(cost_ms[i])) return dcut_fail(c, DCUT_ECOST, "cost_ms[%d] = %g is not a positive finite latency", i, cost_ms[i]);
    DeviceGuard guard(c->device);
    dcut_status st = dcut_check_cuda(c, cudaMemcpy(c->d_cost, cost_ms, sizeof(float) * n, cudaMemcpyHostToDevice), "cudaMemcpy(cost)");
    if (st != DCUT_OK) return st;
    c->cost_n = n;
    c->n_buckets = 0;
    return DCUT_OK;
}

dcut_status dcut_set_cost_buckets(dcut_ctx* c, int B, int gamma, const int* K, const float* cost_ms, int nb) {
    if (!c) return DCUT_EINVAL;
    if (!K || !cost_ms || nb < 1 || B < 1 || gamma < 1) return dcut_fail(c, DCUT_EINVAL, "bad bucket table arguments");
    if (nb > DCUT_MAX_BUCKETS) return dcut_fail(c, DCUT_ECAPACITY, "%d buckets exceed %d", nb, DCUT_MAX_BUCKETS);
    for (int r = 0; r < nb; ++r) {
        if (K[r] < B || K[r] > B * (gamma + 1) || (r > 0 && K[r] <= K[r - 1]))
            return dcut_fail(c, DCUT_EINVAL, "bucket budget K[%d] = %d must ascend within [B, B*(gamma+1)] = [%d, %d]", r, K[r], B, B * (gamma + 1));
        if (bad_cost(cost_ms[r])) return dcut_fail(c, DCUT_ECOST, "cost_ms[%d] = %g is not a positive finite latency", r, cost_ms[r]);
    }
    DeviceGuard guard(c->device);
    dcut_status st = dcut_check_cuda(c, cudaMemcpy(c->d_cost, cost_ms, sizeof(float) * nb, cudaMemcpyHostToDevice), "cudaMemcpy(cost)");
    if (st != DCUT_OK) return st;
    st = dcut_check_cuda(c, cudaMemcpy(c->d_bucket_K, K, sizeof(int) * nb, cudaMemcpyHostToDevice), "cudaMemcpy(bucket_K)");
    if (st != DCUT_OK) return st;
    c->n_buckets = nb;
    c->bucket_B = B;
    c->bucket_gamma = gamma;
    c->cost_n = 0;
    return DCUT_OK;
}

dcut_status dcut_budget_from_ratio(int B, int gamma, int num, int den, int* K) {
    if (!K || B < 0 || gamma < 0 || num < 0 || den <= 0) return DCUT_EINVAL;
    const long long total = (long long)B * (gamma + 1);
    long long k = (total * num + den - 1) / den;
    if (k < B) k = B;
    if (k > total) k = total;
    *K = (int)k;
    return DCUT_OK;
}

static dcut_status select_common(dcut_ctx* c, const float* conf, int B, int gamma, const int* draft_ids, const int* bonus_ids,
                                 const int* ctx_lens, int* depths, int* cu_q, int* tok_req, int* tok_pos, int* tok_id,
                                 dcut_select_info* info, float* scores_out, int* ranks_out, int causal, void* stream) {
    if (!c) return DCUT_EINVAL;
    DCUT_ON_DEVICE(c);
    if (causal && c->n_buckets > 1)
        return dcut_fail(c, DCUT_ECOST, "the causal selector takes a dense cost table or exactly one bucket (a budget fixed beforehand)");
    if (!conf || !depths || !cu_q) return dcut_fail(c, DCUT_EINVAL, "conf, depths and cu_q must not be null");
    if (B < 1 || gamma < 1) return dcut_fail(c, DCUT_EINVAL, "B and gamma must be >= 1");
    if (B > c->lim.max_B || gamma > c->lim.max_gamma) return dcut_fail(c, DCUT_ECAPACITY, "B = %d, gamma = %d exceed the limits (%d, %d)", B, gamma, c->lim.max_B, c->lim.max_gamma);
    if ((long long)B * gamma > DCUT_MAX_KEYS) return dcut_fail(c, DCUT_ECAPACITY, "B * gamma exceeds %d", DCUT_MAX_KEYS);
    if (tok_pos && !ctx_lens) return dcut_fail(c, DCUT_EINVAL, "tok_pos needs ctx_lens");
    if (tok_id && (!draft_ids || !bonus_ids)) return dcut_fail(c, DCUT_EINVAL, "tok_id needs draft_ids and bonus_ids");
    if (c->n_buckets > 0) {
        if (c->bucket_B != B || c->bucket_gamma != gamma) return dcut_fail(c, DCUT_ECOST, "bucket table was set for B = %d, gamma = %d", c->bucket_B, c->bucket_gamma);
    } else if (c->cost_n == 0) {
        return dcut_fail(c, DCUT_ECOST, "no cost table set");
    } else if (c->cost_n < B * (gamma + 1) + 1) {
        return dcut_fail(c, DCUT_ECOST, "dense cost table has %d entries, need %d", c->cost_n, B * (gamma + 1) + 1);
    }
    const int with_plan = c->plan_in_select && ctx_lens && c->lim.n_q_heads > 0;
    dcut_status st = dcut_launch_select(c, conf, B, gamma, draft_ids, bonus_ids, ctx_lens, depths, cu_q, tok_req, tok_pos,
                                        tok_id, info, scores_out, ranks_out, causal, with_plan, static_cast<cudaStream_t>(stream));
    // the attention calls that get these very buffers next use the list instead of building their own
    c->plan_cu_q = (st == DCUT_OK && with_plan) ? cu_q : nullptr;
    c->plan_ctx_lens = ctx_lens;
    c->plan_B = B;
    return st;
}

dcut_status dcut_enable_plan_in_select(dcut_ctx* c, int on) {
    if (!c) return DCUT_EINVAL;
    if (on && c->lim.n_q_heads <= 0) return dcut_fail(c, DCUT_EINVAL, "context was created without attention shapes");
    c->plan_in_select = on ? 1 : 0;
    c->plan_cu_q = nullptr;
    return DCUT_OK;
}

dcut_status dcut_select(dcut_ctx* c, const float* conf, int B, int gamma, const int* draft_ids, const int* bonus_ids,
                        const int* ctx_lens, int* depths, int* cu_q, int* tok_req, int* tok_pos, int* tok_id,
                        dcut_select_info* info, float* scores_out, int* ranks_out, void* stream) {
    return select_common(c, conf, B, gamma, draft_ids, bonus_ids, ctx_lens, depths, cu_q, tok_req, tok_pos, tok_id, info,
                         scores_out, ranks_out, 0, stream);
}

dcut_status dcut_select_causal(dcut_ctx* c, const float* conf, int B, int gamma, const int* draft_ids,
                               const int* bonus_ids, const int* ctx_lens, int* depths, int* cu_q, int* tok_req,
                               int* tok_pos, int* tok_id, dcut_select_info* info, float* scores_out, int* ranks_out,
                               void* stream) {
    return select_common(c, conf, B, gamma, draft_ids, bonus_ids, ctx_lens, depths, cu_q, tok_req, tok_pos, tok_id, info,
                         scores_out, ranks_out, 1, stream);
}

dcut_status dcut_verify_attn(dcut_ctx* c, const void* q, const void* k_cache, const void* v_cache, long long num_pages,
                             const int* block_table, int block_table_stride, const int* ctx_lens, const int* cu_q, int B,
                             int T_cap, float scale, void* out, float* lse, void* stream) {
    if (!c) return DCUT_EINVAL;
    DCUT_ON_DEVICE(c);
    if (c->lim.n_q_heads <= 0) return dcut_fail(c, DCUT_EINVAL, "context was created without attention shapes");
    if (!q || !k_cache || !v_cache || !block_table || !ctx_lens || !cu_q || !out)
        return dcut_fail(c, DCUT_EINVAL, "null pointer argument");
    if (B < 1 || T_cap < B || num_pages < 1) return dcut_fail(c, DCUT_EINVAL, "need B >= 1, T_cap >= B, num_pages >= 1");
    if (B > c->lim.max_B || T_cap > c->lim.max_B * (c->lim.max_gamma + 1))
        return dcut_fail(c, DCUT_ECAPACITY, "B = %d, T_cap = %d exceed the limits", B, T_cap);
    if (block_table_stride < 1 || block_table_stride > c->lim.max_pages_per_req)
        return dcut_fail(c, DCUT_ECAPACITY, "block_table_stride = %d outside [1, %d]", block_table_stride, c->lim.max_pages_per_req);
    if ((reinterpret_cast<uintptr_t>(k_cache) & 127) || (reinterpret_cast<uintptr_t>(v_cache) & 127) ||
        (reinterpret_cast<uintptr_t>(q) & 15) || (reinterpret_cast<uintptr_t>(out) & 15))
        return dcut_fail(c, DCUT_EINVAL, "k_cache / v_cache must be 128-byte aligned, q / out 16-byte aligned");
    if ((num_pages * c->lim.n_kv_heads * c->lim.page_size) >= (1ll << 31))
        return dcut_fail(c, DCUT_ECAPACITY, "cache has too many token rows for 32-bit tile coordinates");
    if (!(scale > 0.0f) || isinf(scale)) return dcut_fail(c, DCUT_EINVAL, "scale must be positive and finite");
    return dcut_launch_verify_attn(c, q, k_cache, v_cache, num_pages, block_table, block_table_stride, ctx_lens, cu_q, B,
                                   T_cap, scale, out, lse, 0, static_cast<cudaStream_t>(stream));
}

dcut_status dcut_accept(dcut_ctx* c, const void* logits, int V, const int* draft_ids, const int* cu_q, int B, int gamma,
                        int T_cap, int* accept_len, int* bonus, int* out_tokens, int* n_accepted_total, void* stream) {
    if (!c) return DCUT_EINVAL;
    DCUT_ON_DEVICE(c);
    if (!logits || !draft_ids || !cu_q || !accept_len || !bonus) return dcut_fail(c, DCUT_EINVAL, "null pointer argument");
    if (B < 1 || gamma < 1 || V < 1 || T_cap < B) return dcut_fail(c, DCUT_EINVAL, "need B, gamma, V >= 1 and T_cap >= B");
    if (B > c->lim.max_B || gamma > c->lim.max_gamma || T_cap > c->lim.max_B * (c->lim.max_gamma + 1))
        return dcut_fail(c, DCUT_ECAPACITY, "B = %d, gamma = %d, T_cap = %d exceed the limits", B, gamma, T_cap);
    if (c->lim.vocab > 0 && V > c->lim.vocab) return dcut_fail(c, DCUT_ECAPACITY, "V = %d exceeds the limit %d", V, c->lim.vocab);
    if (reinterpret_cast<uintptr_t>(logits) & 1) return dcut_fail(c, DCUT_EINVAL, "logits must be 2-byte aligned");
    return dcut_launch_accept(c, logits, V, draft_ids, cu_q, B, gamma, T_cap, accept_len, bonus, out_tokens,
                              n_accepted_total, c->d_row_key, static_cast<cudaStream_t>(stream));
}

dcut_status dcut_accept_rs(dcut_ctx* c, const void* target_logits, const void* draft_logits, int V, const int* draft_ids,
                           const int* cu_q, int B, int gamma, int T_cap, const float* u_accept, const float* u_sample,
                           int* accept_len, int* bonus, int* out_tokens, int* n_accepted_total, float* prob, void* stream) {
    if (!c) return DCUT_EINVAL;
    DCUT_ON_DEVICE(c);
    if (!c->d_rs_scratch) return dcut_fail(c, DCUT_EINVAL, "context was created with vocab = 0");
    if (!target_logits || !draft_logits || !draft_ids || !cu_q || !u_accept || !u_sample || !accept_len || !bonus)
        return dcut_fail(c, DCUT_EINVAL, "null pointer argument");
    if (B < 1 || gamma < 1 || V < 1 || T_cap < B) return dcut_fail(c, DCUT_EINVAL, "need B, gamma, V >= 1 and T_cap >= B");
    if (B > c->lim.max_B || gamma > c->lim.max_gamma || T_cap > c->lim.max_B * (c->lim.max_gamma + 1))
        return dcut_fail(c, DCUT_ECAPACITY, "B = %d, gamma = %d, T_cap = %d exceed the limits", B, gamma, T_cap);
    if (V > c->lim.vocab || V > 262144) return dcut_fail(c, DCUT_ECAPACITY, "V = %d exceeds the limit %d", V, c->lim.vocab < 262144 ? c->lim.vocab : 262144);
    return dcut_launch_accept_rs(c, target_logits, draft_logits, V, draft_ids, cu_q, B, gamma, T_cap, u_accept, u_sample,
                                 accept_len, bonus, out_tokens, n_accepted_total, prob, static_cast<cudaStream_t>(stream));
}

static dcut_status dcut_prepare_rope(dcut_ctx* c, float rope_theta, cudaStream_t stream);

dcut_status dcut_model_verify(dcut_ctx* c, const dcut_model* m, long long num_pages, const int* block_table,
                              int block_table_stride, const int* ctx_lens, const int* cu_q, const int* tok_req,
                              const int* tok_pos, const int* tok_id, const int* draft_ids, int B, int gamma, int T_cap,
                              int* accept_len, int* bonus, int* out_tokens, int* n_accepted_total, int* row_argmax,
                              void* hidden_out, void* stream) {
    if (!c) return DCUT_EINVAL;
    DCUT_ON_DEVICE(c);
    if (c->lim.hidden <= 0 || !c->ly_x[0]) return dcut_fail(c, DCUT_EINVAL, "context was created without layer shapes");
    if (!m || !m->embed || !m->g_final || !m->w_lm || m->n_layers < 0 || (m->n_layers > 0 && (!m->layers || !m->k_caches || !m->v_caches)))
        return dcut_fail(c, DCUT_EINVAL, "incomplete model description");
    if (!block_table || !ctx_lens || !cu_q || !tok_req || !tok_pos || !tok_id || !draft_ids || !accept_len || !bonus)
        return dcut_fail(c, DCUT_EINVAL, "null pointer argument");
    if (m->vocab < 1) return dcut_fail(c, DCUT_EINVAL, "vocab must be >= 1");
    if (B < 1 || B > c->lim.max_B || gamma < 1 || gamma > c->lim.max_gamma || T_cap < B ||
        T_cap > c->lim.max_B * (c->lim.max_gamma + 1))
        return dcut_fail(c, DCUT_ECAPACITY, "B = %d, gamma = %d, T_cap = %d outside the limits", B, gamma, T_cap);
    if (block_table_stride < 1 || block_table_stride > c->lim.max_pages_per_req)
        return dcut_fail(c, DCUT_ECAPACITY, "block_table_stride = %d outside [1, %d]", block_table_stride, c->lim.max_pages_per_req);
    uintptr_t al = reinterpret_cast<uintptr_t>(m->w_lm) | reinterpret_cast<uintptr_t>(m->embed);
    for (int l = 0; l < m->n_layers; ++l) {
        const dcut_layer_weights& w = m->layers[l];
        if (!w.w_qkv || !w.w_o || !w.w_gate || !w.w_up || !w.w_down || !w.g_attn || !w.g_mlp || !m->k_caches[l] || !m->v_caches[l])
            return dcut_fail(c, DCUT_EINVAL, "layer %d: null pointer", l);
        if (!(w.rope_theta > 1.0f) || !(w.rms_eps >= 0.0f) || w.rope_theta != m->layers[0].rope_theta)
            return dcut_fail(c, DCUT_EINVAL, "layer %d: rope_theta must exceed 1 and be the same in every layer, rms_eps >= 0", l);
        if ((reinterpret_cast<uintptr_t>(w.g_attn) | reinterpret_cast<uintptr_t>(w.g_mlp)) & 15)
            return dcut_fail(c, DCUT_EINVAL, "layer %d: gains must be 16-byte aligned", l);
        al |= reinterpret_cast<uintptr_t>(w.w_qkv) | reinterpret_cast<uintptr_t>(w.w_o) | reinterpret_cast<uintptr_t>(w.w_gate) |
              reinterpret_cast<uintptr_t>(w.w_up) | reinterpret_cast<uintptr_t>(w.w_down) |
              reinterpret_cast<uintptr_t>(m->k_caches[l]) | reinterpret_cast<uintptr_t>(m->v_caches[l]);
    }
    if (al & 127) return dcut_fail(c, DCUT_EINVAL, "weights, embedding and caches must be 128-byte aligned");
    if ((reinterpret_cast<uintptr_t>(m->g_final) | reinterpret_cast<uintptr_t>(hidden_out)) & 15)
        return dcut_fail(c, DCUT_EINVAL, "g_final and hidden_out must be 16-byte aligned");
    if (c->lim.vocab > 0 && m->vocab > c->lim.vocab) return dcut_fail(c, DCUT_ECAPACITY, "vocab = %d exceeds the limit %d", m->vocab, c->lim.vocab);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (m->n_layers > 0) {
        dcut_status st = dcut_prepare_rope(c, m->layers[0].rope_theta, s);
        if (st != DCUT_OK) return st;
    }
    return dcut_launch_model(c, m, num_pages, block_table, block_table_stride, ctx_lens, cu_q, tok_req, tok_pos, tok_id, draft_ids,
                             B, gamma, T_cap, accept_len, bonus, out_tokens, n_accepted_total, row_argmax, hidden_out, s);
}

dcut_status dcut_commit(dcut_ctx* c, const int* accept_len, const int* out_tokens, int B, int gamma, int max_ctx,
                        int* ctx_lens, int* bonus_ids, int* stream_tokens, int* stream_len, int stream_cap, void* stream) {
    if (!c) return DCUT_EINVAL;
    DCUT_ON_DEVICE(c);
    if (!accept_len || !out_tokens || !ctx_lens || !bonus_ids) return dcut_fail(c, DCUT_EINVAL, "null pointer argument");
    if ((stream_tokens != nullptr) != (stream_len != nullptr) || (stream_tokens && stream_cap < 1))
        return dcut_fail(c, DCUT_EINVAL, "stream_tokens, stream_len and stream_cap go together");
    if (B < 1 || gamma < 1 || max_ctx < gamma + 1) return dcut_fail(c, DCUT_EINVAL, "need B, gamma >= 1 and max_ctx > gamma");
    if (B > c->lim.max_B || gamma > c->lim.max_gamma) return dcut_fail(c, DCUT_ECAPACITY, "B = %d, gamma = %d exceed the limits", B, gamma);
    return dcut_launch_commit(c, accept_len, out_tokens, B, gamma, max_ctx, ctx_lens, bonus_ids, stream_tokens, stream_len,
                              stream_cap, static_cast<cudaStream_t>(stream));
}

dcut_status dcut_gemm_bf16(dcut_ctx* c, const void* a, const void* w, const void* w2, int mode, int N, int K,
                           const int* cu_q, int B, int T_cap, void* out, const void* residual, void* stream) {
    if (!c) return DCUT_EINVAL;
    DCUT_ON_DEVICE(c);
    if (!c->layer_maps) return dcut_fail(c, DCUT_EINVAL, "context was created without attention shapes (no tensor-map encoder)");
    if (!a || !w || !cu_q || !out || (mode == 2 && !w2) || (mode == 1 && !residual) || mode < 0 || mode > 2)
        return dcut_fail(c, DCUT_EINVAL, "null pointer or bad mode");
    if (B < 1 || T_cap < 1 || K < 64 || K % 64 || N < 1 || N % (mode == 2 ? 128 : 256))
        return dcut_fail(c, DCUT_EINVAL, "need K %% 64 == 0 and N %% 256 == 0 (128 in SwiGLU mode)");
    if ((reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(w) | reinterpret_cast<uintptr_t>(out) |
         reinterpret_cast<uintptr_t>(w2) | reinterpret_cast<uintptr_t>(residual)) & 127)
        return dcut_fail(c, DCUT_EINVAL, "operands must be 128-byte aligned");
    return dcut_launch_gemm(c, a, w, w2, mode, N, K, cu_q, B, T_cap, out, residual, static_cast<cudaStream_t>(stream));
}

dcut_status dcut_lm_head_accept(dcut_ctx* c, const void* x, const void* w_lm, int V, const int* draft_ids,
                                const int* cu_q, int B, int gamma, int T_cap, int* accept_len, int* bonus,
                                int* out_tokens, int* n_accepted_total, int* row_argmax, void* stream) {
    if (!c) return DCUT_EINVAL;
    DCUT_ON_DEVICE(c);
    if (c->lim.hidden <= 0 || !c->layer_maps) return dcut_fail(c, DCUT_EINVAL, "context was created without layer shapes");
    if (!x || !w_lm || !draft_ids || !cu_q || !accept_len || !bonus) return dcut_fail(c, DCUT_EINVAL, "null pointer argument");
    if (V < 1 || c->lim.hidden % 64) return dcut_fail(c, DCUT_EINVAL, "need V >= 1 and hidden %% 64 == 0");
    if (B < 1 || B > c->lim.max_B || gamma < 1 || gamma > c->lim.max_gamma || T_cap < B ||
        T_cap > c->lim.max_B * (c->lim.max_gamma + 1))
        return dcut_fail(c, DCUT_ECAPACITY, "B = %d, gamma = %d, T_cap = %d outside the limits", B, gamma, T_cap);
    if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(w_lm)) & 127)
        return dcut_fail(c, DCUT_EINVAL, "x and w_lm must be 128-byte aligned");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    dcut_status st = dcut_launch_lm_head_argmax(c, x, w_lm, V, c->lim.hidden, cu_q, B, T_cap, c->d_row_key, s);
    if (st != DCUT_OK) return st;
    return dcut_launch_accept_match(c, nullptr, V, draft_ids, cu_q, B, gamma, T_cap, accept_len, bonus, out_tokens,
                                    n_accepted_total, row_argmax, c->d_row_key, s);
}

// first call (or a new theta): build the RoPE inverse-frequency table in fp64, round once to fp32.  The host copy of
// the table lives in the context: if this first call is being captured into a CUDA graph, the copy node reads it again
// at every replay, and the context outlives the graph's use of it.
static dcut_status dcut_prepare_rope(dcut_ctx* c, float rope_theta, cudaStream_t stream) {
    if (c->ly_theta == rope_theta) return DCUT_OK;
    const int half = c->lim.head_dim / 2;
    for (int e = 0; e < half; ++e) c->ly_inv_freq_host[e] = (float)pow((double)rope_theta, -2.0 * e / c->lim.head_dim);
    dcut_status st = dcut_check_cuda(c, cudaMemcpyAsync(c->ly_inv_freq, c->ly_inv_freq_host, sizeof(float) * half,
                                                        cudaMemcpyHostToDevice, stream), "cudaMemcpyAsync(inv_freq)");
    if (st != DCUT_OK) return st;
    c->ly_theta = rope_theta;
    return DCUT_OK;
}

static dcut_status layer_common(dcut_ctx* c, const dcut_layer_weights* w, const void* x, void* y, void* k_cache,
                                void* v_cache, long long num_pages, const int* block_table, int block_table_stride,
                                const int* ctx_lens, const int* cu_q, const int* tok_req, const int* tok_pos, int B,
                                int T_cap, int part, void* stream) {
    if (!c) return DCUT_EINVAL;
    DCUT_ON_DEVICE(c);
    if (c->lim.hidden <= 0 || !c->ly_norm) return dcut_fail(c, DCUT_EINVAL, "context was created without layer shapes");
    const bool attn = part != 2, mlp = part != 1;
    if (!w || !x || !y || !cu_q) return dcut_fail(c, DCUT_EINVAL, "null pointer argument");
    if (attn && (!w->w_qkv || !w->w_o || !w->g_attn || !k_cache || !v_cache || !block_table || !ctx_lens || !tok_req || !tok_pos))
        return dcut_fail(c, DCUT_EINVAL, "null pointer argument");
    if (mlp && (!w->w_gate || !w->w_up || !w->w_down || !w->g_mlp)) return dcut_fail(c, DCUT_EINVAL, "null pointer argument");
    // the tensor-map cache of a layer is keyed by w_qkv and holds all five projections: every weight pointer must be given
    if (!w->w_qkv || !w->w_o || !w->w_gate || !w->w_up || !w->w_down)
        return dcut_fail(c, DCUT_EINVAL, "all five weight pointers of the layer must be set (also for one half of it)");
    if (B < 1 || T_cap < B || B > c->lim.max_B || T_cap > c->lim.max_B * (c->lim.max_gamma + 1))
        return dcut_fail(c, DCUT_ECAPACITY, "B = %d, T_cap = %d outside the limits", B, T_cap);
    if (attn && (block_table_stride < 1 || block_table_stride > c->lim.max_pages_per_req))
        return dcut_fail(c, DCUT_ECAPACITY, "block_table_stride = %d outside [1, %d]", block_table_stride, c->lim.max_pages_per_req);
    if (!(w->rope_theta > 1.0f) || !(w->rms_eps >= 0.0f)) return dcut_fail(c, DCUT_EINVAL, "rope_theta must exceed 1, rms_eps >= 0");
    const uintptr_t al = reinterpret_cast<uintptr_t>(w->w_qkv) | reinterpret_cast<uintptr_t>(w->w_o) |
                         reinterpret_cast<uintptr_t>(w->w_gate) | reinterpret_cast<uintptr_t>(w->w_up) |
                         reinterpret_cast<uintptr_t>(w->w_down) | reinterpret_cast<uintptr_t>(k_cache) |
                         reinterpret_cast<uintptr_t>(v_cache);
    if ((al & 127) || ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y) |
                        reinterpret_cast<uintptr_t>(w->g_attn) | reinterpret_cast<uintptr_t>(w->g_mlp)) & 15))
        return dcut_fail(c, DCUT_EINVAL, "weights and caches must be 128-byte aligned, x / y / gains 16-byte aligned");
    if (attn) {
        dcut_status st = dcut_prepare_rope(c, w->rope_theta, static_cast<cudaStream_t>(stream));
        if (st != DCUT_OK) return st;
    }
    return dcut_launch_layer(c, w, x, y, k_cache, v_cache, num_pages, block_table, block_table_stride, ctx_lens, cu_q,
                             tok_req, tok_pos, B, T_cap, 0, part, static_cast<cudaStream_t>(stream));
}

dcut_status dcut_layer_forward(dcut_ctx* c, const dcut_layer_weights* w, const void* x, void* y, void* k_cache,
                               void* v_cache, long long num_pages, const int* block_table, int block_table_stride,
                               const int* ctx_lens, const int* cu_q, const int* tok_req, const int* tok_pos, int B,
                               int T_cap, void* stream) {
    return layer_common(c, w, x, y, k_cache, v_cache, num_pages, block_table, block_table_stride, ctx_lens, cu_q, tok_req,
                        tok_pos, B, T_cap, 0, stream);
}

dcut_status dcut_layer_attn_part(dcut_ctx* c, const dcut_layer_weights* w, const void* x, void* o_part, void* k_cache,
                                 void* v_cache, long long num_pages, const int* block_table, int block_table_stride,
                                 const int* ctx_lens, const int* cu_q, const int* tok_req, const int* tok_pos, int B,
                                 int T_cap, void* stream) {
    return layer_common(c, w, x, o_part, k_cache, v_cache, num_pages, block_table, block_table_stride, ctx_lens, cu_q, tok_req,
                        tok_pos, B, T_cap, 1, stream);
}

dcut_status dcut_layer_mlp_part(dcut_ctx* c, const dcut_layer_weights* w, const void* h1, void* d_part, const int* cu_q, int B,
                                int T_cap, void* stream) {
    return layer_common(c, w, h1, d_part, nullptr, nullptr, 0, nullptr, 0, nullptr, cu_q, nullptr, nullptr, B, T_cap, 2, stream);
}

dcut_status dcut_residual_add(dcut_ctx* c, const void* a, const void* b, void* out, int width, const int* cu_q, int B,
                              int T_cap, void* stream) {
    if (!c) return DCUT_EINVAL;
    DCUT_ON_DEVICE(c);
    if (!a || !b || !out || !cu_q) return dcut_fail(c, DCUT_EINVAL, "null pointer argument");
    if (B < 1 || T_cap < B || width < 8 || width % 8) return dcut_fail(c, DCUT_EINVAL, "need B >= 1, T_cap >= B, width a positive multiple of 8");
    if ((reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b) | reinterpret_cast<uintptr_t>(out)) & 15)
        return dcut_fail(c, DCUT_EINVAL, "operands must be 16-byte aligned");
    return dcut_launch_residual_add(c, a, b, out, width, cu_q, B, T_cap, static_cast<cudaStream_t>(stream));
}

dcut_status dcut_poll_device_status(dcut_ctx* c, int* code, void* stream) {
    if (!c) return DCUT_EINVAL;
    DeviceGuard guard(c->device);
    int v = 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    dcut_status st = dcut_check_cuda(c, cudaMemcpyAsync(&v, c->d_status, sizeof(int), cudaMemcpyDeviceToHost, s), "cudaMemcpyAsync(status)");
    if (st != DCUT_OK) return st;
    st = dcut_check_cuda(c, cudaStreamSynchronize(s), "cudaStreamSynchronize(status)");
    if (st != DCUT_OK) return st;
    if (v != 0) {
        st = dcut_check_cuda(c, cudaMemsetAsync(c->d_status, 0, sizeof(int), s), "cudaMemsetAsync(status)");
        if (st != DCUT_OK) return st;
        cudaStreamSynchronize(s);
    }
    if (code) *code = v;
    if (v != 0) return dcut_fail(c, DCUT_EDEVICE, "a kernel reported device status %d", v);
    return DCUT_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Whole step from host buffers.

namespace {

dcut_status ensure_host_step_buffers(dcut_ctx* c, int V, bool hidden_form) {
    if (hidden_form && c->hs_ready) {
        if (c->hs_hidden) return DCUT_OK;
        return dmalloc(c, &c->hs_hidden, (size_t)c->lim.max_B * (c->lim.max_gamma + 1) * c->lim.hidden, "cudaMalloc(step hidden)");
    }
    if (c->hs_ready && (hidden_form || c->hs_vocab >= V)) return DCUT_OK;
    const dcut_limits& l = c->lim;
    const size_t max_T = (size_t)l.max_B * (l.max_gamma + 1);
    const size_t keys = (size_t)l.max_B * l.max_gamma;
    dcut_status st;
    if (!c->hs_ready) {
        if ((st = dmalloc(c, &c->hs_conf, keys, "cudaMalloc(step conf)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->hs_draft, keys, "cudaMalloc(step draft)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->hs_bonus, l.max_B, "cudaMalloc(step bonus)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->hs_ctx_lens, l.max_B, "cudaMalloc(step ctx_lens)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->hs_block_table, (size_t)l.max_B * l.max_pages_per_req, "cudaMalloc(step block table)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->hs_depths, l.max_B, "cudaMalloc(step depths)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->hs_cu_q, (size_t)l.max_B + 1, "cudaMalloc(step cu_q)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->hs_accept, (size_t)l.max_B * (l.max_gamma + 3) + 4, "cudaMalloc(step accept)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->hs_q, max_T * l.n_q_heads * l.head_dim, "cudaMalloc(step q)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->hs_out, max_T * l.n_q_heads * l.head_dim, "cudaMalloc(step out)")) != DCUT_OK) return st;
        cudaError_t e = cudaMallocHost(reinterpret_cast<void**>(&c->hs_host_cu_q), sizeof(int) * ((size_t)l.max_B + 1));
        if (e != cudaSuccess) return dcut_check_cuda(c, e, "cudaMallocHost(step cu_q)");
        if ((e = cudaStreamCreateWithFlags(&c->hs_copy_stream, cudaStreamNonBlocking)) != cudaSuccess) return dcut_check_cuda(c, e, "cudaStreamCreate(step copy)");
        if ((e = cudaEventCreateWithFlags(&c->hs_ev_fork, cudaEventDisableTiming)) != cudaSuccess) return dcut_check_cuda(c, e, "cudaEventCreate(step)");
        if ((e = cudaEventCreateWithFlags(&c->hs_ev_join, cudaEventDisableTiming)) != cudaSuccess) return dcut_check_cuda(c, e, "cudaEventCreate(step)");
    }
    if (hidden_form) {
        if (!c->hs_hidden && (st = dmalloc(c, &c->hs_hidden, max_T * (size_t)l.hidden, "cudaMalloc(step hidden)")) != DCUT_OK) return st;
    } else {
        if (c->hs_logits) cudaFree(c->hs_logits);
        c->hs_logits = nullptr;
        if ((st = dmalloc(c, &c->hs_logits, max_T * (size_t)V, "cudaMalloc(step logits)")) != DCUT_OK) return st;
        c->hs_vocab = V;
    }
    c->hs_ready = 1;
    return DCUT_OK;
}

}  // namespace

extern "C" dcut_status dcut_verify_step_host(dcut_ctx* c, const dcut_host_step* s, void* stream) {
    if (!c) return DCUT_EINVAL;
    DCUT_ON_DEVICE(c);
    if (!s || !s->conf || !s->draft_ids || !s->bonus_ids || !s->ctx_lens || !s->block_table || !s->q_rows ||
        !s->k_cache || !s->v_cache || !s->depths || !s->accept_len || !s->bonus || !s->out_tokens || !s->n_accepted_total)
        return dcut_fail(c, DCUT_EINVAL, "null pointer in dcut_host_step");
    const bool hidden_form = s->hidden_rows != nullptr;
    if (hidden_form ? (s->logits_rows != nullptr || !s->w_lm) : !s->logits_rows)
        return dcut_fail(c, DCUT_EINVAL, "dcut_host_step needs either logits_rows, or hidden_rows with w_lm");
    if (hidden_form && (c->lim.hidden <= 0 || !c->layer_maps))
        return dcut_fail(c, DCUT_EINVAL, "the hidden-state form needs a context created with layer shapes");
    const int B = s->B, g = s->gamma, V = s->vocab;
    const dcut_limits& l = c->lim;
    if (B < 1 || g < 1 || V < 1) return dcut_fail(c, DCUT_EINVAL, "need B, gamma, vocab >= 1");
    if (B > l.max_B || g > l.max_gamma || s->block_table_stride > l.max_pages_per_req || s->block_table_stride < 1)
        return dcut_fail(c, DCUT_ECAPACITY, "B, gamma or block_table_stride exceed the limits");
    if (l.n_q_heads <= 0) return dcut_fail(c, DCUT_EINVAL, "context was created without attention shapes");
    dcut_status st = ensure_host_step_buffers(c, V, hidden_form);
    if (st != DCUT_OK) return st;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    // per block position the second stream carries a logits row, or (hidden-state form) a last-hidden-state row
    const size_t q_row = (size_t)l.n_q_heads * l.head_dim * 2, lg_row = hidden_form ? (size_t)l.hidden * 2 : (size_t)V * 2;
    const char* lg_src = static_cast<const char*>(hidden_form ? s->hidden_rows : s->logits_rows);
    char* lg_dst = reinterpret_cast<char*>(hidden_form ? c->hs_hidden : c->hs_logits);
#define DCUT_CP(dst, src, bytes, kind)                                                                   \
    if ((st = dcut_check_cuda(c, cudaMemcpyAsync(dst, src, bytes, kind, cs), "cudaMemcpyAsync(step)")) != DCUT_OK) return st
    DCUT_CP(c->hs_conf, s->conf, sizeof(float) * B * g, cudaMemcpyHostToDevice);
    DCUT_CP(c->hs_draft, s->draft_ids, sizeof(int) * B * g, cudaMemcpyHostToDevice);
    DCUT_CP(c->hs_bonus, s->bonus_ids, sizeof(int) * B, cudaMemcpyHostToDevice);
    DCUT_CP(c->hs_ctx_lens, s->ctx_lens, sizeof(int) * B, cudaMemcpyHostToDevice);
    DCUT_CP(c->hs_block_table, s->block_table, sizeof(int) * (size_t)B * s->block_table_stride, cudaMemcpyHostToDevice);
    st = dcut_select(c, c->hs_conf, B, g, nullptr, nullptr, nullptr, c->hs_depths, c->hs_cu_q, nullptr, nullptr, nullptr,
                     nullptr, nullptr, nullptr, stream);
    if (st != DCUT_OK) return st;
    // the packed shape is resolved on the host: read cu_q back, then copy only the kept prefixes
    DCUT_CP(c->hs_host_cu_q, c->hs_cu_q, sizeof(int) * (B + 1), cudaMemcpyDeviceToHost);
    if ((st = dcut_check_cuda(c, cudaStreamSynchronize(cs), "cudaStreamSynchronize(step)")) != DCUT_OK) return st;
    const int* cu = c->hs_host_cu_q;
    long long h2d = (long long)(sizeof(float) + sizeof(int)) * B * g + 2ll * sizeof(int) * B +
                    (long long)sizeof(int) * B * s->block_table_stride;
    // The logits (the bulk of the bytes) travel on a second stream while the query rows are copied and attention
    // runs on the caller's; acceptance waits for both.  (The previous call ended with a synchronisation, so nothing
    // still reads the buffers that are being overwritten.)
    if ((st = dcut_check_cuda(c, cudaEventRecord(c->hs_ev_fork, cs), "cudaEventRecord(step fork)")) != DCUT_OK) return st;
    if ((st = dcut_check_cuda(c, cudaStreamWaitEvent(c->hs_copy_stream, c->hs_ev_fork, 0), "cudaStreamWaitEvent(step fork)")) != DCUT_OK) return st;
    for (int i = 0; i < B; ++i) {
        const size_t rows = (size_t)(cu[i + 1] - cu[i]);
        DCUT_CP(reinterpret_cast<char*>(c->hs_q) + (size_t)cu[i] * q_row,
                static_cast<const char*>(s->q_rows) + (size_t)i * (g + 1) * q_row, rows * q_row, cudaMemcpyHostToDevice);
        h2d += (long long)(rows * (q_row + lg_row));
    }
    for (int i = 0; i < B; ++i) {
        const size_t rows = (size_t)(cu[i + 1] - cu[i]);
        if ((st = dcut_check_cuda(c, cudaMemcpyAsync(lg_dst + (size_t)cu[i] * lg_row, lg_src + (size_t)i * (g + 1) * lg_row,
                                                     rows * lg_row, cudaMemcpyHostToDevice, c->hs_copy_stream),
                                  "cudaMemcpyAsync(step logits)")) != DCUT_OK) return st;
    }
    if ((st = dcut_check_cuda(c, cudaEventRecord(c->hs_ev_join, c->hs_copy_stream), "cudaEventRecord(step join)")) != DCUT_OK) return st;
    const int T_cap = B * (g + 1);
    st = dcut_verify_attn(c, c->hs_q, s->k_cache, s->v_cache, s->num_pages, c->hs_block_table, s->block_table_stride,
                          c->hs_ctx_lens, c->hs_cu_q, B, T_cap, s->scale, c->hs_out, nullptr, stream);
    if (st != DCUT_OK) return st;
    if ((st = dcut_check_cuda(c, cudaStreamWaitEvent(cs, c->hs_ev_join, 0), "cudaStreamWaitEvent(step join)")) != DCUT_OK) return st;
    int* acc = c->hs_accept;            // [B] accept_len, [B] bonus, [B*(g+1)] tokens, [1] total
    if (hidden_form)
        st = dcut_lm_head_accept(c, c->hs_hidden, s->w_lm, V, c->hs_draft, c->hs_cu_q, B, g, T_cap, acc, acc + B, acc + 2 * B,
                                 acc + 2 * B + B * (g + 1), nullptr, stream);
    else
        st = dcut_accept(c, c->hs_logits, V, c->hs_draft, c->hs_cu_q, B, g, T_cap, acc, acc + B, acc + 2 * B,
                         acc + 2 * B + B * (g + 1), stream);
    if (st != DCUT_OK) return st;
    DCUT_CP(s->depths, c->hs_depths, sizeof(int) * B, cudaMemcpyDeviceToHost);
    DCUT_CP(s->accept_len, acc, sizeof(int) * B, cudaMemcpyDeviceToHost);
    DCUT_CP(s->bonus, acc + B, sizeof(int) * B, cudaMemcpyDeviceToHost);
    DCUT_CP(s->out_tokens, acc + 2 * B, sizeof(int) * B * (g + 1), cudaMemcpyDeviceToHost);
    DCUT_CP(s->n_accepted_total, acc + 2 * B + B * (g + 1), sizeof(int), cudaMemcpyDeviceToHost);
    if (s->attn_out) DCUT_CP(s->attn_out, c->hs_out, (size_t)cu[B] * q_row, cudaMemcpyDeviceToHost);
#undef DCUT_CP
    if ((st = dcut_check_cuda(c, cudaStreamSynchronize(cs), "cudaStreamSynchronize(step end)")) != DCUT_OK) return st;
    if (s->h2d_bytes) *s->h2d_bytes = h2d;
    if (s->d2h_bytes)
        *s->d2h_bytes = (long long)sizeof(int) * (B + 1 + 3 * B + B * (g + 1) + 1) + (s->attn_out ? (long long)cu[B] * q_row : 0);
    return DCUT_OK;
}
