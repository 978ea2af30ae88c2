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

template <typename T>
dcut_status dmalloc(dcut_ctx* ctx, T** p, size_t count, const char* what) {
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(p), sizeof(T) * (count ? count : 1));
    if (e != cudaSuccess) return dcut_check_cuda(ctx, e, what);
    return dcut_check_cuda(ctx, cudaMemset(*p, 0, sizeof(T) * (count ? count : 1)), what);
}

void free_all(dcut_ctx* c) {
    cudaFree(c->d_cost);
    cudaFree(c->d_bucket_K);
    cudaFree(c->d_items);
    cudaFree(c->d_plan);
    cudaFree(c->d_req_part);
    cudaFree(c->d_part_o);
    cudaFree(c->d_part_lse);
    cudaFree(c->d_row_key);
    cudaFree(c->d_status);
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
    if ((st = dcut_init_select(c)) != DCUT_OK) return st;
    if ((st = dcut_init_accept(c)) != DCUT_OK) return st;
    if (has_attn) {
        const char* env = getenv("DCUT_ATTN_TARGET_ITEMS");
        c->target_items = env ? atoi(env) : c->sm_count * 4;
        if (c->target_items < 1) c->target_items = 1;
        c->max_items = lim->max_B * lim->n_kv_heads + c->target_items;
        const int group = lim->n_q_heads / lim->n_kv_heads;
        c->part_rows_cap = (long long)c->max_items * (lim->max_gamma + 1) * group;
        if ((st = dmalloc(c, &c->d_items, c->max_items, "cudaMalloc(items)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->d_plan, 8, "cudaMalloc(plan)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->d_req_part, 2 * (size_t)lim->max_B, "cudaMalloc(req_part)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->d_part_o, (size_t)c->part_rows_cap * lim->head_dim, "cudaMalloc(part_o)")) != DCUT_OK) return st;
        if ((st = dmalloc(c, &c->d_part_lse, (size_t)c->part_rows_cap, "cudaMalloc(part_lse)")) != DCUT_OK) return st;
        if ((st = dcut_init_verify_attn(c)) != DCUT_OK) return st;
    }
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

dcut_status dcut_select(dcut_ctx* c, const float* conf, int B, int gamma, const int* draft_ids, const int* bonus_ids,
                        const int* ctx_lens, int* depths, int* cu_q, int* tok_req, int* tok_pos, int* tok_id,
                        dcut_select_info* info, float* scores_out, int* ranks_out, void* stream) {
    if (!c) return DCUT_EINVAL;
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
    return dcut_launch_select(c, conf, B, gamma, draft_ids, bonus_ids, ctx_lens, depths, cu_q, tok_req, tok_pos, tok_id,
                              info, scores_out, ranks_out, static_cast<cudaStream_t>(stream));
}

dcut_status dcut_verify_attn(dcut_ctx* c, const void* q, const void* k_cache, const void* v_cache, long long num_pages,
                             const int* block_table, int block_table_stride, const int* ctx_lens, const int* cu_q, int B,
                             int T_cap, float scale, void* out, float* lse, void* stream) {
    if (!c) return DCUT_EINVAL;
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
                                   T_cap, scale, out, lse, static_cast<cudaStream_t>(stream));
}

dcut_status dcut_accept(dcut_ctx* c, const void* logits, int V, const int* draft_ids, const int* cu_q, int B, int gamma,
                        int T_cap, int* accept_len, int* bonus, int* out_tokens, int* n_accepted_total, void* stream) {
    if (!c) return DCUT_EINVAL;
    if (!logits || !draft_ids || !cu_q || !accept_len || !bonus) return dcut_fail(c, DCUT_EINVAL, "null pointer argument");
    if (B < 1 || gamma < 1 || V < 1 || T_cap < B) return dcut_fail(c, DCUT_EINVAL, "need B, gamma, V >= 1 and T_cap >= B");
    if (B > c->lim.max_B || gamma > c->lim.max_gamma || T_cap > c->lim.max_B * (c->lim.max_gamma + 1))
        return dcut_fail(c, DCUT_ECAPACITY, "B = %d, gamma = %d, T_cap = %d exceed the limits", B, gamma, T_cap);
    if (c->lim.vocab > 0 && V > c->lim.vocab) return dcut_fail(c, DCUT_ECAPACITY, "V = %d exceeds the limit %d", V, c->lim.vocab);
    if (reinterpret_cast<uintptr_t>(logits) & 1) return dcut_fail(c, DCUT_EINVAL, "logits must be 2-byte aligned");
    return dcut_launch_accept(c, logits, V, draft_ids, cu_q, B, gamma, T_cap, accept_len, bonus, out_tokens,
                              n_accepted_total, c->d_row_key, static_cast<cudaStream_t>(stream));
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
