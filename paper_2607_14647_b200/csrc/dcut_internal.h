// Internal declarations shared by the translation units of libdcut.so (not installed).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dcut.h"

#define DCUT_MAX_KEYS 8192      // B * gamma handled by the single-CTA selector
#define DCUT_MAX_BUCKETS 64

// device status word codes (dcut_poll_device_status)
#define DCUT_DEV_OK 0
#define DCUT_DEV_ATTN_WAIT_TIMEOUT 1   // a bounded mbarrier wait in the attention kernel gave up
#define DCUT_DEV_BAD_PAGE 2            // a block-table entry outside [0, num_pages)
#define DCUT_DEV_PLAN_OVERFLOW 3       // the attention work list did not fit the context's scratch
#define DCUT_DEV_GEMM_WAIT_TIMEOUT 4    // a bounded mbarrier wait in the GEMM kernel gave up
#define DCUT_DEV_COMMIT_OVERFLOW 5      // dcut_commit: a context or a token stream ran out of room
#define DCUT_DEV_BAD_TOKEN 6            // dcut_model_verify: a token id outside [0, vocab)
#define DCUT_DEV_BAD_CU_Q 7             // acceptance: cu_q is not a packing of B requests of 1..gamma+1 rows within T_cap

// One row of the attention work table: a (request, row block of its query tile); it stands for n_kv_heads work items of
// equal cost, one per kv head, each over the request's `pages` KV pages.
struct __align__(16) AttnEntry {
    int32_t req;
    int32_t row0;         // first query row of the block within the request's tile
    int32_t rows;         // query rows of the block
    int32_t pages;        // KV pages of the request (context + retained tokens)
    int32_t q0;           // cu_q[req]: first packed token of the request
    int32_t depth;        // d_i
    int32_t ctx_len;      // L_i
    int32_t tc;           // 1: the items run on the tcgen05 phase of the item kernel, 0: on the warp-level phase
};
// A boundary between two segments of the work stream: before page `p` of the item (entry `e`, kv head `h`).
struct __align__(16) AttnSeg {
    int32_t e, h, p, pad;
};

// What the combine kernel does at boundary b (between segments b - 1 and b): nothing (pieces = 0), or merge the
// `pieces` partial results of the item that boundaries b .. b + pieces - 2 cut (the item begins in segment b - 1).
struct __align__(16) AttnCut {
    int32_t pieces, rows, row0, q0, kv_head, pad[3];
};

// One work item of the attention kernel as a CTA runs it: one (request, kv head, page range).
struct __align__(16) AttnItem {
    int32_t req;
    int32_t kv_head;
    int32_t page_begin;   // first page index (within the request's block-table row)
    int32_t page_end;     // one past the last
    int32_t n_chunks;     // how many chunks the request has
    int32_t part_row;     // first row of this item's partial results in the scratch (-1: writes the output)
    int32_t q0;           // cu_q[req]: first packed token of the request
    int32_t depth;        // d_i
    int32_t ctx_len;      // L_i
    int32_t pad[3];
};

struct dcut_ctx {
    dcut_limits lim;
    int device;
    int sm_count;
    char err[512];

    // cost model
    float* d_cost;          // dense: [cost_n]; bucket: [n_buckets]
    int* d_bucket_K;        // [DCUT_MAX_BUCKETS]
    int cost_n;             // entries of the dense table (0 = none)
    int cost_cap;           // allocated floats
    int n_buckets;          // > 0: bucket mode
    int bucket_B, bucket_gamma;

    // attention scratch
    AttnEntry* d_entries;   // [max_entries] work table (one row per (request, row block))
    AttnSeg* d_segs;        // [sm_count + 1] segment boundaries of the work stream, one segment per CTA of the item kernel
    AttnCut* d_cuts;        // [sm_count] per boundary: the cut item whose pieces the combine kernel merges there
    int* d_plan;            // [16] plan header: n_entries, first warp-level entry, total pages
    float* d_part_o;        // [2 * sm_count slots][144 rows][head_dim] fp32: partial results of the items a boundary cuts
    float* d_part_lse;      // [2 * sm_count slots][144 rows]
    int max_entries;
    int attn_min_chunk_pages;   // no piece of a cut item is shorter than this
    int attn_tc_min_rows;   // items with at least this many query rows use the tcgen05 phase
    int attn_tail_rows;     // a query tile of up to 128 + this many rows stays one item (0: cut at 128)
    // work list left ready by the selector (dcut_enable_plan_in_select): the batch it was made for
    int plan_in_select;
    const int* plan_cu_q;
    const int* plan_ctx_lens;
    int plan_B;

    // accept scratch
    unsigned long long* d_row_key;   // [max_T] packed (ordered max, ~index); zero between calls

    // rejection-sampling acceptance scratch (vocab > 0 only)
    void* d_rs_scratch;
    int rs_n_seg;

    int* d_status;          // device status word

    // tensor-map encoder (driver entry point fetched through the runtime)
    void* encode_tiled;

    // decoder-layer workspace (hidden > 0 only), all [max_T, width] bf16
    __nv_bfloat16 *ly_norm, *ly_qkv, *ly_q, *ly_attn, *ly_h1, *ly_norm2, *ly_act;
    __nv_bfloat16* ly_x[2];   // hidden states between the layers of dcut_model_verify (ping-pong)
    int ly_gemm_pairs;      // clusters of two CTAs the device runs at once
    int ly_gemm_pair_mode;  // 0: the GEMM never runs tiles on pairs of SMs
    int ly_gemm_force;      // experiments: -1 = gemm_plan chooses; 0..6 a width on one SM; 8..14 on a pair
    unsigned ly_gemm_bn_mask;   // tile widths the one-SM mode may choose from (bit i: 256 - 32 i columns)
    float* ly_inv_freq;     // [head_dim / 2]
    float ly_inv_freq_host[64];   // its host copy (head_dim <= 128), the source of the upload
    float ly_theta;         // theta the table was built for (0 = none yet)
    void* layer_maps;       // cached tensor maps (layer.cu)

    // staging of dcut_verify_step_host (allocated by its first call)
    int hs_ready, hs_vocab;
    float* hs_conf;
    int *hs_draft, *hs_bonus, *hs_ctx_lens, *hs_block_table, *hs_depths, *hs_cu_q, *hs_accept;
    unsigned short *hs_q, *hs_out, *hs_logits, *hs_hidden;
    int* hs_host_cu_q;      // pinned
    cudaStream_t hs_copy_stream;   // dcut_verify_step_host: the logits travel on this stream while attention runs
    cudaEvent_t hs_ev_fork, hs_ev_join;
};

#ifdef __CUDACC__
#include <utility>
// Programmatic dependent launch: the kernel may be scheduled while its predecessor in the stream is still running
// (its CTAs take SMs as the predecessor's CTAs leave), which hides launch latency and the kernel's own set-up.  Every
// kernel launched this way calls dcut_pdl_wait() before it touches global memory: the wait returns when the
// predecessor grid has completed, and since the predecessor did the same, everything earlier has completed too.
template <typename... KArgs, typename... Args>
inline cudaError_t dcut_launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                   Args&&... args) {
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = grid;
    lc.blockDim = block;
    lc.dynamicSmemBytes = smem;
    lc.stream = stream;
    lc.attrs = attr;
    lc.numAttrs = 1;
    return cudaLaunchKernelEx(&lc, kernel, std::forward<Args>(args)...);
}
__device__ __forceinline__ void dcut_pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dcut_pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// value order as an unsigned integer: larger float <=> larger code; every non-NaN code is > 0
__device__ __forceinline__ unsigned int dcut_ordered_bits(float f) {
    if (f == 0.0f) f = 0.0f;   // -0 and +0 are the same value
    const unsigned int b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
#endif

dcut_status dcut_fail(dcut_ctx* ctx, dcut_status st, const char* fmt, ...);
dcut_status dcut_check_cuda(dcut_ctx* ctx, cudaError_t e, const char* what);

// per-device set-up (function attributes), called from dcut_create with the device current
dcut_status dcut_init_select(dcut_ctx* ctx);
dcut_status dcut_init_accept(dcut_ctx* ctx);
dcut_status dcut_init_verify_attn(dcut_ctx* ctx);
dcut_status dcut_init_layer(dcut_ctx* ctx);
void dcut_free_layer(dcut_ctx* ctx);

// kernel launchers (one per translation unit)
dcut_status dcut_launch_select(dcut_ctx* ctx, const float* conf, int B, int gamma, const int* draft_ids,
                               const int* bonus_ids, const int* ctx_lens, int* depths, int* cu_q,
                               int* tok_req, int* tok_pos, int* tok_id, dcut_select_info* info,
                               float* scores_out, int* ranks_out, int causal, int with_plan, cudaStream_t stream);
dcut_status dcut_launch_accept(dcut_ctx* ctx, const void* logits, int V, const int* draft_ids,
                               const int* cu_q, int B, int gamma, int T_cap, int* accept_len, int* bonus,
                               int* out_tokens, int* n_accepted_total, unsigned long long* row_key,
                               cudaStream_t stream);
size_t dcut_accept_rs_scratch_bytes(const dcut_ctx* ctx, int n_seg);
dcut_status dcut_init_accept_rs(dcut_ctx* ctx);
dcut_status dcut_launch_accept_rs(dcut_ctx* ctx, const void* target_logits, const void* draft_logits, int V,
                                  const int* draft_ids, const int* cu_q, int B, int gamma, int T_cap,
                                  const float* u_accept, const float* u_sample, int* accept_len, int* bonus,
                                  int* out_tokens, int* n_accepted_total, float* prob, cudaStream_t stream);
dcut_status dcut_launch_verify_attn(dcut_ctx* ctx, const void* q, const void* k_cache, const void* v_cache,
                                    long long num_pages, const int* block_table, int block_table_stride,
                                    const int* ctx_lens, const int* cu_q, int B, int T_cap, float scale,
                                    void* out, float* lse, int reuse_plan, cudaStream_t stream);
dcut_status dcut_launch_gemm(dcut_ctx* ctx, const void* a, const void* w, const void* w2, int mode, int N, int K,
                             const int* cu_q, int B, int T_cap, void* out, const void* residual, cudaStream_t stream);
dcut_status dcut_launch_lm_head_argmax(dcut_ctx* ctx, const void* x, const void* w_lm, int V, int K, const int* cu_q, int B,
                                       int T_cap, unsigned long long* row_key, cudaStream_t stream);
// second half of dcut_accept on per-row words that are already filled (logits may be null: rows without a word give 0)
dcut_status dcut_launch_accept_match(dcut_ctx* ctx, const void* logits, int V, const int* draft_ids, const int* cu_q,
                                     int B, int gamma, int T_cap, int* accept_len, int* bonus, int* out_tokens,
                                     int* n_accepted_total, int* row_argmax, unsigned long long* row_key,
                                     cudaStream_t stream);
dcut_status dcut_launch_model(dcut_ctx* ctx, const dcut_model* m, long long num_pages, const int* block_table,
                              int block_table_stride, const int* ctx_lens, const int* cu_q, const int* tok_req,
                              const int* tok_pos, const int* tok_id, const int* draft_ids, int B, int gamma, int T_cap,
                              int* accept_len, int* bonus, int* out_tokens, int* n_accepted_total, int* row_argmax,
                              void* hidden_out, cudaStream_t stream);
dcut_status dcut_launch_commit(dcut_ctx* ctx, const int* accept_len, const int* out_tokens, int B, int gamma, int max_ctx,
                               int* ctx_lens, int* bonus_ids, int* stream_tokens, int* stream_len, int stream_cap,
                               cudaStream_t stream);
dcut_status dcut_launch_layer(dcut_ctx* ctx, const dcut_layer_weights* w, const void* x, void* y, void* k_cache,
                              void* v_cache, long long num_pages, const int* block_table, int block_table_stride,
                              const int* ctx_lens, const int* cu_q, const int* tok_req, const int* tok_pos, int B,
                              int T_cap, int reuse_plan, int part, cudaStream_t stream);
dcut_status dcut_launch_residual_add(dcut_ctx* ctx, const void* a, const void* b, void* out, int width, const int* cu_q, int B,
                                     int T_cap, cudaStream_t stream);
