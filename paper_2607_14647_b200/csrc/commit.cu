// dcut_commit: the bookkeeping that ends a verify step and starts the next one (Section 3.1: every request commits its
// accepted drafts plus one more token and advances; Appendix A: progress never stalls because the bonus token is
// always kept).
//
// In the paged cache the step appended K/V for the bonus token at position L_i and for the kept drafts at
// L_i + 1 .. L_i + d_i.  Accepted are the bonus token and the first m_i drafts, so the cache is valid up to and
// including position L_i + m_i: the new context length is L_i + m_i + 1.  The rejected drafts' slots need no work:
// the next step writes its own tokens over them ("rolling back" is the shorter context length).  The token the step
// emitted last (the target's own prediction) becomes the next step's bonus token z_{i,0}.
#include "dcut_internal.h"

namespace {

struct CommitArgs {
    const int* accept_len;      // [B] m_i
    const int* out_tokens;      // [B, gamma + 1]: the emitted tokens (m_i drafts, then the closing token), -1 padded
    int B, gamma, max_ctx, stream_cap;
    int* ctx_lens;              // [B] in/out
    int* bonus_ids;             // [B] out: z_{i,0} of the next step
    int* stream;                // [B, stream_cap] or null: every token the request has emitted so far
    int* stream_len;            // [B] in/out (with stream)
    int* status;
};

__global__ void __launch_bounds__(256) commit_kernel(CommitArgs a) {
    const int lane = threadIdx.x & 31;
    const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);   // one warp per request
    if (i >= a.B) return;
    int m = a.accept_len[i];
    m = min(max(m, 0), a.gamma);
    const int* toks = a.out_tokens + (size_t)i * (a.gamma + 1);
    if (a.stream) {
        const int have = a.stream_len[i];
        if (have + m + 1 > a.stream_cap) {
            if (lane == 0) atomicExch(a.status, DCUT_DEV_COMMIT_OVERFLOW);
        } else {
            for (int t = lane; t <= m; t += 32) a.stream[(size_t)i * a.stream_cap + have + t] = toks[t];
            __syncwarp();
            if (lane == 0) a.stream_len[i] = have + m + 1;
        }
    }
    if (lane == 0) {
        const int L = a.ctx_lens[i] + m + 1;
        // the next step appends up to gamma + 1 tokens behind L
        if (L + a.gamma + 1 > a.max_ctx) atomicExch(a.status, DCUT_DEV_COMMIT_OVERFLOW);
        a.ctx_lens[i] = L;
        a.bonus_ids[i] = toks[m];
    }
}

}  // namespace

dcut_status dcut_launch_commit(dcut_ctx* ctx, const int* accept_len, const int* out_tokens, int B, int gamma, int max_ctx,
                               int* ctx_lens, int* bonus_ids, int* stream_tokens, int* stream_len, int stream_cap,
                               cudaStream_t stream) {
    CommitArgs a;
    a.accept_len = accept_len;
    a.out_tokens = out_tokens;
    a.B = B;
    a.gamma = gamma;
    a.max_ctx = max_ctx;
    a.stream_cap = stream_cap;
    a.ctx_lens = ctx_lens;
    a.bonus_ids = bonus_ids;
    a.stream = stream_tokens;
    a.stream_len = stream_len;
    a.status = ctx->d_status;
    commit_kernel<<<(B + 7) / 8, 256, 0, stream>>>(a);
    return dcut_check_cuda(ctx, cudaGetLastError(), "launch commit_kernel");
}
