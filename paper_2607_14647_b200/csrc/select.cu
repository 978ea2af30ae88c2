// dcut_select: cross-request depth selection in one CTA (Eq. 3-5, Algorithm 1).
//
// The whole problem (at most 8192 draft positions, 32 KB of confidences) fits one SM's shared
// memory, and every step depends on the one before, so the kernel is latency-bound: one CTA of
// 1024 threads, no global round trips between the steps.
//   1. prefix products, one thread per request, fp32, left to right           (Eq. 3)
//   2. 64-bit keys (inverted score bits | depth | request) and a bitonic sort held in registers (warp shuffles
//      for short distances, a double-buffered shared array for long ones):
//      ascending key order = score descending, depth ascending, request ascending
//   3. block-wide scan of the fixed-point scores floor(p * 2^40) in int64 (exact in any order)
//   4. objective (B*2^40 + Q_N) / cost for every candidate N, fp64 divide, block argmax with
//      ties toward the smallest N                                            (Eq. 4-5)
//   5. depths by counting kept keys per request, cu_q by a block scan, packed token metadata
#include <limits.h>

#include "dcut_internal.h"
#include "attn_plan.cuh"

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;

struct SelectArgs {
    const float* conf;
    const int* draft_ids;
    const int* bonus_ids;
    const int* ctx_lens;
    const float* cost;      // dense: cost[T]; bucket: cost[c]
    const int* bucket_K;    // bucket mode only
    int n_buckets;          // 0 = dense
    int causal;             // 1: shifted scores (Eq. 7); dense table: early-stopping scan instead of the argmax
    int B, gamma, npad;
    int* depths;
    int* cu_q;
    int* tok_req;
    int* tok_pos;
    int* tok_id;
    dcut_select_info* info;
    float* scores_out;
    int* ranks_out;
    int with_plan;               // also build the attention work list of the packed batch (plan holds its arguments)
    dcut_plan::PlanArgs plan;
};

__device__ __forceinline__ float clamp_conf(float c) {
    if (!(c == c)) return 0.0f;
    if (c < 0.0f) return 0.0f;
    if (c > 1.0f) return 1.0f;
    return c;
}

__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

template <typename T>
__device__ __forceinline__ T warp_inclusive_scan(T v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        T u = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += u;
    }
    return v;
}

// exclusive scan of one value per thread over the CTA; returns the exclusive prefix and writes the
// CTA total to *total_out (same value in every thread).  `ws` is a [kWarps + 1] shared array.
template <typename T>
__device__ __forceinline__ T block_exclusive_scan(T v, T* ws, T* total_out) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    T inc = warp_inclusive_scan(v, lane);
    if (lane == 31) ws[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        T w = ws[lane];
        T winc = warp_inclusive_scan(w, lane);
        ws[lane] = winc - w;
        if (lane == 31) ws[kWarps] = winc;
    }
    __syncthreads();
    T res = ws[warp] + inc - v;
    *total_out = ws[kWarps];
    __syncthreads();
    return res;
}

// keep the smaller (or larger) of own and partner key
__device__ __forceinline__ unsigned long long cx(unsigned long long mine, unsigned long long other, bool keep_min) {
    return ((mine < other) == keep_min) ? mine : other;
}

// order a pair held by one thread: ascending if `up`
__device__ __forceinline__ void cx_pair(unsigned long long& a, unsigned long long& b, bool up) {
    const unsigned long long x = a, y = b;
    const bool swap = (x > y) == up;
    a = swap ? y : x;
    b = swap ? x : y;
}

// Bitonic sort, ascending, of the npad keys in `keys` (shared memory), held in registers meanwhile: KPT consecutive
// keys per thread of the first S / KPT threads (S = max(npad, 32 KPT) keys with padding); the other warps wait at the
// closing barrier.  Compare-exchange distances below KPT stay inside a thread, the next five are warp shuffles, the
// rest cross warps through shared memory: `keys` itself and `alt` (npad words, free during the sort) alternate as the
// exchange buffer, with one named barrier of the sorting warps per stage.  One loop per kind of stage keeps the code
// small: the kernel starts with cold instruction caches in every step, and a network unrolled for each size, though
// a third faster once warm, made the step slower.
template <int KPT>
__device__ __forceinline__ void sort_keys_blocked(unsigned long long* keys, unsigned long long* alt, int npad) {
    const int tid = threadIdx.x;
    int S = 32 * KPT;
    while (S < npad) S <<= 1;
    const int nt = S / KPT;                              // sorting threads: a multiple of 32
    if (tid < nt) {
        unsigned long long k[KPT];
#pragma unroll
        for (int e = 0; e < KPT; ++e) {
            const int idx = KPT * tid + e;
            k[e] = idx < npad ? keys[idx] : ~0ull;
        }
        int p = 0;
        for (int kk = 2; kk <= S; kk <<= 1) {
            const bool up_t = ((KPT * tid) & kk) == 0;   // direction of this thread's keys in the stages across threads
            int j = kk >> 1;
            for (; j >= 32 * KPT; j >>= 1) {             // partner thread in another warp (then S = npad >= 64 KPT)
                const int jt = j / KPT;
                const bool keep_min = up_t == ((tid & jt) == 0);
                unsigned long long* xb = p ? keys : alt;
                unsigned long long o[KPT];
#pragma unroll
                for (int e = 0; e < KPT; ++e) xb[e * nt + tid] = k[e];
                asm volatile("bar.sync 1, %0;" ::"r"(nt) : "memory");
#pragma unroll
                for (int e = 0; e < KPT; ++e) o[e] = xb[e * nt + (tid ^ jt)];
#pragma unroll
                for (int e = 0; e < KPT; ++e) k[e] = cx(k[e], o[e], keep_min);
                p ^= 1;
            }
            for (; j >= KPT; j >>= 1) {                  // partner thread in the same warp; same slot e
                const int jt = j / KPT;
                const bool keep_min = up_t == ((tid & jt) == 0);
                unsigned long long o[KPT];
#pragma unroll
                for (int e = 0; e < KPT; ++e) o[e] = __shfl_xor_sync(0xffffffffu, k[e], jt);
#pragma unroll
                for (int e = 0; e < KPT; ++e) k[e] = cx(k[e], o[e], keep_min);
            }
#pragma unroll
            for (int je = KPT / 2; je >= 1; je >>= 1) {  // partner key in the same thread (constant register indices)
                if (je <= j) {
#pragma unroll
                    for (int e = 0; e < KPT; ++e)
                        if ((e & je) == 0) cx_pair(k[e], k[e | je], ((KPT * tid + e) & kk) == 0);
                }
            }
        }
        // the last exchange buffer may have been `keys`: everybody has read it before the sorted keys go there
        asm volatile("bar.sync 1, %0;" ::"r"(nt) : "memory");
#pragma unroll
        for (int e = 0; e < KPT; ++e) {
            const int idx = KPT * tid + e;
            if (idx < npad) keys[idx] = k[e];
        }
    }
    __syncthreads();
}

__device__ __forceinline__ void sort_keys(unsigned long long* keys, unsigned long long* alt, int npad) {
    if (npad <= 4 * kThreads) sort_keys_blocked<4>(keys, alt, npad);
    else sort_keys_blocked<8>(keys, alt, npad);
}

struct Best {
    double obj;
    int N;
    int cand;
};

__device__ __forceinline__ bool better(const Best& a, const Best& b) {   // is a better than b
    return a.obj > b.obj || (a.obj == b.obj && a.N < b.N);
}

__global__ void __launch_bounds__(kThreads, 1) dcut_select_kernel(SelectArgs a) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int B = a.B, gamma = a.gamma, n = B * gamma, npad = a.npad;
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem);          // [npad]
    long long* qs = reinterpret_cast<long long*>(keys + npad);                       // [npad + 1]
    int* depth_s = reinterpret_cast<int*>(qs + npad + 1);                            // [B]
    int* cu_s = depth_s + B;                                                         // [B + 1]
    __shared__ long long ws64[kWarps + 1];
    __shared__ int ws32[kWarps + 1];
    __shared__ Best wbest[kWarps];
    __shared__ Best best_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    dcut_pdl_wait();
    dcut_pdl_launch_dependents();
    // What the later steps read from global memory, each after a barrier and hence with its full latency exposed:
    // ask for it now (between two steps of a serving loop the KV stream has pushed all of it out of L2).
    {
        const size_t cost_bytes = sizeof(float) * (size_t)(a.n_buckets > 0 ? a.n_buckets : n + 1);
        const char* cost0 = reinterpret_cast<const char*>(a.cost + (a.n_buckets > 0 ? 0 : B));
        for (size_t off = (size_t)tid * 128; off < cost_bytes; off += (size_t)kThreads * 128) prefetch_l2(cost0 + off);
        if (a.draft_ids)      // (the three arrays are optional: a caller that wants only depths and cu_q passes none)
            for (size_t off = (size_t)tid * 128; off < sizeof(int) * (size_t)n; off += (size_t)kThreads * 128)
                prefetch_l2(reinterpret_cast<const char*>(a.draft_ids) + off);
        for (size_t off = (size_t)tid * 128; off < sizeof(int) * (size_t)B; off += (size_t)kThreads * 128) {
            if (a.ctx_lens) prefetch_l2(reinterpret_cast<const char*>(a.ctx_lens) + off);
            if (a.bonus_ids) prefetch_l2(reinterpret_cast<const char*>(a.bonus_ids) + off);
        }
        if (a.n_buckets > 0 && tid == 0) prefetch_l2(a.bucket_K);
    }
    // 1. prefix scores and sort keys.  The confidences come in through shared memory with coalesced loads
    // (the later prefix-sum array is free at this point), so the per-request product chain reads no global memory.
    float* conf_s = reinterpret_cast<float*>(qs);
    for (int e = tid; e < n; e += kThreads) conf_s[e] = a.conf[e];
    __syncthreads();
    for (int i = tid; i < B; i += kThreads) {
        float prev = 1.0f;
        for (int k = 0; k < gamma; ++k) {
            float nxt = __fmul_rn(prev, clamp_conf(conf_s[i * gamma + k]));
            if (nxt == 0.0f) nxt = 0.0f;   // -0 -> +0
            // Eq. 3: the score of depth k + 1 includes its own confidence; Eq. 7 (causal mode): only those before it
            const float p = a.causal ? prev : nxt;
            prev = nxt;
            if (a.scores_out) a.scores_out[(size_t)i * gamma + k] = p;
            const unsigned int bits = __float_as_uint(p);
            keys[i * gamma + k] = ((unsigned long long)(0xffffffffu - bits) << 32) |
                                  ((unsigned long long)k << 16) | (unsigned long long)i;
        }
    }
    for (int r = n + tid; r < npad; r += kThreads) keys[r] = ~0ull;
    for (int i = tid; i < B; i += kThreads) depth_s[i] = 0;
    __syncthreads();
    // 2. bitonic sort, ascending, with the keys held in registers (sort_keys_blocked); the prefix-sum array is free
    // until step 3 and serves as the second exchange buffer
    sort_keys(keys, reinterpret_cast<unsigned long long*>(qs), npad);
    // 3. fixed-point prefix sums Q[0..n]; ranks
    {
        const int per = (npad + kThreads - 1) / kThreads;
        const int r0 = tid * per;
        long long local = 0;
        for (int e = 0; e < per; ++e) {
            const int r = r0 + e;
            if (r < n) {
                const unsigned long long key = keys[r];
                const float p = __uint_as_float(0xffffffffu - (unsigned int)(key >> 32));
                local += __double2ll_rz((double)p * 1099511627776.0);
                if (a.ranks_out) {
                    const int i = (int)(key & 0xffffu), k = (int)((key >> 16) & 0xffffu);
                    a.ranks_out[(size_t)i * gamma + k] = r;
                }
            }
        }
        long long total;
        long long run = block_exclusive_scan<long long>(local, ws64, &total);
        if (tid == 0) qs[0] = 0;
        for (int e = 0; e < per; ++e) {
            const int r = r0 + e;
            if (r < n) {
                const float p = __uint_as_float(0xffffffffu - (unsigned int)(keys[r] >> 32));
                run += __double2ll_rz((double)p * 1099511627776.0);
                qs[r + 1] = run;
            }
        }
    }
    __syncthreads();
    // 4. objective over the candidates
    if (a.causal && a.n_buckets == 0) {
        // Causal early-stopping scan (Appendix B): positions are admitted in ranked order while the objective strictly
        // improves, so N* is the first N whose successor is not better.  A request's shifted scores never increase
        // with depth, so the ranked order is the order in which the frontiers would be exposed.
        const long long bfix = (long long)B << 40;
        int first = n;
        for (int c = tid; c < n; c += kThreads) {
            const double o0 = __ddiv_rn(__ll2double_rn(bfix + qs[c]), (double)a.cost[B + c]);
            const double o1 = __ddiv_rn(__ll2double_rn(bfix + qs[c + 1]), (double)a.cost[B + c + 1]);
            if (!(o1 > o0)) {
                first = c;
                break;          // this thread's later candidates are larger
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) first = min(first, __shfl_xor_sync(0xffffffffu, first, o));
        if (lane == 0) ws32[warp] = first;
        __syncthreads();
        if (warp == 0) {
            first = ws32[lane];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) first = min(first, __shfl_xor_sync(0xffffffffu, first, o));
            if (lane == 0) {
                Best b = {__ddiv_rn(__ll2double_rn(bfix + qs[first]), (double)a.cost[B + first]), first, first};
                best_s = b;
            }
        }
        __syncthreads();
    } else {
        const long long bfix = (long long)B << 40;
        Best b = {-1.0, INT_MAX, -1};
        const int n_cand = a.n_buckets > 0 ? a.n_buckets : n + 1;
        for (int c = tid; c < n_cand; c += kThreads) {
            int N;
            float cost;
            if (a.n_buckets > 0) {
                N = a.bucket_K[c] - B;
                cost = a.cost[c];
            } else {
                N = c;
                cost = a.cost[B + N];
            }
            Best cur = {__ddiv_rn(__ll2double_rn(bfix + qs[N]), (double)cost), N, c};
            if (better(cur, b)) b = cur;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            Best other;
            other.obj = __shfl_xor_sync(0xffffffffu, b.obj, o);
            other.N = __shfl_xor_sync(0xffffffffu, b.N, o);
            other.cand = __shfl_xor_sync(0xffffffffu, b.cand, o);
            if (better(other, b)) b = other;
        }
        if (lane == 0) wbest[warp] = b;
        __syncthreads();
        if (warp == 0) {
            b = wbest[lane];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                Best other;
                other.obj = __shfl_xor_sync(0xffffffffu, b.obj, o);
                other.N = __shfl_xor_sync(0xffffffffu, b.N, o);
                other.cand = __shfl_xor_sync(0xffffffffu, b.cand, o);
                if (better(other, b)) b = other;
            }
            if (lane == 0) best_s = b;
        }
        __syncthreads();
    }
    const int n_star = best_s.N;
    // 5. depths, cu_q, packed token metadata
    for (int r = tid; r < n_star; r += kThreads) atomicAdd(&depth_s[(int)(keys[r] & 0xffffu)], 1);
    __syncthreads();
    {
        const int per = (B + kThreads - 1) / kThreads;
        const int i0 = tid * per;
        int local = 0;
        for (int e = 0; e < per; ++e)
            if (i0 + e < B) local += 1 + depth_s[i0 + e];
        int total;
        int run = block_exclusive_scan<int>(local, ws32, &total);
        for (int e = 0; e < per; ++e) {
            const int i = i0 + e;
            if (i < B) {
                cu_s[i] = run;
                a.cu_q[i] = run;
                a.depths[i] = depth_s[i];
                run += 1 + depth_s[i];
            }
        }
        if (tid == 0) {
            cu_s[B] = total;
            a.cu_q[B] = total;
        }
    }
    __syncthreads();
    const int T = cu_s[B];
    const int cap = B * (gamma + 1);
    for (int idx = tid; idx < cap; idx += kThreads) {
        const int i = idx / (gamma + 1), t = idx - i * (gamma + 1);
        if (t <= depth_s[i]) {
            const int pos = cu_s[i] + t;
            if (a.tok_req) a.tok_req[pos] = i;
            if (a.tok_pos) a.tok_pos[pos] = a.ctx_lens[i] + t;
            if (a.tok_id) a.tok_id[pos] = (t == 0) ? a.bonus_ids[i] : a.draft_ids[(size_t)i * gamma + t - 1];
        }
        if (idx >= T) {
            if (a.tok_req) a.tok_req[idx] = -1;
            if (a.tok_pos) a.tok_pos[idx] = -1;
            if (a.tok_id) a.tok_id[idx] = -1;
        }
    }
    if (tid == 0 && a.info) {
        dcut_select_info out;
        out.n_star = n_star;
        out.t_total = T;
        out.candidate = best_s.cand;
        out.reserved = 0;
        out.sum_fixed = ((long long)B << 40) + qs[n_star];
        out.objective = best_s.obj;
        *a.info = out;
    }
    if (a.with_plan) {
        // 6. the attention work list of the batch just packed: it depends on ctx_lens, cu_q and the shapes only, and
        // this CTA has them at hand, so the attention call that follows need not launch a one-CTA kernel of its own.
        // The sort keys are dead by now: their shared memory holds the plan's ordering keys (npad >= B entries).
        // cu_q is at hand in shared memory (cu_s); ctx_lens joins it in the dead depth array.  The sort keys and the
        // prefix sums are dead too: their contiguous shared memory (16 npad + 8 bytes, npad >= B) holds the plan's
        // 2 B + 1 cost prefixes.
        __syncthreads();            // nobody reads `keys`, `qs` or `depth_s` any more
        int* ctx_s = depth_s;
        for (int i = tid; i < B; i += kThreads) ctx_s[i] = a.ctx_lens[i];
        __syncthreads();
        dcut_plan::PlanArgs pa = a.plan;
        pa.cu_q = cu_s;
        pa.ctx_lens = ctx_s;
        dcut_plan::attn_plan_body(pa, reinterpret_cast<long long*>(keys));
    }
}

size_t select_smem_bytes(int B, int npad) {
    return sizeof(unsigned long long) * (size_t)npad + sizeof(long long) * (size_t)(npad + 1) +
           sizeof(int) * (size_t)(2 * B + 1) + 16;
}

}  // namespace

// Per-device set-up: the selector may use up to ~192 KB of dynamic shared memory.
dcut_status dcut_init_select(dcut_ctx* ctx) {
    cudaError_t e = cudaFuncSetAttribute(dcut_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)select_smem_bytes(DCUT_MAX_KEYS, DCUT_MAX_KEYS));
    return dcut_check_cuda(ctx, e, "cudaFuncSetAttribute(select)");
}

dcut_status dcut_launch_select(dcut_ctx* ctx, const float* conf, int B, int gamma, const int* draft_ids,
                               const int* bonus_ids, const int* ctx_lens, int* depths, int* cu_q,
                               int* tok_req, int* tok_pos, int* tok_id, dcut_select_info* info,
                               float* scores_out, int* ranks_out, int causal, int with_plan, cudaStream_t stream) {
    const int n = B * gamma;
    int npad = 32;
    while (npad < n) npad <<= 1;
    SelectArgs a;
    a.conf = conf;
    a.draft_ids = draft_ids;
    a.bonus_ids = bonus_ids;
    a.ctx_lens = ctx_lens;
    a.cost = ctx->d_cost;
    a.bucket_K = ctx->d_bucket_K;
    a.n_buckets = ctx->n_buckets;
    a.causal = causal;
    a.B = B;
    a.gamma = gamma;
    a.npad = npad;
    a.depths = depths;
    a.cu_q = cu_q;
    a.tok_req = tok_req;
    a.tok_pos = tok_pos;
    a.tok_id = tok_id;
    a.info = info;
    a.scores_out = scores_out;
    a.ranks_out = ranks_out;
    a.with_plan = with_plan;
    if (with_plan) dcut_fill_plan_args(ctx, ctx_lens, cu_q, B, &a.plan);
    const size_t smem = select_smem_bytes(B, npad);
    return dcut_check_cuda(ctx, dcut_launch_pdl(dcut_select_kernel, dim3(1), dim3(kThreads), smem, stream, a), "launch dcut_select_kernel");
}
