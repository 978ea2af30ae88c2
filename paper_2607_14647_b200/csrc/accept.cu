// dcut_accept: greedy acceptance (Sections 3.1-3.2: A_i = 1 + min(L_i, n_i) and the bonus token).
//
// Two launches.
//   accept_argmax_kernel  HBM-bound scan of the bf16 logits [T, V].  Each row is cut into
//       segments, one CTA per (segment, row), so small batches still fill 148 SMs.  Threads read
//       16-byte vectors with streaming loads, several in flight per thread, and keep (max, first
//       index); the CTA result is merged into one 64-bit word per row with atomicMax on
//       (ordered value << 32 | ~index): the largest value wins and, among equals, the lowest
//       index, whatever order the CTAs finish in.
//   accept_match_kernel   one warp per request: longest matching prefix, bonus token, emitted
//       tokens, total; clears the per-row words for the next call.
#include "dcut_internal.h"

namespace {

constexpr int kArgmaxThreads = 256;
constexpr int kUnroll = 8;   // 16-byte loads in flight per thread (4: 35-37 us at T = 600 of the 64-request workload, 8: 30-31; 50 against 51 us at T = 1088)

__device__ __forceinline__ uint4 ld_stream_v4(const uint4* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.L2::256B.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

__device__ __forceinline__ unsigned int ordered_bits(float f) { return dcut_ordered_bits(f); }

__device__ __forceinline__ unsigned int max_bf16x2(unsigned int x, unsigned int y) {   // a NaN operand is ignored
    unsigned int r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(y));
    return r;
}

__device__ __forceinline__ void take(float f, int idx, float& best, int& bidx) {
    if (f > best) {   // strict: the first of equal values stays; NaN never passes
        best = f;
        bidx = idx;
    }
}

__device__ __forceinline__ void take8(const uint4& v, int base, float& best, int& bidx) {
    const unsigned int w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        take(__uint_as_float(w[e] << 16), base + 2 * e, best, bidx);
        take(__uint_as_float(w[e] & 0xffff0000u), base + 2 * e + 1, best, bidx);
    }
}

__global__ void __launch_bounds__(kArgmaxThreads) accept_argmax_kernel(
    const unsigned short* __restrict__ logits, int V, const int* __restrict__ cu_q, int B, int seg_elems,
    unsigned long long* __restrict__ row_key) {
    dcut_pdl_wait();
    dcut_pdl_launch_dependents();
    const int row = blockIdx.y;   // < T_cap, the rows the per-row words are sized for
    if (row >= cu_q[B]) return;
    const int start = blockIdx.x * seg_elems;
    if (start >= V) return;
    const int end = min(V, start + seg_elems);
    const unsigned short* rp = logits + (size_t)row * V;
    float best = -INFINITY;
    int bidx = -1;

    // scalar head up to the first 16-byte boundary, vector body, scalar tail
    const unsigned long long addr = (unsigned long long)(rp + start);
    int head = (int)(((16 - (addr & 15)) & 15) >> 1);
    if (head > end - start) head = end - start;
    const int body0 = start + head;
    const int nvec = (end - body0) >> 3;
    const int tail0 = body0 + (nvec << 3);
    if ((int)threadIdx.x < head)
        take(__uint_as_float((unsigned int)rp[start + threadIdx.x] << 16), start + threadIdx.x, best, bidx);
    // A thread keeps the packed bf16x2 maximum of the vectors it has seen (one max.bf16x2 per 4 bytes, NaNs ignored);
    // only a batch of loads that raises one of its halves can hold a value above `best`, and only such a batch is
    // looked at value by value for (maximum, first index).  After the first few batches that is rare.
    const uint4* vp = reinterpret_cast<const uint4*>(rp + body0);
    unsigned int best2 = 0xff80ff80u;                 // (-inf, -inf)
    int v = threadIdx.x;
    for (; v + (kUnroll - 1) * kArgmaxThreads < nvec; v += kUnroll * kArgmaxThreads) {
        uint4 x[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) x[u] = ld_stream_v4(vp + v + u * kArgmaxThreads);
        unsigned int m2 = best2;
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) m2 = max_bf16x2(m2, max_bf16x2(max_bf16x2(x[u].x, x[u].y), max_bf16x2(x[u].z, x[u].w)));
        if (m2 != best2) {
            best2 = m2;
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) take8(x[u], body0 + ((v + u * kArgmaxThreads) << 3), best, bidx);
        }
    }
    for (; v < nvec; v += kArgmaxThreads) take8(ld_stream_v4(vp + v), body0 + (v << 3), best, bidx);
    // a thread's indices ascend except for the tail, which lies past every body index
    if ((int)threadIdx.x < end - tail0)
        take(__uint_as_float((unsigned int)rp[tail0 + threadIdx.x] << 16), tail0 + threadIdx.x, best, bidx);

    unsigned long long key = 0;   // 0 = nothing above -inf seen
    if (bidx >= 0) key = ((unsigned long long)ordered_bits(best) << 32) | (unsigned long long)(0xffffffffu - (unsigned int)bidx);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, key, o);
        key = other > key ? other : key;
    }
    __shared__ unsigned long long wk[kArgmaxThreads / 32];
    if ((threadIdx.x & 31) == 0) wk[threadIdx.x >> 5] = key;
    __syncthreads();
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 1; w < kArgmaxThreads / 32; ++w) key = wk[w] > key ? wk[w] : key;
        if (key) atomicMax(row_key + row, key);
    }
}

// rows whose maximum is -inf (or that hold only NaN) leave key 0: the first non-NaN index, else 0
__device__ int slow_first_valid(const unsigned short* rp, int V) {
    for (int v = 0; v < V; ++v) {
        const float f = __uint_as_float((unsigned int)rp[v] << 16);
        if (f == f) return v;
    }
    return 0;
}

constexpr int kMatchR = 1;   // requests a warp of the matching kernel has in flight (2: 0.4 us less at B = 64, 0.35 us more at B = 16; 4: slower)

struct MatchArgs {
    const unsigned short* logits;   // only read for rows whose scan found nothing above -inf; may be null
    int V;
    const int* draft_ids;
    const int* cu_q;
    int B, gamma, row_cap;
    unsigned long long* row_key;
    int* accept_len;
    int* bonus;
    int* out_tokens;
    int* n_accepted_total;
    int* row_argmax;
    int* status;
};

// One warp per request: the lanes fetch the row results of t = lane, lane + 32, ... together, a ballot finds the
// first row whose argmax differs from the draft (or the last row), and the per-row words are cleared on the way.
// A warp works on R requests at a time: their loads (offsets, then row words and drafts) are issued together, so the
// two global-memory latencies of the chain are paid once per R requests.
// Only rows below row_cap (the T_cap the words and the scan were sized for) exist: a cu_q that runs past it breaks the
// caller's contract, so those rows are neither read nor cleared, the request's scan ends at the last row that
// exists (a request with none reports accept_len 0 and bonus 0), and the status word, if there is one, says so.
// Returns this lane's share of the accepted-token total (lane 0 of each warp carries it).
template <int R>
__device__ __forceinline__ int match_requests(const MatchArgs& g, int warp, int n_warps, int lane) {
    int local = 0;
    const int gamma = g.gamma;
    for (int i0 = warp * R; i0 < g.B; i0 += n_warps * R) {
        int a_[R], d_[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int i = i0 + r;
            a_[r] = 0;
            d_[r] = -2;                       // -2: no such request
            if (i < g.B) {
                a_[r] = g.cu_q[i];
                d_[r] = g.cu_q[i + 1] - a_[r] - 1;
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if (d_[r] == -2) continue;
            int a = a_[r], d = d_[r];
            if (a < 0 || d < 0 || d > gamma || a + d >= g.row_cap) {
                if (lane == 0 && g.status) atomicExch(g.status, DCUT_DEV_BAD_CU_Q);
                d = min(min(d, gamma), g.row_cap - 1 - a);       // rows [a, a + d] exist; none if d < 0 or a < 0
                if (a < 0 || d < 0) d = -1;
                d_[r] = d;
            }
        }
        unsigned long long key_[R];
        int dr_[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {         // the first 32 rows of each request
            key_[r] = 0;
            dr_[r] = -1;
            if (lane <= d_[r]) {
                key_[r] = __ldcg(g.row_key + a_[r] + lane);
                if (lane < d_[r]) dr_[r] = g.draft_ids[(size_t)(i0 + r) * gamma + lane];
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if (d_[r] == -2) continue;
            const int i = i0 + r, a = a_[r], d = d_[r];
            int m = d < 0 ? 0 : -1, bon = 0;
            for (int t0 = 0; t0 <= d; t0 += 32) {
                const int t = t0 + lane;
                int am = 0;
                bool stop = false;
                if (t <= d) {
                    unsigned long long key;
                    int dr;
                    if (t0 == 0) {
                        key = key_[r];
                        dr = dr_[r];
                    } else {
                        key = __ldcg(g.row_key + a + t);
                        dr = t < d ? g.draft_ids[(size_t)i * gamma + t] : -1;
                    }
                    g.row_key[a + t] = 0;
                    am = key ? (int)(0xffffffffu - (unsigned int)key)
                             : (g.logits ? slow_first_valid(g.logits + (size_t)(a + t) * g.V, g.V) : 0);
                    if (g.row_argmax) g.row_argmax[a + t] = am;
                    stop = (t == d) || am != dr;
                }
                const unsigned int mask = __ballot_sync(0xffffffffu, stop);
                if (m < 0 && mask) {
                    const int first = __ffs(mask) - 1;
                    m = t0 + first;
                    bon = __shfl_sync(0xffffffffu, am, first);
                }
            }
            if (lane == 0) {
                g.accept_len[i] = m;
                g.bonus[i] = bon;
                local += m + 1;
            }
            if (g.out_tokens) {
                int* o = g.out_tokens + (size_t)i * (gamma + 1);
                for (int t = lane; t <= gamma; t += 32)
                    o[t] = t < m ? ((t < 32 && t < d) ? dr_[r] : g.draft_ids[(size_t)i * gamma + t]) : (t == m ? bon : -1);
            }
        }
    }
    return local;
}

__global__ void __launch_bounds__(1024) accept_match_kernel(MatchArgs g) {
    __shared__ int total_s;
    if (threadIdx.x == 0) total_s = 0;
    __syncthreads();
    dcut_pdl_wait();
    dcut_pdl_launch_dependents();
    const int local = match_requests<kMatchR>(g, threadIdx.x >> 5, blockDim.x >> 5, threadIdx.x & 31);
    if (local) atomicAdd(&total_s, local);
    __syncthreads();
    if (threadIdx.x == 0 && g.n_accepted_total) *g.n_accepted_total = total_s;
}

}  // namespace

dcut_status dcut_init_accept(dcut_ctx* ctx) {
    (void)ctx;
    return DCUT_OK;
}

namespace {
MatchArgs match_args(const void* logits, int V, const int* draft_ids, const int* cu_q, int B, int gamma, int T_cap,
                     unsigned long long* row_key, int* accept_len, int* bonus, int* out_tokens, int* n_accepted_total,
                     int* row_argmax, int* status) {
    MatchArgs m;
    m.logits = static_cast<const unsigned short*>(logits);
    m.V = V;
    m.draft_ids = draft_ids;
    m.cu_q = cu_q;
    m.B = B;
    m.gamma = gamma;
    m.row_cap = T_cap;
    m.row_key = row_key;
    m.accept_len = accept_len;
    m.bonus = bonus;
    m.out_tokens = out_tokens;
    m.n_accepted_total = n_accepted_total;
    m.row_argmax = row_argmax;
    m.status = status;
    return m;
}
}  // namespace

dcut_status dcut_launch_accept(dcut_ctx* ctx, const void* logits, int V, const int* draft_ids,
                               const int* cu_q, int B, int gamma, int T_cap, int* accept_len, int* bonus,
                               int* out_tokens, int* n_accepted_total, unsigned long long* row_key,
                               cudaStream_t stream) {
    // segments: at least ~16 KB each, and enough CTAs for a few waves over the SMs
    const int want_ctas = ctx->sm_count * 16;
    int splits = (want_ctas + T_cap - 1) / T_cap;
    const int max_splits = (V + 8191) / 8192;
    if (splits > max_splits) splits = max_splits;
    if (splits < 1) splits = 1;
    int seg = (V + splits - 1) / splits;
    seg = (seg + 7) & ~7;
    splits = (V + seg - 1) / seg;
    dim3 grid(splits, T_cap);
    dcut_status st = dcut_check_cuda(ctx, dcut_launch_pdl(accept_argmax_kernel, grid, dim3(kArgmaxThreads), 0, stream,
                                                          static_cast<const unsigned short*>(logits), V, cu_q, B, seg, row_key),
                                     "launch accept_argmax_kernel");
    if (st != DCUT_OK) return st;
    return dcut_check_cuda(ctx, dcut_launch_pdl(accept_match_kernel, dim3(1), dim3(1024), 0, stream,
                                                match_args(logits, V, draft_ids, cu_q, B, gamma, T_cap, row_key, accept_len, bonus,
                                                           out_tokens, n_accepted_total, nullptr, ctx->d_status)),
                           "launch accept_match_kernel");
}

dcut_status dcut_launch_accept_match(dcut_ctx* ctx, const void* logits, int V, const int* draft_ids, const int* cu_q,
                                     int B, int gamma, int T_cap, int* accept_len, int* bonus, int* out_tokens,
                                     int* n_accepted_total, int* row_argmax, unsigned long long* row_key,
                                     cudaStream_t stream) {
    return dcut_check_cuda(ctx, dcut_launch_pdl(accept_match_kernel, dim3(1), dim3(1024), 0, stream,
                                                match_args(logits, V, draft_ids, cu_q, B, gamma, T_cap, row_key, accept_len, bonus,
                                                           out_tokens, n_accepted_total, row_argmax, ctx->d_status)),
                           "launch accept_match_kernel");
}

// ---------------------------------------------------------------------------------------------
// dcut_accept_static: the same two kernels, with the per-row words in a fixed device array that
// is part of the library image instead of a context allocation.

#include <mutex>
#include <stdio.h>

namespace {

// One 64-bit word per packed logits row.  Every GPU that loads this library carries these 64 KB
// until the process exits.
__device__ __align__(256) static unsigned long long g_static_row_key[DCUT_ACCEPT_STATIC_MAX_ROWS];

constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
unsigned long long* g_static_ptr[kMaxDevices];   // device address of g_static_row_key, per device ordinal
int g_static_sms[kMaxDevices];

void static_msg(char* buf, size_t len, const char* fmt, long long a = 0, long long b = 0) {
    if (buf && len) snprintf(buf, len, fmt, a, b);
}

}  // namespace

extern "C" dcut_status dcut_accept_static(const void* logits, int V, const int* draft_ids, const int* cu_q, int B,
                                          int gamma, int T_cap, int* accept_len, int* bonus, int* out_tokens,
                                          int* n_accepted_total, void* stream, char* errbuf, size_t errbuf_len) {
    if (!logits || !draft_ids || !cu_q || !accept_len || !bonus) {
        static_msg(errbuf, errbuf_len, "dcut_accept_static: null pointer argument");
        return DCUT_EINVAL;
    }
    if (B < 1 || gamma < 1 || V < 1 || T_cap < B) {
        static_msg(errbuf, errbuf_len, "dcut_accept_static: need B, gamma, V >= 1 and T_cap >= B");
        return DCUT_EINVAL;
    }
    if (reinterpret_cast<uintptr_t>(logits) & 1) {
        static_msg(errbuf, errbuf_len, "dcut_accept_static: logits must be 2-byte aligned");
        return DCUT_EINVAL;
    }
    if (T_cap > DCUT_ACCEPT_STATIC_MAX_ROWS || B > 1024 * 64) {
        static_msg(errbuf, errbuf_len,
                   "dcut_accept_static: T_cap = %lld packed rows exceed the fixed scratch of %lld rows; use dcut_accept",
                   T_cap, DCUT_ACCEPT_STATIC_MAX_ROWS);
        return DCUT_ECAPACITY;
    }
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        static_msg(errbuf, errbuf_len, "dcut_accept_static: cudaGetDevice failed or device ordinal %lld out of range", dev);
        return DCUT_ECUDA;
    }
    unsigned long long* keys = nullptr;
    int sms = 0;
    {
        // set-up, once per device and with that device current: in host code the array's name is only a
        // handle, so its device address has to be asked for before a kernel can be given it
        std::lock_guard<std::mutex> lock(g_static_mu);
        if (!g_static_ptr[dev]) {
            unsigned long long* p = nullptr;
            e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_row_key);
            if (e != cudaSuccess || !p) {
                static_msg(errbuf, errbuf_len, "dcut_accept_static: cudaGetSymbolAddress failed (error %lld)", (long long)e);
                return DCUT_ECUDA;
            }
            int n = 0;
            e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
            if (e != cudaSuccess || n < 1) {
                static_msg(errbuf, errbuf_len, "dcut_accept_static: cannot read the SM count (error %lld)", (long long)e);
                return DCUT_ECUDA;
            }
            g_static_sms[dev] = n;
            g_static_ptr[dev] = p;
        }
        keys = g_static_ptr[dev];
        sms = g_static_sms[dev];
    }
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    // the array keeps whatever the last call (of any caller) left: the words must start at zero
    e = cudaMemsetAsync(keys, 0, sizeof(unsigned long long) * (size_t)T_cap, cs);
    if (e != cudaSuccess) {
        static_msg(errbuf, errbuf_len, "dcut_accept_static: cudaMemsetAsync failed (error %lld)", (long long)e);
        return DCUT_ECUDA;
    }
    int splits = (sms * 16 + T_cap - 1) / T_cap;
    const int max_splits = (V + 8191) / 8192;
    if (splits > max_splits) splits = max_splits;
    if (splits < 1) splits = 1;
    int seg = (V + splits - 1) / splits;
    seg = (seg + 7) & ~7;
    splits = (V + seg - 1) / seg;
    dim3 grid(splits, T_cap);
    accept_argmax_kernel<<<grid, kArgmaxThreads, 0, cs>>>(static_cast<const unsigned short*>(logits), V, cu_q, B, seg, keys);
    if ((e = cudaGetLastError()) == cudaSuccess) {
        // rows at or past T_cap are never touched, so nothing outside the first T_cap words of the array is
        accept_match_kernel<<<1, 1024, 0, cs>>>(match_args(logits, V, draft_ids, cu_q, B, gamma, T_cap, keys, accept_len, bonus,
                                                          out_tokens, n_accepted_total, nullptr, nullptr));
        e = cudaGetLastError();
    }
    if (e != cudaSuccess) {
        static_msg(errbuf, errbuf_len, "dcut_accept_static: kernel launch failed (error %lld)", (long long)e);
        return DCUT_ECUDA;
    }
    return DCUT_OK;
}
