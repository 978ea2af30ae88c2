// dcut_accept_rs: rejection-sampling acceptance for the stochastic variant (Appendix B, "Causality under Rejection
// Sampling": accept draft z with probability min(1, p(z)/q(z)); on the first rejection draw from the residual
// distribution proportional to (p - q)+; if every retained draft is accepted, draw the bonus token from the next
// target distribution).  p = softmax of a target logits row, q = softmax of the matching draft logits row, both at
// temperature 1.  The random numbers are inputs.
//
// Three launches.
//   rs_stats_kernel    HBM-bound scan of the bf16 target rows [T, V] and of the draft rows that are in use
//       ((i, t) with t < d_i): every (segment, row) CTA produces the segment's (maximum, sum of exp(x - maximum)).
//   rs_decide_kernel   one warp per request: merges the segments of its rows, walks the drafts in order
//       (u * q(z) < p(z) accepts) and records which distribution ends the request's step.
//   rs_sample_kernel   one CTA per request: inversion sampling over ascending token index from (p - q)+ of the
//       rejected position, or from p of the row after the last accepted draft.  Thread t owns the t-th contiguous
//       slice of the vocabulary; slice sums are scanned in double, the slice that holds u * total is rescanned.
#include "dcut_internal.h"

namespace {

constexpr int kStatThreads = 256;
constexpr int kSampleThreads = 1024;

__device__ __forceinline__ uint4 ld_stream_v4(const uint4* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.L2::256B.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}
__device__ __forceinline__ float bf_at(const unsigned short* p, int v) { return __uint_as_float((unsigned int)p[v] << 16); }

struct RsArgs {
    const unsigned short* target;   // [T, V]
    const unsigned short* draft;    // [B, gamma, V]
    const int* draft_ids;
    const int* cu_q;
    const float* u_accept;          // [B, gamma]
    const float* u_sample;          // [B]
    int V, B, gamma, n_seg, seg_elems;
    float2* stats;                  // [(T_cap + B * gamma) * n_seg]: (max, sum) per segment; draft rows after the target rows
    int T_cap;
    int4* job;                      // [B]: x = target row, y = draft row (-1: sample from p), z = accept_len
    float4* job_stats;              // [B]: (max_p, sum_p, max_q, sum_q) of the job's rows
    int* accept_len;
    int* bonus;
    int* out_tokens;
    int* n_accepted_total;
    float* prob;                    // [B, 2] or null: p(z)/q(z) of the deciding draft, residual mass
};

// (max, sum) of one segment of one row.  Rows: [0, T) target rows; T_cap + i * gamma + t: draft row (i, t), only t < d_i.
__global__ void __launch_bounds__(kStatThreads) rs_stats_kernel(RsArgs a) {
    const int row = blockIdx.y, seg = blockIdx.x;
    const unsigned short* rp;
    if (row < a.T_cap) {
        if (row >= a.cu_q[a.B]) return;
        rp = a.target + (size_t)row * a.V;
    } else {
        const int e = row - a.T_cap, i = e / a.gamma, t = e - i * a.gamma;
        if (t >= a.cu_q[i + 1] - a.cu_q[i] - 1) return;
        rp = a.draft + (size_t)e * a.V;
    }
    const int start = seg * a.seg_elems, end = min(a.V, start + a.seg_elems);
    float m = -INFINITY, s = 0.0f;
    auto take = [&](float x) {
        if (x > m) {
            s = s * __expf(m - x) + 1.0f;   // m = -inf: s is 0, the product is 0 * 0
            m = x;
        } else if (x == x && x > -INFINITY) {   // NaN and -inf carry no mass
            s += __expf(x - m);
        }
    };
    if (start < end) {
        // vector part over the 16-byte aligned middle, scalar head and tail
        const uintptr_t base = reinterpret_cast<uintptr_t>(rp + start);
        int head = (int)(((16 - (base & 15)) & 15) >> 1);
        if (head > end - start) head = end - start;
        for (int v = start + threadIdx.x; v < start + head; v += kStatThreads) take(bf_at(rp, v));
        const int nvec = (end - start - head) >> 3;
        const uint4* vp = reinterpret_cast<const uint4*>(rp + start + head);
        for (int k = threadIdx.x; k < nvec; k += kStatThreads) {
            const uint4 w = ld_stream_v4(vp + k);
            const unsigned int ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                take(__uint_as_float(ws[e] << 16));
                take(__uint_as_float(ws[e] & 0xffff0000u));
            }
        }
        for (int v = start + head + nvec * 8 + threadIdx.x; v < end; v += kStatThreads) take(bf_at(rp, v));
    }
    // merge over the CTA
    auto merge = [](float& m1, float& s1, float m2, float s2) {
        const float mm = fmaxf(m1, m2);
        if (mm == -INFINITY) return;
        s1 = s1 * __expf(m1 - mm) + s2 * __expf(m2 - mm);
        m1 = mm;
    };
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
        merge(m, s, m2, s2);
    }
    __shared__ float2 wp[kStatThreads / 32];
    if ((threadIdx.x & 31) == 0) wp[threadIdx.x >> 5] = make_float2(m, s);
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kStatThreads / 32; ++w) merge(m, s, wp[w].x, wp[w].y);
        a.stats[(size_t)row * a.n_seg + seg] = make_float2(m, s);
    }
}

__device__ __forceinline__ float2 row_stats(const RsArgs& a, int row) {
    float m = -INFINITY, s = 0.0f;
    for (int g = 0; g < a.n_seg; ++g) {
        const float2 p = a.stats[(size_t)row * a.n_seg + g];
        const float mm = fmaxf(m, p.x);
        if (mm == -INFINITY) continue;
        s = s * __expf(m - mm) + p.y * __expf(p.x - mm);
        m = mm;
    }
    return make_float2(m, s);
}

// One warp per request; lane t looks at draft t + 1, a ballot finds the first rejection.
__global__ void __launch_bounds__(1024) rs_decide_kernel(RsArgs a) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    for (int i = warp; i < a.B; i += n_warps) {
        const int r0 = a.cu_q[i], d = a.cu_q[i + 1] - r0 - 1;
        int m = d;
        float ratio = 0.0f;
        float4 st = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int t0 = 0; t0 < d && m == d; t0 += 32) {
            const int t = t0 + lane;
            bool reject = false;
            float my_ratio = 0.0f;
            float4 my_st = make_float4(0.f, 0.f, 0.f, 0.f);
            if (t < d) {
                const float2 sp = row_stats(a, r0 + t), sq = row_stats(a, a.T_cap + i * a.gamma + t);
                const int z = min(max(a.draft_ids[(size_t)i * a.gamma + t], 0), a.V - 1);
                const float pz = __expf(bf_at(a.target + (size_t)(r0 + t) * a.V, z) - sp.x) / sp.y;
                const float qz = __expf(bf_at(a.draft + ((size_t)i * a.gamma + t) * a.V, z) - sq.x) / sq.y;
                reject = !(a.u_accept[(size_t)i * a.gamma + t] * qz < pz);
                my_ratio = pz / qz;
                my_st = make_float4(sp.x, sp.y, sq.x, sq.y);
            }
            const unsigned int mask = __ballot_sync(0xffffffffu, reject);
            const int src = mask ? __ffs(mask) - 1 : min(31, d - 1 - t0);   // first rejection, else the last draft seen
            ratio = __shfl_sync(0xffffffffu, my_ratio, src);
            st.x = __shfl_sync(0xffffffffu, my_st.x, src);
            st.y = __shfl_sync(0xffffffffu, my_st.y, src);
            st.z = __shfl_sync(0xffffffffu, my_st.z, src);
            st.w = __shfl_sync(0xffffffffu, my_st.w, src);
            if (mask) m = t0 + src;
        }
        if (lane == 0) {
            int4 job;
            job.z = m;
            job.w = 0;
            if (m < d) {           // rejected at draft m + 1: residual of target row r0 + m and draft row (i, m)
                job.x = r0 + m;
                job.y = i * a.gamma + m;
            } else {               // all accepted (or d = 0): bonus from the target row after the last draft
                job.x = r0 + d;
                job.y = -1;
                const float2 sp = row_stats(a, r0 + d);
                st = make_float4(sp.x, sp.y, 0.f, 0.f);
            }
            a.job[i] = job;
            a.job_stats[i] = st;
            a.accept_len[i] = m;
            if (a.prob) a.prob[2 * i] = ratio;
        }
    }
}

template <typename T>
__device__ __forceinline__ T block_exclusive_scan_d(T v, T* ws, T* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    T inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const T u = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += u;
    }
    if (lane == 31) ws[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        T w = ws[lane];
        T winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const T u = __shfl_up_sync(0xffffffffu, winc, o);
            if (lane >= o) winc += u;
        }
        ws[lane] = winc - w;
        if (lane == 31) ws[32] = winc;
    }
    __syncthreads();
    const T res = ws[warp] + inc - v;
    *total = ws[32];
    __syncthreads();
    return res;
}

// One CTA per request: the token that ends the request's step.
__global__ void __launch_bounds__(kSampleThreads) rs_sample_kernel(RsArgs a) {
    const int i = blockIdx.x;
    const int4 job = a.job[i];
    const float4 st = a.job_stats[i];
    const unsigned short* tp = a.target + (size_t)job.x * a.V;
    const unsigned short* dp = job.y >= 0 ? a.draft + (size_t)job.y * a.V : nullptr;
    __shared__ double ws[33];
    __shared__ int found_s, last_s;
    const int per = (a.V + kSampleThreads - 1) / kSampleThreads;
    const int v0 = min(a.V, (int)threadIdx.x * per), v1 = min(a.V, v0 + per);
    const float inv_p = 1.0f / st.y, inv_q = dp ? 1.0f / st.w : 0.0f;
    bool use_p = dp == nullptr;
    for (int round = 0; round < 2; ++round) {
        auto weight = [&](int v) -> float {
            const float p = __expf(bf_at(tp, v) - st.x) * inv_p;
            if (use_p) return p == p ? p : 0.0f;
            const float q = __expf(bf_at(dp, v) - st.z) * inv_q;
            const float r = p - q;
            return r > 0.0f ? r : 0.0f;
        };
        if (threadIdx.x == 0) {
            found_s = a.V;
            last_s = -1;
        }
        double local = 0.0;
        int my_last = -1;
        for (int v = v0; v < v1; ++v) {
            const float w = weight(v);
            local += (double)w;
            if (w > 0.0f) my_last = v;
        }
        double total;
        const double before = block_exclusive_scan_d<double>(local, ws, &total);   // also orders the writes above
        if (my_last >= 0) atomicMax(&last_s, my_last);
        if (!(total > 0.0)) {
            // (p - q)+ vanished in this precision: the same draw from p (once)
            if (use_p) break;
            use_p = true;
            continue;
        }
        const double target = (double)a.u_sample[i] * total;
        if (target >= before && target < before + local) {
            double run = before;
            for (int v = v0; v < v1; ++v) {
                run += (double)weight(v);
                if (run > target) {
                    atomicMin(&found_s, v);
                    break;
                }
            }
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            const int tok = found_s < a.V ? found_s : max(last_s, 0);   // rounding left the running sum at the target
            const int m = job.z;
            a.bonus[i] = tok;
            if (a.prob) a.prob[2 * i + 1] = (dp && !use_p) ? (float)total : 0.0f;   // residual mass
            if (a.out_tokens) {
                int* o = a.out_tokens + (size_t)i * (a.gamma + 1);
                for (int t = 0; t <= a.gamma; ++t) o[t] = t < m ? a.draft_ids[(size_t)i * a.gamma + t] : (t == m ? tok : -1);
            }
            if (a.n_accepted_total) atomicAdd(a.n_accepted_total, m + 1);
        }
        return;
    }
    // no positive weight at all (a row of NaN): token 0
    if (threadIdx.x == 0) {
        a.bonus[i] = 0;
        if (a.prob) a.prob[2 * i + 1] = 0.0f;
        if (a.out_tokens) {
            int* o = a.out_tokens + (size_t)i * (a.gamma + 1);
            for (int t = 0; t <= a.gamma; ++t) o[t] = t < job.z ? a.draft_ids[(size_t)i * a.gamma + t] : (t == job.z ? 0 : -1);
        }
        if (a.n_accepted_total) atomicAdd(a.n_accepted_total, job.z + 1);
    }
}

}  // namespace

// scratch layout: per-segment statistics (rounded up to 16 bytes: the job records behind them are 16-byte vectors),
// then one int4 and one float4 per request
static size_t rs_stats_bytes(const dcut_ctx* ctx, int n_seg) {
    const size_t rows = (size_t)ctx->lim.max_B * (ctx->lim.max_gamma + 1) + (size_t)ctx->lim.max_B * ctx->lim.max_gamma;
    return (rows * n_seg * sizeof(float2) + 15) & ~(size_t)15;
}

size_t dcut_accept_rs_scratch_bytes(const dcut_ctx* ctx, int n_seg) {
    return rs_stats_bytes(ctx, n_seg) + (size_t)ctx->lim.max_B * (sizeof(int4) + sizeof(float4));
}

dcut_status dcut_launch_accept_rs(dcut_ctx* ctx, const void* target_logits, const void* draft_logits, int V,
                                  const int* draft_ids, const int* cu_q, int B, int gamma, int T_cap,
                                  const float* u_accept, const float* u_sample, int* accept_len, int* bonus,
                                  int* out_tokens, int* n_accepted_total, float* prob, cudaStream_t stream) {
    RsArgs a;
    a.target = static_cast<const unsigned short*>(target_logits);
    a.draft = static_cast<const unsigned short*>(draft_logits);
    a.draft_ids = draft_ids;
    a.cu_q = cu_q;
    a.u_accept = u_accept;
    a.u_sample = u_sample;
    a.V = V;
    a.B = B;
    a.gamma = gamma;
    a.n_seg = ctx->rs_n_seg;
    a.seg_elems = ((V + a.n_seg - 1) / a.n_seg + 7) & ~7;
    a.T_cap = T_cap;
    unsigned char* base = static_cast<unsigned char*>(ctx->d_rs_scratch);
    a.stats = reinterpret_cast<float2*>(base);
    a.job = reinterpret_cast<int4*>(base + rs_stats_bytes(ctx, a.n_seg));
    a.job_stats = reinterpret_cast<float4*>(reinterpret_cast<unsigned char*>(a.job) + (size_t)ctx->lim.max_B * sizeof(int4));
    a.accept_len = accept_len;
    a.bonus = bonus;
    a.out_tokens = out_tokens;
    a.n_accepted_total = n_accepted_total;
    a.prob = prob;
    if (n_accepted_total) {
        dcut_status st = dcut_check_cuda(ctx, cudaMemsetAsync(n_accepted_total, 0, sizeof(int), stream), "cudaMemsetAsync(total)");
        if (st != DCUT_OK) return st;
    }
    dim3 grid(a.n_seg, T_cap + B * gamma);
    rs_stats_kernel<<<grid, kStatThreads, 0, stream>>>(a);
    dcut_status st = dcut_check_cuda(ctx, cudaGetLastError(), "launch rs_stats_kernel");
    if (st != DCUT_OK) return st;
    rs_decide_kernel<<<1, 1024, 0, stream>>>(a);
    if ((st = dcut_check_cuda(ctx, cudaGetLastError(), "launch rs_decide_kernel")) != DCUT_OK) return st;
    rs_sample_kernel<<<B, kSampleThreads, 0, stream>>>(a);
    return dcut_check_cuda(ctx, cudaGetLastError(), "launch rs_sample_kernel");
}
