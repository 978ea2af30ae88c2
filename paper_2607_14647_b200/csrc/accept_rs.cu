// dcut_accept_rs: rejection-sampling acceptance for the stochastic variant (Appendix B, "Causality under Rejection
// Sampling": accept draft z with probability min(1, p(z)/q(z)); on the first rejection draw from the residual
// distribution proportional to (p - q)+; if every retained draft is accepted, draw the bonus token from the next
// target distribution).  p = softmax of a target logits row, q = softmax of the matching draft logits row, both at
// temperature 1.  The random numbers are inputs.
//
// Two launches (programmatic dependent launch).
//   rs_stats_kernel    HBM-bound scan of the bf16 target rows [T, V] and of the draft rows that are in use
//       ((i, t) with t < d_i): every (segment, row) CTA produces the segment's (maximum, sum of exp(x - maximum)).
//   rs_sample_kernel   one CTA per request.  Its first warp merges the segments of the request's rows, walks the
//       drafts in order (u * q(z) < p(z) accepts) and finds which distribution ends the request's step; the CTA then
//       draws from it by inversion over ascending token index: (p - q)+ of the rejected position, or p of the row
//       after the last accepted draft.  The vocabulary is cut into chunks of 256 tokens; chunk sums are scanned in
//       double, the chunk that holds u * total is rescanned.
#include "dcut_internal.h"

namespace {

constexpr int kStatThreads = 256;
constexpr int kUnroll = 4;
constexpr int kSampleThreads = 256;

__device__ __forceinline__ uint4 ld_stream_v4(const uint4* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.L2::256B.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}
__device__ __forceinline__ float exp2f_fast(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
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
    int* accept_len;
    int* bonus;
    int* out_tokens;
    int* n_accepted_total;
    float* prob;                    // [B, 2] or null: p(z)/q(z) of the deciding draft, residual mass
    double* chunk_sums;             // [B, kMaxChunks] weight of every 256-token chunk of the request's deciding distribution
    int* tickets;                   // [B] parts of the request that have stored their chunk sums (0 between calls)
    int* last_tok;                  // [B] last token with positive weight (-1 between calls)
    int n_parts;                    // CTAs per request in rs_sample_kernel
};

// (max, sum) of one segment of one row.  Rows: [0, T) target rows; T_cap + i * gamma + t: draft row (i, t), only t < d_i.
__global__ void __launch_bounds__(kStatThreads) rs_stats_kernel(RsArgs a) {
    dcut_pdl_wait();
    dcut_pdl_launch_dependents();   // rs_sample_kernel still waits for this grid to finish before it reads the statistics
    const int row = blockIdx.y, seg = blockIdx.x;
    if (row == 0 && seg == 0 && threadIdx.x == 0 && a.n_accepted_total) *a.n_accepted_total = 0;
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
    auto take = [&](float x) {           // scalar head / tail elements
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
        for (int k0 = 0; k0 < nvec; k0 += kUnroll * kStatThreads) {
            // up to four 16-byte vectors in flight per thread, one rescale of the running sum per batch, no
            // data-dependent branch (vectors past the end repeat -inf, which adds nothing)
            uint4 w[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const int k = k0 + u * kStatThreads + threadIdx.x;
                w[u] = k < nvec ? ld_stream_v4(vp + k) : make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
            }
            // Two values per word: NaN is turned into -inf (weight 0) and the batch maximum is taken on the packed
            // words (max.bf16x2 returns the other operand for a NaN), one instruction per two values each
            float x[8 * kUnroll];
            unsigned int wmax = 0xff80ff80u;
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const unsigned int ws[4] = {w[u].x, w[u].y, w[u].z, w[u].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    unsigned int c;
                    asm("max.bf16x2 %0, %1, %2;" : "=r"(c) : "r"(ws[e]), "r"(0xff80ff80u));
                    asm("max.bf16x2 %0, %1, %2;" : "=r"(wmax) : "r"(wmax), "r"(c));
                    x[8 * u + 2 * e] = __uint_as_float(c << 16);
                    x[8 * u + 2 * e + 1] = __uint_as_float(c & 0xffff0000u);
                }
            }
            const float vmax = fmaxf(__uint_as_float(wmax << 16), __uint_as_float(wmax & 0xffff0000u));
            const float mn = fmaxf(m, vmax);
            if (mn > -INFINITY) {
                // exp(x - mn) = 2^(x * log2(e) - mn * log2(e)): one FMA, one special-function operation, one add per
                // value; two partial sums for instruction-level parallelism
                const float kL2e = 1.4426950408889634f, off = -mn * kL2e;
                float add0 = 0.0f, add1 = 0.0f;
#pragma unroll
                for (int e = 0; e < 8 * kUnroll; e += 2) {
                    add0 += exp2f_fast(fmaf(x[e], kL2e, off));
                    add1 += exp2f_fast(fmaf(x[e + 1], kL2e, off));
                }
                s = s * __expf(m - mn) + (add0 + add1);
                m = mn;
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

// Decision for request i by one warp: lane t looks at draft t + 1, a ballot finds the first rejection.  Returns (in every
// lane) the job: x = target row, y = draft row (-1: the draw comes from p), z = accept_len; st = (max_p, sum_p, max_q, sum_q).
__device__ __forceinline__ int4 rs_decide(const RsArgs& a, int i, float4& st, float& ratio) {
    const int lane = threadIdx.x & 31;
    const int r0 = a.cu_q[i], d = a.cu_q[i + 1] - r0 - 1;
    int m = d;
    ratio = 0.0f;
    st = make_float4(0.f, 0.f, 0.f, 0.f);
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
    return job;
}

// One request = n_parts CTAs.  The vocabulary is cut into chunks of 256 tokens; every warp of every part sums the chunks
// assigned to it (16-byte loads, lane l holds tokens 8l .. 8l+7 of the chunk) and stores the sums; the part that
// finishes last (a ticket per request) scans the chunk sums in double and one of its warps rescans the chunk that holds
// u * total.  Chunk sums, scan order and the rescan do not depend on which part does what, so the draw is reproducible.
constexpr int kChunk = 256;
constexpr int kMaxChunks = 1024;   // vocabularies up to 262 144 tokens
constexpr int kBatch = 8;
constexpr int kSampleWarps = kSampleThreads / 32;
constexpr int kPerThread = kMaxChunks / kSampleThreads;

__global__ void __launch_bounds__(kSampleThreads) rs_sample_kernel(RsArgs a) {
    dcut_pdl_wait();
    dcut_pdl_launch_dependents();
    const int i = blockIdx.y, part = blockIdx.x;
    __shared__ int4 job_s;
    __shared__ float4 st_s;
    __shared__ double ws[kSampleWarps + 1];
    __shared__ double base_s;
    __shared__ int found_s, last_s, ticket_s;
    if (threadIdx.x < 32) {           // every part takes the (cheap) decision for itself
        float4 st0;
        float ratio;
        const int4 job0 = rs_decide(a, i, st0, ratio);
        if (threadIdx.x == 0) {
            job_s = job0;
            st_s = st0;
            last_s = -1;
            if (part == 0) {
                a.accept_len[i] = job0.z;
                if (a.prob) a.prob[2 * i] = ratio;
            }
        }
    }
    __syncthreads();
    const int4 job = job_s;
    const float4 st = st_s;
    const unsigned short* tp = a.target + (size_t)job.x * a.V;
    const unsigned short* dp = job.y >= 0 ? a.draft + (size_t)job.y * a.V : nullptr;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n_chunks = (a.V + kChunk - 1) / kChunk;
    const float inv_p = 1.0f / st.y, inv_q = dp ? 1.0f / st.w : 0.0f;
    const bool vec_ok = (a.V & 7) == 0 && (reinterpret_cast<uintptr_t>(a.target) & 15) == 0 &&
                        (reinterpret_cast<uintptr_t>(a.draft) & 15) == 0;   // every row then starts on 16 bytes
    double* csum = a.chunk_sums + (size_t)i * kMaxChunks;
    bool use_p = dp == nullptr;

    auto weight = [&](int v) -> float {
        const float p = __expf(bf_at(tp, v) - st.x) * inv_p;
        if (use_p) return p == p ? p : 0.0f;
        const float q = __expf(bf_at(dp, v) - st.z) * inv_q;
        const float r = p - q;
        return r > 0.0f ? r : 0.0f;
    };
    // the eight weights of this lane in chunk c, in token order; tv / dv: the lane's 16 bytes of the two rows if `vec`
    auto chunk_is_vec = [&](int c) { return vec_ok && c * kChunk + lane * 8 + 8 <= a.V; };
    auto weights_of = [&](int c, bool vec, const uint4& tv, const uint4& dv, float (&w)[8]) {
        const int v0 = c * kChunk + lane * 8;
        if (vec) {
            const unsigned int tw[4] = {tv.x, tv.y, tv.z, tv.w}, dw[4] = {dv.x, dv.y, dv.z, dv.w};
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float xt = __uint_as_float((e & 1) ? (tw[e >> 1] & 0xffff0000u) : (tw[e >> 1] << 16));
                const float p = __expf(xt - st.x) * inv_p;
                if (use_p) {
                    w[e] = p == p ? p : 0.0f;
                } else {
                    const float xd = __uint_as_float((e & 1) ? (dw[e >> 1] & 0xffff0000u) : (dw[e >> 1] << 16));
                    const float r = p - __expf(xd - st.z) * inv_q;
                    w[e] = r > 0.0f ? r : 0.0f;
                }
            }
            return;
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) w[e] = v0 + e < a.V ? weight(v0 + e) : 0.0f;
    };
    auto lane_weights = [&](int c, float (&w)[8]) {
        uint4 tv = make_uint4(0, 0, 0, 0), dv = make_uint4(0, 0, 0, 0);
        const bool vec = chunk_is_vec(c);
        if (vec) {
            tv = *reinterpret_cast<const uint4*>(tp + c * kChunk + lane * 8);
            if (!use_p) dv = *reinterpret_cast<const uint4*>(dp + c * kChunk + lane * 8);
        }
        weights_of(c, vec, tv, dv, w);
    };
    // chunk sums of the chunks first, first + step, ...: lane 31 of the warp stores each; the last token with weight.
    // The loads of kBatch chunks are issued before the first of them is used.
    auto sum_chunks = [&](int first, int step) {
        int my_last = -1;
        for (int c0 = first; c0 < n_chunks; c0 += step * kBatch) {
            uint4 tv[kBatch], dv[kBatch];
#pragma unroll
            for (int k = 0; k < kBatch; ++k) {
                const int c = c0 + k * step;
                tv[k] = dv[k] = make_uint4(0, 0, 0, 0);
                if (c < n_chunks && chunk_is_vec(c)) {
                    tv[k] = ld_stream_v4(reinterpret_cast<const uint4*>(tp + c * kChunk + lane * 8));
                    if (!use_p) dv[k] = ld_stream_v4(reinterpret_cast<const uint4*>(dp + c * kChunk + lane * 8));
                }
            }
#pragma unroll
            for (int k = 0; k < kBatch; ++k) {
                const int c = c0 + k * step;
                if (c >= n_chunks) break;
                float w[8];
                weights_of(c, chunk_is_vec(c), tv[k], dv[k], w);
                double part_sum = 0.0;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    part_sum += (double)w[e];
                    if (w[e] > 0.0f) my_last = c * kChunk + lane * 8 + e;
                }
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {   // inclusive scan over the lanes (fixed order), lane 31 ends with the chunk sum
                    const double u = __shfl_up_sync(0xffffffffu, part_sum, o);
                    if (lane >= o) part_sum += u;
                }
                if (lane == 31) __stcg(csum + c, part_sum);
            }
        }
        if (my_last >= 0) atomicMax(&last_s, my_last);
    };

    sum_chunks(part * kSampleWarps + warp, a.n_parts * kSampleWarps);
    __syncthreads();
    if (threadIdx.x == 0) {
        if (last_s >= 0) atomicMax(a.last_tok + i, last_s);
        __threadfence();                                   // the sums and the maximum before the ticket
        ticket_s = atomicAdd(a.tickets + i, 1);
    }
    __syncthreads();
    if (ticket_s != a.n_parts - 1) return;
    __threadfence();

    // ---- the last part of the request: scan, locate, rescan
    int tok = 0;
    double mass = 0.0;
    for (int round = 0; round < 2; ++round) {
        if (round == 1) {            // (p - q)+ vanished in this precision: the same draw from p, all chunks here
            if (threadIdx.x == 0) last_s = -1;
            __syncthreads();
            sum_chunks(warp, kSampleWarps);
            __syncthreads();
            if (threadIdx.x == 0) a.last_tok[i] = last_s;
        }
        if (threadIdx.x == 0) found_s = n_chunks;
        // thread t owns the chunks kPerThread * t ..: their sums, an exclusive scan over the threads in double
        double mine[kPerThread], own = 0.0;
#pragma unroll
        for (int k = 0; k < kPerThread; ++k) {
            const int c = threadIdx.x * kPerThread + k;
            mine[k] = c < n_chunks ? __ldcg(csum + c) : 0.0;
            own += mine[k];
        }
        double inc = own;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const double u = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += u;
        }
        if (lane == 31) ws[warp] = inc;
        __syncthreads();
        if (threadIdx.x == 0) {
            double run = 0.0;
            for (int w = 0; w < kSampleWarps; ++w) {
                const double t = ws[w];
                ws[w] = run;
                run += t;
            }
            ws[kSampleWarps] = run;
        }
        __syncthreads();
        const double total = ws[kSampleWarps];
        double before = ws[warp] + inc - own;
        if (!(total > 0.0)) {
            if (use_p) break;        // no positive weight at all (a row of NaN): token 0
            use_p = true;
            __syncthreads();
            continue;
        }
        const double target = (double)a.u_sample[i] * total;
#pragma unroll
        for (int k = 0; k < kPerThread; ++k) {
            const int c = threadIdx.x * kPerThread + k;
            if (c < n_chunks && target >= before && target < before + mine[k]) {
                found_s = c;         // at most one chunk satisfies both (the intervals are disjoint)
                base_s = before;
            }
            before += mine[k];
        }
        __syncthreads();
        mass = (dp && !use_p) ? total : 0.0;
        const int c = found_s;
        tok = max(__ldcg(a.last_tok + i), 0);   // if rounding left the running sum at the target: the last token with weight
        if (c < n_chunks && warp == 0) {
            float w[8];
            lane_weights(c, w);
            double part_sum = 0.0;
#pragma unroll
            for (int e = 0; e < 8; ++e) part_sum += (double)w[e];
            double linc = part_sum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double u = __shfl_up_sync(0xffffffffu, linc, o);
                if (lane >= o) linc += u;
            }
            double run = base_s + linc - part_sum;     // weight before this lane's first token
            int hit = -1;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                run += (double)w[e];
                if (hit < 0 && run > target) hit = c * kChunk + lane * 8 + e;
            }
            const unsigned int mask = __ballot_sync(0xffffffffu, hit >= 0);
            if (mask) tok = __shfl_sync(0xffffffffu, hit, __ffs(mask) - 1);
        }
        break;
    }
    if (threadIdx.x == 0) {
        const int m = job.z;
        a.bonus[i] = tok;
        if (a.prob) a.prob[2 * i + 1] = (float)mass;   // residual mass (0 when the draw came from p)
        if (a.out_tokens) {
            int* o = a.out_tokens + (size_t)i * (a.gamma + 1);
            for (int t = 0; t <= a.gamma; ++t) o[t] = t < m ? a.draft_ids[(size_t)i * a.gamma + t] : (t == m ? tok : -1);
        }
        if (a.n_accepted_total) atomicAdd(a.n_accepted_total, m + 1);
        a.tickets[i] = 0;            // ready for the next call on this stream
        a.last_tok[i] = -1;
    }
}

}  // namespace

// scratch layout: per-segment statistics (rounded up to 16 bytes), the chunk sums of every request, tickets, last tokens
static size_t rs_stats_bytes(const dcut_ctx* ctx, int n_seg) {
    const size_t rows = (size_t)ctx->lim.max_B * (ctx->lim.max_gamma + 1) + (size_t)ctx->lim.max_B * ctx->lim.max_gamma;
    return (rows * n_seg * sizeof(float2) + 15) & ~(size_t)15;
}

size_t dcut_accept_rs_scratch_bytes(const dcut_ctx* ctx, int n_seg) {
    return rs_stats_bytes(ctx, n_seg) + (size_t)ctx->lim.max_B * (kMaxChunks * sizeof(double) + 2 * sizeof(int));
}

// tickets = 0 and last tokens = -1: the state rs_sample_kernel expects and leaves behind
dcut_status dcut_init_accept_rs(dcut_ctx* ctx) {
    unsigned char* base = static_cast<unsigned char*>(ctx->d_rs_scratch) + rs_stats_bytes(ctx, ctx->rs_n_seg) +
                          (size_t)ctx->lim.max_B * kMaxChunks * sizeof(double);
    dcut_status st = dcut_check_cuda(ctx, cudaMemset(base, 0, sizeof(int) * ctx->lim.max_B), "cudaMemset(rs tickets)");
    if (st != DCUT_OK) return st;
    return dcut_check_cuda(ctx, cudaMemset(base + sizeof(int) * ctx->lim.max_B, 0xff, sizeof(int) * ctx->lim.max_B), "cudaMemset(rs last)");
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
    // segments: enough CTAs for a few waves over the SMs, at least ~16 KB each, at most what the scratch was sized for
    const int n_rows = T_cap + B * gamma;
    int n_seg = (ctx->sm_count * 16 + n_rows - 1) / n_rows;
    const int max_seg = (V + 8191) / 8192;
    if (n_seg > max_seg) n_seg = max_seg;
    if (n_seg > ctx->rs_n_seg) n_seg = ctx->rs_n_seg;
    if (n_seg < 1) n_seg = 1;
    a.seg_elems = ((V + n_seg - 1) / n_seg + 7) & ~7;
    a.n_seg = (V + a.seg_elems - 1) / a.seg_elems;
    a.T_cap = T_cap;
    unsigned char* base = static_cast<unsigned char*>(ctx->d_rs_scratch);
    a.stats = reinterpret_cast<float2*>(base);
    a.chunk_sums = reinterpret_cast<double*>(base + rs_stats_bytes(ctx, ctx->rs_n_seg));
    a.tickets = reinterpret_cast<int*>(a.chunk_sums + (size_t)ctx->lim.max_B * kMaxChunks);
    a.last_tok = a.tickets + ctx->lim.max_B;
    // Four CTAs per request: each CTA starts with the request's decision (a chain of dependent loads of a few
    // microseconds), so what counts is that all CTAs are resident at once and few, not that each has little to sum
    // (measured at B = 64, V = 151 936, both kernels: 1 part 183 us, 2: 152, 4: 140, 8: 144, 16: 150, 32: 162).
    a.n_parts = 4;
    a.accept_len = accept_len;
    a.bonus = bonus;
    a.out_tokens = out_tokens;
    a.n_accepted_total = n_accepted_total;
    a.prob = prob;
    dcut_status st = dcut_check_cuda(ctx, dcut_launch_pdl(rs_stats_kernel, dim3(a.n_seg, T_cap + B * gamma), dim3(kStatThreads), 0, stream, a),
                                     "launch rs_stats_kernel");
    if (st != DCUT_OK) return st;
    return dcut_check_cuda(ctx, dcut_launch_pdl(rs_sample_kernel, dim3(a.n_parts, B), dim3(kSampleThreads), 0, stream, a),
                           "launch rs_sample_kernel");
}
