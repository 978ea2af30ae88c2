// Work partition of the verification attention, as a device function that runs in ONE CTA: the stand-alone
// attn_plan_kernel of dcut_verify_attn, or the tail of the selector kernel, which has just written cu_q and can leave
// the partition ready for the attention call that follows (dcut_enable_plan_in_select).
//
// The work of a call is a stream of (request, row block, kv head) items, each a run of KV pages; its cost is known
// up front (pages x a per-page weight that depends on how the item runs, plus a fixed cost per item).  The stream is
// cut into one segment of equal cost per SM: a CTA of the persistent item kernel owns a contiguous piece of the
// stream, which may begin or end in the middle of an item.  An item that a boundary cuts is computed in pieces (one
// per segment it touches) whose partial results the combine kernel merges; at most one item is cut per boundary, so
// there are fewer cut items than SMs whatever the batch.  This replaces both the split of long contexts into chunks
// for small batches and a dynamic item queue: every SM ends within the cost model's error of every other, and the
// assignment (hence the rounding of every result) is the same on every run.
//
// The plan only writes the table of entries (one per (request, row block): n_kv_heads items of equal cost) and the
// n_sm + 1 segment boundaries; the item kernel walks its segment and builds its items on the fly.
#pragma once

#include "dcut_internal.h"

namespace dcut_plan {

constexpr int kPage = 16;            // tokens per page
constexpr int kSlotRows = 144;       // rows of a partial-result slot (the largest query tile of an item)
constexpr int kMaxSegs = 256;        // segments (SMs) the plan handles

// Cost model, nanoseconds on B200, fitted to the busy time of the item kernel's CTAs (`%globaltimer` at the start and
// the end of every CTA) against the items and pages of their segments by class of item (least squares over the 148
// CTAs of batches with random depths).  With every SM streaming, a page costs about what the shared HBM gives each SM;
// what differs is how many softmax warps share schedulers with the producer and the MMA issuer.  tcgen05 phase, query
// tiles of up to 96 rows (lane quarter 1 of tensor memory empty, so the issuer has its scheduler to itself): 178 per
// page (fits 178-179 for tiles of <= 32, <= 64, <= 96 rows); 97-128 rows: 197; with tail rows: 204; warp-level phase:
// as the short tiles (163-170 against 166 in the same batches).  Per item, beyond its pages: 3.2-3.8 us up to 96 rows,
// 4.7 to 128, 5.6-7.5 with tail rows (O is single-buffered in tensor memory and the softmax -> PV chain drains at an
// item boundary; the tail warps add their merge), 3.6-4.3 us on the warp-level phase next to tcgen05 CTAs.  Only
// ratios matter for the partition.  With one cost for all tiles up to 128 rows, CTAs whose items had 97-128 rows
// finished 8 % after the mean on workload 3 with mixed depths.
__device__ __forceinline__ int cost_per_page(int rows, int tc) {
    if (tc) return rows > 128 ? 204 : (rows > 96 ? 197 : 178);
    const int mt = (rows + 15) >> 4;                       // m-tiles of the warp-level phase: memory-bound up to two
    return 178 * max(7, 3 * mt) / 7;
}
__device__ __forceinline__ int cost_per_item(int rows, int tc) { return tc ? (rows > 128 ? 6500 : (rows > 96 ? 4700 : 3500)) : 4000; }

struct PlanArgs {
    const int* ctx_lens;
    const int* cu_q;
    int B, n_q_heads, n_kv_heads;
    int n_sm;                           // segments = CTAs of the item kernel
    int min_chunk_pages;                // no piece of a cut item is shorter than this
    int tc_min_rows, max_item_rows;
    int tail_rows;                      // a remainder of at most this many rows rides with the last full row block (0: never)
    int max_entries;
    int* status;
    AttnEntry* entries;                 // [max_entries]
    AttnSeg* segs;                      // [n_sm + 1]
    AttnCut* cuts;                      // [n_sm]: entry b describes the merge the combine kernel does at boundary b
    int* plan;                          // [0] n_entries, [1] first entry of the warp-level part, [2] total pages
};

template <typename T>
__device__ __forceinline__ T plan_warp_scan(T v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        T u = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += u;
    }
    return v;
}

// exclusive scan over the CTA of two counts and two costs per thread at once (one pass of barriers): prefixes in `o`,
// totals in `t`; `w0`..`w3`: 33 values of shared memory each
struct PlanScan4 {
    int n0, n1;
    long long c0, c1;
};
__device__ __forceinline__ void plan_block_exclusive_scan4(const PlanScan4& v, int* w0, int* w1, long long* w2, long long* w3,
                                                           PlanScan4& o, PlanScan4& t) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    PlanScan4 inc;
    inc.n0 = plan_warp_scan(v.n0, lane);
    inc.n1 = plan_warp_scan(v.n1, lane);
    inc.c0 = plan_warp_scan(v.c0, lane);
    inc.c1 = plan_warp_scan(v.c1, lane);
    if (lane == 31) {
        w0[warp] = inc.n0;
        w1[warp] = inc.n1;
        w2[warp] = inc.c0;
        w3[warp] = inc.c1;
    }
    __syncthreads();
    if (warp == 0) {
        const bool in = lane < (int)(blockDim.x >> 5);
        const int a0 = in ? w0[lane] : 0, a1 = in ? w1[lane] : 0;
        const long long a2 = in ? w2[lane] : 0, a3 = in ? w3[lane] : 0;
        const int s0 = plan_warp_scan(a0, lane), s1 = plan_warp_scan(a1, lane);
        const long long s2 = plan_warp_scan(a2, lane), s3 = plan_warp_scan(a3, lane);
        w0[lane] = s0 - a0;
        w1[lane] = s1 - a1;
        w2[lane] = s2 - a2;
        w3[lane] = s3 - a3;
        if (lane == 31) {
            w0[32] = s0;
            w1[32] = s1;
            w2[32] = s2;
            w3[32] = s3;
        }
    }
    __syncthreads();
    o.n0 = w0[warp] + inc.n0 - v.n0;
    o.n1 = w1[warp] + inc.n1 - v.n1;
    o.c0 = w2[warp] + inc.c0 - v.c0;
    o.c1 = w3[warp] + inc.c1 - v.c1;
    t.n0 = w0[32];
    t.n1 = w1[32];
    t.c0 = w2[32];
    t.c1 = w3[32];
}

// Row blocks of a query tile of M rows: full blocks of max_rows rows and one remainder.  A remainder of at most
// tail_rows rows does not become an item of its own (which would stream the request's K/V a second time): it rides
// with the last full block, whose item then has up to max_rows + tail_rows rows (the tail warps of the tcgen05 phase
// take the rows past max_rows from the same staged pages).
__device__ __forceinline__ int plan_row_blocks(int M, int max_rows, int tail_rows) {
    const int n_full = M / max_rows, rem = M - n_full * max_rows;
    return n_full + ((rem > 0 && !(n_full > 0 && rem <= tail_rows)) ? 1 : 0);
}
__device__ __forceinline__ int plan_block_rows(int M, int max_rows, int n_rb, int rb) {
    return rb == n_rb - 1 ? M - rb * max_rows : max_rows;
}

// Every thread of the CTA calls this (it synchronises the CTA).  `prefix` is shared memory for 2 B + 1 64-bit values:
// the cost of the stream before each entry.
__device__ __forceinline__ void attn_plan_body(const PlanArgs& a, long long* prefix) {
    __shared__ long long ws64[33], ws64b[33];
    __shared__ int ws32[33], ws32b[33];
    __shared__ int total_s, w_tc_s, w_mma_s;
    __shared__ AttnSeg seg_s[kMaxSegs + 1];
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int group = a.n_q_heads / a.n_kv_heads;
    if (tid == 0) {
        total_s = 0;
        w_tc_s = 0;
        w_mma_s = 0;
    }
    __syncthreads();
    // pass 1: pages in all, and how they would split over the two phases of the item kernel
    {
        int local = 0, w_tc = 0, w_mma = 0;
        for (int i = tid; i < a.B; i += nthr) {
            const int d = a.cu_q[i + 1] - a.cu_q[i] - 1;
            const int pages = (a.ctx_lens[i] + d + 1 + kPage - 1) / kPage;
            local += pages;
            const int M = (d + 1) * group;
            const int n_rb = plan_row_blocks(M, a.max_item_rows, a.tail_rows);
            int tc_rb = 0;
            for (int rb = 0; rb < n_rb; ++rb) tc_rb += plan_block_rows(M, a.max_item_rows, n_rb, rb) >= a.tc_min_rows ? 1 : 0;
            w_tc += pages * tc_rb;
            w_mma += pages * (n_rb - tc_rb);
        }
        if (local) atomicAdd(&total_s, local);
        if (w_tc) atomicAdd(&w_tc_s, w_tc);
        if (w_mma) atomicAdd(&w_mma_s, w_mma);
    }
    __syncthreads();
    // The item kernel runs a segment's tcgen05 items first and its warp-level items after them.  When the second kind
    // holds only a small part of the pages (a few shallow requests among deep ones), every item takes the tcgen05
    // path: one kind of item, one cost weight, and no switch of phase inside the CTAs.
    const int tc_min_rows = (a.tc_min_rows <= a.max_item_rows && w_tc_s > 0 && 8LL * w_mma_s < (long long)w_tc_s + w_mma_s) ? 1 : a.tc_min_rows;

    // pass 2: entries of each request in either part of the stream, and their cost
    const int per = (a.B + nthr - 1) / nthr;
    const int i0 = tid * per;
    int my_tc = 0, my_mma = 0;
    long long c_tc = 0, c_mma = 0;
    for (int e = 0; e < per; ++e) {
        const int i = i0 + e;
        if (i < a.B) {
            const int d = a.cu_q[i + 1] - a.cu_q[i] - 1;
            const int pages = (a.ctx_lens[i] + d + 1 + kPage - 1) / kPage;
            const int M = (d + 1) * group;
            const int n_rb = plan_row_blocks(M, a.max_item_rows, a.tail_rows);
            for (int rb = 0; rb < n_rb; ++rb) {
                const int rows = plan_block_rows(M, a.max_item_rows, n_rb, rb);
                const int tc = rows >= tc_min_rows;
                const long long c = (long long)a.n_kv_heads * (cost_per_item(rows, tc) + (long long)pages * cost_per_page(rows, tc));
                if (tc) {
                    ++my_tc;
                    c_tc += c;
                } else {
                    ++my_mma;
                    c_mma += c;
                }
            }
        }
    }
    PlanScan4 sc_o, sc_t;
    plan_block_exclusive_scan4(PlanScan4{my_tc, my_mma, c_tc, c_mma}, ws32, ws32b, ws64, ws64b, sc_o, sc_t);
    int off_tc = sc_o.n0, off_mma = sc_o.n1;
    const int n_tc = sc_t.n0, n_mma = sc_t.n1;
    long long pre_tc = sc_o.c0, pre_mma = sc_o.c1;
    const long long tot_tc = sc_t.c0, tot_mma = sc_t.c1;
    const int n_entries = n_tc + n_mma;
    const long long total = tot_tc + tot_mma;
    const bool overflow = n_entries > a.max_entries;      // cannot happen with a context sized for the batch; defensive
    if (tid == 0) {
        a.plan[0] = overflow ? 0 : n_entries;
        a.plan[1] = overflow ? 0 : n_tc;
        a.plan[2] = total_s;
        if (overflow) atomicExch(a.status, DCUT_DEV_PLAN_OVERFLOW);
    }
    if (overflow) {
        for (int s = tid; s <= a.n_sm; s += nthr) {
            a.segs[s] = AttnSeg{0, 0, 0, 0};
            if (s < a.n_sm) a.cuts[s] = AttnCut{0, 0, 0, 0, 0, {0, 0, 0}};
        }
        return;
    }
    off_mma += n_tc;
    pre_mma += tot_tc;
    for (int e = 0; e < per; ++e) {
        const int i = i0 + e;
        if (i < a.B) {
            const int q0 = a.cu_q[i];
            const int d = a.cu_q[i + 1] - q0 - 1;
            const int ctx_len = a.ctx_lens[i];
            const int pages = (ctx_len + d + 1 + kPage - 1) / kPage;
            const int M = (d + 1) * group;
            const int n_rb = plan_row_blocks(M, a.max_item_rows, a.tail_rows);
            for (int rb = 0; rb < n_rb; ++rb) {
                const int rows = plan_block_rows(M, a.max_item_rows, n_rb, rb);
                const int tc = rows >= tc_min_rows;
                const long long c = (long long)a.n_kv_heads * (cost_per_item(rows, tc) + (long long)pages * cost_per_page(rows, tc));
                AttnEntry en;
                en.req = i;
                en.row0 = rb * a.max_item_rows;
                en.rows = rows;
                en.pages = pages;
                en.q0 = q0;
                en.depth = d;
                en.ctx_len = ctx_len;
                en.tc = tc;
                const int idx = tc ? off_tc++ : off_mma++;
                a.entries[idx] = en;
                prefix[idx] = tc ? pre_tc : pre_mma;
                if (tc) pre_tc += c; else pre_mma += c;
            }
        }
    }
    if (tid == 0) prefix[n_entries] = total;
    __syncthreads();
    // segment boundaries: position s / n_sm of the total cost, mapped to (entry, kv head, page) and moved to the nearest
    // place where an item may be cut (no piece shorter than min_chunk_pages; tcgen05 items at multiples of 4 pages)
    for (int s = tid; s <= a.n_sm; s += nthr) {
        AttnSeg sg = {n_entries, 0, 0, 0};
        if (s == 0) {
            sg.e = 0;                                        // the stream's beginning, whatever its first item looks like
        } else if (s < a.n_sm && n_entries > 0) {
            const long long pos = (total / a.n_sm) * s + (total % a.n_sm) * s / a.n_sm;
            int lo = 0, hi = n_entries;                      // largest e < n_entries with prefix[e] <= pos
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (prefix[mid] <= pos) lo = mid; else hi = mid;
            }
            int e = lo;
            const AttnEntry en = a.entries[e];               // written by this CTA before the barrier above
            const long long item_cost = (prefix[e + 1] - prefix[e]) / a.n_kv_heads;
            const long long rem = pos - prefix[e];
            int h = (int)(rem / item_cost);
            if (h >= a.n_kv_heads) h = a.n_kv_heads - 1;
            const long long in_item = rem - (long long)h * item_cost - cost_per_item(en.rows, en.tc);
            // Cuts inside an item fall on multiples of min_chunk_pages.  Two boundaries must never cut an item at the same
            // page (the segment between them would hold an empty piece that nobody writes): consecutive positions are
            // at least total / n_sm apart, so they land on different multiples as long as a segment is worth at least
            // min_chunk_pages of this item; below that (tiny batches) the item is not cut at all.
            const long long quantum = (long long)a.min_chunk_pages * cost_per_page(en.rows, en.tc);
            int p = (in_item <= 0 || total / a.n_sm < quantum) ? 0 : (int)(in_item / quantum) * a.min_chunk_pages;
            if (en.pages - p < a.min_chunk_pages) {          // the rest is too short to be a piece: the boundary moves to the next item
                p = 0;
                if (++h == a.n_kv_heads) {
                    h = 0;
                    ++e;
                }
            }
            sg.e = e;
            sg.h = h;
            sg.p = p;
        }
        a.segs[s] = sg;
        seg_s[s] = sg;
    }
    __syncthreads();
    // what the combine kernel merges at each boundary: the item a boundary cuts is merged at the first boundary inside it
    for (int b = tid; b < a.n_sm; b += nthr) {
        AttnCut cut = {0, 0, 0, 0, 0, {0, 0, 0}};
        const AttnSeg sg = seg_s[b];
        if (b > 0 && sg.p > 0 && sg.e < n_entries) {
            const AttnSeg pv = seg_s[b - 1];
            if (!(pv.e == sg.e && pv.h == sg.h && pv.p > 0)) {
                int m = 1;                                    // boundaries b .. b + m - 1 cut the item: m + 1 pieces
                while (b + m < a.n_sm && seg_s[b + m].e == sg.e && seg_s[b + m].h == sg.h && seg_s[b + m].p > 0) ++m;
                const AttnEntry en = a.entries[sg.e];
                cut.pieces = m + 1;
                cut.rows = en.rows;
                cut.row0 = en.row0;
                cut.q0 = en.q0;
                cut.kv_head = sg.h;
            }
        }
        a.cuts[b] = cut;
    }
}

}  // namespace dcut_plan

// fills the arguments of the partition builder for this batch from the context's shapes and scratch (verify_attn.cu)
void dcut_fill_plan_args(dcut_ctx* ctx, const int* ctx_lens, const int* cu_q, int B, dcut_plan::PlanArgs* pa);
