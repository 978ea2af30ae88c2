// Work list of the verification attention (split-KV flash-decoding plan), as a device function that runs in ONE CTA:
// the stand-alone attn_plan_kernel of dcut_verify_attn, or the tail of the selector kernel, which has just written
// cu_q and can leave the list ready for the attention call that follows (dcut_enable_plan_in_select).
#pragma once

#include "dcut_internal.h"

namespace dcut_plan {

constexpr int kPage = 16;            // tokens per page

struct PlanArgs {
    const int* ctx_lens;
    const int* cu_q;
    int B, n_q_heads, n_kv_heads;
    int target_items, min_chunk_pages, max_items, npad, tc_min_rows, max_item_rows;
    int tail_rows;                      // a remainder of at most this many rows rides with the last full row block (0: never)
    int tail_req_div, tail_min_pages;   // the shortest B / tail_req_div requests are cut finer (0: none)
    long long part_rows_cap;
    int* status;
    AttnItem* items;
    int* plan;       // [0] n_items, [1] chunk_pages, [2] total_pages, [3] partial rows used, [4] overflow, [5] n_tc, [8], [9] queue heads
    int* req_part;   // [B][2]: first partial row, n_chunks
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

// three exclusive scans over the CTA at once (one value of each per thread): prefixes in o0..o2, totals in t0..t2
__device__ __forceinline__ void plan_block_exclusive_scan3(int v0, int v1, int v2, int (*ws)[33], int& o0, int& o1, int& o2,
                                                           int& t0, int& t1, int& t2) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int i0 = plan_warp_scan(v0, lane), i1 = plan_warp_scan(v1, lane), i2 = plan_warp_scan(v2, lane);
    if (lane == 31) {
        ws[0][warp] = i0;
        ws[1][warp] = i1;
        ws[2][warp] = i2;
    }
    __syncthreads();
    if (warp < 3) {
        const int w = lane < (int)(blockDim.x >> 5) ? ws[warp][lane] : 0;
        const int winc = plan_warp_scan(w, lane);
        ws[warp][lane] = winc - w;
        if (lane == 31) ws[warp][32] = winc;
    }
    __syncthreads();
    o0 = ws[0][warp] + i0 - v0;
    o1 = ws[1][warp] + i1 - v1;
    o2 = ws[2][warp] + i2 - v2;
    t0 = ws[0][32];
    t1 = ws[1][32];
    t2 = ws[2][32];
}

// ascending bitonic sort of 32 E keys by one warp: lane l holds elements e * 32 + l
template <int E>
__device__ __forceinline__ void plan_warp_sort(unsigned long long* keys, int lane) {
    unsigned long long k[E];
#pragma unroll
    for (int e = 0; e < E; ++e) k[e] = keys[e * 32 + lane];
#pragma unroll
    for (int kk = 2; kk <= 32 * E; kk <<= 1) {
#pragma unroll
        for (int j = kk >> 1; j > 0; j >>= 1) {
            if (j >= 32) {                          // partner in the same lane
                const int je = j >> 5;
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    if ((e & je) == 0) {
                        const bool up = (((e * 32 + lane) & kk) == 0);
                        const unsigned long long x = k[e], y = k[e | je];
                        const bool swap = (x > y) == up;
                        k[e] = swap ? y : x;
                        k[e | je] = swap ? x : y;
                    }
                }
            } else {                                // partner in another lane
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    const unsigned long long other = __shfl_xor_sync(0xffffffffu, k[e], j);
                    const bool keep_min = (((e * 32 + lane) & kk) == 0) == ((lane & j) == 0);
                    k[e] = ((k[e] < other) == keep_min) ? k[e] : other;
                }
            }
        }
    }
#pragma unroll
    for (int e = 0; e < E; ++e) keys[e * 32 + lane] = k[e];
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

// Requests are ordered by the estimated duration of their items, longest first, so the CTAs that
// start last are the short ones (the hardware hands items to SMs in index order as SMs free up).
// Every thread of the CTA calls this (it synchronises the CTA).  `order` is shared memory for a.npad 64-bit keys:
// (inverted cost << 32 | request), sorted ascending.
__device__ __forceinline__ void attn_plan_body(const PlanArgs& a, unsigned long long* order) {
    __shared__ int ws3[3][33];
    __shared__ int total_s, tail_s, w_tc_s, w_mma_s;
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int group = a.n_q_heads / a.n_kv_heads;
    if (tid == 0) {
        total_s = 0;
        tail_s = 0;
        w_tc_s = 0;
        w_mma_s = 0;
    }
    __syncthreads();
    int local = 0, w_tc = 0, w_mma = 0;   // pages in all; pages whose items would go to the tcgen05 / warp-level queue
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
    __syncthreads();
    const int total_pages = total_s;
    const long long units = (long long)total_pages * a.n_kv_heads;
    int chunk_pages = (int)((units + a.target_items - 1) / a.target_items);
    if (chunk_pages < a.min_chunk_pages) chunk_pages = a.min_chunk_pages;

    for (int i = tid; i < a.npad; i += nthr) {
        unsigned long long key = ~0ull;
        if (i < a.B) {
            const int d = a.cu_q[i + 1] - a.cu_q[i] - 1;
            const int pages = (a.ctx_lens[i] + d + 1 + kPage - 1) / kPage;
            const int nc = (pages + chunk_pages - 1) / chunk_pages;
            const int cp = (pages + nc - 1) / nc;
            const int MT = ((d + 1) * group + 15) >> 4;
            // per page: memory-bound below about two m-tiles, then time grows with the m-tiles
            const unsigned int cost = (unsigned int)cp * (unsigned int)max(7, 3 * MT);
            key = ((unsigned long long)(0xffffffffu - cost) << 32) | (unsigned int)i;
        }
        order[i] = key;
    }
    __syncthreads();
    if (a.npad <= 256) {
        // up to 256 requests: one warp sorts the keys in registers (element e * 32 + lane), without a single barrier
        if (tid < 32) {
            if (a.npad <= 32) plan_warp_sort<1>(order, tid);
            else if (a.npad <= 64) plan_warp_sort<2>(order, tid);
            else if (a.npad <= 128) plan_warp_sort<4>(order, tid);
            else plan_warp_sort<8>(order, tid);
        }
        __syncthreads();
    } else {
        for (int k = 2; k <= a.npad; k <<= 1)
            for (int j = k >> 1; j > 0; j >>= 1) {
                for (int t = tid; t < (a.npad >> 1); t += nthr) {
                    const int i = 2 * t - (t & (j - 1)), l = i + j;
                    const bool up = (i & k) == 0;
                    const unsigned long long x = order[i], y = order[l];
                    if ((x > y) == up) {
                        order[i] = y;
                        order[l] = x;
                    }
                }
                __syncthreads();
            }
    }

    // The items that start last decide how unevenly the SMs finish: the requests at the end of the order are cut
    // into about target_items pieces altogether, so every SM ends on a short item.
    const int n_tail = a.tail_req_div > 0 ? (a.B + a.tail_req_div - 1) / a.tail_req_div : 0;
    const int tail_from = a.B - n_tail;
    if (n_tail > 0) {   // (the same answer in every thread)
        for (int j = tail_from + tid; j < a.B; j += nthr) {
            const int i = (int)(order[j] & 0xffffffffu);
            const int d = a.cu_q[i + 1] - a.cu_q[i] - 1;
            atomicAdd(&tail_s, (a.ctx_lens[i] + d + 1 + kPage - 1) / kPage);
        }
        __syncthreads();
    }
    int tail_chunk = (int)(((long long)tail_s * a.n_kv_heads + a.target_items - 1) / a.target_items);
    if (tail_chunk < a.tail_min_pages) tail_chunk = a.tail_min_pages;
    if (tail_chunk > chunk_pages) tail_chunk = chunk_pages;

    // The item kernel works through the tcgen05 queue first and the warp-level queue after it.  When the second
    // holds only a small part of the pages (a few shallow requests among deep ones), its few long items would start
    // late on a few SMs with the rest idle (measured at B = 64: +15 us per call while 3-8 % of the pages were in
    // it): below one eighth of the pages everything goes to the tcgen05 queue.
    const int tc_min_rows = (a.tc_min_rows <= a.max_item_rows && w_tc_s > 0 && 8LL * w_mma_s < (long long)w_tc_s + w_mma_s) ? 1 : a.tc_min_rows;

    const int per = (a.B + nthr - 1) / nthr;
    const int j0 = tid * per;
    int my_tc = 0, my_mma = 0, my_rows = 0;
    for (int e = 0; e < per; ++e) {
        const int j = j0 + e;
        if (j < a.B) {
            const int i = (int)(order[j] & 0xffffffffu);
            const int d = a.cu_q[i + 1] - a.cu_q[i] - 1;
            const int pages = (a.ctx_lens[i] + d + 1 + kPage - 1) / kPage;
            const int cpj = j >= tail_from ? tail_chunk : chunk_pages;
            const int nc = (pages + cpj - 1) / cpj;
            // row blocks of the query tile: full blocks of max_item_rows rows and one remainder; each goes to the
            // tcgen05 queue or to the warp-level queue by its number of rows
            const int M = (d + 1) * group;
            const int n_rb = plan_row_blocks(M, a.max_item_rows, a.tail_rows);
            int tc_rb = 0;
            for (int rb = 0; rb < n_rb; ++rb) tc_rb += plan_block_rows(M, a.max_item_rows, n_rb, rb) >= tc_min_rows ? 1 : 0;
            my_tc += nc * a.n_kv_heads * tc_rb;
            my_mma += nc * a.n_kv_heads * (n_rb - tc_rb);
            if (nc > 1) my_rows += nc * (d + 1) * a.n_q_heads;
        }
    }
    int n_tc, n_mma, n_rows;
    int tc_off, mma_off, row_off;
    plan_block_exclusive_scan3(my_tc, my_mma, my_rows, ws3, tc_off, mma_off, row_off, n_tc, n_mma, n_rows);
    const int n_items = n_tc + n_mma;
    mma_off += n_tc;
    const bool overflow = n_items > a.max_items || (long long)n_rows > a.part_rows_cap;
    if (tid == 0) {
        a.plan[0] = overflow ? 0 : n_items;
        a.plan[1] = chunk_pages;
        a.plan[2] = total_pages;
        a.plan[3] = n_rows;
        a.plan[4] = overflow ? 1 : 0;
        a.plan[5] = overflow ? 0 : n_tc;     // items [0, n_tc): tcgen05 queue; [n_tc, n_items): warp-level queue
        a.plan[8] = 0;                       // next item of the tcgen05 queue (claimed by the CTAs of the item kernel)
        a.plan[9] = overflow ? 0 : n_tc;     // next item of the warp-level queue
        if (overflow) atomicExch(a.status, DCUT_DEV_PLAN_OVERFLOW);
    }
    if (overflow) return;
    for (int e = 0; e < per; ++e) {
        const int j = j0 + e;
        if (j < a.B) {
            const int i = (int)(order[j] & 0xffffffffu);
            const int q0 = a.cu_q[i];
            const int d = a.cu_q[i + 1] - q0 - 1;
            const int ctx_len = a.ctx_lens[i];
            const int pages = (ctx_len + d + 1 + kPage - 1) / kPage;
            const int cpj = j >= tail_from ? tail_chunk : chunk_pages;
            const int nc = (pages + cpj - 1) / cpj;
            const int cp = (pages + nc - 1) / nc;   // near-equal chunks
            const int M = (d + 1) * group;
            a.req_part[2 * i] = row_off;
            a.req_part[2 * i + 1] = nc;
            // a query tile above max_item_rows (+ tail_rows) rows is cut into row blocks, each its own item over the
            // same pages
            const int n_rb = plan_row_blocks(M, a.max_item_rows, a.tail_rows);
            for (int c = 0; c < nc; ++c)
                for (int h = 0; h < a.n_kv_heads; ++h)
                    for (int rb = 0; rb < n_rb; ++rb) {
                        const int row0 = rb * a.max_item_rows, rows = plan_block_rows(M, a.max_item_rows, n_rb, rb);
                        AttnItem it;
                        it.req = i;
                        it.kv_head = h;
                        it.page_begin = c * cp;
                        it.page_end = min(pages, (c + 1) * cp);
                        it.n_chunks = nc;
                        it.part_row = nc > 1 ? row_off + (c * a.n_kv_heads + h) * M + row0 : -1;
                        it.q0 = q0;
                        it.depth = d;
                        it.ctx_len = ctx_len;
                        const bool tc = rows >= tc_min_rows;
                        it.pad[0] = tc ? 1 : 0;   // which queue the item is in
                        it.pad[1] = row0;         // first query row of the item within the request's tile
                        it.pad[2] = rows;         // query rows of the item
                        a.items[tc ? tc_off++ : mma_off++] = it;
                    }
            if (nc > 1) row_off += nc * (d + 1) * a.n_q_heads;
        }
    }
}

}  // namespace dcut_plan

// fills the arguments of the work-list builder for this batch from the context's shapes and scratch (verify_attn.cu)
void dcut_fill_plan_args(dcut_ctx* ctx, const int* ctx_lens, const int* cu_q, int B, dcut_plan::PlanArgs* pa);
