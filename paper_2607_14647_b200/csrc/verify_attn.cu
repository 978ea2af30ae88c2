// dcut_verify_attn: ragged causal multi-token attention over a paged bf16 KV cache.
//
// HBM-bound by design: every K/V byte of every request is read once per step, so the kernels are organised around
// keeping 100-200 KB of page loads in flight per SM, all the time.
//
//   work partition       one CTA (attn_plan.cuh): the tail of the selector kernel, or the stand-alone attn_plan_kernel.
//                        The call's work is a stream of (request, row block, kv head) items, each a run of KV pages of
//                        known cost; it is cut into one segment of equal cost per SM.  A segment may begin or end inside
//                        an item: that item is computed in pieces.  Query tiles of 17+ rows form the tcgen05 part of the
//                        stream, smaller ones the warp-level part.
//   attn_item_kernel     persistent, one CTA per SM.  A CTA walks its segment: its tcgen05 items, then its warp-level
//                        items.  In both phases the TMA producer warp builds the next item from the work table as soon
//                        as it has issued the current item's last load and keeps streaming into the same ring of
//                        stages (stages, tensor-memory buffers and their mbarriers are numbered through consecutive
//                        items), so the loads never pause at an item boundary.
//       tcgen05 phase    Q and P in tensor memory, page groups of four (64 keys), S = Q K^T and O += P V as tcgen05.mma,
//                        softmax by two threads per row (see tc_phase).
//       warp-level phase 8 consumer warps + 1 producer warp; the query tile is cut into 16-row m-tiles, warp w owns
//                        m-tile (w mod MT) and page slot (w div MT) and runs S = Q K^T, online softmax and O += P V on
//                        every nslots-th page (mma.sync m16n8k16 bf16, fp32 accumulate, ldmatrix from the swizzled
//                        tiles), in order from its slot's sub-ring; the slots' (m, l, O) are merged through shared
//                        memory (see mma_phase).
//       output           an item that no segment boundary cuts writes bf16 output directly, a piece of a cut item
//                        normalised fp32 partials and their log-sum-exp.
//   attn_combine_kernel  merges the pieces of the cut items (one per boundary at most).
//
// The three kernels are chained with programmatic dependent launch.  Every mbarrier wait is bounded; on expiry the CTA
// sets the device status word and every role leaves at a point where none is left waiting at a named barrier.
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdlib.h>
#include <type_traits>

#include "dcut_internal.h"
#include "attn_plan.cuh"

namespace {

constexpr int kThreads = 384;        // tcgen05 phase: TMA warp, MMA warp, 8 softmax warps, 2 tail-row warps; warp-level phase: 8 consumer warps + 1 producer
constexpr int kMmaWarps = 8;         // consumer warps of the warp-level MMA phase
constexpr int kMmaThreads = kMmaWarps * 32;
constexpr int kMmaStages = 16;       // page stages in its ring (8 KB each at head_dim 128)
constexpr int kMaxProducerLanes = 8;
constexpr int kPage = dcut_plan::kPage;   // tokens per page
constexpr int kMaxMTiles = 8;        // query rows per item <= 128
constexpr int kPlanThreads = 1024;
constexpr int kSpinLimit = 1 << 21;   // bounded waits: ~1 s, then the CTA reports and leaves

// ------------------------------------------------------------------------------------------------
// PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// bounded wait: false if the phase did not complete within the spin limit, or another warp of the
// CTA has already given up
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    for (int it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (it > 4096) {
            __nanosleep(128);
            if ((it & 255) == 0 && *abort_flag) return false;
        }
    }
    return false;
}
// one (page, kv head) tile: box {64 columns, 16 token rows, head_dim/64 column halves}
__device__ __forceinline__ void tma_load_tile(uint32_t dst, const CUtensorMap* map, int row, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(0), "r"(row), "r"(0), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// the same without `volatile`: a pure function of its operands, which the compiler may move across the loads around it
__device__ __forceinline__ void mma_bf16_pure(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// transposes an 8 x 8 matrix of 16-bit elements held one row per four lanes (lane 4 g + t: row g, elements 2 t, 2 t + 1)
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t v) {
    uint32_t r;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(r) : "r"(v));
    return r;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// 2^x on the special-function unit (2 ulp; -inf -> 0); far inside the output tolerance of bf16
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Two fp32 values in one 64-bit register and the sm_100 instructions that work on both at once: the softmax warps of
// the tcgen05 phase are short of issue slots, not of arithmetic.
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma_f32x2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ unsigned long long add_f32x2(unsigned long long a, unsigned long long b) {
    unsigned long long r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
// maximum of three (one instruction on sm_100)
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
// byte offset of 16-byte chunk `c16` (0 .. DH/8-1) of token/row `r` (0..15) inside a swizzled
// [DH/64][16][64] bf16 tile (what two 64-column TMA boxes with 128-byte swizzle produce)
__device__ __forceinline__ uint32_t tile_off(int r, int c16) {
    return (uint32_t)(((c16 >> 3) << 11) + (r << 7) + (((c16 & 7) ^ (r & 7)) << 4));
}

// the same for a K page of the tcgen05 phase, which one 4-D TMA box delivers as [8-row group][half][8 rows][64 columns]
__device__ __forceinline__ uint32_t tile_off_k4(int r, int c16) {
    return (uint32_t)(((r >> 3) << 11) + ((c16 >> 3) << 10) + ((r & 7) << 7) + (((c16 & 7) ^ (r & 7)) << 4));
}

// ------------------------------------------------------------------------------------------------
// plan (the body lives in attn_plan.cuh: the selector kernel can run it too)

using dcut_plan::PlanArgs;

__global__ void __launch_bounds__(kPlanThreads) attn_plan_kernel(PlanArgs a) {
    extern __shared__ long long plan_prefix[];                        // [2 B + 1] cost prefixes, then cu_q [B + 1] and ctx_lens [B]
    dcut_pdl_wait();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the item kernel's CTAs may take their SMs now
    // the body reads every request's cu_q and ctx_lens several times: from shared memory, not through L2
    int* cu_s = reinterpret_cast<int*>(plan_prefix + 2 * a.B + 1);
    int* ctx_s = cu_s + a.B + 1;
    for (int i = threadIdx.x; i <= a.B; i += blockDim.x) cu_s[i] = a.cu_q[i];
    for (int i = threadIdx.x; i < a.B; i += blockDim.x) ctx_s[i] = a.ctx_lens[i];
    __syncthreads();
    a.cu_q = cu_s;
    a.ctx_lens = ctx_s;
    dcut_plan::attn_plan_body(a, plan_prefix);                        // 256 threads for small batches: cheaper barriers
}

// ------------------------------------------------------------------------------------------------
// tcgen05 phase: items with many query rows (head_dim 128, 17 <= rows <= 128).
//
// With 3+ m-tiles the warp-level MMA path is bound by the tensor pipe and by operand traffic through
// registers, not by HBM.  Here the query tile is padded to 128 rows (row = tensor-memory lane) and lives in
// tensor memory for the whole item; pages are handled in groups of four (64 keys):
//   S[128, 64]  = Q . K_group^T     8 MMAs (M128 N64 K16): A = Q from tensor memory, B = the group's K tiles,
//                 which TMA lays out contiguously so the 64 key rows form one K-major operand;
//                 accumulator in tensor memory, three buffers;
//   softmax     two teams of 128 threads take the groups alternately; a thread owns a row: tcgen05.ld of the
//                 row, mask, running max and sum without any shuffle; P goes back as bf16 into the columns S
//                 occupied (tcgen05.st), so it never touches shared memory; the team's O is only rescaled when
//                 a row's maximum grows by more than 2^8; the teams' (m, l, O) are merged in the item's epilogue;
//   O_team[128, 128] += P . V_page  one MMA (M128 N128 K16) per page: A = P from tensor memory, B = the V tile
//                 read MN-major (transposed by its descriptor); one accumulator per team in tensor memory.
// Both MMAs therefore stream only K and V from shared memory.  Warp 0: TMA producer (lanes 0-3 look up the
// group's pages, one elected lane issues its loads), warp 1: MMA issuer and tensor-memory owner, warps 2-3: tail rows
// (below), warps 4-7 and 8-11: the two softmax teams, which also write the output (why this order: tc_phase).
//   tail rows   a query tile of 129..144 rows (8 q heads per kv head at depth 16: 136) does not fit the 128 lanes of
//                 tensor memory.  Cutting it into two items would stream the request's K/V twice; instead the item
//                 keeps all its rows and warps 2-3 take rows 128.. as one m16 tile of warp-level MMAs
//                 (mma.sync, as in the warp-level phase) on the very pages the ring holds for the tcgen05 MMAs: the
//                 two warps take the item's pages alternately and merge their (m, l, O) at the end of the item.  A
//                 ring stage is released by three arrivals: the commit of its last PV MMA and the two tail warps
//                 (which arrive as soon as the stage is full when the item has no tail rows; with shapes that
//                 never give more than 128 rows they take no part and the commit alone releases a stage).
constexpr int kTcGroupStages = 6;                  // ring of page groups (192 KB in flight)
constexpr int kTcSBufs = 3;                        // S/P buffers in tensor memory: groups in flight between QK^T and PV
constexpr int kTcSoftmaxThreads = 256;             // two teams of 128: one thread per row and team
constexpr int kTcTailWarps = 2;                    // warps 2, 3: query rows 128..143 of an item, by warp-level MMA
constexpr int kTcTailRows = 16;                    // one m16 tile
constexpr int kTcTailStride = 128 + 8;             // floats per row of the tail warps' merge buffer
constexpr int kTcTailBytes = (kTcTailRows * kTcTailStride + kTcTailRows * 2) * 4;
static_assert(kThreads == 64 + kTcSoftmaxThreads + 32 * kTcTailWarps, "roles of the tcgen05 phase");
constexpr int kTcPageBytes = kPage * 128 * 2;      // 4 KB: one K or V page tile
constexpr int kTcGroupBytes = 8 * kTcPageBytes;    // K of 4 pages (16 KB, [half][64 rows][64]) + V of 4 pages
constexpr int kTcRingBytes = kTcGroupStages * kTcGroupBytes;
constexpr int kTcCols = 512;                       // O of team 0: 0..127, of team 1: 128..255, S/P buffers: 256..447, Q: 448..511
constexpr int kTcColOB = 128, kTcColS = 256, kTcColQ = kTcColS + 64 * kTcSBufs;
static_assert(kTcColQ + 64 <= kTcCols, "tensor-memory columns");
constexpr float kRescaleLog2 = 8.0f;

// One lane of a converged warp.  Issuing tcgen05.mma / tcgen05.commit under this predicate (not under `lane == 0`)
// lets the compiler keep the operands in uniform registers: on B200 the issuing thread then needs ~47 cycles for
// an M128 N64 K16 MMA with A in tensor memory and ~73 for N128, against 96+ from a lane-0-only branch.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(pred));
    return pred != 0;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[tmem] . B[smem descriptor]
__device__ __forceinline__ void tc_mma_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t db, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(tmem_d), "r"(tmem_a), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]),
          "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]),
          "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]), "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar) : "memory");
}

// K-major tile with 128-byte rows and 128-byte swizzle: 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t addr) {
    return (uint64_t)((addr & 0x3ffff) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
           ((uint64_t)2 << 61);
}
// the same with the 8-row groups 2048 bytes apart: the two 64-column halves of a 128-wide K row sit side by side
// (group, half, row), which is the order one 4-D TMA box per page delivers
__device__ __forceinline__ uint64_t desc_kmajor_2k(uint32_t addr) {
    return (uint64_t)((addr & 0x3ffff) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(2048 >> 4) << 32) | ((uint64_t)1 << 46) |
           ((uint64_t)2 << 61);
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar) : "memory");
}
// MN-major tile (rows = K index, 128 bytes = 64 consecutive MN elements per row): the next 64 MN elements are
// 2048 bytes on (leading byte offset), the next 8 K rows 1024 bytes on (stride byte offset)
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t addr) {
    return (uint64_t)((addr & 0x3ffff) >> 4) | ((uint64_t)(2048 >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// instruction descriptors: fp32 accumulate, bf16 operands, M = 128; QK^T: B K-major, N = 16 per page in the group;
// PV: B MN-major, N = 128
constexpr uint32_t kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 4) << 24);
constexpr uint32_t kIdescPV = kIdescBase | (1u << 16) | ((128u >> 3) << 17);

// ------------------------------------------------------------------------------------------------
// persistent item kernel: shared declarations

struct AttnArgs {
    const __nv_bfloat16* q;
    const int* block_table;
    int block_table_stride;
    const int* ctx_lens;
    const int* cu_q;
    const AttnEntry* entries;  // work table and segment boundaries (attn_plan.cuh)
    const AttnSeg* segs;
    const int* plan;
    int n_q_heads, n_kv_heads;
    long long num_pages;
    float scale_log2;          // softmax scale * log2(e)
    int q_row_bytes;           // head_dim * 2
    int tail_on;               // query tiles above 128 rows can occur with this context's shapes: the tail warps take part
    __nv_bfloat16* out;
    float* lse;                // [T, Hq] or null
    float* part_o;
    float* part_lse;
    int* status;
};

// Control block of a CTA (shared memory, behind the data region).  Every cross-role hand-over goes through an
// mbarrier with a bounded wait; the two phases of the kernel use separate scheduler barriers.
struct __align__(16) Ctrl {
    unsigned long long ring_full[kMmaStages], ring_empty[kMmaStages];   // the tcgen05 phase uses the first kTcGroupStages
    unsigned long long s_full[kTcSBufs], p_full[kTcSBufs], pv_done[kTcSBufs];
    unsigned long long q_ready, o_free;
    unsigned long long sched_full[2][2], sched_empty[2][2];             // [phase][slot]
    unsigned long long geom_a, geom_b;                                  // ring re-initialisation of the warp-level phase
    AttnItem item[2];
    int item_idx[2];
    uint32_t tmem_base;
    int abort;
};

#define ABORTED(c) (*(volatile int*)&(c)->abort)

template <int DH>
struct MmaSmem {
    static constexpr int kPageBytes = kPage * DH * 2;            // one K or V page tile
    static constexpr int kStageBytes = 2 * kPageBytes;
    static constexpr int kRingBytes = kMmaStages * kStageBytes;
    static constexpr int kQBytes = kMaxMTiles * 16 * DH * 2;
    static constexpr int kMergeStride = DH + 8;                  // floats per merged row
    static constexpr int kMergeBytes = kMmaWarps * 16 * kMergeStride * 4;
    static constexpr int kMergeOrQ = kMergeBytes > kQBytes ? kMergeBytes : kQBytes;   // Q staging reuses the merge buffer
    static constexpr int kMLBytes = kMmaWarps * 16 * 2 * 4;
    static constexpr int kTotal = kRingBytes + kMergeOrQ + kMLBytes;
};

// barrier + OR-reduction over the threads of a named barrier: the result is the same in every thread
__device__ __forceinline__ bool bar_any(int id, int nthreads, bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %3, 0;\n\t"
        "barrier.cta.red.or.pred q, %1, %2, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r) : "r"(id), "r"(nthreads), "r"((uint32_t)pred) : "memory");
    return r != 0;
}

// Position in the work stream (entry, kv head, page), and the end of what this CTA runs in the current phase.
struct SegCursor {
    int e, h, p;
    int e1, h1, p1;
};
__device__ __forceinline__ bool seg_before(int e, int h, int p, int e1, int h1, int p1) {
    return e < e1 || (e == e1 && (h < h1 || (h == h1 && p < p1)));
}
// the part of this CTA's segment [s0, s1) that lies in [lo, hi) entries of the table (one phase of the kernel)
__device__ __forceinline__ SegCursor seg_range(const AttnSeg& s0, const AttnSeg& s1, int e_lo, int e_hi) {
    SegCursor c;
    if (s0.e < e_lo) { c.e = e_lo; c.h = 0; c.p = 0; } else { c.e = s0.e; c.h = s0.h; c.p = s0.p; }
    if (s1.e >= e_hi) { c.e1 = e_hi; c.h1 = 0; c.p1 = 0; } else { c.e1 = s1.e; c.h1 = s1.h; c.p1 = s1.p; }
    return c;
}

// Scheduler, producer side (whole warp, converged): builds the next item of this CTA's segment and posts it in slot
// n & 1 of the CTA's queue.  idx = -1 when the phase has no items left.  An item that a segment boundary cuts covers
// only this segment's pages of it and leaves a partial result in one of the segment's two slots: slot 2 s when the
// item began in an earlier segment, slot 2 s + 1 when it begins here and continues in the next.
__device__ __forceinline__ bool sched_fetch(Ctrl* c, const AttnArgs& a, int phase, int n, SegCursor& cur,
                                            AttnItem& it, int& idx) {
    const int slot = n & 1, lane = threadIdx.x & 31;
    if (n >= 2 && !__all_sync(0xffffffffu, mbar_wait(smem_u32(&c->sched_empty[phase][slot]), ((n >> 1) - 1) & 1, &c->abort)))
        return false;
    idx = seg_before(cur.e, cur.h, cur.p, cur.e1, cur.h1, cur.p1) ? n : -1;
    if (idx >= 0) {
        const AttnEntry en = a.entries[cur.e];
        const bool last = cur.e == cur.e1 && cur.h == cur.h1;      // the segment ends inside this item
        it.req = en.req;
        it.kv_head = cur.h;
        it.page_begin = cur.p;
        it.page_end = last ? cur.p1 : en.pages;
        const bool whole = it.page_begin == 0 && it.page_end == en.pages;
        it.n_chunks = whole ? 1 : 2;
        it.part_row = whole ? -1 : (2 * (int)blockIdx.x + (cur.p > 0 ? 0 : 1)) * dcut_plan::kSlotRows;
        it.q0 = en.q0;
        it.depth = en.depth;
        it.ctx_len = en.ctx_len;
        it.pad[0] = en.tc;
        it.pad[1] = en.row0;      // first query row of the item within the request's tile
        it.pad[2] = en.rows;      // query rows of the item
        {
            // the item's query rows will be fetched when the item before it ends: ask L2 for them now (256 bytes per
            // row at head_dim 128; rows of one token are contiguous across the group's heads)
            const int group = a.n_q_heads / a.n_kv_heads, dh_bytes = (int)(a.q_row_bytes);
            for (int r = lane; r < en.rows; r += 32) {
                const int t = (en.row0 + r) / group, hl = (en.row0 + r) - t * group;
                const char* p = reinterpret_cast<const char*>(a.q) + ((size_t)(en.q0 + t) * a.n_q_heads + cur.h * group + hl) * dh_bytes;
                for (int o = 0; o < dh_bytes; o += 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(p + o));
            }
        }
        if (last) {
            cur.p = cur.p1;
        } else {
            cur.p = 0;
            if (++cur.h == a.n_kv_heads) {
                cur.h = 0;
                ++cur.e;
            }
        }
    }
    if (lane == 0) {
        c->item_idx[slot] = idx;
        if (idx >= 0) c->item[slot] = it;
        mbar_arrive(smem_u32(&c->sched_full[phase][slot]));
    }
    __syncwarp();
    return true;
}
// consumer side: idx = -2 when the wait gave up
__device__ __forceinline__ int sched_wait(Ctrl* c, int phase, int n, AttnItem& it) {
    if (!mbar_wait(smem_u32(&c->sched_full[phase][n & 1]), (n >> 1) & 1, &c->abort)) return -2;
    const int idx = c->item_idx[n & 1];
    if (idx >= 0) it = c->item[n & 1];
    return idx;
}
__device__ __forceinline__ void sched_release(Ctrl* c, int phase, int n) {
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(smem_u32(&c->sched_empty[phase][n & 1]));
}

// ------------------------------------------------------------------------------------------------
// warp-level MMA phase (items with few query rows, or any item when head_dim is not 128)
//
// kMmaWarps consumer warps + one producer warp.  The ring of page stages is cut into one sub-ring per page slot
// (nslots = kMmaWarps / m-tiles of the item); page p of an item goes to slot p mod nslots, and every slot's pages are
// numbered through consecutive items, so the producer keeps loading the next item's pages while the consumers still
// merge the current one and an item's result does not depend on what its CTA worked on before (the same bits on
// every run).  Only when the number of m-tiles changes between two items is the ring drained and its barriers set
// up again.

template <int DH>
__device__ __forceinline__ void mma_phase(const CUtensorMap& k_map, const CUtensorMap& v_map, const AttnArgs& a,
                                          unsigned char* smem, Ctrl* c, SegCursor cur) {
    using L = MmaSmem<DH>;
    unsigned char* ring = smem;
    float* merge = reinterpret_cast<float*>(smem + L::kRingBytes);
    unsigned char* q_s = smem + L::kRingBytes;
    float* ml_s = reinterpret_cast<float*>(smem + L::kRingBytes + L::kMergeOrQ);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int group = a.n_q_heads / a.n_kv_heads;
    const uint32_t full_bar = smem_u32(c->ring_full), empty_bar = smem_u32(c->ring_empty);
    const uint32_t geom_a = smem_u32(&c->geom_a), geom_b = smem_u32(&c->geom_b);
    constexpr int kPhase = 1;

    if (warp > kMmaWarps) return;               // spare warps of the CTA

    AttnItem item;
    int cur_mt = -1, n_geom = 0;
    long long slot_pages = 0;                   // producer lanes: pages of this lane's slot since the ring was last set up
    bool failed = false;

    if (warp == kMmaWarps) {
        // ---------------------------------------------------------------- producer warp
        for (int n = 0;; ++n) {
            int idx;
            if (!sched_fetch(c, a, kPhase, n, cur, item, idx)) {
                failed = true;
                break;
            }
            if (idx < 0) break;
            const int MT = (item.pad[2] + 15) >> 4;
            const int nslots = kMmaWarps / MT, depth_s = kMmaStages / nslots, ring_n = nslots * depth_s;
            if (MT != cur_mt) {
                // every consumer has finished the previous item (nothing of this one is in flight yet)
                if (lane == 0) mbar_arrive(geom_a);
                if (!__all_sync(0xffffffffu, mbar_wait(geom_b, n_geom & 1, &c->abort))) {
                    failed = true;
                    break;
                }
                ++n_geom;
                cur_mt = MT;
                slot_pages = 0;
            }
            const int n_pages = item.page_end - item.page_begin;
            static_assert(kMaxProducerLanes == 8 && kMmaStages == 16, "lane / slot / stage arithmetic below");
            (void)ring_n;
            if (lane < kMaxProducerLanes) {
                // Page p of the item belongs to slot p mod nslots, whatever came before it (the split of an item's
                // pages over the slots, and with it the rounding of its result, must not depend on which items this
                // CTA happened to take earlier).  A slot's pages go through its sub-ring in order; the slot is served
                // by 8 / nslots lanes, lane l = slot + nslots j taking the slot's positions q with q mod (8 / nslots)
                // = j: a stage is always refilled by the same lane, whose waits on it are therefore ordered.
                const int sl = lane % nslots, ksub = kMaxProducerLanes / nslots, jsub = lane / nslots;
                const int cnt = sl < n_pages ? (n_pages - sl + nslots - 1) / nslots : 0;   // this item's pages of the slot
                const int* bt = a.block_table + (size_t)item.req * a.block_table_stride + item.page_begin;
                int k = (int)((jsub - slot_pages % ksub + ksub) % ksub);
                int next = k < cnt ? bt[sl + nslots * k] : 0;
                for (; k < cnt; k += ksub) {
                    int page_id = next;
                    if (k + ksub < cnt) next = bt[sl + nslots * (k + ksub)];
                    const long long q = slot_pages + k;               // position in the slot's sub-ring since it was set up
                    const int r = (int)(q % depth_s);
                    const long long use = q / depth_s;
                    const int stage = sl * depth_s + r;
                    if (use > 0 && !mbar_wait(empty_bar + 8 * stage, (uint32_t)((use - 1) & 1), &c->abort)) {
                        failed = true;
                        break;
                    }
                    if (page_id < 0 || page_id >= a.num_pages) {
                        atomicExch(a.status, DCUT_DEV_BAD_PAGE);
                        page_id = 0;
                    }
                    const uint32_t bar = full_bar + 8 * stage;
                    const uint32_t dst = smem_u32(ring + stage * L::kStageBytes);
                    const int row = (page_id * a.n_kv_heads + item.kv_head) * kPage;
                    mbar_arrive_expect_tx(bar, L::kStageBytes);
                    tma_load_tile(dst, &k_map, row, bar);
                    tma_load_tile(dst + L::kPageBytes, &v_map, row, bar);
                }
            }
            __syncwarp();
            if (__any_sync(0xffffffffu, failed) || c->abort) {
                failed = true;
                break;
            }
            {
                const int sl = lane % nslots;
                slot_pages += sl < n_pages ? (n_pages - sl + nslots - 1) / nslots : 0;
            }
        }
        if (failed) {
            atomicExch(a.status, DCUT_DEV_ATTN_WAIT_TIMEOUT);
            c->abort = 1;
        }
        return;
    }

    // -------------------------------------------------------------------- consumer warps
    int r_stage = 0, parity = 0;                // position of this warp in its slot's sub-ring
    for (int n = 0;; ++n) {
        const int idx = sched_wait(c, kPhase, n, item);
        if (idx == -2) failed = true;
        if (bar_any(1, kMmaThreads, failed || c->abort)) break;   // also: the previous merge has been read by everyone
        if (idx < 0) break;
        const int q0 = item.q0, ctx_len = item.ctx_len, kvh = item.kv_head;
        const int row0 = item.pad[1], M = item.pad[2];   // this item's rows of the request's query tile
        const int MT = (M + 15) >> 4;
        const int nslots = kMmaWarps / MT, depth_s = kMmaStages / nslots;
        const int n_pages = item.page_end - item.page_begin;
        if (MT != cur_mt) {
            // set the ring up for this number of m-tiles; the producer waits for it before it loads anything
            __syncwarp();
            if (lane == 0) mbar_arrive(geom_a);
            if (tid == 0) {
                if (mbar_wait(geom_a, n_geom & 1, &c->abort)) {
                    for (int s = 0; s < kMmaStages; ++s) {
                        asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(full_bar + 8 * s) : "memory");
                        asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(empty_bar + 8 * s) : "memory");
                        mbar_init(full_bar + 8 * s, 1);
                        mbar_init(empty_bar + 8 * s, MT);   // the m-tile warps of the stage's slot
                    }
                    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    mbar_arrive(geom_b);
                } else {
                    c->abort = 1;
                }
            }
            if (!mbar_wait(geom_b, n_geom & 1, &c->abort)) failed = true;
            ++n_geom;
            cur_mt = MT;
            r_stage = 0;
            parity = 0;
        }
        // stage the query tile: row R = t * group + hl  <->  q[(q0 + t), kvh * group + hl, :]
        {
            constexpr int kChunks = DH / 8;
            const int rows_padded = MT * 16;
            for (int i = tid; i < rows_padded * kChunks; i += kMmaThreads) {
                const int R = i / kChunks, c16 = i - R * kChunks;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (R < M) {
                    const int t = (row0 + R) / group, hl = (row0 + R) - t * group;
                    v = *reinterpret_cast<const uint4*>(a.q + ((size_t)(q0 + t) * a.n_q_heads + kvh * group + hl) * DH + c16 * 8);
                }
                *reinterpret_cast<uint4*>(q_s + (R >> 4) * (16 * DH * 2) + tile_off(R & 15, c16)) = v;
            }
        }
        if (bar_any(1, kMmaThreads, failed)) break;

        const int mt = warp % MT, slot = warp / MT;
        const bool active = slot < nslots;
        float o[DH / 8][4];
#pragma unroll
        for (int j = 0; j < DH / 8; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.0f;
        float m_run[2] = {-INFINITY, -INFINITY};
        float l_run[2] = {0.0f, 0.0f};

        if (active) {
            uint32_t qf[DH / 16][4];
            {
                const int mat = lane >> 3;
                const int r = ((mat & 1) << 3) + (lane & 7);
                const uint32_t qbase = smem_u32(q_s + mt * (16 * DH * 2));
#pragma unroll
                for (int ks = 0; ks < DH / 16; ++ks) ldmatrix_x4(qbase + tile_off(r, 2 * ks + (mat >> 1)), qf[ks]);
            }
            // causal limit per row: query token t sees cache positions j <= ctx_len + t
            const int R_lo = mt * 16 + (lane >> 2), R_hi = R_lo + 8;
            const int jmax_lo = ctx_len + (row0 + min(R_lo, M - 1)) / group;
            const int jmax_hi = ctx_len + (row0 + min(R_hi, M - 1)) / group;
            // per-lane ldmatrix row/chunk selectors
            const int kmat = lane >> 3;
            const int k_tok = ((kmat >> 1) << 3) + (lane & 7);
            const int k_chunk = kmat & 1;
            const int v_tok = ((kmat & 1) << 3) + (lane & 7);
            const int v_chunk = kmat >> 1;

            // this warp's pages of the item: p = slot modulo nslots, in order through the slot's sub-ring
            const float c_log2 = a.scale_log2;
            for (int p = slot; p < n_pages; p += nslots) {
                const int stage = slot * depth_s + r_stage;
                if (!mbar_wait(full_bar + 8 * stage, parity, &c->abort)) {
                    failed = true;
                    break;
                }
                if (++r_stage == depth_s) {
                    r_stage = 0;
                    parity ^= 1;
                }
                const uint32_t k_base = smem_u32(ring + stage * L::kStageBytes);
                const uint32_t v_base = k_base + L::kPageBytes;

                float s[2][4];
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.0f;
#pragma unroll
                for (int ks = 0; ks < DH / 16; ++ks) {
                    uint32_t kf[4];
                    ldmatrix_x4(k_base + tile_off(k_tok, 2 * ks + k_chunk), kf);
                    mma_bf16(s[0], qf[ks], kf[0], kf[1]);
                    mma_bf16(s[1], qf[ks], kf[2], kf[3]);
                }
                // causal mask: only pages that reach past the cached context can hold hidden positions
                const int j0 = (item.page_begin + p) * kPage + ((lane & 3) << 1);
                if ((item.page_begin + p) * kPage + kPage - 1 > ctx_len) {
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int j = j0 + nt * 8 + (e & 1);
                            const int jmax = (e < 2) ? jmax_lo : jmax_hi;
                            if (j > jmax) s[nt][e] = -INFINITY;
                        }
                    }
                }
                // online softmax for the two rows this thread holds; running max kept on the raw scores,
                // the softmax scale folded into the exponent: p = 2^(s*c - m*c)
                float mx[2] = {fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1])),
                               fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]))};
                float alpha[2], mc[2];
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
                    mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
                    const float m_new = fmaxf(m_run[r], mx[r]);
                    const float msafe = (m_new == -INFINITY) ? 0.0f : m_new;
                    alpha[r] = fast_exp2((m_run[r] - msafe) * c_log2);
                    mc[r] = msafe * c_log2;
                    m_run[r] = m_new;
                }
                float ps[2][4];
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    ps[nt][0] = fast_exp2(fmaf(s[nt][0], c_log2, -mc[0]));
                    ps[nt][1] = fast_exp2(fmaf(s[nt][1], c_log2, -mc[0]));
                    ps[nt][2] = fast_exp2(fmaf(s[nt][2], c_log2, -mc[1]));
                    ps[nt][3] = fast_exp2(fmaf(s[nt][3], c_log2, -mc[1]));
                }
                l_run[0] = l_run[0] * alpha[0] + (ps[0][0] + ps[0][1] + ps[1][0] + ps[1][1]);
                l_run[1] = l_run[1] * alpha[1] + (ps[0][2] + ps[0][3] + ps[1][2] + ps[1][3]);
                if (__any_sync(0xffffffffu, alpha[0] != 1.0f || alpha[1] != 1.0f)) {
#pragma unroll
                    for (int j = 0; j < DH / 8; ++j) {
                        o[j][0] *= alpha[0];
                        o[j][1] *= alpha[0];
                        o[j][2] *= alpha[1];
                        o[j][3] *= alpha[1];
                    }
                }
                uint32_t pf[4] = {pack_bf16(ps[0][0], ps[0][1]), pack_bf16(ps[0][2], ps[0][3]),
                                  pack_bf16(ps[1][0], ps[1][1]), pack_bf16(ps[1][2], ps[1][3])};
#pragma unroll
                for (int jj = 0; jj < DH / 16; ++jj) {
                    uint32_t vf[4];
                    ldmatrix_x4_trans(v_base + tile_off(v_tok, 2 * jj + v_chunk), vf);
                    mma_bf16(o[2 * jj], pf, vf[0], vf[1]);
                    mma_bf16(o[2 * jj + 1], pf, vf[2], vf[3]);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty_bar + 8 * stage);
            }
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
                l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
            }
        }
        if (failed) c->abort = 1;

        // ---------------------------------------------------------------- merge the slots
        // (the merge buffer is not part of the ring: the producer is already loading the next item)
        if (active) {
            float* mo = merge + (size_t)warp * 16 * L::kMergeStride;
            const int r_lo = lane >> 2, c0 = (lane & 3) << 1;
#pragma unroll
            for (int j = 0; j < DH / 8; ++j) {
                *reinterpret_cast<float2*>(mo + r_lo * L::kMergeStride + j * 8 + c0) = make_float2(o[j][0], o[j][1]);
                *reinterpret_cast<float2*>(mo + (r_lo + 8) * L::kMergeStride + j * 8 + c0) = make_float2(o[j][2], o[j][3]);
            }
            if ((lane & 3) == 0) {
                ml_s[(warp * 16 + r_lo) * 2] = m_run[0];
                ml_s[(warp * 16 + r_lo) * 2 + 1] = l_run[0];
                ml_s[(warp * 16 + r_lo + 8) * 2] = m_run[1];
                ml_s[(warp * 16 + r_lo + 8) * 2 + 1] = l_run[1];
            }
        }
        if (bar_any(1, kMmaThreads, failed || ABORTED(c))) break;
        {
            constexpr int kVec = DH / 4;   // float4 per row
            for (int i = tid; i < M * kVec; i += kMmaThreads) {
                const int R = i / kVec, c4 = i - R * kVec;
                const int tile = R >> 4, r = R & 15;
                float m_all = -INFINITY;
                for (int sl = 0; sl < nslots; ++sl) m_all = fmaxf(m_all, ml_s[((sl * MT + tile) * 16 + r) * 2]);
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                float l_all = 0.0f;
                for (int sl = 0; sl < nslots; ++sl) {
                    const int w = sl * MT + tile;
                    const float m_w = ml_s[(w * 16 + r) * 2];
                    const float wgt = (m_w == -INFINITY) ? 0.0f : exp2f((m_w - m_all) * a.scale_log2);
                    l_all += wgt * ml_s[(w * 16 + r) * 2 + 1];
                    const float4 v = *reinterpret_cast<const float4*>(merge + ((size_t)w * 16 + r) * L::kMergeStride + c4 * 4);
                    acc.x += wgt * v.x;
                    acc.y += wgt * v.y;
                    acc.z += wgt * v.z;
                    acc.w += wgt * v.w;
                }
                const float inv = l_all > 0.0f ? 1.0f / l_all : 0.0f;
                acc.x *= inv;
                acc.y *= inv;
                acc.z *= inv;
                acc.w *= inv;
                const float lse_nat = l_all > 0.0f ? (m_all * a.scale_log2 + log2f(l_all)) * 0.6931471805599453f : -INFINITY;
                const int t = (row0 + R) / group, hl = (row0 + R) - t * group;
                const size_t orow = (size_t)(q0 + t) * a.n_q_heads + kvh * group + hl;
                if (item.n_chunks == 1) {
                    uint2 pk;
                    pk.x = pack_bf16(acc.x, acc.y);
                    pk.y = pack_bf16(acc.z, acc.w);
                    *reinterpret_cast<uint2*>(a.out + orow * DH + c4 * 4) = pk;
                    if (a.lse && c4 == 0) a.lse[orow] = lse_nat;
                } else {
                    const size_t prow = (size_t)item.part_row + R;
                    *reinterpret_cast<float4*>(a.part_o + prow * DH + c4 * 4) = acc;
                    if (c4 == 0) a.part_lse[prow] = lse_nat;
                }
            }
        }
        sched_release(c, kPhase, n);
    }
    if (failed) {
        atomicExch(a.status, DCUT_DEV_ATTN_WAIT_TIMEOUT);
        c->abort = 1;
    }
}

// One persistent pass over the tcgen05-path items of this CTA.  Ring stages, S/P buffers and their barriers are
// numbered through consecutive items (running group number), so the producer streams the next item's pages while the
// current item is still being finished; only Q and O (single-buffered in tensor memory) serialise at an item boundary,
// through the q_ready and o_free barriers.
__device__ __forceinline__ void tc_phase(const CUtensorMap& k2_map, const CUtensorMap& v_map, const AttnArgs& a,
                                         unsigned char* ring, float* tail_buf, Ctrl* c, float (*xm)[128],
                                         float (*xl)[128], SegCursor cur) {
    constexpr int kPhase = 0;
    const uint32_t full_bar = smem_u32(c->ring_full), empty_bar = smem_u32(c->ring_empty);
    const uint32_t s_full = smem_u32(c->s_full), p_full = smem_u32(c->p_full), pv_done = smem_u32(c->pv_done);
    const uint32_t q_ready = smem_u32(&c->q_ready), o_free = smem_u32(&c->o_free);
    const int tid = threadIdx.x, lane = tid & 31;
    // Roles: warp 0 TMA producer, warp 1 MMA issuer, warps 2-3 tail rows, warps 4-11 softmax (team 0: 4-7, team 1: 8-11).
    // A softmax warp's number mod 4 is its lane quarter of tensor memory and its scheduler, and a scheduler prefers its
    // lower-numbered warps.  Query row r lives in lane (r + 64) mod 128: rows 0-63, which every tcgen05 item has, belong
    // to quarters 2 and 3, so the producer and the issuer (schedulers 0 and 1, first in line there) share a scheduler
    // only with the softmax warps of rows 64-127, which short query tiles (32q/8kv at depth 16: 68 rows; pruned
    // batches) leave idle.  With row r in lane r the issuer and the producer shared schedulers 0 and 1 with the softmax
    // warps that always have rows, and one scheduler issued 6 % of the time on 68-row tiles.
    const int warp = tid >> 5;
    const int group = a.n_q_heads / a.n_kv_heads;
    const uint32_t tmem_o = c->tmem_base;
    AttnItem item;
    bool failed = false;
    int G0 = 0;                                  // groups of the earlier items: running group number = G0 + g

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        // The whole warp walks the groups; lanes 0-3 look up the group's four pages one group ahead, and one elected
        // lane issues all of the group's tile loads (uniform operands: a divergent lane needs about twice as long per
        // load, which made the producer the slowest role).
        for (int n = 0;; ++n) {
            int idx;
            if (!sched_fetch(c, a, kPhase, n, cur, item, idx)) {
                failed = true;
                break;
            }
            if (idx < 0) break;
            const int n_pages = item.page_end - item.page_begin;
            const int n_groups = (n_pages + 3) >> 2;
            const int* bt = a.block_table + (size_t)item.req * a.block_table_stride + item.page_begin;
            int next = (lane < 4 && lane < n_pages) ? bt[lane] : 0;
            for (int g = 0; g < n_groups; ++g) {
                int page_id = next;
                const int pn = 4 * (g + 1) + lane;
                if (lane < 4 && pn < n_pages) next = bt[pn];
                const int gc = G0 + g, gs = gc % kTcGroupStages, use = gc / kTcGroupStages;
                if (use > 0 && !__all_sync(0xffffffffu, mbar_wait(empty_bar + 8 * gs, (use - 1) & 1, &c->abort))) {
                    failed = true;
                    break;
                }
                const int np = min(4, n_pages - 4 * g);
                if (lane < np && (page_id < 0 || page_id >= a.num_pages)) {
                    atomicExch(a.status, DCUT_DEV_BAD_PAGE);
                    page_id = 0;
                }
                const int row = (page_id * a.n_kv_heads + item.kv_head) * kPage;
                const int r0 = __shfl_sync(0xffffffffu, row, 0), r1 = __shfl_sync(0xffffffffu, row, 1);
                const int r2 = __shfl_sync(0xffffffffu, row, 2), r3 = __shfl_sync(0xffffffffu, row, 3);
                if (elect_one()) {
                    const uint32_t bar = full_bar + 8 * gs;
                    const uint32_t dst = smem_u32(ring + gs * kTcGroupBytes);
                    mbar_arrive_expect_tx(bar, (uint32_t)np * 2 * kTcPageBytes);
                    const int rows[4] = {r0, r1, r2, r3};
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (j < np) {
                            // page j of K as one 4 KB box: (two 8-row groups) x (two 64-column halves) x 8 rows x 128 bytes
                            tma_load_4d(dst + j * 4096, &k2_map, 0, 0, 0, rows[j] >> 3, bar);
                            tma_load_tile(dst + 4 * kTcPageBytes + j * kTcPageBytes, &v_map, rows[j], bar);
                        }
                }
                __syncwarp();
            }
            if (failed || ABORTED(c)) {
                failed = true;
                break;
            }
            G0 += n_groups;
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        // The whole warp walks the schedule and waits on the barriers; one elected lane issues.
        const uint32_t tmem_q = tmem_o + kTcColQ;
        for (int n = 0; !failed; ++n) {
            const int idx = sched_wait(c, kPhase, n, item);
            if (idx == -2) failed = true;
            if (__any_sync(0xffffffffu, failed) || idx < 0) break;
            const int n_pages = item.page_end - item.page_begin;
            const int n_groups = (n_pages + 3) >> 2;
            // this item's query tile is in tensor memory
            if (!__all_sync(0xffffffffu, mbar_wait(q_ready, n & 1, &c->abort))) {
                failed = true;
                break;
            }
            tc_fence_after();
            auto issue_qk = [&](int g) -> bool {
                const int gc = G0 + g;
                const int np = min(4, n_pages - 4 * g), gs = gc % kTcGroupStages, b = gc % kTcSBufs;
                // the S/P buffer was last used by the running group gc - kTcSBufs
                if (gc >= kTcSBufs && !__all_sync(0xffffffffu, mbar_wait(pv_done + 8 * b, ((gc / kTcSBufs) - 1) & 1, &c->abort))) return false;
                if (!__all_sync(0xffffffffu, mbar_wait(full_bar + 8 * gs, (gc / kTcGroupStages) & 1, &c->abort))) return false;
                tc_fence_after();
                if (elect_one()) {
                    const uint32_t k_addr = smem_u32(ring + gs * kTcGroupBytes);
                    const uint32_t d = tmem_o + kTcColS + 64 * b;
                    const uint32_t idesc = kIdescBase | ((uint32_t)(np * kPage >> 3) << 17);
                    const uint64_t dk0 = desc_kmajor_2k(k_addr), dk1 = desc_kmajor_2k(k_addr + 1024);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)    // 16 head-dim elements = 8 words of Q, 32 bytes along a K row
                        tc_mma_ts(d, tmem_q + ks * 8, dk0 + 2 * ks, idesc, ks ? 1u : 0u);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        tc_mma_ts(d, tmem_q + (4 + ks) * 8, dk1 + 2 * ks, idesc, 1u);
                    tc_commit(s_full + 8 * b);
                }
                __syncwarp();
                return true;
            };
            // QK^T runs kTcSBufs - 1 groups ahead of PV
            bool ok = true;
            for (int g = 0; ok && g < kTcSBufs - 1 && g < n_groups; ++g) ok = issue_qk(g);
            for (int g = 0; ok && g < n_groups; ++g) {
                const int ga = g + kTcSBufs - 1;
                if (ga < n_groups && !issue_qk(ga)) { ok = false; break; }
                const int gc = G0 + g, b = gc % kTcSBufs;
                if (!__all_sync(0xffffffffu, mbar_wait(p_full + 8 * b, (gc / kTcSBufs) & 1, &c->abort))) { ok = false; break; }
                // the first PV of an item overwrites O: the previous item's epilogue must have read it
                if (g == 0 && n > 0 && !__all_sync(0xffffffffu, mbar_wait(o_free, (n - 1) & 1, &c->abort))) { ok = false; break; }
                tc_fence_after();
                if (elect_one()) {
                    const int np = min(4, n_pages - 4 * g), gs = gc % kTcGroupStages;
                    const uint32_t tmem_p = tmem_o + kTcColS + 64 * b;
                    const uint32_t tmem_ov = tmem_o + kTcColOB * (g & 1);   // the O accumulator of the team that owns group g
                    const uint64_t dv = desc_mnmajor(smem_u32(ring + gs * kTcGroupBytes) + 4 * kTcPageBytes);
                    if (np == 4) {
#pragma unroll
                        for (int j = 0; j < 4; ++j)        // 16 keys = 8 words of P; the next V tile is 4 KB = 256 units on
                            tc_mma_ts(tmem_ov, tmem_p + 8 * j, dv + 256 * j, kIdescPV, ((g >> 1) | j) ? 1u : 0u);
                    } else {
                        for (int j = 0; j < np; ++j)
                            tc_mma_ts(tmem_ov, tmem_p + 8 * j, dv + 256 * j, kIdescPV, ((g >> 1) | j) ? 1u : 0u);
                    }
                    tc_commit(empty_bar + 8 * gs);         // the group's K and V tiles are free again
                    tc_commit(pv_done + 8 * b);
                }
                __syncwarp();
            }
            if (!ok) {
                failed = true;
                break;
            }
            sched_release(c, kPhase, n);
            G0 += n_groups;
        }
    } else if (warp >= 2 + kTcTailWarps) {
        // ---------------------------------------------------------------- softmax + epilogue
        // Two teams of 128 threads (warps 4-7 and 8-11) take the page groups of an item alternately; each has its own
        // running (maximum, sum) per row and its own O accumulator, so while one team works through the latency chain
        // of its group (tcgen05.ld, maximum, exponentials, tcgen05.st) the other team's group is in flight too.
        // Row R sits in tensor-memory lane (R + 64) mod 128; a thread owns the whole row (64 columns) of its team's S tiles.  The two threads
        // of a row (one per team) meet at a named barrier at the top and at the end of an item only.
        const uint32_t tmem_q = tmem_o + kTcColQ;
        const int quarter = warp & 3, team = (warp - 2 - kTcTailWarps) >> 2;   // lane quarter of tensor memory; team 0 / 1
        const int R = (quarter * 32 + lane + 64) & 127;            // the query row in this thread's lane
        const uint32_t t_lane = tmem_o + ((uint32_t)(quarter * 32) << 16);
        const uint32_t t_mine = t_lane + kTcColOB * team, t_other = t_lane + kTcColOB * (team ^ 1);
        const float cs = a.scale_log2;
        // an item's query tile goes to tensor memory: row R into this thread's lane, 128 bf16 = 64 words, 32 per team
        auto store_q = [&](const AttnItem& it) {
            uint32_t qw[32];
            const int rows = min(it.pad[2], 128);
            if (R < rows) {
                const int t = (it.pad[1] + R) / group, hl = (it.pad[1] + R) - t * group;
                const uint4* src = reinterpret_cast<const uint4*>(a.q + ((size_t)(it.q0 + t) * a.n_q_heads + it.kv_head * group + hl) * 128) + 8 * team;
#pragma unroll
                for (int cc = 0; cc < 8; ++cc) {
                    const uint4 v = src[cc];
                    qw[4 * cc] = v.x; qw[4 * cc + 1] = v.y; qw[4 * cc + 2] = v.z; qw[4 * cc + 3] = v.w;
                }
            } else {
#pragma unroll
                for (int cc = 0; cc < 32; ++cc) qw[cc] = 0;
            }
            tc_st32(tmem_q + ((uint32_t)(quarter * 32) << 16) + 32 * team, qw);
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(q_ready);
        };
        bool q_staged = false;                   // this item's query tile was stored while the previous item was finishing
        for (int n = 0;; ++n) {
            const int idx = sched_wait(c, kPhase, n, item);
            if (idx == -2) failed = true;
            if (bar_any(2 + quarter, 64, failed || ABORTED(c))) {
                failed = true;
                break;
            }
            if (idx < 0) break;
            const int q0 = item.q0, ctx_len = item.ctx_len, kvh = item.kv_head;
            const int row0 = item.pad[1], M = min(item.pad[2], 128);   // this item's rows of the request's query tile (rows past 128: tail warps)
            const int n_pages = item.page_end - item.page_begin;
            const int n_groups = (n_pages + 3) >> 2;
            if (!q_staged) store_q(item);
            q_staged = false;
            const int jmax = ctx_len + (row0 + min(R, M - 1)) / group;  // last visible cache position
            const bool live = ((quarter * 32 + 64) & 127) < M;           // (warp-uniform) some of this warp's rows exist
            float m_run = -INFINITY, l_run = 0.0f;
            for (int g = team; g < n_groups; g += 2) {
                const int gc = G0 + g, b = gc % kTcSBufs;
                if (!failed && !mbar_wait(s_full + 8 * b, (gc / kTcSBufs) & 1, &c->abort)) failed = true;
                failed = __any_sync(0xffffffffu, failed);
                if (failed) break;
                if (!live) {
                    // None of this warp's 32 rows exists (a query tile of at most 96, 64 or 32 rows): nothing to compute.
                    // Its lanes of P keep the raw scores and its rows of O whatever the MMAs make of them; rows of
                    // the accumulators are independent and these are never read.
                    mbar_arrive(p_full + 8 * b);
                    continue;
                }
                const uint32_t t_s = t_lane + kTcColS + 64 * b;
                uint32_t sr[64];
                tc_fence_after();
                tc_ld32(t_s, sr);
                tc_ld32(t_s + 32, sr + 32);
                tc_wait_ld();
                float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
                const int ncols = min(4, n_pages - 4 * g) * kPage;
                const int j0 = (item.page_begin + 4 * g) * kPage;
                if (ncols < 64 || j0 + 63 > ctx_len) {                  // a partial group or one that holds hidden keys
                    const int lim = min(ncols - 1, jmax - j0);          // columns 0..lim are visible
#pragma unroll
                    for (int e = 0; e < 64; ++e) sr[e] = e <= lim ? sr[e] : 0xff800000u;   // -inf
                }
#pragma unroll
                for (int e = 0; e < 64; e += 8)
#pragma unroll
                    for (int k = 0; k < 4; ++k) mx4[k] = fmax3(mx4[k], __uint_as_float(sr[e + k]), __uint_as_float(sr[e + 4 + k]));
                const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                // the running maximum only moves (and O is only rescaled) when it would grow by more than 2^8
                float alpha = 1.0f;
                bool moved = false;
                if (mx > m_run && (m_run == -INFINITY || (mx - m_run) * cs > kRescaleLog2)) {
                    alpha = fast_exp2((m_run - mx) * cs);                 // 0 when nothing was visible before
                    m_run = mx;
                    l_run *= alpha;
                    moved = g >= 2;                                       // this team's O holds its earlier groups
                }
                if (g >= 2 && __any_sync(0xffffffffu, moved)) {
                    // this team's O is being updated by its previous group's MMAs: wait for them, then scale the row
                    if (!mbar_wait(pv_done + 8 * ((gc - 2) % kTcSBufs), ((gc - 2) / kTcSBufs) & 1, &c->abort)) failed = true;
                    failed = __any_sync(0xffffffffu, failed);
                    if (failed) break;
                    tc_fence_after();
#pragma unroll 1
                    for (int cc = 0; cc < 128; cc += 32) {
                        uint32_t o[32];
                        tc_ld32(t_mine + cc, o);
                        tc_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                        tc_st32(t_mine + cc, o);
                    }
                    tc_wait_st();
                }
                const float mc = (m_run == -INFINITY ? 0.0f : m_run) * cs;
                const unsigned long long cs2 = pack_f32x2(cs, cs), nmc2 = pack_f32x2(-mc, -mc);
                unsigned long long sum2[2] = {0ull, 0ull};                // four partial sums, two per register
                uint32_t pw[32];
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    float x0, x1;
                    unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(sr[2 * e]), __uint_as_float(sr[2 * e + 1])), cs2, nmc2), x0, x1);
                    const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
                    sum2[e & 1] = add_f32x2(sum2[e & 1], pack_f32x2(p0, p1));
                    pw[e] = pack_bf16(p0, p1);
                }
                {
                    float s0, s1, s2, s3;
                    unpack_f32x2(sum2[0], s0, s1);
                    unpack_f32x2(sum2[1], s2, s3);
                    l_run += (s0 + s1) + (s2 + s3);
                }
                tc_st32(t_s, pw);                                         // P over the columns S occupied
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(p_full + 8 * b);
            }
            const int gl = G0 + n_groups - 1;
            // The next item's query tile, before this item's epilogue: Q's columns are free as soon as the last QK^T of
            // this item has completed (s_full of its last group; the team that did not own that group waits for it
            // here), and the scheduler posted the next item when it issued this item's last load.  The MMA warp can
            // then issue the next item's first QK^T products while the epilogue below runs, instead of after it.
            if (!failed) {
                AttnItem nxt;
                const int idx_n = sched_wait(c, kPhase, n + 1, nxt);
                if (idx_n == -2) failed = true;
                if (idx_n >= 0 && !mbar_wait(s_full + 8 * (gl % kTcSBufs), (gl / kTcSBufs) & 1, &c->abort)) failed = true;
                if (!__any_sync(0xffffffffu, failed) && idx_n >= 0) {
                    tc_fence_after();
                    store_q(nxt);
                    q_staged = true;
                }
            }
            // epilogue: every MMA of the item has completed once its last PV has; the two teams' (m, l, O) are merged
            // and normalised; this thread writes columns [64 * team, 64 * team + 64) of its row
            if (!failed && !mbar_wait(pv_done + 8 * (gl % kTcSBufs), (gl / kTcSBufs) & 1, &c->abort)) failed = true;
            failed = __any_sync(0xffffffffu, failed);
            tc_fence_after();
            xm[team][R] = m_run;
            xl[team][R] = l_run;
            if (failed) c->abort = 1;
            if (bar_any(2 + quarter, 64, failed)) {
                failed = true;
                break;
            }
            const float m_o = xm[team ^ 1][R], l_o = xl[team ^ 1][R];
            const float m_all = fmaxf(m_run, m_o);
            const float w_s = m_run == -INFINITY ? 0.0f : fast_exp2((m_run - m_all) * cs);
            const float w_o = m_o == -INFINITY ? 0.0f : fast_exp2((m_o - m_all) * cs);
            const float l_all = l_run * w_s + l_o * w_o;
            const float inv = l_all > 0.0f ? 1.0f / l_all : 0.0f;
            const float lse_nat = l_all > 0.0f ? (m_all * cs + log2f(l_all)) * 0.6931471805599453f : -INFINITY;
            const float f_s = w_s * inv, f_o = w_o * inv;
            const int t = (row0 + R) / group, hl = (row0 + R) - t * group;
            const size_t orow = (size_t)(q0 + t) * a.n_q_heads + kvh * group + hl;
            if (!live) {
                tc_fence_before();
                mbar_arrive(o_free);
            }
#pragma unroll 1
            for (int hh = 0; live && hh < 2; ++hh) {
                const int cc = 64 * team + 32 * hh;
                uint32_t os[32], oo[32];
                tc_ld32(t_mine + cc, os);
                tc_ld32(t_other + cc, oo);
                tc_wait_ld();
                if (hh == 1) {
                    tc_fence_before();
                    mbar_arrive(o_free);                                  // both O accumulators may be overwritten by the next item
                }
                float v[32];
#pragma unroll
                for (int e = 0; e < 32; ++e)   // a team without groups (or without visible keys) has weight 0: its O is not read as a number
                    v[e] = (w_s > 0.0f ? __uint_as_float(os[e]) * f_s : 0.0f) + (w_o > 0.0f ? __uint_as_float(oo[e]) * f_o : 0.0f);
                if (R < M) {
                    if (item.n_chunks == 1) {
#pragma unroll
                        for (int e = 0; e < 32; e += 8) {
                            uint32_t w[4];
#pragma unroll
                            for (int j = 0; j < 4; ++j) w[j] = pack_bf16(v[e + 2 * j], v[e + 2 * j + 1]);
                            *reinterpret_cast<uint4*>(a.out + orow * 128 + cc + e) = make_uint4(w[0], w[1], w[2], w[3]);
                        }
                    } else {
                        float* po = a.part_o + ((size_t)item.part_row + R) * 128 + cc;
#pragma unroll
                        for (int e = 0; e < 32; e += 4) *reinterpret_cast<float4*>(po + e) = make_float4(v[e], v[e + 1], v[e + 2], v[e + 3]);
                    }
                }
            }
            if (R < M && team == 0) {
                if (item.n_chunks == 1) {
                    if (a.lse) a.lse[orow] = lse_nat;
                } else {
                    a.part_lse[(size_t)item.part_row + R] = lse_nat;
                }
            }
            sched_release(c, kPhase, n);
            G0 += n_groups;
        }
    } else if (a.tail_on) {
        // ---------------------------------------------------------------- tail rows (128 .. 143 of the item)
        // (with shapes whose query tiles never exceed 128 rows these two warps have no part in the phase: no stage and
        // no item waits for them)
        // One m16 tile by warp-level MMA on the staged pages; warp tw takes the item's pages p with p mod 2 = tw.
        // Both warps walk every group of every item, because every stage of the ring waits for their arrival.
        const int tw = warp - 2;
        const float cs = a.scale_log2;
        float* t_o = tail_buf;
        float* t_ml = tail_buf + kTcTailRows * kTcTailStride;
        const int r_lo = lane >> 2, c0 = (lane & 3) << 1;
        const int kmat = lane >> 3;
        const int k_tok = ((kmat >> 1) << 3) + (lane & 7), k_chunk = kmat & 1;
        const int v_tok = ((kmat & 1) << 3) + (lane & 7), v_chunk = kmat >> 1;
        for (int n = 0;; ++n) {
            const int idx = sched_wait(c, kPhase, n, item);
            if (idx == -2) failed = true;
            // also: the first tail warp has read what the second left in the merge buffer for the previous item
            if (bar_any(6, 32 * kTcTailWarps, failed || ABORTED(c))) {
                failed = true;
                break;
            }
            if (idx < 0) break;
            const int q0 = item.q0, ctx_len = item.ctx_len, kvh = item.kv_head;
            const int row0 = item.pad[1] + 128, M = item.pad[2] - 128;   // the tail's first row within the request's tile, its rows
            const int n_pages = item.page_end - item.page_begin;
            const int n_groups = (n_pages + 3) >> 2;
            const bool has_tail = M > 0;
            uint32_t qf[8][4];
            float o[16][4];
            float m_run[2] = {-INFINITY, -INFINITY};
            float l_run[2] = {0.0f, 0.0f};
            int jmax_lo = 0, jmax_hi = 0;
            // A tail of at most 8 rows (8 q heads per kv head at depth 16) runs with the operands swapped: S^T = K Q^T and
            // O^T = V^T P^T, the tail rows as the MMA's n = 8 and the keys / head dimension as its m = 16, which takes half
            // the MMAs of a 16-row tile that is half padding.
            const bool swapped = has_tail && M <= 8;
            if (swapped) {
                // B fragments of Q^T: lane 4 g + t holds row g, head-dim elements 2 t, 2 t + 1 (+ 8) of every k-step
                const int R = row0 + min(r_lo, M - 1), tq = R / group;
                const uint32_t* qr = reinterpret_cast<const uint32_t*>(a.q + ((size_t)(q0 + tq) * a.n_q_heads + kvh * group + (R - tq * group)) * 128);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    qf[ks][0] = qr[ks * 8 + (lane & 3)];
                    qf[ks][1] = qr[ks * 8 + 4 + (lane & 3)];
                }
                // the two rows whose scores this lane holds: 2 t and 2 t + 1
                jmax_lo = ctx_len + (row0 + min(c0, M - 1)) / group;
                jmax_hi = ctx_len + (row0 + min(c0 + 1, M - 1)) / group;
#pragma unroll
                for (int j = 0; j < 8; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.0f;
            } else if (has_tail) {
                // A fragments straight from global memory (16 rows of 256 bytes, once per item); rows past the tail
                // repeat its last row and are never written
                const int R_lo = row0 + min(r_lo, M - 1), R_hi = row0 + min(r_lo + 8, M - 1);
                const int t_l = R_lo / group, t_h = R_hi / group;
                const uint32_t* q_l = reinterpret_cast<const uint32_t*>(a.q + ((size_t)(q0 + t_l) * a.n_q_heads + kvh * group + (R_lo - t_l * group)) * 128);
                const uint32_t* q_h = reinterpret_cast<const uint32_t*>(a.q + ((size_t)(q0 + t_h) * a.n_q_heads + kvh * group + (R_hi - t_h * group)) * 128);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    qf[ks][0] = q_l[ks * 8 + (lane & 3)];
                    qf[ks][1] = q_h[ks * 8 + (lane & 3)];
                    qf[ks][2] = q_l[ks * 8 + 4 + (lane & 3)];
                    qf[ks][3] = q_h[ks * 8 + 4 + (lane & 3)];
                }
                jmax_lo = ctx_len + t_l;     // query token t sees cache positions j <= ctx_len + t
                jmax_hi = ctx_len + t_h;
#pragma unroll
                for (int j = 0; j < 16; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.0f;
            }
            // NP pages (8 KB apart in the stage: this warp's page of the group and the one two further on) = 16 NP keys.
            // The ldmatrix loads run one step ahead of the MMAs that use them (a warp issues in order, and with two
            // tail warps per SM nothing else hides the shared-memory latency).
            auto tail_step = [&](auto npc, uint32_t k_base, int pg) {
                constexpr int NP = decltype(npc)::value, NT = 2 * NP;
                float s[NT][4];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) s[nt][e] = 0.0f;
                {
                    uint32_t kf[2][NP][4];
#pragma unroll
                    for (int pp = 0; pp < NP; ++pp) ldmatrix_x4(k_base + pp * 2 * kTcPageBytes + tile_off_k4(k_tok, k_chunk), kf[0][pp]);
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        if (ks + 1 < 8) {
#pragma unroll
                            for (int pp = 0; pp < NP; ++pp)
                                ldmatrix_x4(k_base + pp * 2 * kTcPageBytes + tile_off_k4(k_tok, 2 * (ks + 1) + k_chunk), kf[(ks + 1) & 1][pp]);
                        }
#pragma unroll
                        for (int pp = 0; pp < NP; ++pp) {
                            mma_bf16_pure(s[2 * pp], qf[ks], kf[ks & 1][pp][0], kf[ks & 1][pp][1]);
                            mma_bf16_pure(s[2 * pp + 1], qf[ks], kf[ks & 1][pp][2], kf[ks & 1][pp][3]);
                        }
                    }
                }
                if ((pg + 2 * (NP - 1)) * kPage + kPage - 1 > ctx_len) {   // only pages that reach past the cached context hold hidden keys
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const int j0 = (pg + 2 * (nt >> 1)) * kPage + (nt & 1) * 8 + c0;
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if (j0 + (e & 1) > ((e < 2) ? jmax_lo : jmax_hi)) s[nt][e] = -INFINITY;
                    }
                }
                float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    mx[0] = fmaxf(mx[0], fmaxf(s[nt][0], s[nt][1]));
                    mx[1] = fmaxf(mx[1], fmaxf(s[nt][2], s[nt][3]));
                }
                float alpha[2], mc[2];
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
                    mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
                    const float m_new = fmaxf(m_run[r], mx[r]);
                    const float msafe = (m_new == -INFINITY) ? 0.0f : m_new;
                    alpha[r] = fast_exp2((m_run[r] - msafe) * cs);
                    mc[r] = msafe * cs;
                    m_run[r] = m_new;
                }
                // the first V fragments travel while the exponentials are computed
                const uint32_t v_base = k_base + 4 * kTcPageBytes;
                constexpr int NV = 8 * NP;               // V fragment loads of the step: (page pp, 16 columns jj)
                uint32_t vf[3][4];
                ldmatrix_x4_trans(v_base + tile_off(v_tok, v_chunk), vf[0]);
                ldmatrix_x4_trans(v_base + tile_off(v_tok, 2 + v_chunk), vf[1]);
                float sum[2] = {0.0f, 0.0f};
                uint32_t pf[NP][4];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const float p0 = fast_exp2(fmaf(s[nt][0], cs, -mc[0])), p1 = fast_exp2(fmaf(s[nt][1], cs, -mc[0]));
                    const float p2 = fast_exp2(fmaf(s[nt][2], cs, -mc[1])), p3 = fast_exp2(fmaf(s[nt][3], cs, -mc[1]));
                    sum[0] += p0 + p1;
                    sum[1] += p2 + p3;
                    pf[nt >> 1][2 * (nt & 1)] = pack_bf16(p0, p1);
                    pf[nt >> 1][2 * (nt & 1) + 1] = pack_bf16(p2, p3);
                }
                l_run[0] = l_run[0] * alpha[0] + sum[0];
                l_run[1] = l_run[1] * alpha[1] + sum[1];
                if (__any_sync(0xffffffffu, alpha[0] != 1.0f || alpha[1] != 1.0f)) {
#pragma unroll
                    for (int jo = 0; jo < 16; ++jo) {
                        o[jo][0] *= alpha[0];
                        o[jo][1] *= alpha[0];
                        o[jo][2] *= alpha[1];
                        o[jo][3] *= alpha[1];
                    }
                }
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    const int pp = i >> 3, jj = i & 7;
                    if (i + 2 < NV) {
                        const int pn = (i + 2) >> 3, jn = (i + 2) & 7;
                        ldmatrix_x4_trans(v_base + pn * 2 * kTcPageBytes + tile_off(v_tok, 2 * jn + v_chunk), vf[(i + 2) % 3]);
                    }
                    mma_bf16_pure(o[2 * jj], pf[pp], vf[i % 3][0], vf[i % 3][1]);
                    mma_bf16_pure(o[2 * jj + 1], pf[pp], vf[i % 3][2], vf[i % 3][3]);
                }
            };
            // The same step with the operands swapped (tails of at most 8 rows).  S^T[16 keys, 8 rows] per page: A = the K
            // page (keys x head dim, as stored), B = Q^T; this lane holds keys g and g + 8 of rows 2 t and 2 t + 1, so
            // a row's maximum is taken over the lanes of equal t.  P^T becomes the B operand of O^T += V^T P^T through
            // movmatrix (key-major pairs -> row-major pairs); A = the V page read transposed (head dim x keys).
            // o[mt] holds O^T: head-dim elements 16 mt + g and + 8 of rows 2 t and 2 t + 1.
            auto tail_step8 = [&](auto npc, uint32_t k_base, int pg) {
                constexpr int NP = decltype(npc)::value;   // consecutive pages of the group
                constexpr int DK = 4, DV = 6;              // fragment loads in flight ahead of the MMAs
                float s[NP][4];
#pragma unroll
                for (int pp = 0; pp < NP; ++pp)
#pragma unroll
                    for (int e = 0; e < 4; ++e) s[pp][e] = 0.0f;
                {
                    uint32_t kf[DK][NP][4];
#pragma unroll
                    for (int ks = 0; ks < DK - 1; ++ks)
#pragma unroll
                        for (int pp = 0; pp < NP; ++pp) ldmatrix_x4(k_base + pp * kTcPageBytes + tile_off_k4(v_tok, 2 * ks + v_chunk), kf[ks][pp]);
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        if (ks + DK - 1 < 8) {
#pragma unroll
                            for (int pp = 0; pp < NP; ++pp)
                                ldmatrix_x4(k_base + pp * kTcPageBytes + tile_off_k4(v_tok, 2 * (ks + DK - 1) + v_chunk), kf[(ks + DK - 1) % DK][pp]);
                        }
#pragma unroll
                        for (int pp = 0; pp < NP; ++pp) mma_bf16_pure(s[pp], kf[ks % DK][pp], qf[ks][0], qf[ks][1]);
                    }
                }
                if ((pg + NP - 1) * kPage + kPage - 1 > ctx_len) {
#pragma unroll
                    for (int pp = 0; pp < NP; ++pp) {
                        const int j0 = (pg + pp) * kPage + r_lo;
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if (j0 + ((e >> 1) << 3) > ((e & 1) ? jmax_hi : jmax_lo)) s[pp][e] = -INFINITY;
                    }
                }
                float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
                for (int pp = 0; pp < NP; ++pp) {
                    mx[0] = fmaxf(mx[0], fmaxf(s[pp][0], s[pp][2]));
                    mx[1] = fmaxf(mx[1], fmaxf(s[pp][1], s[pp][3]));
                }
#pragma unroll
                for (int sh = 4; sh < 32; sh <<= 1) {
                    mx[0] = fmaxf(mx[0], __shfl_xor_sync(0xffffffffu, mx[0], sh));
                    mx[1] = fmaxf(mx[1], __shfl_xor_sync(0xffffffffu, mx[1], sh));
                }
                float alpha[2], mc[2];
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    const float m_new = fmaxf(m_run[r], mx[r]);
                    const float msafe = (m_new == -INFINITY) ? 0.0f : m_new;
                    alpha[r] = fast_exp2((m_run[r] - msafe) * cs);
                    mc[r] = msafe * cs;
                    m_run[r] = m_new;
                }
                // the first V fragments travel while the exponentials are computed
                const uint32_t v_base = k_base + 4 * kTcPageBytes;
                constexpr int NV = 8 * NP;               // V fragment loads of the step: (page pp, 16 head-dim elements mt)
                uint32_t vf[DV][4];
#pragma unroll
                for (int i = 0; i < DV - 1; ++i) ldmatrix_x4_trans(v_base + (i >> 3) * kTcPageBytes + tile_off(k_tok, 2 * (i & 7) + k_chunk), vf[i]);
                float sum[2] = {0.0f, 0.0f};
                uint32_t pb[NP][2];
#pragma unroll
                for (int pp = 0; pp < NP; ++pp) {
                    const float p0 = fast_exp2(fmaf(s[pp][0], cs, -mc[0])), p1 = fast_exp2(fmaf(s[pp][1], cs, -mc[1]));
                    const float p2 = fast_exp2(fmaf(s[pp][2], cs, -mc[0])), p3 = fast_exp2(fmaf(s[pp][3], cs, -mc[1]));
                    sum[0] += p0 + p2;
                    sum[1] += p1 + p3;
                    pb[pp][0] = movmatrix_trans(pack_bf16(p0, p1));      // keys 0-7: (row g; keys 2 t, 2 t + 1)
                    pb[pp][1] = movmatrix_trans(pack_bf16(p2, p3));      // keys 8-15
                }
                l_run[0] = l_run[0] * alpha[0] + sum[0];                 // this lane's keys only; summed over the lanes at the end
                l_run[1] = l_run[1] * alpha[1] + sum[1];
                if (__any_sync(0xffffffffu, alpha[0] != 1.0f || alpha[1] != 1.0f)) {
#pragma unroll
                    for (int mt = 0; mt < 8; ++mt) {
                        o[mt][0] *= alpha[0];
                        o[mt][1] *= alpha[1];
                        o[mt][2] *= alpha[0];
                        o[mt][3] *= alpha[1];
                    }
                }
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    const int pp = i >> 3, mt = i & 7;
                    if (i + DV - 1 < NV) {
                        const int in = i + DV - 1;
                        ldmatrix_x4_trans(v_base + (in >> 3) * kTcPageBytes + tile_off(k_tok, 2 * (in & 7) + k_chunk), vf[in % DV]);
                    }
                    mma_bf16_pure(o[mt], vf[i % DV], pb[pp][0], pb[pp][1]);
                }
            };
            for (int g = 0; g < n_groups; ++g) {
                const int gc = G0 + g, gs = gc % kTcGroupStages;
                if (!__all_sync(0xffffffffu, mbar_wait(full_bar + 8 * gs, (gc / kTcGroupStages) & 1, &c->abort))) {
                    failed = true;
                    break;
                }
                if (swapped) {
                    const int np = min(4, n_pages - 4 * g);
                    const uint32_t k_grp = smem_u32(ring + gs * kTcGroupBytes);
                    // the warps take the groups alternately, a whole group (64 keys) per softmax step
                    if ((g & 1) == tw) {
                        if (np == 4) tail_step8(std::integral_constant<int, 4>(), k_grp, item.page_begin + 4 * g);
                        else
                            for (int j = 0; j < np; ++j) tail_step8(std::integral_constant<int, 1>(), k_grp + j * kTcPageBytes, item.page_begin + 4 * g + j);
                    }
                } else if (has_tail) {
                    const int np = min(4, n_pages - 4 * g);
                    const uint32_t k_grp = smem_u32(ring + gs * kTcGroupBytes);
                    // this warp's pages of the group, tw and tw + 2, go through one softmax step together: twice as
                    // many independent MMA chains per step and half as many steps
                    if (tw + 2 < np) tail_step(std::integral_constant<int, 2>(), k_grp + tw * kTcPageBytes, item.page_begin + 4 * g + tw);
                    else if (tw < np) tail_step(std::integral_constant<int, 1>(), k_grp + tw * kTcPageBytes, item.page_begin + 4 * g + tw);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty_bar + 8 * gs);     // this warp is done with the group's stage
            }
            if (failed) c->abort = 1;
            if (swapped) {
                // both warps leave (m, l, O) in the merge buffer: [warp][row][head dim]
#pragma unroll
                for (int sh = 4; sh < 32; sh <<= 1) {
                    l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], sh);
                    l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], sh);
                }
                float* mo = t_o + tw * 8 * kTcTailStride;
#pragma unroll
                for (int mt = 0; mt < 8; ++mt) {
                    mo[c0 * kTcTailStride + 16 * mt + r_lo] = o[mt][0];
                    mo[(c0 + 1) * kTcTailStride + 16 * mt + r_lo] = o[mt][1];
                    mo[c0 * kTcTailStride + 16 * mt + r_lo + 8] = o[mt][2];
                    mo[(c0 + 1) * kTcTailStride + 16 * mt + r_lo + 8] = o[mt][3];
                }
                if (r_lo == 0) {
                    t_ml[(tw * 8 + c0) * 2] = m_run[0];
                    t_ml[(tw * 8 + c0) * 2 + 1] = l_run[0];
                    t_ml[(tw * 8 + c0 + 1) * 2] = m_run[1];
                    t_ml[(tw * 8 + c0 + 1) * 2 + 1] = l_run[1];
                }
            } else if (has_tail) {
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
                    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
                }
                if (tw == 1) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        *reinterpret_cast<float2*>(t_o + r_lo * kTcTailStride + j * 8 + c0) = make_float2(o[j][0], o[j][1]);
                        *reinterpret_cast<float2*>(t_o + (r_lo + 8) * kTcTailStride + j * 8 + c0) = make_float2(o[j][2], o[j][3]);
                    }
                    if ((lane & 3) == 0) {
                        t_ml[2 * r_lo] = m_run[0];
                        t_ml[2 * r_lo + 1] = l_run[0];
                        t_ml[2 * (r_lo + 8)] = m_run[1];
                        t_ml[2 * (r_lo + 8) + 1] = l_run[1];
                    }
                }
            }
            if (bar_any(6, 32 * kTcTailWarps, failed)) {
                failed = true;
                break;
            }
            if (swapped) {
                // the 64 threads merge the two warps' rows and write them out, four head-dim elements at a time
                for (int i = tw * 32 + lane; i < M * 32; i += 32 * kTcTailWarps) {
                    const int rr = i >> 5, c4 = (i & 31) << 2;
                    const float m0 = t_ml[rr * 2], l0 = t_ml[rr * 2 + 1], m1 = t_ml[(8 + rr) * 2], l1 = t_ml[(8 + rr) * 2 + 1];
                    const float m_all = fmaxf(m0, m1);
                    const float w0 = m0 == -INFINITY ? 0.0f : fast_exp2((m0 - m_all) * cs);
                    const float w1 = m1 == -INFINITY ? 0.0f : fast_exp2((m1 - m_all) * cs);
                    const float l_all = l0 * w0 + l1 * w1;
                    const float inv = l_all > 0.0f ? 1.0f / l_all : 0.0f;
                    const float f0 = w0 * inv, f1 = w1 * inv;
                    const float4 v0 = *reinterpret_cast<const float4*>(t_o + rr * kTcTailStride + c4);
                    const float4 v1 = *reinterpret_cast<const float4*>(t_o + (8 + rr) * kTcTailStride + c4);
                    const float4 v = make_float4(v0.x * f0 + v1.x * f1, v0.y * f0 + v1.y * f1, v0.z * f0 + v1.z * f1, v0.w * f0 + v1.w * f1);
                    const int R = row0 + rr;
                    const int t = R / group, hl = R - t * group;
                    const size_t orow = (size_t)(q0 + t) * a.n_q_heads + kvh * group + hl;
                    const float lse_nat = l_all > 0.0f ? (m_all * cs + log2f(l_all)) * 0.6931471805599453f : -INFINITY;
                    if (item.n_chunks == 1) {
                        *reinterpret_cast<uint2*>(a.out + orow * 128 + c4) = make_uint2(pack_bf16(v.x, v.y), pack_bf16(v.z, v.w));
                        if (a.lse && c4 == 0) a.lse[orow] = lse_nat;
                    } else {
                        const size_t prow = (size_t)item.part_row + 128 + rr;
                        *reinterpret_cast<float4*>(a.part_o + prow * 128 + c4) = v;
                        if (c4 == 0) a.part_lse[prow] = lse_nat;
                    }
                }
            } else if (has_tail && tw == 0) {
                // each lane merges the elements it holds with the ones the same lane of the other warp held
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    const int rr = r_lo + 8 * r;
                    const float m_o = t_ml[2 * rr], l_o = t_ml[2 * rr + 1];
                    const float m_all = fmaxf(m_run[r], m_o);
                    const float w_s = m_run[r] == -INFINITY ? 0.0f : fast_exp2((m_run[r] - m_all) * cs);
                    const float w_o = m_o == -INFINITY ? 0.0f : fast_exp2((m_o - m_all) * cs);
                    const float l_all = l_run[r] * w_s + l_o * w_o;
                    const float inv = l_all > 0.0f ? 1.0f / l_all : 0.0f;
                    const float f_s = w_s * inv, f_o = w_o * inv;
                    if (rr < M) {
                        const int R = row0 + rr;
                        const int t = R / group, hl = R - t * group;
                        const size_t orow = (size_t)(q0 + t) * a.n_q_heads + kvh * group + hl;
                        const float lse_nat = l_all > 0.0f ? (m_all * cs + log2f(l_all)) * 0.6931471805599453f : -INFINITY;
                        const float* po = t_o + rr * kTcTailStride + c0;
                        if (item.n_chunks == 1) {
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const float2 v = *reinterpret_cast<const float2*>(po + j * 8);
                                *reinterpret_cast<uint32_t*>(a.out + orow * 128 + j * 8 + c0) =
                                    pack_bf16(o[j][2 * r] * f_s + v.x * f_o, o[j][2 * r + 1] * f_s + v.y * f_o);
                            }
                            if (a.lse && (lane & 3) == 0) a.lse[orow] = lse_nat;
                        } else {
                            const size_t prow = (size_t)item.part_row + 128 + rr;
                            float* pd = a.part_o + prow * 128 + c0;
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const float2 v = *reinterpret_cast<const float2*>(po + j * 8);
                                *reinterpret_cast<float2*>(pd + j * 8) = make_float2(o[j][2 * r] * f_s + v.x * f_o, o[j][2 * r + 1] * f_s + v.y * f_o);
                            }
                            if ((lane & 3) == 0) a.part_lse[prow] = lse_nat;
                        }
                    }
                }
            }
            sched_release(c, kPhase, n);
            G0 += n_groups;
        }
    }
    if (failed) {
        atomicExch(a.status, DCUT_DEV_ATTN_WAIT_TIMEOUT);
        c->abort = 1;
    }
}


template <int DH>
constexpr int kDataBytes = (DH == 128 && kTcRingBytes > MmaSmem<DH>::kTotal) ? kTcRingBytes : MmaSmem<DH>::kTotal;
template <int DH>
constexpr int kTailPad = DH == 128 ? ((kTcTailBytes + 1023) / 1024) * 1024 : 0;   // merge buffer of the tcgen05 phase's tail warps
template <int DH>
constexpr int kSmemBytes = kDataBytes<DH> + kTailPad<DH> + 1024 /* alignment slack */ + 1024 /* control block */;
static_assert(sizeof(Ctrl) <= 1024, "control block");

// Persistent kernel: one CTA per SM runs its segment of the work stream, first its tcgen05-path items, then its
// warp-level-MMA items.
template <int DH>
__global__ void __launch_bounds__(kThreads, 1)
attn_item_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map,
                 const __grid_constant__ CUtensorMap k2_map, AttnArgs a) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Ctrl* c = reinterpret_cast<Ctrl*>(smem + kDataBytes<DH> + kTailPad<DH>);
    __shared__ float xm[2][128];       // [team][row]: the teams' running maxima at the end of an item (tcgen05 phase)
    __shared__ float xl[2][128];       // [team][row]: their running sums
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kMmaStages; ++s) {
            mbar_init(smem_u32(&c->ring_full[s]), 1);    // tcgen05 phase: one arrival (with the group's byte count)
            mbar_init(smem_u32(&c->ring_empty[s]), 1 + (a.tail_on ? kTcTailWarps : 0));   // the commit of the stage's last MMA + the tail warps
        }
        for (int b = 0; b < kTcSBufs; ++b) {
            mbar_init(smem_u32(&c->s_full[b]), 1);
            mbar_init(smem_u32(&c->p_full[b]), kTcSoftmaxThreads / 2);   // the team that owns the group
            mbar_init(smem_u32(&c->pv_done[b]), 1);
        }
        mbar_init(smem_u32(&c->q_ready), kTcSoftmaxThreads);
        mbar_init(smem_u32(&c->o_free), kTcSoftmaxThreads);
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&c->sched_full[0][s]), 1);
            mbar_init(smem_u32(&c->sched_full[1][s]), 1);
            mbar_init(smem_u32(&c->sched_empty[0][s]), 1 + kTcSoftmaxThreads / 32 + (a.tail_on ? kTcTailWarps : 0));   // MMA warp + softmax warps + tail warps
            mbar_init(smem_u32(&c->sched_empty[1][s]), kMmaWarps);
        }
        mbar_init(smem_u32(&c->geom_a), kMmaWarps + 1);
        mbar_init(smem_u32(&c->geom_b), 1);
        c->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (DH == 128 && warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&c->tmem_base)), "n"(kTcCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // launched with programmatic stream serialization: everything above overlaps the plan kernel; nothing it writes
    // is read before this wait
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // this CTA's segment of the work stream: its tcgen05 items first, then its warp-level items
    const int n_entries = a.plan[0], e_split = a.plan[1];
    const AttnSeg s0 = a.segs[blockIdx.x], s1 = a.segs[blockIdx.x + 1];
    const SegCursor tc_cur = seg_range(s0, s1, 0, e_split), mma_cur = seg_range(s0, s1, e_split, n_entries);
    if (DH == 128 && seg_before(tc_cur.e, tc_cur.h, tc_cur.p, tc_cur.e1, tc_cur.h1, tc_cur.p1)) {
        tc_phase(k2_map, v_map, a, smem, reinterpret_cast<float*>(smem + kDataBytes<DH>), c, xm, xl, tc_cur);
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    }
    if (seg_before(mma_cur.e, mma_cur.h, mma_cur.p, mma_cur.e1, mma_cur.h1, mma_cur.p1) && !ABORTED(c))
        mma_phase<DH>(k_map, v_map, a, smem, c, mma_cur);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the combine kernel may take this SM
    tc_fence_before();
    __syncthreads();
    if (DH == 128 && warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(c->tmem_base), "n"(kTcCols) : "memory");
    }
}

// ------------------------------------------------------------------------------------------------
// combine the pieces of the items that segment boundaries cut: one CTA per boundary

struct CombineArgs {
    const AttnCut* cuts;
    const float* part_o;
    const float* part_lse;
    int n_q_heads, n_kv_heads;
    __nv_bfloat16* out;
    float* lse;
};

template <int DH>
__global__ void __launch_bounds__(1024) attn_combine_kernel(CombineArgs a) {
    // grid: x: boundary b = blockIdx.x + 1 between segments b - 1 and b; y: block of 32 query rows; a warp merges one row
    // (the loads of a row depend on one another, so the rows must not queue up behind each other).
    // Launched with programmatic stream serialization (see attn_item_kernel).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int b = blockIdx.x + 1;
    const AttnCut en = a.cuts[b];
    if (en.pieces == 0 || (int)blockIdx.y * 32 >= en.rows) return;   // no item to merge at this boundary, or no rows for this block
    const int m = en.pieces - 1;
    struct { int h; } sg = {en.kv_head};
    const int group = a.n_q_heads / a.n_kv_heads;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int kPer = DH / 32;
    for (int R = blockIdx.y * 32 + warp; R < en.rows; R += 32 * gridDim.y) {
        // piece 0 is in segment b - 1 (the item begins there: its second slot); piece c >= 1 in segment b + c - 1 (first slot)
        const int t = (en.row0 + R) / group, hl = (en.row0 + R) - t * group;
        const size_t orow = (size_t)(en.q0 + t) * a.n_q_heads + sg.h * group + hl;
        __nv_bfloat16* op = a.out + orow * DH + lane * kPer;
        if (m == 1) {
            // two pieces (nearly every cut): the four loads leave together, one trip to L2 instead of two per piece;
            // the same arithmetic in the same order as the general loop below
            const size_t r0 = (size_t)(2 * (b - 1) + 1) * dcut_plan::kSlotRows + R, r1 = (size_t)(2 * b) * dcut_plan::kSlotRows + R;
            const float l0 = __ldcg(a.part_lse + r0), l1 = __ldcg(a.part_lse + r1);
            float o0[kPer], o1[kPer];
#pragma unroll
            for (int e = 0; e < kPer; ++e) {
                o0[e] = __ldcg(a.part_o + r0 * DH + lane * kPer + e);
                o1[e] = __ldcg(a.part_o + r1 * DH + lane * kPer + e);
            }
            const float m_all = fmaxf(l0, l1);
            const float w0 = (l0 == -INFINITY) ? 0.0f : __expf(l0 - m_all), w1 = (l1 == -INFINITY) ? 0.0f : __expf(l1 - m_all);
            const float wsum = (0.0f + w0) + w1;
            const float inv = wsum > 0.0f ? 1.0f / wsum : 0.0f;
#pragma unroll
            for (int e = 0; e < kPer; e += 2) {
                const float x0 = fmaf(w1, o1[e], fmaf(w0, o0[e], 0.0f)), x1 = fmaf(w1, o1[e + 1], fmaf(w0, o0[e + 1], 0.0f));
                *reinterpret_cast<uint32_t*>(op + e) = pack_bf16(x0 * inv, x1 * inv);
            }
            if (a.lse && lane == 0) a.lse[orow] = wsum > 0.0f ? m_all + logf(wsum) : -INFINITY;
            continue;
        }
        float m_all = -INFINITY;
        for (int c = 0; c <= m; ++c) {
            const size_t prow = (size_t)(c == 0 ? 2 * (b - 1) + 1 : 2 * (b + c - 1)) * dcut_plan::kSlotRows + R;
            m_all = fmaxf(m_all, a.part_lse[prow]);
        }
        float acc[kPer];
#pragma unroll
        for (int e = 0; e < kPer; ++e) acc[e] = 0.0f;
        float wsum = 0.0f;
        for (int c = 0; c <= m; ++c) {
            const size_t prow = (size_t)(c == 0 ? 2 * (b - 1) + 1 : 2 * (b + c - 1)) * dcut_plan::kSlotRows + R;
            const float l = a.part_lse[prow];
            const float w = (l == -INFINITY) ? 0.0f : __expf(l - m_all);
            wsum += w;
            const float* po = a.part_o + prow * DH + lane * kPer;
#pragma unroll
            for (int e = 0; e < kPer; ++e) acc[e] += w * po[e];
        }
        const float inv = wsum > 0.0f ? 1.0f / wsum : 0.0f;
#pragma unroll
        for (int e = 0; e < kPer; e += 2) *reinterpret_cast<uint32_t*>(op + e) = pack_bf16(acc[e] * inv, acc[e + 1] * inv);
        if (a.lse && lane == 0) a.lse[orow] = wsum > 0.0f ? m_all + logf(wsum) : -INFINITY;
    }
}

// ------------------------------------------------------------------------------------------------
// host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

dcut_status make_cache_map(dcut_ctx* ctx, CUtensorMap* map, const void* base, long long num_pages) {
    // The cache seen as a 3-D tensor {64 columns, token rows, head_dim / 64 column halves}: one box
    // {64, 16, halves} is a whole (page, kv head) tile and lands in shared memory as
    // [half][16 rows][64 columns] with the 128-byte swizzle the ldmatrix addressing expects.
    const int DH = ctx->lim.head_dim;
    cuuint64_t dims[3] = {64, (cuuint64_t)num_pages * ctx->lim.n_kv_heads * kPage, (cuuint64_t)(DH / 64)};
    cuuint64_t strides[2] = {(cuuint64_t)DH * 2, 128};
    cuuint32_t box[3] = {64, kPage, (cuuint32_t)(DH / 64)};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
        map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return dcut_fail(ctx, DCUT_ECUDA, "cuTensorMapEncodeTiled failed (%d)", (int)r);
    return DCUT_OK;
}

template <int DH>
dcut_status launch_t(dcut_ctx* ctx, const CUtensorMap& km, const CUtensorMap& vm, const CUtensorMap& k2m, const AttnArgs& aa,
                     const CombineArgs& ca, int T_cap, cudaStream_t stream) {
    // Both kernels may be scheduled before their predecessor has finished (they wait on the device before reading
    // its results), which hides the launch latency between the three kernels of the call.
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(ctx->sm_count);   // persistent: one CTA per SM
    lc.blockDim = dim3(kThreads);
    lc.dynamicSmemBytes = kSmemBytes<DH>;
    lc.stream = stream;
    lc.attrs = attr;
    lc.numAttrs = 1;
    dcut_status st = dcut_check_cuda(ctx, cudaLaunchKernelEx(&lc, attn_item_kernel<DH>, km, vm, k2m, aa), "launch attn_item_kernel");
    if (st != DCUT_OK) return st;
    (void)T_cap;
    if (ctx->sm_count < 2) return DCUT_OK;      // one segment: no boundary, nothing to merge
    lc.gridDim = dim3(ctx->sm_count - 1, (dcut_plan::kSlotRows + 31) / 32);
    lc.blockDim = dim3(1024);
    lc.dynamicSmemBytes = 0;
    return dcut_check_cuda(ctx, cudaLaunchKernelEx(&lc, attn_combine_kernel<DH>, ca), "launch attn_combine_kernel");
}

}  // namespace

dcut_status dcut_init_verify_attn(dcut_ctx* ctx) {
    cudaError_t e = cudaFuncSetAttribute(attn_item_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes<128>);
    if (e != cudaSuccess) return dcut_check_cuda(ctx, e, "cudaFuncSetAttribute(attn 128)");
    e = cudaFuncSetAttribute(attn_item_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes<64>);
    if (e != cudaSuccess) return dcut_check_cuda(ctx, e, "cudaFuncSetAttribute(attn 64)");
    {
        const char* env = getenv("DCUT_ATTN_TC_MIN_ROWS");   // query rows from which an item goes to the tcgen05 kernel
        ctx->attn_tc_min_rows = env ? atoi(env) : 17;
        env = getenv("DCUT_ATTN_TAIL_ROWS");     // 0: a query tile above 128 rows becomes two items (experiments)
        ctx->attn_tail_rows = env ? (atoi(env) > 0 ? kTcTailRows : 0) : kTcTailRows;
    }
    e = cudaFuncSetAttribute(attn_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 8 * (2 * DCUT_MAX_KEYS + 1) + 4 * (2 * DCUT_MAX_KEYS + 1));
    if (e != cudaSuccess) return dcut_check_cuda(ctx, e, "cudaFuncSetAttribute(attn plan)");
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn)
        return dcut_fail(ctx, DCUT_ECUDA, "cuTensorMapEncodeTiled entry point not available");
    ctx->encode_tiled = fn;
    return DCUT_OK;
}

void dcut_fill_plan_args(dcut_ctx* ctx, const int* ctx_lens, const int* cu_q, int B, dcut_plan::PlanArgs* out) {
    dcut_plan::PlanArgs& pa = *out;
    pa.ctx_lens = ctx_lens;
    pa.cu_q = cu_q;
    pa.B = B;
    pa.n_q_heads = ctx->lim.n_q_heads;
    pa.n_kv_heads = ctx->lim.n_kv_heads;
    pa.n_sm = ctx->sm_count;
    pa.min_chunk_pages = ctx->attn_min_chunk_pages;
    pa.status = ctx->d_status;
    pa.tc_min_rows = ctx->lim.head_dim == 128 ? ctx->attn_tc_min_rows : 1 << 30;
    pa.max_item_rows = 128;
    // (no tail-row items when the shapes cannot need them: the item kernel then runs without its tail warps)
    const bool tail_on = ctx->attn_tail_rows > 0 && (ctx->lim.max_gamma + 1) * (ctx->lim.n_q_heads / ctx->lim.n_kv_heads) > 128;
    pa.tail_rows = (ctx->lim.head_dim == 128 && ctx->attn_tc_min_rows <= 128 && tail_on) ? ctx->attn_tail_rows : 0;
    pa.max_entries = ctx->max_entries;
    pa.entries = ctx->d_entries;
    pa.segs = ctx->d_segs;
    pa.cuts = ctx->d_cuts;
    pa.plan = ctx->d_plan;
}

dcut_status dcut_launch_verify_attn(dcut_ctx* ctx, const void* q, const void* k_cache, const void* v_cache,
                                    long long num_pages, const int* block_table, int block_table_stride,
                                    const int* ctx_lens, const int* cu_q, int B, int T_cap, float scale,
                                    void* out, float* lse, int reuse_plan, cudaStream_t stream) {
    CUtensorMap km, vm, k2m;
    dcut_status st = make_cache_map(ctx, &km, k_cache, num_pages);
    if (st != DCUT_OK) return st;
    st = make_cache_map(ctx, &vm, v_cache, num_pages);
    if (st != DCUT_OK) return st;
    k2m = km;
    if (ctx->lim.head_dim == 128) {
        // The K cache for the tcgen05 phase: token rows of 128 columns seen as (64 columns, 8 rows, 2 halves, groups of
        // 8 rows), so that a {64, 8, 2, 2} box (one page: 16 rows, 4 KB) arrives as [group][half][row][64 columns]:
        // each half is a K-major tile of 128-byte rows whose 8-row groups are 2048 bytes apart.
        cuuint64_t dims[4] = {64, 8, 2, (cuuint64_t)num_pages * ctx->lim.n_kv_heads * kPage / 8};
        cuuint64_t strides[3] = {256, 128, 2048};
        cuuint32_t box[4] = {64, 8, 2, 2}, estr[4] = {1, 1, 1, 1};
        CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
            &k2m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(k_cache), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return dcut_fail(ctx, DCUT_ECUDA, "cuTensorMapEncodeTiled failed (%d)", (int)r);
    }

    PlanArgs pa;
    dcut_fill_plan_args(ctx, ctx_lens, cu_q, B, &pa);
    // the selector may have left the work list of exactly this batch ready (dcut_enable_plan_in_select)
    if (ctx->plan_in_select && ctx->plan_cu_q == cu_q && ctx->plan_ctx_lens == ctx_lens && ctx->plan_B == B) reuse_plan = 1;
    if (!reuse_plan) {   // reuse_plan: the previous launch on this stream had the same ctx_lens, cu_q and B (its work list stands)
        ctx->plan_cu_q = nullptr;   // the list now belongs to this call's batch
        st = dcut_check_cuda(ctx, dcut_launch_pdl(attn_plan_kernel, dim3(1), dim3(B <= 256 ? 256 : kPlanThreads),
                                                  sizeof(long long) * (2 * B + 1) + sizeof(int) * (2 * B + 1), stream, pa),
                             "launch attn_plan_kernel");
        if (st != DCUT_OK) return st;
    }

    AttnArgs aa;
    aa.q = static_cast<const __nv_bfloat16*>(q);
    aa.block_table = block_table;
    aa.block_table_stride = block_table_stride;
    aa.ctx_lens = ctx_lens;
    aa.cu_q = cu_q;
    aa.entries = ctx->d_entries;
    aa.segs = ctx->d_segs;
    aa.plan = ctx->d_plan;
    aa.n_q_heads = ctx->lim.n_q_heads;
    aa.n_kv_heads = ctx->lim.n_kv_heads;
    aa.num_pages = num_pages;
    aa.scale_log2 = scale * 1.4426950408889634f;
    aa.q_row_bytes = ctx->lim.head_dim * 2;
    aa.tail_on = ctx->attn_tail_rows > 0 && (ctx->lim.max_gamma + 1) * (ctx->lim.n_q_heads / ctx->lim.n_kv_heads) > 128;
    aa.out = static_cast<__nv_bfloat16*>(out);
    aa.lse = lse;
    aa.part_o = ctx->d_part_o;
    aa.part_lse = ctx->d_part_lse;
    aa.status = ctx->d_status;

    CombineArgs ca;
    ca.cuts = ctx->d_cuts;
    ca.part_o = ctx->d_part_o;
    ca.part_lse = ctx->d_part_lse;
    ca.n_q_heads = ctx->lim.n_q_heads;
    ca.n_kv_heads = ctx->lim.n_kv_heads;
    ca.out = static_cast<__nv_bfloat16*>(out);
    ca.lse = lse;

    if (ctx->lim.head_dim == 128) return launch_t<128>(ctx, km, vm, k2m, aa, ca, T_cap, stream);
    return launch_t<64>(ctx, km, vm, k2m, aa, ca, T_cap, stream);
}
