// dcut_layer_forward: one pre-norm decoder layer over the ragged packed batch (full-layer workload).
//
//   h1 = x + Wo . Attn(RoPE(Wqkv . RMSNorm(x)))        y = h1 + Wd . (SiLU(Wg . n2) * (Wu . n2)),  n2 = RMSNorm(h1)
//
// Kernels in this file
//   rmsnorm_kernel        one CTA per packed token, fp32 sum of squares, bf16 out
//   rope_append_kernel    rotate-half RoPE on q and k heads, K/V of the new tokens written into the paged cache at
//                         position L_i + t, q written as the attention kernel's [T, Hq, Dh] input
//   gemm_tcgen05_kernel   C[M, N] = A[M, K] . B[N, K]^T on the 5th-generation tensor cores.  Persistent; launched as
//                         clusters of two CTAs.  After reading the packed length it looks up how to run: 128-row
//                         tiles on single SMs (tcgen05.mma M128 K16), 256-row tiles on pairs of SMs (cta_group::2,
//                         M256, each CTA loading half of B), or a pair sharing one 128-row tile with half of K each;
//                         and how wide the tile is (256, 224, ..., 64 columns = the MMA's N).  Operands
//                         are staged by TMA as 128-byte-swizzled K-major tiles (BK = 64); one elected lane issues the
//                         MMAs and releases stages with tcgen05.commit; two accumulators in tensor memory let the four
//                         epilogue warps (tcgen05.ld) work on one tile while the next is being multiplied.
//                         Epilogues: plain bf16, + residual, SwiGLU (the B tile is 128 gate rows and the 128 matching
//                         up rows, so silu(g) * u is formed in registers and the [T, 2I] intermediate never exists),
//                         or row argmax (the LM head fused with acceptance: the logits are never stored).
// M is ragged and known only on the device (T = cu_q[B]): grids are sized for T_cap, CTAs without work fall through,
// rows past T are computed on whatever the buffers hold and never stored.  Every kernel is launched with programmatic
// dependent launch and waits for its predecessor before touching global memory.
#include <cuda.h>
#include <cuda_bf16.h>
#include <limits.h>
#include <math.h>
#include <stdlib.h>

#include "dcut_internal.h"

namespace {

constexpr int BM = 128, BN = 256, BK = 64, kGemmStages = 4;
constexpr int kATile = BM * BK * 2;            // 16 KB
constexpr int kBTile = BN * BK * 2;            // 32 KB
constexpr int kGemmStageBytes = kATile + kBTile;
constexpr int kGemmThreads = 192;              // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2-5: epilogue
constexpr int kTmemCols = 512;              // two 128 x 256 fp32 accumulators
constexpr int kMaxStages = 12;                 // a narrow tile's stage is smaller: more of them fit the same operand area
constexpr int kGemmSmem = kGemmStages * kGemmStageBytes + 1024 /* align */ + 512 /* two sets of barriers, tmem ptr */;
constexpr int kWaitLimit = 1 << 22;

enum GemmMode { kPlain = 0, kResidual = 1, kSwiGLU = 2, kArgmax = 3 };

// Widths of the output tile that the one-SM mode may use: 256, 224, ..., 64 columns.  A narrower tile costs a little
// efficiency per flop and buys more tiles, which is what a GEMM with fewer than one wave of 128 x 256 tiles needs
// (T = 600, N = 4096: 80 tiles for 148 SMs at width 256, 130 at width 160).  One tensor map of the weight per width
// (box = half the width in rows: a B tile is loaded as two halves, which is also how the SwiGLU tile is put together).
constexpr int kNumBn = 7;
__host__ __device__ constexpr int bn_of(int i) { return BN - 32 * i; }
struct BMaps {
    CUtensorMap m[kNumBn];
};
// The activations' tensor map with the full 128-row box and with a 64-row box: with at most 64 packed rows a tile's
// lower half would only be fetched to be ignored (at T = 64 the A tiles were more than half of what the SMs took in).
struct AMaps {
    CUtensorMap full, half;
};
constexpr unsigned kBnMaskAll = (1u << kNumBn) - 1;
constexpr int kPlanRows = 72;
constexpr int kSplitCost = 50;             // gemm_plan: what the exchange of partial sums between the two SMs costs
constexpr unsigned kBnMaskSwiGLU = 0x55;   // widths whose halves are whole 32-column epilogue steps: 256, 192, 128, 64

// ------------------------------------------------------------------------------------------------ PTX

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (int it = 0; it < kWaitLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (it > 8192) __nanosleep(64);
    }
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// One lane of a converged warp.  Issuing tcgen05 / TMA instructions under this predicate (rather than under
// `lane == 0`) lets the compiler keep their operands in uniform registers; measured on B200 this halves the
// cycles per tcgen05.mma of the issuing thread.
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
// D[tmem] (+)= A[smem desc] . B[smem desc]^T, M128 N256 K16, bf16 in, fp32 accumulate
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes (64 bf16) with the 128-byte
// swizzle: 8-row groups are 1024 bytes apart (stride byte offset), descriptor version 1, layout type 2.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3ffff) >> 4);          // start address, 16-byte units
    d |= (uint64_t)1 << 16;                               // leading byte offset: unused with this swizzle
    d |= (uint64_t)(1024 >> 4) << 32;                     // stride byte offset
    d |= (uint64_t)1 << 46;                               // descriptor version
    d |= (uint64_t)2 << 61;                               // SWIZZLE_128B
    return d;
}
// Instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, N = 256, M = 128.
constexpr uint32_t kIdescNoN = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BM >> 4) << 24);   // N >> 3 goes to bits 17..22

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// ------------------------------------------------------------------------------------------------ GEMM

struct GemmArgs {
    const int* cu_q;   // T = cu_q[B]
    int B;
    int N_out;         // columns of the output (kSwiGLU: the intermediate size I; otherwise N)
    int K;
    int n_tiles;       // output tiles along N
    __nv_bfloat16* out;
    const __nv_bfloat16* residual;   // [T, N_out] or null
    unsigned long long* row_key;     // kArgmax: one packed (ordered maximum, ~column) word per row
    int V;                           // kArgmax: live columns (rows of the weight)
    int pairs;                       // launched as clusters of two CTAs: the pair mode may be chosen
    unsigned bn_mask;                // tile widths whose tensor maps were supplied (bit i: bn_of(i)); bit 0 always
    int force;                       // experiments: -1 = let gemm_plan choose, 0..6 = that width on one SM, 8..14 = on a pair
    unsigned char plan_by_m[kPlanRows];   // gemm_plan for 1, 2, ... row blocks of 128 (the last entry serves all larger counts)
    int* status;
};

// the map of width index i; every address is formed statically (kernel parameter space)
__device__ __forceinline__ const CUtensorMap* pick_map(const BMaps& s, int i) {
    switch (i) {
        case 1: return &s.m[1];
        case 2: return &s.m[2];
        case 3: return &s.m[3];
        case 4: return &s.m[4];
        case 5: return &s.m[5];
        case 6: return &s.m[6];
        default: return &s.m[0];
    }
}

// Epilogue of one 128 x bn accumulator (this thread: tensor-memory lane = output row `row`), for every mode.  Columns
// past N_out (a ragged last tile of a narrow width) were computed on zero weight rows and are not stored.
template <int MODE>
__device__ __forceinline__ void gemm_epilogue(const GemmArgs& g, int T, int row, int n_tile, uint32_t t_row, int bn) {
    if (MODE == kSwiGLU) {
        const int half = bn >> 1, col0 = n_tile * half;
        __nv_bfloat16* orow = g.out + (size_t)row * g.N_out + col0;
#pragma unroll 1
        for (int c = 0; c < half; c += 32) {
            uint32_t gt[32], up[32];
            tc_ld32(t_row + c, gt);
            tc_ld32(t_row + half + c, up);
            tc_wait_ld();
            if (row < T) {
#pragma unroll
                for (int e = 0; e < 32; e += 8) {
                    if (col0 + c + e >= g.N_out) break;
                    uint32_t o[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float g0 = __uint_as_float(gt[e + 2 * j]), g1 = __uint_as_float(gt[e + 2 * j + 1]);
                        const float u0 = __uint_as_float(up[e + 2 * j]), u1 = __uint_as_float(up[e + 2 * j + 1]);
                        o[j] = pack_bf16(g0 / (1.0f + __expf(-g0)) * u0, g1 / (1.0f + __expf(-g1)) * u1);
                    }
                    *reinterpret_cast<uint4*>(orow + c + e) = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
        }
    } else if (MODE == kArgmax) {
        // The bf16 logits an unfused path would store are formed in registers and reduced to the row's
        // (maximum, first column) over this tile; rows merge across tiles with a 64-bit atomicMax on
        // (ordered value << 32 | ~column): largest value, lowest column, whatever order the tiles finish in.
        float best = -INFINITY;
        int bidx = -1;
        const int col0 = n_tile * bn;
#pragma unroll 1
        for (int c = 0; c < bn; c += 32) {
            uint32_t av[32];
            tc_ld32(t_row + c, av);
            tc_wait_ld();
            if (col0 + c < g.V) {
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    const uint32_t pk = pack_bf16(__uint_as_float(av[e]), __uint_as_float(av[e + 1]));
                    const float f0 = bf_lo(pk), f1 = bf_hi(pk);
                    const int col = col0 + c + e;
                    if (col < g.V && f0 > best) {        // strict: the first of equal values stays; NaN never passes
                        best = f0;
                        bidx = col;
                    }
                    if (col + 1 < g.V && f1 > best) {
                        best = f1;
                        bidx = col + 1;
                    }
                }
            }
        }
        if (row < T && bidx >= 0)
            atomicMax(g.row_key + row, ((unsigned long long)dcut_ordered_bits(best) << 32) | (0xffffffffu - (unsigned int)bidx));
    } else {
        const int col0 = n_tile * bn;
        __nv_bfloat16* orow = g.out + (size_t)row * g.N_out + col0;
        const __nv_bfloat16* rrow = MODE == kResidual ? g.residual + (size_t)row * g.N_out + col0 : nullptr;
#pragma unroll 1
        for (int c = 0; c < bn; c += 32) {
            uint32_t av[32];
            tc_ld32(t_row + c, av);
            tc_wait_ld();
            if (row < T) {
#pragma unroll
                for (int e = 0; e < 32; e += 8) {
                    if (col0 + c + e >= g.N_out) break;
                    uint4 res = make_uint4(0, 0, 0, 0);
                    if (MODE == kResidual) res = *reinterpret_cast<const uint4*>(rrow + c + e);
                    const uint32_t rw[4] = {res.x, res.y, res.z, res.w};
                    uint32_t o[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        o[j] = pack_bf16(__uint_as_float(av[e + 2 * j]) + bf_lo(rw[j]),
                                         __uint_as_float(av[e + 2 * j + 1]) + bf_hi(rw[j]));
                    *reinterpret_cast<uint4*>(orow + c + e) = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------ GEMM, pair mode
//
// Pair mode of the GEMM kernel (a cluster of two SMs, tcgen05 cta_group::2): a pair owns a 256 x 256 output tile,
// each CTA its 128 rows.  Each CTA loads its own A tile and HALF of the B tile (128 of the 256 weight rows; for
// SwiGLU the leader's half is the gate rows, the peer's the up rows); the leader's MMA warp issues M256 N256 K16 MMAs
// that read both halves, so an MMA streams 8 KB per SM from shared memory instead of 12 KB and a stage is 32 KB
// instead of 48 KB (six stages fit).  Hand-overs: both CTAs' TMA loads complete on the LEADER's full barrier; the
// leader's commits are multicast to both CTAs' empty / accumulator-full barriers; the peer's epilogue threads arrive
// on the leader's accumulator-empty barrier through distributed shared memory.
// Measured against the one-CTA kernel: 74 us against 86 us for the down projection at T = 512-640 (K = 12288), 81 against
// 90 us for gate/up + SwiGLU at T = 512, but 135 against 92 us for the down projection at T = 1088, where 5 x 16 = 80
// pair tiles need two waves on 74 pairs (and 1280 padded rows are computed instead of 1152): the mode is therefore
// chosen per launch (gemm_plan).

constexpr int kG2Stages = 6;
constexpr int kG2StageBytes = kATile + kBTile / 2;     // 32 KB
constexpr uint32_t kIdesc2NoN = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)((2 * BM) >> 4) << 24);

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_rank(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA tile load whose completion is signalled on a barrier of either CTA of the pair
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar_cluster_addr) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void tc_mma2(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}
// arrives on the barrier at the same offset in both CTAs of the pair once the MMAs issued so far have completed
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((unsigned short)3) : "memory");
}

// One persistent kernel, three ways of running a GEMM and seven tile widths, looked up on the device from the packed
// length (the same answer in every CTA).
//   One SM per tile: a CTA walks the 128 x bn output tiles b, b + gridDim.x, ... (m fastest, so the CTAs running
//   together share weight tiles in L2); a stage holds the tile's A and B bytes, 4 (bn = 256) to 12 stages.
//   A pair of SMs per tile (see above): 256 x bn tiles, six 32 KB stages.  Fewer bytes per flop from L2, but rows
//   padded to 256 and half as many, larger work items.
//   A pair per 128 x bn tile, half of K each (below): for launches whose tiles all fit one wave of pairs.
// In the first two the operand ring and its barriers continue across tiles and the accumulator is double-buffered in
// tensor memory (2 x 256 columns), so the epilogue of one tile overlaps the main loop of the next.
// The cheapest way to run this launch under a model fitted to measurements on the four projections of an 8B-class
// layer at 17 packed lengths from 64 to 1088 (every width, every mode): time = waves x (4 bn + 1664) on one SM per
// tile, waves x (7 bn + 800) on a pair, half a one-SM tile + kSplitCost for a pair splitting K.  (A pair tile moves two
// thirds of the bytes per flop from L2 and its MMAs are issued at about 0.57 of the one-SM rate per column; the
// constants stand for what a tile costs whatever its width.)  Over those 68 cases the pick reaches the best measured
// single choice to within a percent (geometric mean).  Returns the width index, + kPlanPair or + kPlanSplit; the
// wider tile wins ties.
// The choice depends on T only through the number of 128-row blocks, so the host tabulates it per launch
// (GemmArgs::plan_by_m) and the kernel looks it up after reading T.
constexpr int kPlanPair = 8, kPlanSplit = 16;
inline int gemm_plan(int m1, int N_out, unsigned bn_mask, bool pairs, bool may_split, int force, bool swiglu, int grid) {
    if (force >= 0) return force;
    const int m2 = (m1 + 1) / 2;
    const int n_pairs = pairs ? grid >> 1 : 0;
    int best = 0, best_cost = INT_MAX;
    for (int i = 0; i < kNumBn; ++i) {
        if (!((bn_mask >> i) & 1)) continue;
        const int bn = bn_of(i), per = swiglu ? bn >> 1 : bn, n_tiles = (N_out + per - 1) / per;
        const int cost1 = ((m1 * n_tiles + grid - 1) / grid) * (4 * bn + 1664);
        if (cost1 < best_cost) {
            best_cost = cost1;
            best = i;
        }
        if (n_pairs > 0) {
            const int cost2 = ((m2 * n_tiles + n_pairs - 1) / n_pairs) * (7 * bn + 800);
            if (cost2 < best_cost) {
                best_cost = cost2;
                best = kPlanPair + i;
            }
            // both SMs of a pair on one 128-row tile, half of K each (only as a single wave: a tile per pair)
            if (may_split && m1 * n_tiles <= n_pairs) {
                const int cost3 = (4 * bn + 1664) / 2 + kSplitCost;
                if (cost3 < best_cost) {
                    best_cost = cost3;
                    best = kPlanSplit + i;
                }
            }
        }
    }
    return best;
}

static_assert(kGemmStages * kGemmStageBytes == kG2Stages * kG2StageBytes, "both modes use the same operand area");

template <int MODE>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_tcgen05_kernel(const __grid_constant__ AMaps a_maps, const __grid_constant__ BMaps b_maps,
                    const __grid_constant__ BMaps b2_maps, GemmArgs g) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + kGemmStages * kGemmStageBytes);
    unsigned long long* bars2 = bars + 2 * kMaxStages + 4;                  // the pair mode's set
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars2 + 2 * kG2Stages + 4);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_kb = g.K / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(smem_u32(bars + s), 1);
            mbar_init(smem_u32(bars + kMaxStages + s), 1);
        }
        for (int s = 0; s < kG2Stages; ++s) {
            mbar_init(smem_u32(bars2 + s), 1);                 // the leader's expect_tx arrival (bytes of both CTAs)
            mbar_init(smem_u32(bars2 + kG2Stages + s), 1);     // the leader's multicast commit
        }
        for (int k = 0; k < 2; ++k) {
            mbar_init(smem_u32(bars + 2 * kMaxStages + k), 1);
            mbar_init(smem_u32(bars + 2 * kMaxStages + 2 + k), 128);   // the four epilogue warps
            mbar_init(smem_u32(bars2 + 2 * kG2Stages + k), 1);          // the leader's multicast commit
            mbar_init(smem_u32(bars2 + 2 * kG2Stages + 2 + k), 256);    // (leader's copy) the epilogue threads of both CTAs
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    cluster_sync_all();                          // the peer's barriers exist before anything is signalled on them
    // everything above overlaps the previous kernel of the stream; nothing it wrote is read before this wait
    dcut_pdl_wait();
    dcut_pdl_launch_dependents();
    const int T = g.cu_q[g.B];
    // rows 64..127 of the A tile are not loaded when no row of them exists: they hold whatever shared memory held, and
    // the accumulator rows computed from them are never stored (one-SM and split modes; a pair always loads full boxes)
    const bool a_half = T <= BM / 2;
    const CUtensorMap* a_map1 = a_half ? &a_maps.half : &a_maps.full;
    const uint32_t a_bytes = a_half ? kATile / 2 : kATile;
    const int m_blocks = (T + BM - 1) / BM;
    const int plan_all = m_blocks > 0 ? g.plan_by_m[(m_blocks < kPlanRows ? m_blocks : kPlanRows) - 1] : 0;
    const bool split = plan_all >= kPlanSplit;                      // the pair shares one 128-row tile, half of K each
    const bool pairs = plan_all >= kPlanPair && !split;
    const int plan = plan_all & 7;                                  // width index
    const int bn = bn_of(plan), half_rows = bn >> 1;                // tile width; a B tile is loaded as two halves
    const int per = MODE == kSwiGLU ? half_rows : bn;               // output columns per tile
    const int n_tiles = (g.N_out + per - 1) / per;
    // one-SM and split modes: a stage is this tile's A and B bytes, and as many stages as fit the operand area (a
    // 64-wide tile at T <= 64 moves 8 KB of weights per stage: with four stages too few bytes were in flight per SM to
    // cover the DRAM latency)
    const uint32_t stage_stride = a_bytes + (uint32_t)bn * BK * 2;                         // multiples of 1 KB
    const int n_stages = min(kMaxStages, (int)((uint32_t)(kGemmStages * kGemmStageBytes) / stage_stride));
    if (warp == 1) {   // tensor memory: two 128 x 256 fp32 accumulators (per CTA; allocated for the pair in pair mode)
        if (pairs) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "n"(kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "n"(kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (pairs) cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    bool failed = false;

    if (split) {
        // ------------------------------------------------------------------ one tile per pair of SMs, K cut in two
        // Each CTA runs the one-SM main loop over its half of the k-blocks into its own accumulator.  Then the two
        // exchange: a CTA sends the columns the other one will finish (fp32, through distributed shared memory into
        // the other's idle operand ring) and finishes its own columns with what it received.  Every thread of both
        // CTAs passes the same two cluster barriers whatever happened before, so a wait that gave up cannot strand
        // the peer.
        const int m_tiles = (T + BM - 1) / BM;
        const int w = blockIdx.x >> 1;                              // the pair's tile
        const bool has_tile = w < m_tiles * n_tiles;
        const uint32_t rank = cluster_ctarank();
        const int n_tile = has_tile ? w / m_tiles : 0, m0 = has_tile ? (w - n_tile * m_tiles) * BM : 0;
        const int kb_mid = (n_kb + 1) >> 1, kb0 = rank ? kb_mid : 0, kb1 = rank ? n_kb : kb_mid;
        const uint32_t full_bar = smem_u32(bars), empty_bar = smem_u32(bars + kMaxStages);
        const uint32_t acc_full = smem_u32(bars + 2 * kMaxStages);
        if (has_tile && warp == 0) {
            const CUtensorMap* b_map = pick_map(b_maps, plan);
            const uint32_t stage_tx = a_bytes + bn * BK * 2;
            for (int kb = kb0, kc = 0, s = 0, use = 0; kb < kb1; ++kb, ++kc) {
                if (use > 0 && !__all_sync(0xffffffffu, mbar_wait(empty_bar + 8 * s, (use - 1) & 1))) {
                    failed = true;
                    break;
                }
                if (elect_one()) {
                    const uint32_t a_dst = smem_u32(smem + s * stage_stride), b_dst = a_dst + a_bytes;
                    const uint32_t bar = full_bar + 8 * s;
                    mbar_arrive_expect_tx(bar, stage_tx);
                    tma_load_2d(a_dst, a_map1, kb * BK, m0, bar);
                    tma_load_2d(b_dst, b_map, kb * BK, n_tile * bn, bar);
                    tma_load_2d(b_dst + half_rows * BK * 2, b_map, kb * BK, n_tile * bn + half_rows, bar);
                }
                __syncwarp();
                if (++s == n_stages) {
                    s = 0;
                    ++use;
                }
            }
        } else if (has_tile && warp == 1) {
            const uint32_t idesc = kIdescNoN | ((uint32_t)(bn >> 3) << 17);
            for (int kb = kb0, kc = 0, s = 0, use = 0; kb < kb1; ++kb, ++kc) {
                if (!__all_sync(0xffffffffu, mbar_wait(full_bar + 8 * s, use & 1))) {
                    failed = true;
                    break;
                }
                tc_fence_after();
                if (elect_one()) {
                    const uint32_t a_addr = smem_u32(smem + s * stage_stride);
                    const uint64_t da = umma_desc_sw128(a_addr), db = umma_desc_sw128(a_addr + a_bytes);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k) tc_mma(tmem_base, da + 2 * k, db + 2 * k, idesc, (kc | k) ? 1u : 0u);
                    tc_commit(empty_bar + 8 * s);
                }
                __syncwarp();
                if (++s == n_stages) {
                    s = 0;
                    ++use;
                }
            }
            if (!failed && elect_one()) tc_commit(acc_full);    // this CTA's partial sums are complete
            __syncwarp();
        } else if (has_tile) {
            if (!__all_sync(0xffffffffu, mbar_wait(acc_full, 0))) failed = true;   // ... and its operand ring is idle
            tc_fence_after();
        }
        // columns [0, cut) are finished by rank 0, [cut, bn) by rank 1
        const int cut = (bn >> 6) << 5;
        const int own0 = rank ? cut : 0, own1 = rank ? bn : cut, send0 = rank ? 0 : cut, send1 = rank ? cut : bn;
        const int quarter = warp & 3, row_in_tile = quarter * 32 + lane;
        const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const uint32_t stage_local = smem_u32(smem);              // [column / 4][row] vectors of four fp32: 64 KB at most
        tc_fence_before();
        cluster_sync_all();                                       // both accumulators complete, both rings idle
        tc_fence_after();
        if (has_tile && warp >= 2 && !failed) {
            asm volatile("fence.proxy.async;" ::: "memory");      // the ring was last written and read through the async proxy
            const uint32_t stage_peer = mapa_rank(stage_local, rank ^ 1);
#pragma unroll 1
            for (int c = send0; c < send1; c += 32) {
                uint32_t av[32];
                tc_ld32(t_row + c, av);
                tc_wait_ld();
#pragma unroll
                for (int v = 0; v < 8; ++v) {
                    const uint32_t dst = stage_peer + (uint32_t)((((c - send0) >> 2) + v) * BM + row_in_tile) * 16;
                    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(av[4 * v]), "r"(av[4 * v + 1]),
                                 "r"(av[4 * v + 2]), "r"(av[4 * v + 3]) : "memory");
                }
            }
        }
        tc_fence_before();
        cluster_sync_all();                                       // the peer's partial sums have arrived
        tc_fence_after();
        if (has_tile && warp >= 2 && !failed) {
            const int row = m0 + row_in_tile, col0 = n_tile * bn;
            __nv_bfloat16* orow = g.out + (size_t)row * g.N_out + col0;
            const __nv_bfloat16* rrow = MODE == kResidual ? g.residual + (size_t)row * g.N_out + col0 : nullptr;
#pragma unroll 1
            for (int c = own0; c < own1; c += 32) {
                uint32_t av[32];
                tc_ld32(t_row + c, av);
                tc_wait_ld();
                if (row < T) {
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        if (col0 + c + e >= g.N_out) break;
                        float add[8];
#pragma unroll
                        for (int v = 0; v < 2; ++v) {
                            const uint32_t src = stage_local + (uint32_t)((((c - own0 + e) >> 2) + v) * BM + row_in_tile) * 16;
                            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                         : "=f"(add[4 * v]), "=f"(add[4 * v + 1]), "=f"(add[4 * v + 2]), "=f"(add[4 * v + 3]) : "r"(src));
                        }
                        uint4 res = make_uint4(0, 0, 0, 0);
                        if (MODE == kResidual) res = *reinterpret_cast<const uint4*>(rrow + c + e);
                        const uint32_t rw[4] = {res.x, res.y, res.z, res.w};
                        uint32_t o[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j)   // (rank 0's half of K) + (rank 1's), then the residual
                            o[j] = pack_bf16((rank ? add[2 * j] + __uint_as_float(av[e + 2 * j]) : __uint_as_float(av[e + 2 * j]) + add[2 * j]) + bf_lo(rw[j]),
                                             (rank ? add[2 * j + 1] + __uint_as_float(av[e + 2 * j + 1]) : __uint_as_float(av[e + 2 * j + 1]) + add[2 * j + 1]) + bf_hi(rw[j]));
                        *reinterpret_cast<uint4*>(orow + c + e) = make_uint4(o[0], o[1], o[2], o[3]);
                    }
                }
            }
        }
    } else if (!pairs) {
        const int m_tiles = (T + BM - 1) / BM;
        const int n_work = m_tiles * n_tiles;                      // (a CTA without work falls through the loops below)
        const uint32_t full_bar = smem_u32(bars), empty_bar = smem_u32(bars + kMaxStages);
        const uint32_t acc_full = smem_u32(bars + 2 * kMaxStages), acc_empty = acc_full + 16;
        if (warp == 0) {
            // ---------------------------------------------------------------- TMA producer (whole warp walks, one lane issues)
            const CUtensorMap* b_map = pick_map(b_maps, plan);
            const CUtensorMap* b2_map = pick_map(b2_maps, plan);
            const uint32_t stage_tx = a_bytes + bn * BK * 2;
            int s = 0, use = 0;   // stage of the next k-block, and how often the ring has gone round (over all tiles)
            for (int w = blockIdx.x; w < n_work && !failed; w += gridDim.x) {
                const int n_tile = w / m_tiles, m0 = (w - n_tile * m_tiles) * BM;
                for (int kb = 0; kb < n_kb; ++kb) {
                    if (use > 0 && !__all_sync(0xffffffffu, mbar_wait(empty_bar + 8 * s, (use - 1) & 1))) {
                        failed = true;
                        break;
                    }
                    if (elect_one()) {
                        const uint32_t a_dst = smem_u32(smem + s * stage_stride), b_dst = a_dst + a_bytes;
                        const uint32_t bar = full_bar + 8 * s;
                        mbar_arrive_expect_tx(bar, stage_tx);
                        tma_load_2d(a_dst, a_map1, kb * BK, m0, bar);
                        if (MODE == kSwiGLU) {   // the gate rows, then the up rows of the same features
                            tma_load_2d(b_dst, b_map, kb * BK, n_tile * half_rows, bar);
                            tma_load_2d(b_dst + half_rows * BK * 2, b2_map, kb * BK, n_tile * half_rows, bar);
                        } else {                 // (weight rows past N read as zeros)
                            tma_load_2d(b_dst, b_map, kb * BK, n_tile * bn, bar);
                            tma_load_2d(b_dst + half_rows * BK * 2, b_map, kb * BK, n_tile * bn + half_rows, bar);
                        }
                    }
                    __syncwarp();
                    if (++s == n_stages) {
                        s = 0;
                        ++use;
                    }
                }
            }
        } else if (warp == 1) {
            // ---------------------------------------------------------------- MMA issuer (whole warp walks, one lane issues)
            const uint32_t idesc = kIdescNoN | ((uint32_t)(bn >> 3) << 17);
            int s = 0, use = 0, it = 0;
            for (int w = blockIdx.x; w < n_work && !failed; w += gridDim.x, ++it) {
                const int acc = it & 1;
                // the epilogue must have drained this accumulator (used by tile it - 2)
                if (it >= 2 && !__all_sync(0xffffffffu, mbar_wait(acc_empty + 8 * acc, ((it >> 1) - 1) & 1))) {
                    failed = true;
                    break;
                }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + acc * BN;
                for (int kb = 0; kb < n_kb; ++kb) {
                    if (!__all_sync(0xffffffffu, mbar_wait(full_bar + 8 * s, use & 1))) {
                        failed = true;
                        break;
                    }
                    tc_fence_after();
                    if (elect_one()) {
                        const uint32_t a_addr = smem_u32(smem + s * stage_stride);
                        const uint64_t da = umma_desc_sw128(a_addr), db = umma_desc_sw128(a_addr + a_bytes);
    #pragma unroll
                        for (int k = 0; k < BK / 16; ++k)   // 32 bytes along K per step = 2 descriptor address units
                            tc_mma(tmem_d, da + 2 * k, db + 2 * k, idesc, (kb | k) ? 1u : 0u);
                        tc_commit(empty_bar + 8 * s);       // the stage is free once these MMAs have read it
                    }
                    __syncwarp();
                    if (++s == n_stages) {
                        s = 0;
                        ++use;
                    }
                }
                if (failed) break;
                if (elect_one()) tc_commit(acc_full + 8 * acc);   // accumulator complete
                __syncwarp();
            }
        } else {
            // ---------------------------------------------------------------- epilogue warps
            const int quarter = warp & 3;               // tensor-memory lanes 32 * quarter .. + 31
            int it = 0;
            for (int w = blockIdx.x; w < n_work && !failed; w += gridDim.x, ++it) {
                const int n_tile = w / m_tiles, m0 = (w - n_tile * m_tiles) * BM;
                const int acc = it & 1;
                const int row = m0 + quarter * 32 + lane;
                if (!mbar_wait(acc_full + 8 * acc, (it >> 1) & 1)) {
                    failed = true;
                    break;
                }
                tc_fence_after();
                const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN;
                gemm_epilogue<MODE>(g, T, row, n_tile, t_row, bn);
                // this accumulator may be overwritten once all four epilogue warps have read it
                tc_fence_before();
                mbar_arrive(acc_empty + 8 * acc);
            }
        }
    } else {
        const int m_tiles = (T + 2 * BM - 1) / (2 * BM);          // 256-row tiles of the pair
        const int n_work = m_tiles * n_tiles;
        const uint32_t rank = cluster_ctarank();                   // 0: leader
        const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
        const uint32_t full_bar = smem_u32(bars2), empty_bar = smem_u32(bars2 + kG2Stages);
        const uint32_t acc_full = smem_u32(bars2 + 2 * kG2Stages), acc_empty = acc_full + 16;
        if (warp == 0) {
            // ---------------------------------------------------------------- TMA producer (both CTAs)
            const uint32_t lead_full = mapa_rank(full_bar, 0);
            const CUtensorMap* b_map = pick_map(b_maps, plan);
            const CUtensorMap* b2_map = pick_map(b2_maps, plan);
            const uint32_t pair_tx = 2 * (kATile + half_rows * BK * 2);   // both CTAs' A tile and half of the B tile
            int kc = 0;
            for (int w = pair; w < n_work && !failed; w += n_pairs) {
                const int n_tile = w / m_tiles, m0 = (w - n_tile * m_tiles) * (2 * BM) + (int)rank * BM;
                for (int kb = 0; kb < n_kb; ++kb, ++kc) {
                    const int s = kc % kG2Stages;
                    if (kc >= kG2Stages && !__all_sync(0xffffffffu, mbar_wait(empty_bar + 8 * s, ((kc / kG2Stages) - 1) & 1))) {
                        failed = true;
                        break;
                    }
                    if (elect_one()) {
                        const uint32_t a_dst = smem_u32(smem + s * kG2StageBytes), b_dst = a_dst + kATile;
                        if (rank == 0) mbar_arrive_expect_tx(full_bar + 8 * s, pair_tx);
                        const uint32_t bar = lead_full + 8 * s;
                        tma_load_2d_pair(a_dst, &a_maps.full, kb * BK, m0, bar);
                        if (MODE == kSwiGLU)      // the leader's half: 128 gate rows; the peer's: the 128 up rows of the same features
                            tma_load_2d_pair(b_dst, rank == 0 ? b_map : b2_map, kb * BK, n_tile * half_rows, bar);
                        else
                            tma_load_2d_pair(b_dst, b_map, kb * BK, n_tile * bn + (int)rank * half_rows, bar);
                    }
                    __syncwarp();
                }
            }
        } else if (warp == 1) {
            // ---------------------------------------------------------------- MMA issuer (leader CTA only)
            if (rank == 0) {
                const uint32_t idesc2 = kIdesc2NoN | ((uint32_t)(bn >> 3) << 17);
                int kc = 0, it = 0;
                for (int w = pair; w < n_work && !failed; w += n_pairs, ++it) {
                    const int acc = it & 1;
                    // the epilogues of both CTAs must have drained this accumulator (used by tile it - 2)
                    if (it >= 2 && !__all_sync(0xffffffffu, mbar_wait(acc_empty + 8 * acc, ((it >> 1) - 1) & 1))) {
                        failed = true;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t tmem_d = tmem_base + acc * BN;
                    for (int kb = 0; kb < n_kb; ++kb, ++kc) {
                        const int s = kc % kG2Stages;
                        if (!__all_sync(0xffffffffu, mbar_wait(full_bar + 8 * s, (kc / kG2Stages) & 1))) {
                            failed = true;
                            break;
                        }
                        tc_fence_after();
                        if (elect_one()) {
                            const uint32_t a_addr = smem_u32(smem + s * kG2StageBytes);
                            const uint64_t da = umma_desc_sw128(a_addr), db = umma_desc_sw128(a_addr + kATile);
    #pragma unroll
                            for (int k = 0; k < BK / 16; ++k)
                                tc_mma2(tmem_d, da + 2 * k, db + 2 * k, idesc2, (kb | k) ? 1u : 0u);
                            tc_commit_pair(empty_bar + 8 * s);     // the stage is free in both CTAs once these MMAs have read it
                        }
                        __syncwarp();
                    }
                    if (failed) break;
                    if (elect_one()) tc_commit_pair(acc_full + 8 * acc);   // accumulator complete, in both CTAs
                    __syncwarp();
                }
            }
        } else {
            // ---------------------------------------------------------------- epilogue warps (both CTAs)
            const int quarter = warp & 3;
            const uint32_t lead_acc_empty = mapa_rank(acc_empty, 0);
            int it = 0;
            for (int w = pair; w < n_work && !failed; w += n_pairs, ++it) {
                const int n_tile = w / m_tiles, m0 = (w - n_tile * m_tiles) * (2 * BM) + (int)rank * BM;
                const int acc = it & 1;
                const int row = m0 + quarter * 32 + lane;
                if (!mbar_wait(acc_full + 8 * acc, (it >> 1) & 1)) {
                    failed = true;
                    break;
                }
                tc_fence_after();
                const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN;
                gemm_epilogue<MODE>(g, T, row, n_tile, t_row, bn);
                tc_fence_before();
                mbar_arrive_remote(lead_acc_empty + 8 * acc);
            }
        }
    }
    if (failed) atomicExch(g.status, DCUT_DEV_GEMM_WAIT_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                          // nobody leaves while the other CTA may still signal its barriers
    if (warp == 1) {
        tc_fence_after();
        if (pairs)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(kTmemCols) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(kTmemCols) : "memory");
    }
}

// ------------------------------------------------------------------------------------------------ RMSNorm

__global__ void __launch_bounds__(256) rmsnorm_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ gain,
                                                      const int* __restrict__ cu_q, int B, int hidden, float eps,
                                                      __nv_bfloat16* __restrict__ y) {
    dcut_pdl_wait();
    dcut_pdl_launch_dependents();
    const int row = blockIdx.x;
    if (row >= cu_q[B]) return;
    const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)row * hidden);
    const uint4* gr = reinterpret_cast<const uint4*>(gain);
    uint4* yr = reinterpret_cast<uint4*>(y + (size_t)row * hidden);
    const int nvec = hidden >> 3;
    float ss = 0.0f;
    for (int v = threadIdx.x; v < nvec; v += 256) {
        const uint4 a = xr[v];
        const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) ss += bf_lo(w[j]) * bf_lo(w[j]) + bf_hi(w[j]) * bf_hi(w[j]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    __shared__ float wsum[8];
    if ((threadIdx.x & 31) == 0) wsum[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.0f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += wsum[w];
    const float inv = rsqrtf(tot / (float)hidden + eps);
    for (int v = threadIdx.x; v < nvec; v += 256) {
        const uint4 a = xr[v], gq = gr[v];
        const uint32_t w[4] = {a.x, a.y, a.z, a.w}, gw[4] = {gq.x, gq.y, gq.z, gq.w};
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) o[j] = pack_bf16(bf_lo(w[j]) * inv * bf_lo(gw[j]), bf_hi(w[j]) * inv * bf_hi(gw[j]));
        yr[v] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// ------------------------------------------------------------------------------------------------ RoPE + KV append

struct RopeArgs {
    const __nv_bfloat16* qkv;   // [T, (Hq + 2 Hkv) * Dh]: q heads, k heads, v heads
    const int* cu_q;
    const int* tok_req;
    const int* tok_pos;
    const int* block_table;
    int block_table_stride;
    const float* inv_freq;      // [Dh / 2] = theta^(-2e/Dh)
    int B, n_q_heads, n_kv_heads, head_dim;
    long long num_pages;
    __nv_bfloat16* q_out;       // [T, Hq, Dh]
    __nv_bfloat16* k_cache;
    __nv_bfloat16* v_cache;
    int* status;
};

__global__ void __launch_bounds__(256) rope_append_kernel(RopeArgs a) {
    dcut_pdl_wait();
    dcut_pdl_launch_dependents();
    const int tok = blockIdx.x;
    if (tok >= a.cu_q[a.B]) return;
    const int Dh = a.head_dim, half = Dh >> 1;
    const int req = a.tok_req[tok], pos = a.tok_pos[tok];
    int page = a.block_table[(size_t)req * a.block_table_stride + pos / 16];
    if (page < 0 || page >= a.num_pages) {
        if (threadIdx.x == 0) atomicExch(a.status, DCUT_DEV_BAD_PAGE);
        return;
    }
    const int slot = pos & 15;
    const int row_w = (a.n_q_heads + 2 * a.n_kv_heads) * Dh;
    const __nv_bfloat16* row = a.qkv + (size_t)tok * row_w;
    // A thread keeps its two rotation pairs (e, e + 1) and walks the heads: one sincos pair per thread, 4-byte accesses.
    // (head_dim is a multiple of 16, so half is even and rows are 4-byte aligned.)
    const int lanes_per_head = half >> 1;                      // threads that cover one head
    const int heads_per_pass = blockDim.x / lanes_per_head;
    const int e = (threadIdx.x % lanes_per_head) * 2;
    float sn0, cs0, sn1, cs1;
    sincosf((float)pos * a.inv_freq[e], &sn0, &cs0);
    sincosf((float)pos * a.inv_freq[e + 1], &sn1, &cs1);
    if ((int)threadIdx.x < heads_per_pass * lanes_per_head) {
        for (int h = threadIdx.x / lanes_per_head; h < a.n_q_heads + a.n_kv_heads; h += heads_per_pass) {
            const uint32_t lo = *reinterpret_cast<const uint32_t*>(row + h * Dh + e);
            const uint32_t hi = *reinterpret_cast<const uint32_t*>(row + h * Dh + e + half);
            const float a0 = bf_lo(lo), a1 = bf_hi(lo), b0 = bf_lo(hi), b1 = bf_hi(hi);
            const uint32_t y_lo = pack_bf16(a0 * cs0 - b0 * sn0, a1 * cs1 - b1 * sn1);
            const uint32_t y_hi = pack_bf16(b0 * cs0 + a0 * sn0, b1 * cs1 + a1 * sn1);
            __nv_bfloat16* dst = h < a.n_q_heads
                                     ? a.q_out + ((size_t)tok * a.n_q_heads + h) * Dh
                                     : a.k_cache + (((size_t)page * a.n_kv_heads + (h - a.n_q_heads)) * 16 + slot) * Dh;
            *reinterpret_cast<uint32_t*>(dst + e) = y_lo;
            *reinterpret_cast<uint32_t*>(dst + e + half) = y_hi;
        }
    }
    const uint4* vrow = reinterpret_cast<const uint4*>(row + (a.n_q_heads + a.n_kv_heads) * Dh);   // 16-byte aligned: Dh % 8 == 0
    const int vec_per_head = Dh >> 3;
    for (int idx = threadIdx.x; idx < a.n_kv_heads * vec_per_head; idx += blockDim.x) {
        const int h = idx / vec_per_head, v = idx - h * vec_per_head;
        reinterpret_cast<uint4*>(a.v_cache + (((size_t)page * a.n_kv_heads + h) * 16 + slot) * Dh)[v] = vrow[idx];
    }
}

// ------------------------------------------------------------------------------------------------ host

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// K-major bf16 matrix [rows, cols] as a 2-D tensor map with a {64 columns, box_rows} box and 128-byte swizzle
dcut_status make_kmajor_map(dcut_ctx* ctx, CUtensorMap* map, const void* base, long long rows, long long cols, int box_rows) {
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
        map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return dcut_fail(ctx, DCUT_ECUDA, "cuTensorMapEncodeTiled failed for a GEMM operand (%d)", (int)r);
    return DCUT_OK;
}

dcut_status make_act_maps(dcut_ctx* ctx, AMaps* maps, const void* base, long long rows, long long cols) {
    dcut_status st = make_kmajor_map(ctx, &maps->full, base, rows, cols, BM);
    if (st != DCUT_OK) return st;
    return make_kmajor_map(ctx, &maps->half, base, rows, cols, BM / 2);
}

// The weight's tensor maps for the tile widths in `mask` (box = half the width in rows)
dcut_status make_weight_maps(dcut_ctx* ctx, BMaps* maps, const void* w, long long rows, long long cols, unsigned mask) {
    for (int i = 0; i < kNumBn; ++i) {
        if (!((mask >> i) & 1)) continue;
        dcut_status st = make_kmajor_map(ctx, &maps->m[i], w, rows, cols, bn_of(i) / 2);
        if (st != DCUT_OK) return st;
    }
    return DCUT_OK;
}

template <int MODE>
dcut_status launch_gemm(dcut_ctx* ctx, const AMaps& a, const BMaps& b, const BMaps& b2, int n_tiles,
                        int T_cap, unsigned bn_mask, const GemmArgs& g, cudaStream_t stream) {
    GemmArgs ga = g;
    ga.n_tiles = n_tiles;
    ga.bn_mask = bn_mask | 1u;

    // work items at the narrowest width that may be chosen (the widest has n_tiles per row block)
    int narrow = 0;
    for (int i = 0; i < kNumBn; ++i)
        if ((ga.bn_mask >> i) & 1) narrow = i;
    const int n_work = ((T_cap + BM - 1) / BM) * ((n_tiles * BN + bn_of(narrow) - 1) / bn_of(narrow));
    int grid = n_work < ctx->sm_count ? n_work : ctx->sm_count;   // persistent: at most one CTA per SM
    ga.pairs = 0;
    ga.force = ctx->ly_gemm_force >= 0 && ctx->ly_gemm_force < kNumBn && ((ga.bn_mask >> ctx->ly_gemm_force) & 1) ? ctx->ly_gemm_force : -1;
    if (ctx->ly_gemm_pairs > 0) {
        // always launched as clusters of two CTAs (the kernel holds cta_group::2 instructions); the pair mode itself
        // can be switched off
        grid = 2 * (n_work < ctx->ly_gemm_pairs ? n_work : ctx->ly_gemm_pairs);   // room for either mode
        ga.pairs = ctx->ly_gemm_pair_mode;
        ga.force = ctx->ly_gemm_force;
        if (ga.force >= 0 && (ga.force > 22 || (ga.force & 7) == 7 || !((ga.bn_mask >> (ga.force & 7)) & 1) || (ga.force >= 8 && !ga.pairs) ||
                              (ga.force >= 16 && !((MODE == kPlain || MODE == kResidual) && ga.K >= 2 * BK))))
            ga.force = -1;
        const int m_cap = (T_cap + BM - 1) / BM;   // no launch has more row blocks than that: the rest of the table repeats
        for (int m = 1; m <= kPlanRows; ++m)
            ga.plan_by_m[m - 1] = m > m_cap && m > 1 ? ga.plan_by_m[m - 2]
                                                    : (unsigned char)gemm_plan(m, ga.N_out, ga.bn_mask, ga.pairs != 0,
                                                                               ga.pairs != 0 && (MODE == kPlain || MODE == kResidual) && ga.K >= 2 * BK,
                                                                               ga.force, MODE == kSwiGLU, grid);
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cudaLaunchConfig_t lc = {};
        lc.gridDim = dim3(grid);
        lc.blockDim = dim3(kGemmThreads);
        lc.dynamicSmemBytes = kGemmSmem;
        lc.stream = stream;
        lc.attrs = attr;
        lc.numAttrs = 2;
        return dcut_check_cuda(ctx, cudaLaunchKernelEx(&lc, gemm_tcgen05_kernel<MODE>, a, b, b2, ga), "launch gemm_tcgen05_kernel");
    }
    for (int m = 1; m <= kPlanRows; ++m)
        ga.plan_by_m[m - 1] = m > (T_cap + BM - 1) / BM && m > 1
                                  ? ga.plan_by_m[m - 2]
                                  : (unsigned char)gemm_plan(m, ga.N_out, ga.bn_mask, false, false, ga.force, MODE == kSwiGLU, grid);
    return dcut_check_cuda(ctx, dcut_launch_pdl(gemm_tcgen05_kernel<MODE>, dim3(grid), dim3(kGemmThreads), kGemmSmem, stream, a, b, b2, ga),
                           "launch gemm_tcgen05_kernel");
}

// Tensor maps of the layers seen so far: the weights' (for every tile width) in a small direct-mapped cache keyed by the
// layer's w_qkv pointer, so that a model forward does not encode 36 x 31 maps on every call
struct WeightMaps {
    const void* w[5];
    BMaps m[5];         // w_qkv, w_o, w_gate, w_up, w_down
};
constexpr int kLayerCache = 64;
struct LayerMaps {
    AMaps act[4];       // norm out, attention out, norm-2 out, mlp activation
    bool act_ready;
    WeightMaps cache[kLayerCache];
};

}  // namespace

dcut_status dcut_init_layer(dcut_ctx* ctx) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tcgen05_kernel<kPlain>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tcgen05_kernel<kResidual>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tcgen05_kernel<kSwiGLU>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tcgen05_kernel<kArgmax>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmem);
    if (e != cudaSuccess) return dcut_check_cuda(ctx, e, "cudaFuncSetAttribute(gemm)");
    {
        // The GEMM is launched as clusters of two CTAs so that it can run tiles on pairs of SMs where that pays
        // (DCUT_GEMM_2CTA=0: never).  ly_gemm_pairs = how many such clusters the device runs at once.
        const char* env = getenv("DCUT_GEMM_2CTA");
        ctx->ly_gemm_pair_mode = (!env || atoi(env) != 0) ? 1 : 0;
        const char* envf = getenv("DCUT_GEMM_FORCE");
        ctx->ly_gemm_force = envf ? atoi(envf) : -1;
        const char* envw = getenv("DCUT_GEMM_WIDTHS");   // bit i allows tile width 256 - 32 i in the one-SM mode
        ctx->ly_gemm_bn_mask = ((envw ? (unsigned)strtoul(envw, nullptr, 0) : kBnMaskAll) & kBnMaskAll) | 1u;
        ctx->ly_gemm_pairs = 0;
        {
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = 2;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cudaLaunchConfig_t lc = {};
            lc.gridDim = dim3(2 * ctx->sm_count);
            lc.blockDim = dim3(kGemmThreads);
            lc.dynamicSmemBytes = kGemmSmem;
            lc.attrs = attr;
            lc.numAttrs = 1;
            int n_clusters = 0;
            if (cudaOccupancyMaxActiveClusters(&n_clusters, gemm_tcgen05_kernel<kPlain>, &lc) == cudaSuccess && n_clusters > 0)
                ctx->ly_gemm_pairs = n_clusters;
            else
                (void)cudaGetLastError();
        }
    }
    ctx->layer_maps = calloc(1, sizeof(LayerMaps));
    return ctx->layer_maps ? DCUT_OK : dcut_fail(ctx, DCUT_EINVAL, "out of host memory");
}

void dcut_free_layer(dcut_ctx* ctx) { free(ctx->layer_maps); }

// x[t, :] = embed[tok_id[t], :] for the packed tokens (ids outside [0, V) read row 0 and set the status word)
__global__ void __launch_bounds__(128) embed_kernel(const __nv_bfloat16* __restrict__ embed, const int* __restrict__ tok_id,
                                                    const int* __restrict__ cu_q, int B, int hidden, int V,
                                                    __nv_bfloat16* __restrict__ x, int* __restrict__ status) {
    dcut_pdl_wait();
    dcut_pdl_launch_dependents();
    const int row = blockIdx.x;
    if (row >= cu_q[B]) return;
    int id = tok_id[row];
    if (id < 0 || id >= V) {
        if (threadIdx.x == 0) atomicExch(status, DCUT_DEV_BAD_TOKEN);
        id = 0;
    }
    const uint4* src = reinterpret_cast<const uint4*>(embed + (size_t)id * hidden);
    uint4* dst = reinterpret_cast<uint4*>(x + (size_t)row * hidden);
    for (int v = threadIdx.x; v < hidden / 8; v += 128) dst[v] = src[v];
}

// The whole verification forward of a small model: embedding, n_layers decoder layers (each with its own paged
// cache), final RMSNorm, LM head fused with acceptance.
dcut_status dcut_launch_model(dcut_ctx* ctx, const dcut_model* m, long long num_pages, const int* block_table,
                              int block_table_stride, const int* ctx_lens, const int* cu_q, const int* tok_req,
                              const int* tok_pos, const int* tok_id, const int* draft_ids, int B, int gamma, int T_cap,
                              int* accept_len, int* bonus, int* out_tokens, int* n_accepted_total, int* row_argmax,
                              void* hidden_out, cudaStream_t stream) {
    const int H = ctx->lim.hidden;
    __nv_bfloat16* user = static_cast<__nv_bfloat16*>(hidden_out);
    dcut_status st = dcut_check_cuda(ctx, dcut_launch_pdl(embed_kernel, dim3(T_cap), dim3(128), 0, stream,
                                                          static_cast<const __nv_bfloat16*>(m->embed), tok_id, cu_q, B, H, m->vocab,
                                                          (m->n_layers == 0 && user) ? user : ctx->ly_x[0], ctx->d_status),
                                     "launch embed_kernel");
    if (st != DCUT_OK) return st;
    __nv_bfloat16* x = (m->n_layers == 0 && user) ? user : ctx->ly_x[0];
    for (int l = 0; l < m->n_layers; ++l) {   // ping-pong between the context's two buffers; the last layer may write to the caller
        __nv_bfloat16* y = (l == m->n_layers - 1 && user) ? user : ctx->ly_x[(l + 1) & 1];
        st = dcut_launch_layer(ctx, &m->layers[l], x, y, m->k_caches[l], m->v_caches[l], num_pages,
                               block_table, block_table_stride, ctx_lens, cu_q, tok_req, tok_pos, B, T_cap,
                               l > 0 /* the attention work list of layer 0 serves every layer */, 0, stream);
        if (st != DCUT_OK) return st;
        x = y;
    }
    const float eps = m->n_layers > 0 ? m->layers[0].rms_eps : 1e-6f;
    if ((st = dcut_check_cuda(ctx, dcut_launch_pdl(rmsnorm_kernel, dim3(T_cap), dim3(256), 0, stream,
                                                   static_cast<const __nv_bfloat16*>(x),
                                                   static_cast<const __nv_bfloat16*>(m->g_final), cu_q, B, H, eps, ctx->ly_norm),
                              "launch rmsnorm_kernel")) != DCUT_OK) return st;
    if ((st = dcut_launch_lm_head_argmax(ctx, ctx->ly_norm, m->w_lm, m->vocab, H, cu_q, B, T_cap, ctx->d_row_key, stream)) != DCUT_OK) return st;
    return dcut_launch_accept_match(ctx, nullptr, m->vocab, draft_ids, cu_q, B, gamma, T_cap, accept_len, bonus, out_tokens,
                                    n_accepted_total, row_argmax, ctx->d_row_key, stream);
}

// logits = x . w_lm^T reduced on the fly to one (maximum, first column) word per row: the [T, V] logits never exist
dcut_status dcut_launch_lm_head_argmax(dcut_ctx* ctx, const void* x, const void* w_lm, int V, int K, const int* cu_q, int B,
                                       int T_cap, unsigned long long* row_key, cudaStream_t stream) {
    AMaps am;
    BMaps bm;
    dcut_status st = make_act_maps(ctx, &am, x, T_cap, K);
    if (st != DCUT_OK) return st;
    // rows past V read as zeros; hundreds of tiles per row block: only the full width is offered
    if ((st = make_weight_maps(ctx, &bm, w_lm, V, K, 1u)) != DCUT_OK) return st;
    for (int i = 1; i < kNumBn; ++i) bm.m[i] = bm.m[0];
    GemmArgs g;
    g.cu_q = cu_q;
    g.B = B;
    g.N_out = V;
    g.K = K;
    g.out = nullptr;
    g.residual = nullptr;
    g.row_key = row_key;
    g.V = V;
    g.status = ctx->d_status;
    return launch_gemm<kArgmax>(ctx, am, bm, bm, (V + BN - 1) / BN, T_cap, 1u, g, stream);
}

dcut_status dcut_launch_gemm(dcut_ctx* ctx, const void* a, const void* w, const void* w2, int mode, int N, int K,
                             const int* cu_q, int B, int T_cap, void* out, const void* residual, cudaStream_t stream) {
    // generic entry used by dcut_gemm_bf16 (tests, benchmarks): encodes its maps on every call
    AMaps am;
    BMaps bm, b2m;
    dcut_status st = make_act_maps(ctx, &am, a, T_cap, K);
    if (st != DCUT_OK) return st;
    const unsigned mask = (mode == kSwiGLU ? ctx->ly_gemm_bn_mask & kBnMaskSwiGLU : ctx->ly_gemm_bn_mask) | 1u;
    for (int i = 0; i < kNumBn; ++i) bm.m[i] = am.full;   // entries outside the mask are never used; keep them defined
    if ((st = make_weight_maps(ctx, &bm, w, N, K, mask)) != DCUT_OK) return st;
    b2m = bm;
    if (mode == kSwiGLU && (st = make_weight_maps(ctx, &b2m, w2, N, K, mask)) != DCUT_OK) return st;
    GemmArgs g;
    g.cu_q = cu_q;
    g.B = B;
    g.N_out = N;
    g.K = K;
    g.out = static_cast<__nv_bfloat16*>(out);
    g.residual = static_cast<const __nv_bfloat16*>(residual);
    g.row_key = nullptr;
    g.V = 0;
    g.status = ctx->d_status;
    if (mode == kSwiGLU) return launch_gemm<kSwiGLU>(ctx, am, bm, b2m, N / (BN / 2), T_cap, mask, g, stream);
    if (mode == kResidual) return launch_gemm<kResidual>(ctx, am, bm, b2m, N / BN, T_cap, mask, g, stream);
    return launch_gemm<kPlain>(ctx, am, bm, b2m, N / BN, T_cap, mask, g, stream);
}

dcut_status dcut_launch_layer(dcut_ctx* ctx, const dcut_layer_weights* w, const void* x, void* y, void* k_cache,
                              void* v_cache, long long num_pages, const int* block_table, int block_table_stride,
                              const int* ctx_lens, const int* cu_q, const int* tok_req, const int* tok_pos, int B,
                              int T_cap, int reuse_plan, int part, cudaStream_t stream) {
    // part 0: the whole layer.  Tensor-parallel halves (a rank's shard of the heads / of the intermediate width, the
    // projections that close a half WITHOUT the residual, so that the ranks' outputs can be summed first):
    // part 1: y = Attn(RoPE(Wqkv . RMSNorm(x))) . Wo^T;  part 2: y = (SiLU(Wg . n) * (Wu . n)) . Wd^T with n = RMSNorm(x).
    const dcut_limits& l = ctx->lim;
    const int H = l.hidden, I = l.intermediate, Dh = l.head_dim;
    const int qkv_w = (l.n_q_heads + 2 * l.n_kv_heads) * Dh, q_w = l.n_q_heads * Dh;
    const int max_T = l.max_B * (l.max_gamma + 1);
    LayerMaps* lm = static_cast<LayerMaps*>(ctx->layer_maps);
    dcut_status st;
    if (!lm->act_ready) {
        if ((st = make_act_maps(ctx, &lm->act[0], ctx->ly_norm, max_T, H)) != DCUT_OK) return st;
        if ((st = make_act_maps(ctx, &lm->act[1], ctx->ly_attn, max_T, q_w)) != DCUT_OK) return st;
        if ((st = make_act_maps(ctx, &lm->act[2], ctx->ly_norm2, max_T, H)) != DCUT_OK) return st;
        if ((st = make_act_maps(ctx, &lm->act[3], ctx->ly_act, max_T, I)) != DCUT_OK) return st;
        lm->act_ready = true;
    }
    const void* wp[5] = {w->w_qkv, w->w_o, w->w_gate, w->w_up, w->w_down};
    const long long wr[5] = {qkv_w, H, I, I, H}, wc[5] = {H, q_w, H, H, I};
    const unsigned mask = ctx->ly_gemm_bn_mask, wmask[5] = {mask, mask, mask & kBnMaskSwiGLU, mask & kBnMaskSwiGLU, mask};
    WeightMaps* wm = &lm->cache[(reinterpret_cast<uintptr_t>(w->w_qkv) >> 8) % kLayerCache];
    for (int i = 0; i < 5; ++i)
        if (wm->w[i] != wp[i]) {
            if ((st = make_weight_maps(ctx, &wm->m[i], wp[i], wr[i], wc[i], wmask[i] | 1u)) != DCUT_OK) return st;
            wm->w[i] = wp[i];
        }
    GemmArgs g;
    g.cu_q = cu_q;
    g.B = B;
    g.row_key = nullptr;
    g.V = 0;
    g.status = ctx->d_status;

    if (part != 2) {
    // 1. n = RMSNorm(x)
    if ((st = dcut_check_cuda(ctx, dcut_launch_pdl(rmsnorm_kernel, dim3(T_cap), dim3(256), 0, stream, static_cast<const __nv_bfloat16*>(x),
                                                   static_cast<const __nv_bfloat16*>(w->g_attn), cu_q, B, H, w->rms_eps, ctx->ly_norm),
                              "launch rmsnorm_kernel")) != DCUT_OK) return st;
    // 2. qkv = n . Wqkv^T
    g.N_out = qkv_w; g.K = H; g.out = ctx->ly_qkv; g.residual = nullptr;
    if ((st = launch_gemm<kPlain>(ctx, lm->act[0], wm->m[0], wm->m[0], qkv_w / BN, T_cap, wmask[0], g, stream)) != DCUT_OK) return st;
    // 3. RoPE, append the new K/V to the paged cache
    RopeArgs r;
    r.qkv = ctx->ly_qkv; r.cu_q = cu_q; r.tok_req = tok_req; r.tok_pos = tok_pos; r.block_table = block_table;
    r.block_table_stride = block_table_stride; r.inv_freq = ctx->ly_inv_freq; r.B = B; r.n_q_heads = l.n_q_heads;
    r.n_kv_heads = l.n_kv_heads; r.head_dim = Dh; r.num_pages = num_pages; r.q_out = ctx->ly_q;
    r.k_cache = static_cast<__nv_bfloat16*>(k_cache); r.v_cache = static_cast<__nv_bfloat16*>(v_cache); r.status = ctx->d_status;
    if ((st = dcut_check_cuda(ctx, dcut_launch_pdl(rope_append_kernel, dim3(T_cap), dim3(256), 0, stream, r), "launch rope_append_kernel")) != DCUT_OK) return st;
    // 4. attention
    st = dcut_launch_verify_attn(ctx, ctx->ly_q, k_cache, v_cache, num_pages, block_table, block_table_stride, ctx_lens,
                                 cu_q, B, T_cap, 1.0f / sqrtf((float)Dh), ctx->ly_attn, nullptr, reuse_plan, stream);
    if (st != DCUT_OK) return st;
    // 5. h1 = x + attn . Wo^T   (a tensor-parallel half: the rank's partial product alone, into y)
    g.N_out = H; g.K = q_w;
    if (part == 1) {
        g.out = static_cast<__nv_bfloat16*>(y); g.residual = nullptr;
        return launch_gemm<kPlain>(ctx, lm->act[1], wm->m[1], wm->m[1], H / BN, T_cap, wmask[1], g, stream);
    }
    g.out = ctx->ly_h1; g.residual = static_cast<const __nv_bfloat16*>(x);
    if ((st = launch_gemm<kResidual>(ctx, lm->act[1], wm->m[1], wm->m[1], H / BN, T_cap, wmask[1], g, stream)) != DCUT_OK) return st;
    }
    // 6. n2 = RMSNorm(h1)   (the MLP half of a tensor-parallel layer starts here, from the caller's h1)
    const __nv_bfloat16* h1 = part == 2 ? static_cast<const __nv_bfloat16*>(x) : ctx->ly_h1;
    if ((st = dcut_check_cuda(ctx, dcut_launch_pdl(rmsnorm_kernel, dim3(T_cap), dim3(256), 0, stream, h1,
                                                   static_cast<const __nv_bfloat16*>(w->g_mlp), cu_q, B, H, w->rms_eps, ctx->ly_norm2),
                              "launch rmsnorm_kernel")) != DCUT_OK) return st;
    // 7. act = SiLU(n2 . Wg^T) * (n2 . Wu^T)
    g.N_out = I; g.K = H; g.out = ctx->ly_act; g.residual = nullptr;
    if ((st = launch_gemm<kSwiGLU>(ctx, lm->act[2], wm->m[2], wm->m[3], I / (BN / 2), T_cap, wmask[2], g, stream)) != DCUT_OK) return st;
    // 8. y = h1 + act . Wd^T
    g.N_out = H; g.K = I; g.out = static_cast<__nv_bfloat16*>(y);
    if (part == 2) {
        g.residual = nullptr;
        return launch_gemm<kPlain>(ctx, lm->act[3], wm->m[4], wm->m[4], H / BN, T_cap, wmask[4], g, stream);
    }
    g.residual = ctx->ly_h1;
    return launch_gemm<kResidual>(ctx, lm->act[3], wm->m[4], wm->m[4], H / BN, T_cap, wmask[4], g, stream);
}

namespace {
// out = a + b over the rows in use (bf16, one 16-byte vector per thread and step)
__global__ void __launch_bounds__(256) residual_add_kernel(const uint4* __restrict__ a, const uint4* __restrict__ b, uint4* __restrict__ out,
                                                           const int* __restrict__ cu_q, int B, int vec_per_row) {
    dcut_pdl_wait();
    dcut_pdl_launch_dependents();
    const long long n = (long long)cu_q[B] * vec_per_row;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        const uint4 x = a[i], y = b[i];
        const uint32_t xs[4] = {x.x, x.y, x.z, x.w}, ys[4] = {y.x, y.y, y.z, y.w};
        uint32_t r[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const __nv_bfloat162 u = *reinterpret_cast<const __nv_bfloat162*>(&xs[e]), v = *reinterpret_cast<const __nv_bfloat162*>(&ys[e]);
            const __nv_bfloat162 s = __floats2bfloat162_rn(__low2float(u) + __low2float(v), __high2float(u) + __high2float(v));
            r[e] = *reinterpret_cast<const uint32_t*>(&s);
        }
        out[i] = make_uint4(r[0], r[1], r[2], r[3]);
    }
}
}  // namespace

dcut_status dcut_launch_residual_add(dcut_ctx* ctx, const void* a, const void* b, void* out, int width, const int* cu_q, int B,
                                     int T_cap, cudaStream_t stream) {
    const long long cap = (long long)T_cap * (width / 8);
    int grid = (int)((cap + 255) / 256);
    if (grid > 4 * ctx->sm_count) grid = 4 * ctx->sm_count;
    if (grid < 1) grid = 1;
    return dcut_check_cuda(ctx, dcut_launch_pdl(residual_add_kernel, dim3(grid), dim3(256), 0, stream, static_cast<const uint4*>(a),
                                                static_cast<const uint4*>(b), static_cast<uint4*>(out), cu_q, B, width / 8),
                           "launch residual_add_kernel");
}
