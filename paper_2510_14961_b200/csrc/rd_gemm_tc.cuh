// Weight-streaming GEMM on the 5th-generation tensor cores (tcgen05 + TMEM, operands by TMA).
//
//   acc[r, o] = sum_k X[r, k] * W[o, k],   X: [rows, K] bf16,  W: [n_out, K] bf16
//
// The W positions in flight share the weights, so one step is a dense contraction; below ~250 rows
// it is bound by streaming W from HBM once.  Mapping: the WEIGHT tile is the UMMA M operand
// (128 output features x 64 k), the activation rows are the N operand (16..256 rows x 64 k), both
// K-major with the 128-byte swizzle TMA writes; the accumulator D[feature, row] lives in TMEM
// (128 lanes x BN columns, fp32, two buffers).
//
// Persistent stream-K schedule: the (row tile, feature tile, k-block) units are numbered tile by
// tile, all feature tiles of the first row tile before those of the second, and cut into one
// contiguous share per CTA (two CTAs per SM while the row tile is at most 128 wide), so every SM
// streams the same number of weight bytes through long-lived rings whatever n_out is.  With two row tiles (prefill chunks) the CTA half a grid away therefore
// streams the same weight tile at the same moment for the other row tile, and one of the two reads
// hits L2; numbered with the row tiles of a feature tile next to each other, a CTA came back to a
// weight tile a whole tile later, with more than an L2's worth of other weights streamed in between.
// A share is a list of segments (tile, k-block range):
//   warp 0 / lane 0   TMA producer: fills a ring of STAGES {A,B} stages, mbarrier complete_tx
//   warp 1 / lane 0   issues tcgen05.mma (4 per stage, K = 16 each); tcgen05.commit frees the stage
//                     and, at the end of a segment, publishes the accumulator buffer
//   warps 2-5         tcgen05.ld of their 32 TMEM lanes, coalesced stores; the next segment's MMAs
//                     run meanwhile in the other accumulator buffer
// The kernel does not finish the sums.  Each segment's fp32 partial sums go to their own slot of a
// scratch buffer (rd_partial.cuh), and the kernel that consumes the GEMM's result (normalisation,
// rotary embedding + cache write, SwiGLU, sampling) adds a tile's slots in ascending k order while
// it reads.  So there are no float atomics, no fences, no counters, nobody waits for another CTA,
// and results are bit-reproducible.  (Measured on B200: finishing split tiles inside the kernel,
// last arriver adds, cost 8-11 us per launch; the kernels here run 15-110 us.)
//
// Programmatic dependent launch: the kernel lets its successor start at once, and itself starts
// while its predecessor still runs: it sets up, requests its first ring of weight tiles (weights
// do not depend on earlier kernels), and only then waits for the predecessor before touching
// activations or the scratch buffer.
//
// Tiles of 128 and 256 rows run on CTA pairs (gemm_tc_pair_kernel, tcgen05 cta_group::2): the two CTAs of a
// cluster each stage one 128-feature weight tile and half of the rows, and one MMA of M = 256 spans
// both SMs.  Same units, slots and consumers.
//
// Every wait on an mbarrier is bounded; on time-out the kernel raises a status word, drains the
// copies it issued, frees its TMEM and returns.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>

#include "../../include/rd.h"
#include "rd_common.cuh"
#include "rd_partial.cuh"

namespace rd {

constexpr int TC_BM = 128;       // output features per tile (UMMA M)
constexpr int TC_BK = 64;        // k per stage: 64 bf16 = one 128-byte swizzle row
constexpr int TC_THREADS = 192;
constexpr uint32_t TC_SPIN_LIMIT = 1u << 22;

struct TcParamsFuse {
    __nv_bfloat16* act_out;
    int act_ld, n_rows, inner;
};

struct TcWeight {
    CUtensorMap map;             // box of 128 output features
    CUtensorMap map2;            // box of 256 output features (two tiles per unit, see TC_MT)
    bool valid = false;
    int n_out = 0, K = 0;
};
// Activation operand: one descriptor per row-tile height (the TMA box is part of the descriptor).
struct TcAct {
    CUtensorMap map[5];          // BN = 16, 32, 64, 128, 256
    bool valid = false;
    int rows = 0, K = 0;
};

typedef CUresult (*PFN_encodeTiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static PFN_encodeTiled g_encode_tiled = nullptr;

static inline int tc_init_driver() {
    if (g_encode_tiled) return RD_OK;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess)
        return RD_E_CUDA;
    g_encode_tiled = (PFN_encodeTiled)fn;
    return RD_OK;
}

// 2-D bf16 tensor [rows, K] (K contiguous), box {64 k, box_rows}, 128-byte swizzle, zero fill
// outside the tensor (a ragged last k-block or feature tile contributes zeros).
static inline int tc_encode(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t K, uint32_t box_rows) {
    if (!g_encode_tiled) return RD_E_STATE;
    if ((K * 2) % 16 != 0 || ((uintptr_t)ptr & 15) != 0) return RD_E_INVALID_ARG;
    const cuuint64_t dims[2] = {K, rows};
    const cuuint64_t strides[1] = {K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)TC_BK, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides,
                                      box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? RD_OK : RD_E_CUDA;
}
static inline int tc_make_weight(TcWeight* w, const void* ptr, int n_out, int K) {
    w->valid = false;
    int rc = tc_encode(&w->map, ptr, (uint64_t)n_out, (uint64_t)K, TC_BM);
    if (rc) return rc;
    rc = tc_encode(&w->map2, ptr, (uint64_t)n_out, (uint64_t)K, 2 * TC_BM);
    if (rc) return rc;
    w->n_out = n_out; w->K = K; w->valid = true;
    return RD_OK;
}
static inline int tc_make_act(TcAct* a, const void* ptr, int rows, int K) {
    a->valid = false;
    for (int i = 0; i < 5; i++) {
        const int rc = tc_encode(&a->map[i], ptr, (uint64_t)rows, (uint64_t)K, 16u << i);
        if (rc) return rc;
    }
    a->rows = rows; a->K = K; a->valid = true;
    return RD_OK;
}

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false when `limit` polls ran out.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, uint32_t limit = TC_SPIN_LIMIT) {
    for (uint32_t i = 0; i < limit; i++) {
        if (mbar_test(bar, parity)) return true;
        if (i > 64) __nanosleep(64);
    }
    return false;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// ---- CTA-pair (cta_group::2) forms: two CTAs of a cluster, one on each SM of a pair, run one MMA
// of M = 256; the even-ranked CTA (the leader) issues it and owns the barriers the loads signal ----
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of the same variable in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_rank(const void* p, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load into this CTA's shared memory whose bytes are counted on a barrier of the pair's leader
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* map, int x, int y, uint32_t leader_bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(leader_bar) : "memory");
}
// issued by the same warp of both CTAs of the pair, with the same shared-memory offset for the result
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// arrives, once the pair's MMAs issued so far have completed, on the barrier at this offset in both CTAs
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar) {
    const uint16_t both = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"(both) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* v) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// 32 columns of this warp's 32 lanes in one instruction (fewer load/wait round trips per segment)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* v) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void named_bar_sync(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes (64 bf16), stored as
// TMA's 128-byte swizzle writes them: 8-row groups 1024 bytes apart (stride offset), descriptor
// version 1, layout type SWIZZLE_128B.  Successive K = 16 slices start 32 bytes further on.
__device__ __forceinline__ uint64_t umma_desc_k128(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = bn.
__host__ __device__ constexpr uint32_t umma_idesc(int bn, int m = TC_BM) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// SwiGLU on 32 accumulator columns (= rows) of this lane's feature.  Lanes 2i and 2i+1 hold gate i and
// up i of the same inner feature; the pair splits the columns between them (even lane: even columns,
// odd lane: odd columns), so every lane computes and stores 16 values.
//   raw: 32 columns of this lane; row0: row of column 0; feat: inner feature of the lane pair.
__device__ __forceinline__ void swiglu_store32(const uint32_t* raw, int lane, int row0, int feat, const TcParamsFuse& f) {
    const bool odd = lane & 1;
#pragma unroll
    for (int j = 0; j < 32; j += 2) {
        const float a = __uint_as_float(raw[j]), b = __uint_as_float(raw[j + 1]);
        const float got = __shfl_xor_sync(0xffffffffu, odd ? a : b, 1);
        const float g = odd ? got : a;            // even lane: its own gate of column j; odd lane: the partner's gate of column j+1
        const float u = odd ? b : got;
        const int row = row0 + j + (odd ? 1 : 0);
        if (row < f.n_rows && feat < f.inner)
            f.act_out[(size_t)row * f.act_ld + feat] = __float2bfloat16_rn((g / (1.0f + expf(-g))) * u);
    }
}

#ifndef RD_TC_RING_KB
#define RD_TC_RING_KB 100
#endif
#ifndef RD_TC_2CTA_MAX_BN
#define RD_TC_2CTA_MAX_BN 128
#endif
constexpr int TC_CTAS_PER_SM = 2;   // while BN <= RD_TC_2CTA_MAX_BN

// Feature tiles per unit.  At 256 rows a stage would otherwise move 32 KB of activations from L2 for
// 16 KB of weights and the SM's L2 port (about 120 GB/s) becomes the limit; two feature tiles share
// one activation tile there (two accumulators of 256 columns = all of TMEM, no double buffering).
template <int BN> struct TcTiles { static constexpr int MT = BN == 256 ? 2 : 1; };

template <int BN> struct TcCfg {
    static constexpr int MT = TcTiles<BN>::MT;
    static constexpr int A_BYTES = MT * TC_BM * TC_BK * 2;            // 16 KB per feature tile
    static constexpr int B_BYTES = BN * TC_BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    // Two CTAs per SM with about 100 KB of ring each (measured: two independent producer / MMA
    // pipelines per SM stream at the HBM peak, one with a ring twice as deep at 80 % of it).
    // Measured at 128 rows: 5.65 TB/s with two CTAs of 3 stages, 4.8 TB/s with one of 6.  The
    // 256-row tile (48 KB per stage) takes the whole SM.
    static constexpr int RING_KB = BN <= RD_TC_2CTA_MAX_BN ? RD_TC_RING_KB : 200;
    static constexpr int STAGES = (RING_KB * 1024) / STAGE_BYTES > 12 ? 12 : (RING_KB * 1024) / STAGE_BYTES;
    static constexpr int SMEM = STAGES * STAGE_BYTES + 1024 /*align*/ + 256 /*barriers*/;
    static constexpr int ACC_COLS = BN < 32 ? 32 : BN;                // columns of one accumulator
    static constexpr int NBUF = MT == 1 ? 2 : 1;                      // accumulator sets (a set = MT accumulators)
    static constexpr int TMEM_COLS = NBUF * MT * ACC_COLS;            // power of two, 64..512
};

struct TcParams {
    int kb;                    // k-blocks per tile
    int n_tiles_m;             // feature tiles of a unit's width; tile number = row tile * n_tiles_m + feature tile / MT
    long long units;           // tiles * kb
    int per;                   // units per CTA
    int max_seg;               // scratch slots per CTA
    float* scratch;            // [gridDim.x * max_seg][MT][BN][128] partial sums
    int* status;
    // Fused SwiGLU epilogue (gate/up projection with rows interleaved: feature 2j = gate j, 2j+1 = up j).
    // Non-null act_out: every CTA's share is whole tiles (per is a multiple of kb), nothing goes to the
    // scratch buffer, and the epilogue writes silu(gate) * up as bf16 to act_out[row * act_ld + j].
    TcParamsFuse fuse;         // fuse.act_out; rows >= fuse.n_rows and inner features >= fuse.inner are not written
    uint32_t spin_limit;       // polls a wait on a pipeline barrier may take (TC_SPIN_LIMIT)
    int skip_unit;             // -1.  Test aid (rd_debug_expire_next_wait): CTA 0's producer leaves this unit of
                               // its share out, so that the barrier the unit would complete is never completed
                               // and the waits on it run out
};

template <int BN>
__global__ void __launch_bounds__(TC_THREADS)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x, const TcParams p) {
    using C = TcCfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* full = (uint64_t*)(smem + C::STAGES * C::STAGE_BYTES);
    uint64_t* empty = full + C::STAGES;
    uint64_t* acc_full = empty + C::STAGES;     // [2]
    uint64_t* acc_empty = acc_full + 2;         // [2]
    uint32_t* tmem_slot = (uint32_t*)(acc_empty + 2);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long u0 = (long long)blockIdx.x * p.per;
    const long long u1 = min(p.units, u0 + p.per);
    pdl_trigger();
    if (u0 >= u1) { pdl_wait(); return; }       // no share for this CTA (uniform for the whole CTA)
    const int n_units = (int)(u1 - u0);

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::STAGES; s++) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; b++) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 4); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    if (warp == 0) {
        if (lane == 0) {
            // ---- TMA producer ----
            // Weights do not depend on the previous kernel: the first ring of A tiles is requested
            // before the dependency wait, the matching B tiles after it.
            const int pre = min(n_units, C::STAGES);
            const int skip = blockIdx.x == 0 ? p.skip_unit : -1;   // test aid: a unit among the first `pre` that is never loaded
            for (int i = 0; i < pre; i++) {
                if (i == skip) continue;
                const long long u = u0 + i;
                const int tile = (int)(u / p.kb), kblk = (int)(u % p.kb);
                mbar_expect_tx(&full[i], C::STAGE_BYTES);
                tma_load_2d(smem + i * C::STAGE_BYTES, &tmap_w, kblk * TC_BK, (tile % p.n_tiles_m) * TC_BM * C::MT, &full[i]);
            }
            pdl_wait();
            for (int i = 0; i < pre; i++) {
                if (i == skip) continue;
                const long long u = u0 + i;
                const int tile = (int)(u / p.kb), kblk = (int)(u % p.kb);
                tma_load_2d(smem + i * C::STAGE_BYTES + C::A_BYTES, &tmap_x, kblk * TC_BK, (tile / p.n_tiles_m) * BN, &full[i]);
            }
            int issued = pre;
            for (int i = pre; i < n_units; i++) {
                const int s = i % C::STAGES;
                if (*abort_flag || !mbar_wait(&empty[s], ((i / C::STAGES) - 1) & 1, p.spin_limit)) { *abort_flag = 1; break; }
                const long long u = u0 + i;
                const int tile = (int)(u / p.kb), kblk = (int)(u % p.kb);
                mbar_expect_tx(&full[s], C::STAGE_BYTES);
                uint8_t* a = smem + s * C::STAGE_BYTES;
                tma_load_2d(a, &tmap_w, kblk * TC_BK, (tile % p.n_tiles_m) * TC_BM * C::MT, &full[s]);
                tma_load_2d(a + C::A_BYTES, &tmap_x, kblk * TC_BK, (tile / p.n_tiles_m) * BN, &full[s]);
                issued = i + 1;
            }
            if (*abort_flag) {
                // drain: every stage this thread armed must land before the CTA's memory is released
                for (int i = max(0, issued - C::STAGES); i < issued; i++) mbar_wait(&full[i % C::STAGES], (i / C::STAGES) & 1, p.spin_limit);
            }
        } else {
            pdl_wait();
        }
    } else {
        if (warp == 1) tmem_alloc(tmem_slot, C::TMEM_COLS);
        tc_fence_before();
        named_bar_sync(1, TC_THREADS - 32);
        tc_fence_after();
        const uint32_t tmem_base = *tmem_slot;
        pdl_wait();
        if (warp == 1) {
            if (lane == 0) {
                // ---- MMA issuer ----
                constexpr uint32_t idesc = umma_idesc(BN);
                int i = 0, seg = 0;
                bool ok = true;
                while (i < n_units && ok) {
                    const long long u = u0 + i;
                    const int ka = (int)(u % p.kb);
                    const int len = min(p.kb - ka, n_units - i);
                    const int buf = seg % C::NBUF, use = seg / C::NBUF;
                    if (use >= 1 && !mbar_wait(&acc_empty[buf], (use - 1) & 1, p.spin_limit)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t d = tmem_base + (uint32_t)(buf * C::MT * C::ACC_COLS);
                    for (int j = 0; j < len; j++, i++) {
                        const int s = i % C::STAGES;
                        if (*abort_flag || !mbar_wait(&full[s], (i / C::STAGES) & 1, p.spin_limit)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t a = smem_u32(smem + s * C::STAGE_BYTES);
                        const uint64_t adesc = umma_desc_k128(a), bdesc = umma_desc_k128(a + C::A_BYTES);
#pragma unroll
                        for (int k = 0; k < TC_BK / 16; k++)
#pragma unroll
                            for (int mt = 0; mt < C::MT; mt++)   // the mt-th feature tile starts 16 KB further on
                                umma_bf16(d + (uint32_t)(mt * C::ACC_COLS), adesc + (uint64_t)(mt * 1024 + k * 2),
                                          bdesc + (uint64_t)(k * 2), idesc, (j | k) ? 1u : 0u);
                        umma_commit(&empty[s]);          // stage reusable once these MMAs have read it
                    }
                    if (!ok) break;
                    umma_commit(&acc_full[buf]);         // this segment's sums are complete
                    seg++;
                }
                if (!ok) *abort_flag = 1;
            }
        } else {
            // ---- warps 2..5 move finished segments from TMEM to their scratch slot ----
            const int quad = warp & 3;                    // TMEM lane quadrant a warp may read
            int i = 0, seg = 0;
            bool ok = true;
            while (i < n_units && ok) {
                const long long u = u0 + i;
                const int ka = (int)(u % p.kb);
                const int len = min(p.kb - ka, n_units - i);
                const int buf = seg % C::NBUF;
                if (*abort_flag || !mbar_wait(&acc_full[buf], (seg / C::NBUF) & 1, p.spin_limit)) { ok = false; break; }
                tc_fence_after();
                const uint32_t t = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * C::MT * C::ACC_COLS);
                // the share's seg-th segment (= seg-th tile it touches) -> slot blockIdx.x * max_seg + seg
                float* slot = p.scratch + ((size_t)blockIdx.x * p.max_seg + seg) * (size_t)(C::MT * BN * TC_BM) + quad * 32 + lane;
                if (p.fuse.act_out) {
                    // whole tile (ka == 0, len == kb): SwiGLU straight from the accumulator
                    const int tile = (int)(u / p.kb);
                    const int ftu = tile % p.n_tiles_m, rt = tile / p.n_tiles_m;
                    if constexpr (BN >= 32) {
#pragma unroll 1
                        for (int c = 0; c < C::MT * BN; c += 32) {
                            uint32_t raw[32];
                            tmem_ld32(t + (uint32_t)((c / BN) * C::ACC_COLS + c % BN), raw);
                            const int feat = ((ftu * C::MT + c / BN) * TC_BM + quad * 32 + lane) >> 1;
                            swiglu_store32(raw, lane, rt * BN + c % BN, feat, p.fuse);
                        }
                    } else {
                        uint32_t raw[32];
                        tmem_ld16(t, raw);
#pragma unroll
                        for (int j = 16; j < 32; j++) raw[j] = 0;
                        TcParamsFuse f16 = p.fuse;
                        f16.n_rows = min(f16.n_rows, rt * BN + 16);          // columns 16.. do not exist
                        swiglu_store32(raw, lane, rt * BN, ((ftu * TC_BM) + quad * 32 + lane) >> 1, f16);
                    }
                } else if constexpr (BN >= 32) {
#pragma unroll 1
                    for (int c = 0; c < C::MT * BN; c += 32) {  // column c = (feature tile in the unit) * BN + row
                        uint32_t raw[32];
                        tmem_ld32(t + (uint32_t)((c / BN) * C::ACC_COLS + c % BN), raw);
#pragma unroll
                        for (int j = 0; j < 32; j++) slot[(size_t)(c + j) * TC_BM] = __uint_as_float(raw[j]);
                    }
                } else {
                    uint32_t raw[16];
                    tmem_ld16(t, raw);
#pragma unroll
                    for (int j = 0; j < 16; j++) slot[(size_t)j * TC_BM] = __uint_as_float(raw[j]);
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&acc_empty[buf]);     // accumulator buffer may be overwritten
                i += len;
                seg++;
            }
            if (!ok) *abort_flag = 1;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) atomicExch(p.status, 1);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(*tmem_slot, C::TMEM_COLS);
    }
}

// Position of a unit in (row tile, feature tile [pair], k-block) order, advanced without division.
struct UnitCursor {
    int ft, rt, kblk;
    __device__ UnitCursor(long long u, int kb, int n_tiles_m) {
        const long long tile = u / kb;
        kblk = (int)(u % kb);
        ft = (int)(tile % n_tiles_m);
        rt = (int)(tile / n_tiles_m);
    }
    __device__ __forceinline__ void next(int kb, int n_tiles_m) {
        if (++kblk == kb) {
            kblk = 0;
            if (++ft == n_tiles_m) { ft = 0; rt++; }
        }
    }
};

// ---------------------------------------------------------------------------------------------
// 128- and 256-row tiles on a CTA pair.  Two CTAs of a cluster (one per SM of a pair) share every unit: a
// unit is (256 output features, BN rows, one k-block); CTA `rank` loads the rank-th 128-feature weight
// tile and the rank-th half of the rows of the activation tile, the leader (rank 0) issues one MMA of
// M = 256, N = BN per K = 16 slice, and each CTA's TMEM receives its own 128 features x BN rows.
// Against one CTA running two M = 128 MMAs over a full 256-row activation tile, each SM stages half
// the activation bytes per weight byte (32 KB instead of 48 KB of shared-memory writes per k-block and
// each half of the activation tile is read from shared memory once for both tensor cores), and the ring is 6 deep.
//   full[s]       leader's, 1 arrival + the bytes of both CTAs' loads (the loads of the other CTA name
//                 the leader's barrier)
//   empty[s]      one in each CTA, released by the leader's tcgen05.commit to both
//   acc_full[b]   one in each CTA, same
//   acc_empty[b]  leader's, 8 arrivals: the four TMEM-reading warps of both CTAs
// Slots, segments and the consumer side are those of gemm_tc_kernel<256>, with a pair in place of a CTA.
// ---------------------------------------------------------------------------------------------
template <int BN_> struct TcPairCfg {
    static constexpr int BN = BN_;                                    // rows of a unit (UMMA N): 128 or 256
    static constexpr int A_BYTES = TC_BM * TC_BK * 2;                 // this CTA's weight tile, 16 KB
    static constexpr int B_BYTES = (BN / 2) * TC_BK * 2;              // this CTA's half of the rows
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;             // 32 KB / 24 KB
    static constexpr int STAGES = (200 * 1024) / STAGE_BYTES;         // 6 / 8
    static constexpr int SMEM = STAGES * STAGE_BYTES + 1024 /*align*/ + 256 /*barriers*/;
    static constexpr int ACC_COLS = BN;
    static constexpr int NBUF = 2;
    static constexpr int TMEM_COLS = NBUF * ACC_COLS;                 // 512 / 256; one CTA per SM
};

template <int BN>
__global__ void __launch_bounds__(TC_THREADS)
gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x, const TcParams p) {
    using C = TcPairCfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* full = (uint64_t*)(smem + C::STAGES * C::STAGE_BYTES);
    uint64_t* empty = full + C::STAGES;
    uint64_t* acc_full = empty + C::STAGES;     // [2]
    uint64_t* acc_empty = acc_full + 2;         // [2]
    uint32_t* tmem_slot = (uint32_t*)(acc_empty + 2);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();       // 0: leader
    const int pair = blockIdx.x >> 1;
    const long long u0 = (long long)pair * p.per;
    const long long u1 = min(p.units, u0 + p.per);
    pdl_trigger();
    if (u0 >= u1) { pdl_wait(); return; }       // no share for this pair (both CTAs leave together)
    const int n_units = (int)(u1 - u0);

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::STAGES; s++) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; b++) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 8); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    cluster_sync_all();                         // both CTAs' barriers exist before anything signals them

    if (warp == 0) {
        if (lane == 0) {
            // ---- TMA producer (one in each CTA) ----
            const int pre = min(n_units, C::STAGES);
            for (int i = 0; i < pre; i++) {
                const long long u = u0 + i;
                const int tile = (int)(u / p.kb), kblk = (int)(u % p.kb);
                if (rank == 0) mbar_expect_tx(&full[i], 2 * C::STAGE_BYTES);
                tma_load_2d_pair(smem + i * C::STAGE_BYTES, &tmap_w, kblk * TC_BK,
                                 ((tile % p.n_tiles_m) * 2 + (int)rank) * TC_BM, map_to_rank(&full[i], 0));
            }
            pdl_wait();
            for (int i = 0; i < pre; i++) {
                const long long u = u0 + i;
                const int tile = (int)(u / p.kb), kblk = (int)(u % p.kb);
                tma_load_2d_pair(smem + i * C::STAGE_BYTES + C::A_BYTES, &tmap_x, kblk * TC_BK,
                                 (tile / p.n_tiles_m) * C::BN + (int)rank * (C::BN / 2), map_to_rank(&full[i], 0));
            }
            int issued = pre;
            // no division in this loop: it sets the pace of the pair (measured: 665 -> 320 cycles per unit)
            UnitCursor cur(u0 + pre, p.kb, p.n_tiles_m);
            int s = pre % C::STAGES;
            uint32_t parity = (uint32_t)(((pre / C::STAGES) - 1) & 1);
            for (int i = pre; i < n_units; i++) {
                if (*abort_flag || !mbar_wait(&empty[s], parity, p.spin_limit)) { *abort_flag = 1; break; }
                if (rank == 0) mbar_expect_tx(&full[s], 2 * C::STAGE_BYTES);
                uint8_t* a = smem + s * C::STAGE_BYTES;
                const uint32_t bar = map_to_rank(&full[s], 0);
                tma_load_2d_pair(a, &tmap_w, cur.kblk * TC_BK, (cur.ft * 2 + (int)rank) * TC_BM, bar);
                tma_load_2d_pair(a + C::A_BYTES, &tmap_x, cur.kblk * TC_BK, cur.rt * C::BN + (int)rank * (C::BN / 2), bar);
                issued = i + 1;
                cur.next(p.kb, p.n_tiles_m);
                if (++s == C::STAGES) { s = 0; parity ^= 1; }
            }
            if (*abort_flag && rank == 0) {
                // drain: the stages the leader armed count both CTAs' bytes
                for (int i = max(0, issued - C::STAGES); i < issued; i++) mbar_wait(&full[i % C::STAGES], (i / C::STAGES) & 1, p.spin_limit);
            }
        } else {
            pdl_wait();
        }
    } else {
        if (warp == 1) tmem_alloc_pair(tmem_slot, C::TMEM_COLS);
        tc_fence_before();
        named_bar_sync(1, TC_THREADS - 32);
        tc_fence_after();
        const uint32_t tmem_base = *tmem_slot;
        pdl_wait();
        if (warp == 1) {
            if (lane == 0 && rank == 0) {
                // ---- MMA issuer (leader only) ----
                constexpr uint32_t idesc = umma_idesc(C::BN, 2 * TC_BM);
                int i = 0, seg = 0, s = 0;
                uint32_t parity = 0;
                bool ok = true;
                while (i < n_units && ok) {
                    const long long u = u0 + i;
                    const int ka = (int)(u % p.kb);
                    const int len = min(p.kb - ka, n_units - i);
                    const int buf = seg % C::NBUF, use = seg / C::NBUF;
                    if (use >= 1 && !mbar_wait(&acc_empty[buf], (use - 1) & 1, p.spin_limit)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t d = tmem_base + (uint32_t)(buf * C::ACC_COLS);
                    for (int j = 0; j < len; j++, i++) {
                        if (*abort_flag || !mbar_wait(&full[s], parity, p.spin_limit)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t a = smem_u32(smem + s * C::STAGE_BYTES);
                        const uint64_t adesc = umma_desc_k128(a), bdesc = umma_desc_k128(a + C::A_BYTES);
#pragma unroll
                        for (int k = 0; k < TC_BK / 16; k++)
                            umma_bf16_pair(d, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, (j | k) ? 1u : 0u);
                        umma_commit_pair(&empty[s]);         // both CTAs' stage s reusable once these MMAs have read it
                        if (++s == C::STAGES) { s = 0; parity ^= 1; }
                    }
                    if (!ok) break;
                    umma_commit_pair(&acc_full[buf]);        // this segment's sums are complete in both CTAs
                    seg++;
                }
                if (!ok) *abort_flag = 1;
            }
        } else {
            // ---- warps 2..5 of both CTAs move their 128 features of a finished segment to its slot ----
            const int quad = warp & 3;
            const uint32_t leader_empty0 = map_to_rank(&acc_empty[0], 0), leader_empty1 = map_to_rank(&acc_empty[1], 0);
            int i = 0, seg = 0;
            bool ok = true;
            while (i < n_units && ok) {
                const long long u = u0 + i;
                const int ka = (int)(u % p.kb);
                const int len = min(p.kb - ka, n_units - i);
                const int buf = seg % C::NBUF;
                if (*abort_flag || !mbar_wait(&acc_full[buf], (seg / C::NBUF) & 1, p.spin_limit)) { ok = false; break; }
                tc_fence_after();
                const uint32_t t = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * C::ACC_COLS);
                // slot of the pair's seg-th segment; this CTA's feature tile is the rank-th of the unit's two
                float* slot = p.scratch + ((size_t)pair * p.max_seg + seg) * (size_t)(2 * C::BN * TC_BM) +
                              (size_t)rank * (C::BN * TC_BM) + quad * 32 + lane;
                if (p.fuse.act_out) {
                    // whole tile: SwiGLU straight from this CTA's 128 features of the accumulator
                    const int tile = (int)(u / p.kb);
                    const int ft = (tile % p.n_tiles_m) * 2 + (int)rank, rt = tile / p.n_tiles_m;
                    const int feat = (ft * TC_BM + quad * 32 + lane) >> 1;
#pragma unroll 1
                    for (int c = 0; c < C::BN; c += 32) {
                        uint32_t raw[32];
                        tmem_ld32(t + (uint32_t)c, raw);
                        swiglu_store32(raw, lane, rt * C::BN + c, feat, p.fuse);
                    }
                } else {
#pragma unroll 1
                    for (int c = 0; c < C::BN; c += 32) {
                        uint32_t raw[32];
                        tmem_ld32(t + (uint32_t)c, raw);
#pragma unroll
                        for (int j = 0; j < 32; j++) slot[(size_t)(c + j) * TC_BM] = __uint_as_float(raw[j]);
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(buf ? leader_empty1 : leader_empty0);
                i += len;
                seg++;
            }
            if (!ok) *abort_flag = 1;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) {
        atomicExch(p.status, 1);
        // the other CTA's loads into its own memory are counted on the leader's barriers only:
        // give copies still in flight time to land before this CTA's memory is released
        if (rank != 0) for (int i = 0; i < 200; i++) __nanosleep(1000);
    }
    __syncthreads();
    cluster_sync_all();                         // nobody signals or reads a CTA that has left
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(*tmem_slot, C::TMEM_COLS);
    }
}

static inline int tc_pick_bn(int n_rows) { return n_rows <= 16 ? 0 : n_rows <= 32 ? 1 : n_rows <= 64 ? 2 : n_rows <= 128 ? 3 : 4; }

struct TcPlan {
    int bn_idx, bn, mt, kb, n_tiles_m, n_tiles_n, per, grid, max_seg;
    bool pair;
    long long units;
    size_t scratch_elems;
};
// Every CTA gets `per` consecutive units (the last ones possibly fewer).
// `pair`: tiles of 128 and 256 rows go to CTA pairs (gemm_tc_pair_kernel) instead of single CTAs.
constexpr int TC_PAIR_MIN_BN = 128;
// `whole_tiles`: a share is a whole number of tiles (for the fused SwiGLU epilogue, which needs finished sums).
static inline TcPlan tc_plan(int K, int n_out, int n_rows, int n_sms, bool pair = true, bool whole_tiles = false) {
    TcPlan pl;
    pl.bn_idx = tc_pick_bn(n_rows);
    pl.bn = 16 << pl.bn_idx;
    pl.pair = pair && pl.bn >= TC_PAIR_MIN_BN;
    if (pl.pair) n_sms /= 2;                            // a CTA pair per two SMs takes a share
    else if (pl.bn <= RD_TC_2CTA_MAX_BN) n_sms *= TC_CTAS_PER_SM;
    pl.kb = (K + TC_BK - 1) / TC_BK;
    pl.mt = pl.pair || pl.bn == 256 ? 2 : 1;            // feature tiles per unit (= TcTiles<bn>::MT for single CTAs)
    pl.n_tiles_m = (n_out + pl.mt * TC_BM - 1) / (pl.mt * TC_BM);   // units cover mt feature tiles
    pl.n_tiles_n = (n_rows + pl.bn - 1) / pl.bn;
    pl.units = (long long)pl.n_tiles_m * pl.n_tiles_n * pl.kb;
    const long long g = std::min<long long>(n_sms, pl.units);
    pl.per = (int)((pl.units + g - 1) / g);
    if (whole_tiles) {
        const long long tiles = (long long)pl.n_tiles_m * pl.n_tiles_n;
        const long long gt = std::min<long long>(n_sms, tiles);
        pl.per = (int)((tiles + gt - 1) / gt) * pl.kb;
    }
    pl.grid = (int)((pl.units + pl.per - 1) / pl.per);
    pl.max_seg = (pl.per + pl.kb - 1) / pl.kb + 1;      // tiles a run of `per` units can touch
    pl.scratch_elems = (size_t)pl.grid * pl.max_seg * pl.mt * pl.bn * TC_BM;
    return pl;
}

template <int BN>
static int tc_launch(cudaStream_t st, const CUtensorMap& mw, const CUtensorMap& mx, const TcParams& p, int grid, bool chained) {
    return launch_chained(gemm_tc_kernel<BN>, dim3(grid), dim3(TC_THREADS), TcCfg<BN>::SMEM, st, chained, mw, mx, p) == cudaSuccess
               ? RD_OK : RD_E_CUDA;
}

template <int BN>
static int tc_launch_pair(cudaStream_t st, const CUtensorMap& mw, const CUtensorMap& mx, const TcParams& p, int pairs, bool chained) {
    return launch_chained_cluster(gemm_tc_pair_kernel<BN>, dim3(2 * pairs), dim3(TC_THREADS), TcPairCfg<BN>::SMEM, st, chained, 2, mw, mx, p) ==
                   cudaSuccess ? RD_OK : RD_E_CUDA;
}

// Opt-in to more than 48 KB of dynamic shared memory for every GEMM kernel, on the CURRENT device
// (the attribute is kept per device: call once for each device a session is created on).
static inline int tc_configure_device() {
    cudaError_t e = cudaSuccess;
    auto set = [&](auto* kern, int smem) {
        if (e == cudaSuccess) e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    };
    set(gemm_tc_kernel<16>, TcCfg<16>::SMEM);
    set(gemm_tc_kernel<32>, TcCfg<32>::SMEM);
    set(gemm_tc_kernel<64>, TcCfg<64>::SMEM);
    set(gemm_tc_kernel<128>, TcCfg<128>::SMEM);
    set(gemm_tc_kernel<256>, TcCfg<256>::SMEM);
    set(gemm_tc_pair_kernel<128>, TcPairCfg<128>::SMEM);
    set(gemm_tc_pair_kernel<256>, TcPairCfg<256>::SMEM);
    return e == cudaSuccess ? RD_OK : RD_E_CUDA;
}

// Launches the GEMM; *out describes where a consumer finds the sums.  Returns RD_E_INVALID_ARG when
// the shape is not taken (caller falls back to the SIMT kernels).
static inline int tc_gemm(cudaStream_t st, const TcAct& ta, const TcWeight& tw, int K, int n_out, int n_rows,
                          float* scratch, size_t scratch_elems, int n_sms, int* status, bool chained, PartialSums* out,
                          bool pair = true, bool* expire_wait = nullptr, const TcParamsFuse* fuse = nullptr) {
    if (ta.K != K || tw.K != K || tw.n_out != n_out || n_rows < 1 || n_rows > ta.rows) return RD_E_INVALID_ARG;
    const TcPlan pl = tc_plan(K, n_out, n_rows, n_sms, pair, fuse != nullptr);
    if (!fuse && pl.scratch_elems > scratch_elems) return RD_E_INVALID_ARG;
    TcParams p;
    p.kb = pl.kb; p.n_tiles_m = pl.n_tiles_m; p.units = pl.units; p.per = pl.per; p.max_seg = pl.max_seg;
    p.scratch = scratch; p.status = status;
    p.fuse = fuse ? *fuse : TcParamsFuse{nullptr, 0, 0, 0};
    p.spin_limit = TC_SPIN_LIMIT; p.skip_unit = -1;
    if (expire_wait && *expire_wait && !pl.pair) {
        // test aid, one launch: CTA 0 never loads the first unit of its share and every wait of the
        // launch gives up after a few thousand polls; the kernel then raises the status word
        p.spin_limit = 1u << 12; p.skip_unit = 0;
        *expire_wait = false;
    }
    out->scratch = scratch; out->kb = pl.kb; out->per = pl.per; out->n_tiles_m = pl.n_tiles_m; out->bn = pl.bn;
    out->max_seg = pl.max_seg; out->mt_shift = pl.mt == 2 ? 1 : 0;
    switch (pl.bn_idx) {
        case 0: return tc_launch<16>(st, tw.map, ta.map[0], p, pl.grid, chained);
        case 1: return tc_launch<32>(st, tw.map, ta.map[1], p, pl.grid, chained);
        case 2: return tc_launch<64>(st, tw.map, ta.map[2], p, pl.grid, chained);
        case 3:
            if (pl.pair) return tc_launch_pair<128>(st, tw.map, ta.map[2], p, pl.grid, chained);   // 64 rows per CTA
            return tc_launch<128>(st, tw.map, ta.map[3], p, pl.grid, chained);
        default:
            if (pl.pair) return tc_launch_pair<256>(st, tw.map, ta.map[3], p, pl.grid, chained);   // 128 rows per CTA
            return tc_launch<256>(st, tw.map2, ta.map[4], p, pl.grid, chained);
    }
}

}  // namespace rd
