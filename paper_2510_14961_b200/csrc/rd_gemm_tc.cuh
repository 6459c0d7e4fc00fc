// Weight-streaming GEMM on the 5th-generation tensor cores (tcgen05 + TMEM, operands by TMA).
//
//   Y[r, o] = sum_k X[r, k] * W[o, k]  (+ resid[r, o]),   X: [rows, K] bf16,  W: [n_out, K] bf16
//
// The W positions in flight share the weights, so one step is a dense contraction; at W <= 256 rows
// it is bound by streaming W from HBM once.  Mapping: the WEIGHT tile is the UMMA M operand
// (128 output features x 64 k), the activation rows are the N operand (16..256 rows x 64 k), both
// K-major with the 128-byte swizzle TMA writes; the accumulator D[feature, row] lives in TMEM
// (128 lanes x BN columns, fp32).  One CTA computes one (feature tile, row tile, K range) unit:
//   warp 0 / lane 0   TMA producer: fills a ring of STAGES {A,B} stages, mbarrier complete_tx
//   warp 1 / lane 0   issues tcgen05.mma (4 per stage, K = 16 each); tcgen05.commit frees the stage
//   warps 0-3         epilogue: tcgen05.ld of their 32 TMEM lanes, coalesced stores along features
// Split-K units write fp32 partials [split][row][feature]; a second kernel adds them in split order
// (no float atomics: results are bit-reproducible).
// Every wait on an mbarrier is bounded; on time-out the kernel raises a status word, drains the
// copies it issued, frees its TMEM and returns.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>

#include "../../include/rd.h"

namespace rd {

constexpr int TC_BM = 128;       // output features per tile (UMMA M)
constexpr int TC_BK = 64;        // k per stage: 64 bf16 = one 128-byte swizzle row
constexpr int TC_MAX_SPLITS = 8;
constexpr uint32_t TC_SPIN_LIMIT = 1u << 22;

struct TcWeight {
    CUtensorMap map;
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
    const int rc = tc_encode(&w->map, ptr, (uint64_t)n_out, (uint64_t)K, TC_BM);
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
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false when the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    for (uint32_t i = 0; i < TC_SPIN_LIMIT; i++) {
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

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes (64 bf16), stored as
// TMA's 128-byte swizzle writes them: 8-row groups 1024 bytes apart (stride offset), descriptor
// version 1, layout type SWIZZLE_128B.  Successive K = 16 slices start 32 bytes further on.
__device__ __forceinline__ uint64_t umma_desc_k128(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = bn.
__host__ __device__ constexpr uint32_t umma_idesc(int bn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
}

template <int BN> struct TcCfg {
    static constexpr int A_BYTES = TC_BM * TC_BK * 2;                 // 16 KB
    static constexpr int B_BYTES = BN * TC_BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES = BN <= 16 ? 6 : BN <= 32 ? 5 : BN <= 64 ? 4 : BN <= 128 ? 3 : 4;
    static constexpr int SMEM = STAGES * STAGE_BYTES + 1024 /*align*/ + 256 /*barriers*/;
    static constexpr int TMEM_COLS = BN < 32 ? 32 : BN;
};

struct TcParams {
    int K, n_out, n_rows;
    int kb_total, kb_per_split, n_splits;
    float* Y; size_t ldy;             // used when n_splits == 1
    const float* resid;
    float* partial;                   // [split][rows_pad][n_out] when n_splits > 1
    int rows_pad;
    int* status;
};

template <int BN>
__global__ void __launch_bounds__(128)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x, const TcParams p) {
    using C = TcCfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* full = (uint64_t*)(smem + C::STAGES * C::STAGE_BYTES);
    uint64_t* empty = full + C::STAGES;
    uint64_t* accum = empty + C::STAGES;
    uint32_t* tmem_slot = (uint32_t*)(accum + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * TC_BM;
    const int split = blockIdx.y;
    const int n0 = blockIdx.z * BN;
    const int kb0 = split * p.kb_per_split;
    const int kb1 = min(p.kb_total, kb0 + p.kb_per_split);
    const int nkb = kb1 - kb0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::STAGES; s++) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(accum, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(tmem_slot, C::TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (threadIdx.x == 0) {
        // ---- TMA producer ----
        int issued = 0;
        for (int i = 0; i < nkb; i++) {
            const int s = i % C::STAGES;
            if (i >= C::STAGES && !mbar_wait(&empty[s], ((i / C::STAGES) - 1) & 1)) { *abort_flag = 1; break; }
            if (*abort_flag) break;
            mbar_expect_tx(&full[s], C::STAGE_BYTES);
            uint8_t* a = smem + s * C::STAGE_BYTES;
            tma_load_2d(a, &tmap_w, (kb0 + i) * TC_BK, m0, &full[s]);
            tma_load_2d(a + C::A_BYTES, &tmap_x, (kb0 + i) * TC_BK, n0, &full[s]);
            issued = i + 1;
        }
        if (*abort_flag) {
            // drain: every stage this thread armed must land before the CTA's memory is released
            for (int i = max(0, issued - C::STAGES); i < issued; i++) mbar_wait(&full[i % C::STAGES], (i / C::STAGES) & 1);
        }
    } else if (threadIdx.x == 32) {
        // ---- MMA issuer ----
        constexpr uint32_t idesc = umma_idesc(BN);
        bool ok = true;
        for (int i = 0; i < nkb && ok; i++) {
            const int s = i % C::STAGES;
            if (*abort_flag || !mbar_wait(&full[s], (i / C::STAGES) & 1)) { *abort_flag = 1; ok = false; break; }
            tc_fence_after();
            const uint32_t a = smem_u32(smem + s * C::STAGE_BYTES);
            const uint64_t adesc = umma_desc_k128(a), bdesc = umma_desc_k128(a + C::A_BYTES);
#pragma unroll
            for (int k = 0; k < TC_BK / 16; k++)
                umma_bf16(tmem_base, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, (i | k) ? 1u : 0u);
            umma_commit(&empty[s]);          // stage reusable once these MMAs have read it
        }
        umma_commit(accum);                  // accumulator complete (arrives even after an abort)
    }
    // ---- epilogue: all four warps ----
    __syncwarp();
    const bool done = mbar_wait(accum, 0);
    tc_fence_after();
    if (!done) *abort_flag = 1;
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0) atomicExch(p.status, 1);
    } else if (nkb > 0) {
        const int m = m0 + warp * 32 + lane;              // TMEM lane = output feature
#pragma unroll 1
        for (int c = 0; c < BN; c += 16) {
            uint32_t v[16];
            tmem_ld16(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)c, v);
            if (m < p.n_out) {
#pragma unroll
                for (int j = 0; j < 16; j++) {
                    const int r = n0 + c + j;
                    if (r < p.n_rows) {
                        const float acc = __uint_as_float(v[j]);
                        if (p.n_splits == 1) {
                            const size_t o = (size_t)r * p.ldy + m;
                            p.Y[o] = p.resid ? p.resid[o] + acc : acc;
                        } else {
                            p.partial[((size_t)split * p.rows_pad + r) * p.n_out + m] = acc;
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, C::TMEM_COLS);
}

// Y[r, o] = resid[r, o] + sum_s partial[s][r][o], s ascending.
__global__ void splitk_reduce_kernel(const float* __restrict__ partial, int n_splits, int rows_pad, int n_rows,
                                     int n_out, float* __restrict__ Y, size_t ldy, const float* __restrict__ resid) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)n_rows * n_out) return;
    const size_t r = i / n_out, o = i % n_out;
    float acc = 0.f;
    for (int s = 0; s < n_splits; s++) acc += partial[((size_t)s * rows_pad + r) * n_out + o];
    const size_t y = r * ldy + o;
    Y[y] = resid ? resid[y] + acc : acc;
}

static inline int tc_pick_bn(int n_rows) { return n_rows <= 16 ? 0 : n_rows <= 32 ? 1 : n_rows <= 64 ? 2 : n_rows <= 128 ? 3 : 4; }

// Number of K splits for a GEMM: enough (feature tile x row tile x split) units to fill the 148
// SMs twice over, never fewer than 8 k-blocks per unit.
static inline void tc_plan(int K, int n_out, int n_rows, int* bn_idx, int* n_splits, int* kb_per_split, int* kb_total) {
    *bn_idx = tc_pick_bn(n_rows);
    const int bn = 16 << *bn_idx;
    const int tiles = ((n_out + TC_BM - 1) / TC_BM) * ((n_rows + bn - 1) / bn);
    const int kb = (K + TC_BK - 1) / TC_BK;
    int s = (2 * 148 + tiles - 1) / tiles;
    s = s > TC_MAX_SPLITS ? TC_MAX_SPLITS : s;
    const int max_by_k = kb / 8 > 1 ? kb / 8 : 1;
    s = s > max_by_k ? max_by_k : s;
    const int per = (kb + s - 1) / s;
    *kb_per_split = per;
    *n_splits = (kb + per - 1) / per;
    *kb_total = kb;
}

// Scratch the split-K partials of this model need at `rows` rows.
static inline size_t tc_partial_elems(size_t rows, const rd_config& c) {
    const int shapes[6][2] = {{c.hidden, 3 * c.hidden}, {c.hidden, c.hidden}, {c.hidden, 2 * c.mlp_inner},
                              {c.mlp_inner, c.hidden}, {2 * c.hidden, c.hidden}, {c.hidden, c.vocab}};
    size_t need = 16;
    for (int n = 1; n <= (int)rows; n = n < 16 ? 16 : n * 2) {
        const int nr = n > (int)rows ? (int)rows : n;
        for (auto& sh : shapes) {
            int bi, ns, per, kb;
            tc_plan(sh[0], sh[1], nr, &bi, &ns, &per, &kb);
            const int bn = 16 << bi;
            const size_t rows_pad = (size_t)((nr + bn - 1) / bn) * bn;
            if (ns > 1) need = std::max(need, (size_t)ns * rows_pad * sh[1]);
        }
        if (n >= (int)rows) break;
    }
    return need;
}

template <int BN>
static int tc_launch(cudaStream_t st, const CUtensorMap& mw, const CUtensorMap& mx, const TcParams& p, dim3 grid) {
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(gemm_tc_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, TcCfg<BN>::SMEM) != cudaSuccess)
            return RD_E_CUDA;
        attr_set = true;
    }
    gemm_tc_kernel<BN><<<grid, 128, TcCfg<BN>::SMEM, st>>>(mw, mx, p);
    return cudaGetLastError() == cudaSuccess ? RD_OK : RD_E_CUDA;
}

// Returns RD_E_INVALID_ARG when the shape is not taken (caller falls back to the SIMT kernel).
static inline int tc_gemm(cudaStream_t st, const TcAct& ta, const TcWeight& tw, int K, int n_out, float* Y, size_t ldy,
                          const float* resid, int n_rows, float* partial, size_t partial_elems, int* status,
                          uint64_t* launches) {
    if (ta.K != K || tw.K != K || tw.n_out != n_out || n_rows < 1 || n_rows > ta.rows) return RD_E_INVALID_ARG;
    TcParams p;
    int bi;
    tc_plan(K, n_out, n_rows, &bi, &p.n_splits, &p.kb_per_split, &p.kb_total);
    const int bn = 16 << bi;
    const int n_tiles = (n_rows + bn - 1) / bn;
    p.K = K; p.n_out = n_out; p.n_rows = n_rows;
    p.Y = Y; p.ldy = ldy; p.resid = resid; p.partial = partial; p.status = status;
    p.rows_pad = n_tiles * bn;
    if (p.n_splits > 1 && (size_t)p.n_splits * p.rows_pad * n_out > partial_elems) return RD_E_INVALID_ARG;
    const dim3 grid((n_out + TC_BM - 1) / TC_BM, p.n_splits, n_tiles);
    int rc;
    switch (bi) {
        case 0: rc = tc_launch<16>(st, tw.map, ta.map[0], p, grid); break;
        case 1: rc = tc_launch<32>(st, tw.map, ta.map[1], p, grid); break;
        case 2: rc = tc_launch<64>(st, tw.map, ta.map[2], p, grid); break;
        case 3: rc = tc_launch<128>(st, tw.map, ta.map[3], p, grid); break;
        default: rc = tc_launch<256>(st, tw.map, ta.map[4], p, grid); break;
    }
    if (rc) return rc;
    (*launches)++;
    if (p.n_splits > 1) {
        const size_t n = (size_t)n_rows * n_out;
        splitk_reduce_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(partial, p.n_splits, p.rows_pad, n_rows, n_out,
                                                                          Y, ldy, resid);
        if (cudaGetLastError() != cudaSuccess) return RD_E_CUDA;
        (*launches)++;
    }
    return RD_OK;
}

}  // namespace rd
