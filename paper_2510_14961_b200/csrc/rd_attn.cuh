// Windowed flash-decode attention for the bf16 path.
//
// One CTA takes one (query group, head, KV split).  A query group is a set of up to 128 rows of ONE
// sequence (the in-flight wavefront of a sequence during decode, 128 consecutive prompt positions
// during prefill); a CTA has one warp per 16 queries of the largest group it takes (4 or 8 warps).  The row at position p attends cache entries 0..p of its sequence: committed
// prefix and the in-flight rows <= p as overwritten this pass (shared KV cache, Section 3.2;
// causal, left to right only).  K and V tiles of 64 keys stream through shared memory once per CTA
// (16-byte cp.async, double buffered) and are reused by every query of the group, so the KV
// prefix is read once per (sequence, head) for the whole wavefront.  Each warp owns 16 queries:
// S = Q K^T and O += P V run on mma.sync m16n8k16 (bf16 in, fp32 accumulate) with an online
// softmax in fp32; P is rounded to bf16 for the second product.  The KV splits of one (group, head)
// form a thread-block cluster: each leaves its (m, l, O) partials in its own shared memory, and
// after a cluster barrier every block merges the partials of its share of the queries, in split
// order (deterministic), reading the other blocks' shared memory directly.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cooperative_groups.h>
#include <stdint.h>

#include "rd_common.cuh"

namespace rd {

constexpr int ATT_KT = 64;          // keys per tile
constexpr int ATT_QMAX = 128;       // queries per group (the paper's default maximum wavefront)
constexpr int ATT_MAX_SPLITS = 8;    // = portable cluster size

__device__ __forceinline__ void cp_async16(void* dst, const void* src, bool valid) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst);
    const int sz = valid ? 16 : 0;                      // 0 bytes read => 16 bytes of zeros written
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t* r, const void* p) {
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t* r, const void* p) {
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void mma_bf16_16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

template <int D, int NW> struct AttCfg {
    static constexpr int LD = D + 8;    // padded row (elements): ldmatrix rows fall in distinct banks
    static constexpr int QMAX = 16 * NW;   // queries a CTA of NW warps holds
    static constexpr int SMEM = (QMAX * LD + 4 * ATT_KT * LD) * 2 + 2 * QMAX * 4;   // Q, K/V double buffer, positions, row indices
};

// Grid (splits, heads, groups), clusters of `splits` blocks along x.  out: [rows, hidden] bf16.
// KW = keys of a 64-key tile one warp takes.  KW = 64: the NW warps are NW blocks of 16 queries
// (groups of up to 16 NW rows: 64 with four warps, 128 with eight).  KW = 32, for groups of at most 32 rows: warps 0,1 take the two query
// blocks on the tile's first 32 keys, warps 2,3 the same queries on its last 32, and the two halves
// are merged (first half, then second) through shared memory before the cluster merge.
// Groups in the order the hardware should start them (blockIdx.z counts through it): the host
// puts the longest contexts first so that the blocks that run longest do not start last.
constexpr int ATT_MAX_ORDERED = 64;
struct GroupOrder {
    unsigned char idx[ATT_MAX_ORDERED];
    int n;                              // 0: groups in index order
};

template <int D, int KW, int NW>
__global__ void __launch_bounds__(32 * NW)
attn_window_kernel(const GroupOrder order, const __nv_bfloat16* __restrict__ q_t, const int* __restrict__ row_pos,
                   const int* __restrict__ row_seq, const int* __restrict__ grp_index, int rows_per_group, int n_rows,
                   const __nv_bfloat16* __restrict__ Kc, const __nv_bfloat16* __restrict__ Vc, size_t seq_stride,
                   size_t head_stride, int hidden, float scale_log2, __nv_bfloat16* __restrict__ out) {
    constexpr int LD = AttCfg<D, NW>::LD;
    constexpr int QMAX = AttCfg<D, NW>::QMAX;
    constexpr int NT = 32 * NW;
    constexpr int CH = D / 8;           // 16-byte chunks per row
    static_assert(KW == 64 || NW == 4, "half-tile warps only with four warps");
    extern __shared__ __align__(16) uint8_t att_smem[];
    __nv_bfloat16* Qs = (__nv_bfloat16*)att_smem;
    __nv_bfloat16* Ks = Qs + QMAX * LD;                   // [2][KT][LD]
    __nv_bfloat16* Vs = Ks + 2 * ATT_KT * LD;             // [2][KT][LD]
    int* pos_s = (int*)(Vs + 2 * ATT_KT * LD);
    int* ridx_s = pos_s + QMAX;

    pdl_enter();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int sp = blockIdx.x, n_splits = gridDim.x, hd = blockIdx.y;
    const int grp = order.n ? (int)order.idx[blockIdx.z] : (int)blockIdx.z;
    const int r0 = grp * rows_per_group;
    // rows of the group: consecutive rows r0 .. of the row table, or (pooled slots) the rows grp_index lists
    const int nq = grp_index ? rows_per_group : min(rows_per_group, n_rows - r0);
    // positions of the group's rows; kv_len = 1 + the largest of them
    __shared__ int warp_max[NW];
    const int my_row = (tid < QMAX && tid < nq) ? (grp_index ? grp_index[r0 + tid] : r0 + tid) : -1;
    const int my_pos = my_row >= 0 ? row_pos[my_row] : -1;
    if (tid < QMAX) { pos_s[tid] = my_pos; ridx_s[tid] = my_row; }
    const int wmax = __reduce_max_sync(0xffffffffu, my_pos);
    if (lane == 0) warp_max[warp] = wmax;
    __syncthreads();
    int kv_len = 0;
#pragma unroll
    for (int w = 0; w < NW; w++) kv_len = max(kv_len, warp_max[w] + 1);
    const int n_tiles = (kv_len + ATT_KT - 1) / ATT_KT;
    const int t0 = (int)((long long)sp * n_tiles / n_splits), t1 = (int)((long long)(sp + 1) * n_tiles / n_splits);
    const int seq = grp_index ? grp : row_seq[r0];          // pooled slots: group = sequence
    // cache layout [sequence][head][position][D]: this head's keys are one contiguous stream
    const __nv_bfloat16* kbase = Kc + (size_t)seq * seq_stride + (size_t)hd * head_stride;
    const __nv_bfloat16* vbase = Vc + (size_t)seq * seq_stride + (size_t)hd * head_stride;

    for (int c = tid; c < QMAX * CH; c += NT) {
        const int r = c / CH, ch = c % CH;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (r < nq && pos_s[r] >= 0) v = *reinterpret_cast<const uint4*>(q_t + (size_t)ridx_s[r] * hidden + hd * D + ch * 8);
        *reinterpret_cast<uint4*>(Qs + r * LD + ch * 8) = v;
    }
    auto load_tile = [&](int t, int buf) {
        const int key0 = t * ATT_KT;
        for (int c = tid; c < ATT_KT * CH; c += NT) {
            const int r = c / CH, ch = c % CH;
            const int key = key0 + r;
            const bool ok = key < kv_len;
            const size_t off = (size_t)(ok ? key : 0) * D + ch * 8;
            cp_async16(Ks + (buf * ATT_KT + r) * LD + ch * 8, kbase + off, ok);
            cp_async16(Vs + (buf * ATT_KT + r) * LD + ch * 8, vbase + off, ok);
        }
        cp_async_commit();
    };

    const int qblk = KW == 64 ? warp : (warp & 1);        // block of 16 queries this warp takes
    const int koff = KW == 64 ? 0 : (warp >> 1) * KW;     // first key of the tile this warp takes
    const bool active = qblk * 16 < nq;
    const int g = lane >> 2, tq = lane & 3;
    const int qa = qblk * 16 + g, qb = qa + 8;            // this thread's two query rows
    float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f;
    float o[D / 8][4];
#pragma unroll
    for (int j = 0; j < D / 8; j++) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }

    if (t0 < t1) load_tile(t0, 0);
    __syncthreads();                                       // Qs and pos_s visible
    const int pa = pos_s[qa], pb = pos_s[qb];
    uint32_t qf[D / 16][4];
    if (active) {
#pragma unroll
        for (int kk = 0; kk < D / 16; kk++)
            ldsm_x4(qf[kk], Qs + (qblk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * LD + kk * 16 + (lane >> 4) * 8);
    }
    for (int t = t0; t < t1; t++) {
        const int buf = (t - t0) & 1;
        if (t + 1 < t1) { load_tile(t + 1, buf ^ 1); cp_async_wait<1>(); } else { cp_async_wait<0>(); }
        __syncthreads();
        if (active) {
            const __nv_bfloat16* Kt = Ks + (buf * ATT_KT + koff) * LD;
            const __nv_bfloat16* Vt = Vs + (buf * ATT_KT + koff) * LD;
            float s[KW / 8][4];
#pragma unroll
            for (int j = 0; j < KW / 8; j++) { s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f; }
#pragma unroll
            for (int kk = 0; kk < D / 16; kk++) {
#pragma unroll
                for (int jn = 0; jn < KW / 16; jn++) {
                    uint32_t kb[4];
                    ldsm_x4(kb, Kt + (jn * 16 + (lane & 7) + (lane >> 4) * 8) * LD + kk * 16 + ((lane >> 3) & 1) * 8);
                    mma_bf16_16816(s[2 * jn], qf[kk], kb[0], kb[1]);
                    mma_bf16_16816(s[2 * jn + 1], qf[kk], kb[2], kb[3]);
                }
            }
            // scale, causal mask, running max
            const int key0 = t * ATT_KT + koff;
            float mx_a = -INFINITY, mx_b = -INFINITY;
#pragma unroll
            for (int j = 0; j < KW / 8; j++) {
                const int k0 = key0 + j * 8 + 2 * tq;
                s[j][0] = (k0 <= pa) ? s[j][0] * scale_log2 : -INFINITY;
                s[j][1] = (k0 + 1 <= pa) ? s[j][1] * scale_log2 : -INFINITY;
                s[j][2] = (k0 <= pb) ? s[j][2] * scale_log2 : -INFINITY;
                s[j][3] = (k0 + 1 <= pb) ? s[j][3] * scale_log2 : -INFINITY;
                mx_a = fmaxf(mx_a, fmaxf(s[j][0], s[j][1]));
                mx_b = fmaxf(mx_b, fmaxf(s[j][2], s[j][3]));
            }
            mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 1));
            mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 2));
            mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 1));
            mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 2));
            const float mn_a = fmaxf(m_a, mx_a), mn_b = fmaxf(m_b, mx_b);
            const float ua = mn_a == -INFINITY ? 0.f : mn_a, ub = mn_b == -INFINITY ? 0.f : mn_b;
            const float ca = exp2f(m_a - ua), cb = exp2f(m_b - ub);
            m_a = mn_a; m_b = mn_b;
            float sa = 0.f, sb = 0.f;
            uint32_t pf[KW / 16][4];
#pragma unroll
            for (int j = 0; j < KW / 8; j++) {
                const float p0 = exp2f(s[j][0] - ua), p1 = exp2f(s[j][1] - ua);
                const float p2 = exp2f(s[j][2] - ub), p3 = exp2f(s[j][3] - ub);
                sa += p0 + p1;
                sb += p2 + p3;
                pf[j >> 1][(j & 1) * 2] = pack_bf16(p0, p1);
                pf[j >> 1][(j & 1) * 2 + 1] = pack_bf16(p2, p3);
            }
            l_a = l_a * ca + sa;
            l_b = l_b * cb + sb;
#pragma unroll
            for (int j = 0; j < D / 8; j++) { o[j][0] *= ca; o[j][1] *= ca; o[j][2] *= cb; o[j][3] *= cb; }
#pragma unroll
            for (int kk = 0; kk < KW / 16; kk++) {
#pragma unroll
                for (int jn = 0; jn < D / 16; jn++) {
                    uint32_t vb[4];
                    ldsm_x4_t(vb, Vt + (kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * LD + jn * 16 + (lane >> 4) * 8);
                    mma_bf16_16816(o[2 * jn], pf[kk], vb[0], vb[1]);
                    mma_bf16_16816(o[2 * jn + 1], pf[kk], vb[2], vb[3]);
                }
            }
        }
        __syncthreads();                                   // buffer may be refilled next round
    }
    // ---- partials to shared memory (the K/V buffers are free now), merge across the cluster ----
    float* Os = reinterpret_cast<float*>(att_smem);          // [QMAX][D] unnormalised outputs
    float* MLs = Os + QMAX * D;                               // [QMAX][2] (max in the log2 domain, sum)
    __syncthreads();
    if (KW != 64) {
        // the warps of the second key half hand (m, l, O) to the warps of the first half, thread to thread
        constexpr int PER = D / 2 + 4;
        float* st = MLs + QMAX * 2 + (size_t)(qblk * 32 + lane) * PER;
        if (warp >= 2) {
#pragma unroll
            for (int j = 0; j < D / 8; j++)
                *reinterpret_cast<float4*>(st + j * 4) = make_float4(o[j][0], o[j][1], o[j][2], o[j][3]);
            *reinterpret_cast<float4*>(st + D / 2) = make_float4(m_a, l_a, m_b, l_b);
        }
        __syncthreads();
        if (warp < 2) {
            const float4 ml = *reinterpret_cast<const float4*>(st + D / 2);
            const float Ma = fmaxf(m_a, ml.x), Mb = fmaxf(m_b, ml.z);
            const float ua = Ma == -INFINITY ? 0.f : Ma, ub = Mb == -INFINITY ? 0.f : Mb;
            const float a0 = exp2f(m_a - ua), a1 = exp2f(ml.x - ua), b0 = exp2f(m_b - ub), b1 = exp2f(ml.z - ub);
#pragma unroll
            for (int j = 0; j < D / 8; j++) {
                const float4 v = *reinterpret_cast<const float4*>(st + j * 4);
                o[j][0] = o[j][0] * a0 + v.x * a1;
                o[j][1] = o[j][1] * a0 + v.y * a1;
                o[j][2] = o[j][2] * b0 + v.z * b1;
                o[j][3] = o[j][3] * b0 + v.w * b1;
            }
            l_a = l_a * a0 + ml.y * a1;
            l_b = l_b * b0 + ml.w * b1;
            m_a = Ma; m_b = Mb;
        }
        __syncthreads();                                      // the staging area overlaps nothing read later
    }
    if (active && (KW == 64 || warp < 2)) {
        // row sums live spread over the quad
        l_a += __shfl_xor_sync(0xffffffffu, l_a, 1);
        l_a += __shfl_xor_sync(0xffffffffu, l_a, 2);
        l_b += __shfl_xor_sync(0xffffffffu, l_b, 1);
        l_b += __shfl_xor_sync(0xffffffffu, l_b, 2);
#pragma unroll
        for (int half = 0; half < 2; half++) {
            const int q = half ? qb : qa;
            float* po = Os + q * D;
#pragma unroll
            for (int j = 0; j < D / 8; j++)
                *reinterpret_cast<float2*>(po + j * 8 + 2 * tq) = make_float2(o[j][half * 2], o[j][half * 2 + 1]);
            if (tq == 0) {
                MLs[q * 2] = half ? m_b : m_a;
                MLs[q * 2 + 1] = half ? l_b : l_a;
            }
        }
    }
    cooperative_groups::cluster_group cluster = cooperative_groups::this_cluster();
    cluster.sync();
    // block `sp` merges queries sp, sp + n_splits, ...; one thread per 4 output elements
    constexpr int Q4 = D / 4;
    const int mine = nq > sp ? (nq - sp + n_splits - 1) / n_splits : 0;
    for (int item = tid; item < mine * Q4; item += NT) {
        const int q = sp + (item / Q4) * n_splits, e = (item % Q4) * 4;
        if (ridx_s[q] < 0) continue;                          // no row behind this entry of the group
        __nv_bfloat16* dst = out + (size_t)ridx_s[q] * hidden + hd * D + e;
        float2 ml[ATT_MAX_SPLITS];
        float4 po[ATT_MAX_SPLITS];
#pragma unroll
        for (int s2 = 0; s2 < ATT_MAX_SPLITS; s2++) {
            if (s2 < n_splits) {
                ml[s2] = *reinterpret_cast<const float2*>(cluster.map_shared_rank(MLs, s2) + q * 2);
                po[s2] = *reinterpret_cast<const float4*>(cluster.map_shared_rank(Os, s2) + q * D + e);
            }
        }
        float M = -INFINITY;
#pragma unroll
        for (int s2 = 0; s2 < ATT_MAX_SPLITS; s2++)
            if (s2 < n_splits) M = fmaxf(M, ml[s2].x);
        float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
        float den = 0.f;
#pragma unroll
        for (int s2 = 0; s2 < ATT_MAX_SPLITS; s2++) {
            if (s2 >= n_splits || ml[s2].x == -INFINITY) continue;
            const float w = exp2f(ml[s2].x - M);
            num.x += po[s2].x * w; num.y += po[s2].y * w; num.z += po[s2].z * w; num.w += po[s2].w * w;
            den += ml[s2].y * w;
        }
        const float inv = (pos_s[q] >= 0 && den > 0.f) ? 1.0f / den : 0.f;     // unused slot: zeros
        dst[0] = __float2bfloat16_rn(num.x * inv);
        dst[1] = __float2bfloat16_rn(num.y * inv);
        dst[2] = __float2bfloat16_rn(num.z * inv);
        dst[3] = __float2bfloat16_rn(num.w * inv);
    }
    cluster.sync();                                           // shared memory stays until everyone has read it
}


// ---------------------------------------------------------------------------------------------
// The same attention with K and V brought in by TMA through a ring of mbarrier-guarded stages.
//
// A stage holds one tile of 64 keys: K and V each as D/64 sub-tiles of 64 columns (rows of 128 bytes,
// 128-byte swizzle) followed, when D is not a multiple of 64, by one sub-tile of 32 columns (rows of 64
// bytes, 64-byte swizzle): TMA writes them swizzled, ldmatrix reads them with the same XOR, so no
// padding is needed and no bank conflicts arise.  The cache of one block is one 2-D tensor
// [layers * sequences * heads * max_context rows, D]; a tile that reaches past a head's last position
// reads rows of the next head (or zeros beyond the tensor), which the causal mask removes.
// One thread keeps STAGES - 1 tiles in flight beside the one being used: at the start of iteration i it
// refills the stage of tile i - 1 (released by every warp through an `empty` barrier) with tile
// i - 1 + STAGES.  Every wait is
// bounded; a wait that runs out raises the status word and the block goes on to the merge with
// whatever it has (all threads still meet at the cluster barriers).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t att_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void att_mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(att_smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void att_mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(att_smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void att_mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(att_smem_u32(bar)) : "memory");
}
constexpr uint32_t ATT_SPIN_LIMIT = 1u << 22;
__device__ __forceinline__ bool att_mbar_wait(uint64_t* bar, uint32_t parity) {
    for (uint32_t i = 0; i < ATT_SPIN_LIMIT; i++) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(att_smem_u32(bar)), "r"(parity) : "memory");
        if (ok) return true;
        if (i > 64) __nanosleep(32);
    }
    return false;
}
__device__ __forceinline__ void att_tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(att_smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(att_smem_u32(bar)) : "memory");
}

// Layout of one 64-key tile of K or V in a stage.
template <int D> struct AttTile {
    static_assert(D % 32 == 0, "head_dim a multiple of 32");
    static constexpr int NA = D / 64;            // sub-tiles of 64 columns (128-byte swizzle)
    static constexpr int NB = (D % 64) / 32;     // 0 or 1 sub-tile of 32 columns (64-byte swizzle)
    static constexpr int A_BYTES = ATT_KT * 128, B_BYTES = ATT_KT * 64;
    static constexpr int BYTES = NA * A_BYTES + NB * B_BYTES;      // = ATT_KT * D * 2
    // byte offset of the 16-byte chunk holding (row, col), col a multiple of 8
    __device__ static __forceinline__ uint32_t off(int row, int col) {
        if (col < 64 * NA) {
            const uint32_t o = (uint32_t)(row * 128 + (col & 63) * 2);
            return (uint32_t)(col >> 6) * A_BYTES + (o ^ (((o >> 7) & 7u) << 4));
        }
        const uint32_t o = (uint32_t)(row * 64 + (col - 64 * NA) * 2);
        return (uint32_t)NA * A_BYTES + (o ^ (((o >> 7) & 3u) << 4));
    }
};

template <int D, int NW> struct AttTmaCfg {
    static constexpr int LD = D + 8;                        // padded query row
    static constexpr int QMAX = 16 * NW;
    // Two stages with four warps (62 KB at head_dim 96: three blocks per SM, and the kernel is bound by
    // the latency of each warp's QK^T -> softmax -> PV chain, so resident warps count for more than tiles
    // in flight: four stages, two blocks per SM, measured 4.07 against 4.73 TB/s at 8k keys); three with eight.
    static constexpr int STAGES = NW == 4 ? 2 : 3;
    static constexpr int STAGE_BYTES = 2 * AttTile<D>::BYTES;    // K tile, V tile
    static constexpr int RING = STAGES * STAGE_BYTES;
    static constexpr int Q_BYTES = QMAX * LD * 2;
    // ring (1024-aligned) | Q | positions | barriers
    static constexpr int SMEM = 1024 + RING + Q_BYTES + 2 * QMAX * 4 + 2 * STAGES * 8 + 16;
    static_assert(QMAX * D * 4 + QMAX * 8 + 64 * (D / 2 + 4) * 4 <= RING, "merge area fits in the ring");
};

struct AttMaps {
    CUtensorMap k64, k32, v64, v32;     // boxes of 64 and of 32 columns over the K and the V cache of a block
};

// Grid (splits, heads, groups), clusters of `splits` blocks along x; 32 * NW threads.
// row_base: first row of this layer in the block's tensor (layer * sequences * heads * max_context).
template <int D, int KW, int NW>
__global__ void __launch_bounds__(32 * NW, NW == 4 ? 3 : 1)
attn_tma_kernel(const __grid_constant__ AttMaps maps, const GroupOrder order, const __nv_bfloat16* __restrict__ q_t,
                const int* __restrict__ row_pos, const int* __restrict__ row_seq, const int* __restrict__ grp_index,
                int rows_per_group, int n_rows, int row_base, int n_heads, int max_context, int hidden, float scale_log2,
                __nv_bfloat16* __restrict__ out, int* __restrict__ status) {
    using C = AttTmaCfg<D, NW>;
    using T = AttTile<D>;
    constexpr int LD = C::LD, QMAX = C::QMAX, NT = 32 * NW, CH = D / 8, S = C::STAGES;
    static_assert(KW == 64 || NW == 4, "half-tile warps only with four warps");
    extern __shared__ uint8_t att_raw[];
    uint8_t* ring = (uint8_t*)(((uintptr_t)att_raw + 1023) & ~(uintptr_t)1023);
    __nv_bfloat16* Qs = (__nv_bfloat16*)(ring + C::RING);
    int* pos_s = (int*)(ring + C::RING + C::Q_BYTES);
    int* ridx_s = pos_s + QMAX;
    uint64_t* full = (uint64_t*)(ridx_s + QMAX);
    uint64_t* empty = full + S;
    __shared__ int warp_max[NW];
    __shared__ int abort_s;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        // the descriptors do not depend on the previous kernel: fetch them before the dependency wait
        asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.k64) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.v64) : "memory");
        if (T::NB) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.k32) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.v32) : "memory");
        }
        for (int s = 0; s < S; s++) { att_mbar_init(&full[s], 1); att_mbar_init(&empty[s], NW); }
        abort_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    pdl_enter();
    const int sp = blockIdx.x, n_splits = gridDim.x, hd = blockIdx.y;
    const int grp = order.n ? (int)order.idx[blockIdx.z] : (int)blockIdx.z;
    const int r0 = grp * rows_per_group;
    const int nq = grp_index ? rows_per_group : min(rows_per_group, n_rows - r0);
    const int my_row = (tid < QMAX && tid < nq) ? (grp_index ? grp_index[r0 + tid] : r0 + tid) : -1;
    const int my_pos = my_row >= 0 ? row_pos[my_row] : -1;
    if (tid < QMAX) { pos_s[tid] = my_pos; ridx_s[tid] = my_row; }
    const int wmax = __reduce_max_sync(0xffffffffu, my_pos);
    if (lane == 0) warp_max[warp] = wmax;
    __syncthreads();                                       // barriers initialised, positions visible
    int kv_len = 0;
#pragma unroll
    for (int w = 0; w < NW; w++) kv_len = max(kv_len, warp_max[w] + 1);
    const int n_tiles = (kv_len + ATT_KT - 1) / ATT_KT;
    const int t0 = (int)((long long)sp * n_tiles / n_splits), t1 = (int)((long long)(sp + 1) * n_tiles / n_splits);
    const int nt = t1 - t0;
    const int seq = grp_index ? grp : row_seq[r0];          // pooled slots: group = sequence
    const int head_row0 = row_base + (seq * n_heads + hd) * max_context;   // row of this head's position 0

    auto issue = [&](int it) {                              // issuing thread: tile t0 + it into stage it % S
        const int s = it % S;
        uint8_t* kdst = ring + s * C::STAGE_BYTES;
        uint8_t* vdst = kdst + T::BYTES;
        const int y = head_row0 + (t0 + it) * ATT_KT;
        att_mbar_expect_tx(&full[s], C::STAGE_BYTES);
#pragma unroll
        for (int a = 0; a < T::NA; a++) {
            att_tma_load_2d(kdst + a * T::A_BYTES, &maps.k64, a * 64, y, &full[s]);
            att_tma_load_2d(vdst + a * T::A_BYTES, &maps.v64, a * 64, y, &full[s]);
        }
        if (T::NB) {
            att_tma_load_2d(kdst + T::NA * T::A_BYTES, &maps.k32, T::NA * 64, y, &full[s]);
            att_tma_load_2d(vdst + T::NA * T::A_BYTES, &maps.v32, T::NA * 64, y, &full[s]);
        }
    };
    // the thread that issues the copies: lane 0 of the LAST warp, which has no queries of its own when
    // the group is small (one row per sequence in the sequential decoder) and then acts as a producer
    const bool issuer = tid == NT - 32;
    int issued = 0;
    if (issuer) {
        issued = min(S - 1, nt);
        for (int it = 0; it < issued; it++) issue(it);
    }
    for (int c = tid; c < QMAX * CH; c += NT) {
        const int r = c / CH, ch = c % CH;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (r < nq && pos_s[r] >= 0) v = *reinterpret_cast<const uint4*>(q_t + (size_t)ridx_s[r] * hidden + hd * D + ch * 8);
        *reinterpret_cast<uint4*>(Qs + r * LD + ch * 8) = v;
    }
    const int qblk = KW == 64 ? warp : (warp & 1);        // block of 16 queries this warp takes
    const int koff = KW == 64 ? 0 : (warp >> 1) * KW;     // first key of the tile this warp takes
    const bool active = qblk * 16 < nq;
    const int g = lane >> 2, tq = lane & 3;
    const int qa = qblk * 16 + g, qb = qa + 8;            // this thread's two query rows
    float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f;
    float o[D / 8][4];
#pragma unroll
    for (int j = 0; j < D / 8; j++) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
    __syncthreads();                                       // Qs visible
    const int pa = pos_s[qa], pb = pos_s[qb];
    uint32_t qf[D / 16][4];
    if (active) {
#pragma unroll
        for (int kk = 0; kk < D / 16; kk++)
            ldsm_x4(qf[kk], Qs + (qblk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * LD + kk * 16 + (lane >> 4) * 8);
    }
    bool ok = true;
    for (int it = 0; it < nt; it++) {
        const int s = it % S;
        if (issuer && issued < nt && ok) {
            // keep S - 1 tiles in flight: the stage of tile it - 1 (or a fresh one) takes tile `issued`
            const int is = issued % S;
            if (issued >= S && !att_mbar_wait(&empty[is], ((issued / S) - 1) & 1)) { abort_s = 1; ok = false; }
            else { issue(issued); issued++; }
        }
        if (!att_mbar_wait(&full[s], (it / S) & 1)) { abort_s = 1; ok = false; }
        if (!ok || *(volatile int*)&abort_s) break;
        if (active) {
            const uint8_t* Kt = ring + s * C::STAGE_BYTES;
            const uint8_t* Vt = Kt + T::BYTES;
            float sc[KW / 8][4];
#pragma unroll
            for (int j = 0; j < KW / 8; j++) { sc[j][0] = sc[j][1] = sc[j][2] = sc[j][3] = 0.f; }
#pragma unroll
            for (int kk = 0; kk < D / 16; kk++) {
#pragma unroll
                for (int jn = 0; jn < KW / 16; jn++) {
                    uint32_t kb[4];
                    ldsm_x4(kb, Kt + T::off(koff + jn * 16 + (lane & 7) + (lane >> 4) * 8, kk * 16 + ((lane >> 3) & 1) * 8));
                    mma_bf16_16816(sc[2 * jn], qf[kk], kb[0], kb[1]);
                    mma_bf16_16816(sc[2 * jn + 1], qf[kk], kb[2], kb[3]);
                }
            }
            const int key0 = (t0 + it) * ATT_KT + koff;
            float mx_a = -INFINITY, mx_b = -INFINITY;
#pragma unroll
            for (int j = 0; j < KW / 8; j++) {
                const int k0 = key0 + j * 8 + 2 * tq;
                sc[j][0] = (k0 <= pa) ? sc[j][0] * scale_log2 : -INFINITY;
                sc[j][1] = (k0 + 1 <= pa) ? sc[j][1] * scale_log2 : -INFINITY;
                sc[j][2] = (k0 <= pb) ? sc[j][2] * scale_log2 : -INFINITY;
                sc[j][3] = (k0 + 1 <= pb) ? sc[j][3] * scale_log2 : -INFINITY;
                mx_a = fmaxf(mx_a, fmaxf(sc[j][0], sc[j][1]));
                mx_b = fmaxf(mx_b, fmaxf(sc[j][2], sc[j][3]));
            }
            mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 1));
            mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 2));
            mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 1));
            mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 2));
            const float mn_a = fmaxf(m_a, mx_a), mn_b = fmaxf(m_b, mx_b);
            const float ua = mn_a == -INFINITY ? 0.f : mn_a, ub = mn_b == -INFINITY ? 0.f : mn_b;
            const float ca = exp2f(m_a - ua), cb = exp2f(m_b - ub);
            m_a = mn_a; m_b = mn_b;
            float sa = 0.f, sb = 0.f;
            uint32_t pf[KW / 16][4];
#pragma unroll
            for (int j = 0; j < KW / 8; j++) {
                const float p0 = exp2f(sc[j][0] - ua), p1 = exp2f(sc[j][1] - ua);
                const float p2 = exp2f(sc[j][2] - ub), p3 = exp2f(sc[j][3] - ub);
                sa += p0 + p1;
                sb += p2 + p3;
                pf[j >> 1][(j & 1) * 2] = pack_bf16(p0, p1);
                pf[j >> 1][(j & 1) * 2 + 1] = pack_bf16(p2, p3);
            }
            l_a = l_a * ca + sa;
            l_b = l_b * cb + sb;
#pragma unroll
            for (int j = 0; j < D / 8; j++) { o[j][0] *= ca; o[j][1] *= ca; o[j][2] *= cb; o[j][3] *= cb; }
#pragma unroll
            for (int kk = 0; kk < KW / 16; kk++) {
#pragma unroll
                for (int jn = 0; jn < D / 16; jn++) {
                    uint32_t vb[4];
                    ldsm_x4_t(vb, Vt + T::off(koff + kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, jn * 16 + (lane >> 4) * 8));
                    mma_bf16_16816(o[2 * jn], pf[kk], vb[0], vb[1]);
                    mma_bf16_16816(o[2 * jn + 1], pf[kk], vb[2], vb[3]);
                }
            }
        }
        __syncwarp();
        if (lane == 0) att_mbar_arrive(&empty[s]);            // this warp is done with the stage
    }
    __syncthreads();
    if (abort_s) {
        // a wait ran out: let every copy this block issued land before its memory is reused or released
        if (issuer) {
            for (int it = max(0, issued - S); it < issued; it++) att_mbar_wait(&full[it % S], (it / S) & 1);
            atomicExch(status, 1);
        }
        __syncthreads();
    }
    // ---- partials to shared memory (the ring is free now), merge across the cluster ----
    float* Os = reinterpret_cast<float*>(ring);              // [QMAX][D] unnormalised outputs
    float* MLs = Os + QMAX * D;                               // [QMAX][2] (max in the log2 domain, sum)
    if (KW != 64) {
        // the warps of the second key half hand (m, l, O) to the warps of the first half, thread to thread
        constexpr int PER = D / 2 + 4;
        float* st = MLs + QMAX * 2 + (size_t)(qblk * 32 + lane) * PER;
        if (warp >= 2) {
#pragma unroll
            for (int j = 0; j < D / 8; j++)
                *reinterpret_cast<float4*>(st + j * 4) = make_float4(o[j][0], o[j][1], o[j][2], o[j][3]);
            *reinterpret_cast<float4*>(st + D / 2) = make_float4(m_a, l_a, m_b, l_b);
        }
        __syncthreads();
        if (warp < 2) {
            const float4 ml = *reinterpret_cast<const float4*>(st + D / 2);
            const float Ma = fmaxf(m_a, ml.x), Mb = fmaxf(m_b, ml.z);
            const float ua = Ma == -INFINITY ? 0.f : Ma, ub = Mb == -INFINITY ? 0.f : Mb;
            const float a0 = exp2f(m_a - ua), a1 = exp2f(ml.x - ua), b0 = exp2f(m_b - ub), b1 = exp2f(ml.z - ub);
#pragma unroll
            for (int j = 0; j < D / 8; j++) {
                const float4 v = *reinterpret_cast<const float4*>(st + j * 4);
                o[j][0] = o[j][0] * a0 + v.x * a1;
                o[j][1] = o[j][1] * a0 + v.y * a1;
                o[j][2] = o[j][2] * b0 + v.z * b1;
                o[j][3] = o[j][3] * b0 + v.w * b1;
            }
            l_a = l_a * a0 + ml.y * a1;
            l_b = l_b * b0 + ml.w * b1;
            m_a = Ma; m_b = Mb;
        }
        __syncthreads();                                      // the staging area overlaps nothing read later
    }
    if (active && (KW == 64 || warp < 2)) {
        l_a += __shfl_xor_sync(0xffffffffu, l_a, 1);
        l_a += __shfl_xor_sync(0xffffffffu, l_a, 2);
        l_b += __shfl_xor_sync(0xffffffffu, l_b, 1);
        l_b += __shfl_xor_sync(0xffffffffu, l_b, 2);
#pragma unroll
        for (int half = 0; half < 2; half++) {
            const int q = half ? qb : qa;
            float* po = Os + q * D;
#pragma unroll
            for (int j = 0; j < D / 8; j++)
                *reinterpret_cast<float2*>(po + j * 8 + 2 * tq) = make_float2(o[j][half * 2], o[j][half * 2 + 1]);
            if (tq == 0) {
                MLs[q * 2] = half ? m_b : m_a;
                MLs[q * 2 + 1] = half ? l_b : l_a;
            }
        }
    }
    cooperative_groups::cluster_group cluster = cooperative_groups::this_cluster();
    cluster.sync();
    // block `sp` merges queries sp, sp + n_splits, ...; one thread per 4 output elements
    constexpr int Q4 = D / 4;
    const int mine = nq > sp ? (nq - sp + n_splits - 1) / n_splits : 0;
    for (int item = tid; item < mine * Q4; item += NT) {
        const int q = sp + (item / Q4) * n_splits, e = (item % Q4) * 4;
        if (ridx_s[q] < 0) continue;                          // no row behind this entry of the group
        __nv_bfloat16* dst = out + (size_t)ridx_s[q] * hidden + hd * D + e;
        float2 ml[ATT_MAX_SPLITS];
        float4 po[ATT_MAX_SPLITS];
#pragma unroll
        for (int s2 = 0; s2 < ATT_MAX_SPLITS; s2++) {
            if (s2 < n_splits) {
                ml[s2] = *reinterpret_cast<const float2*>(cluster.map_shared_rank(MLs, s2) + q * 2);
                po[s2] = *reinterpret_cast<const float4*>(cluster.map_shared_rank(Os, s2) + q * D + e);
            }
        }
        float M = -INFINITY;
#pragma unroll
        for (int s2 = 0; s2 < ATT_MAX_SPLITS; s2++)
            if (s2 < n_splits) M = fmaxf(M, ml[s2].x);
        float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
        float den = 0.f;
#pragma unroll
        for (int s2 = 0; s2 < ATT_MAX_SPLITS; s2++) {
            if (s2 >= n_splits || ml[s2].x == -INFINITY) continue;
            const float w = exp2f(ml[s2].x - M);
            num.x += po[s2].x * w; num.y += po[s2].y * w; num.z += po[s2].z * w; num.w += po[s2].w * w;
            den += ml[s2].y * w;
        }
        const float inv = (pos_s[q] >= 0 && den > 0.f) ? 1.0f / den : 0.f;     // unused slot: zeros
        dst[0] = __float2bfloat16_rn(num.x * inv);
        dst[1] = __float2bfloat16_rn(num.y * inv);
        dst[2] = __float2bfloat16_rn(num.z * inv);
        dst[3] = __float2bfloat16_rn(num.w * inv);
    }
    cluster.sync();                                           // shared memory stays until everyone has read it
}

}  // namespace rd
