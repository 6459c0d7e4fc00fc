// SIMT kernels of the recurrent-depth sampler: everything on the step that is not a tensor-core
// GEMM (row planning, embedding, RMSNorm, rotary + KV write, attention, SwiGLU, sampling, the
// convergence test of Eq. 3, the freeze/commit/advance logic of Algorithms 1-2), plus a plain
// FFMA GEMM that serves the float32 configuration and acts as fallback for shapes the tensor-core
// kernel does not take.  All reductions run in a fixed order: results are bit-reproducible.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cooperative_groups.h>
#include <stdint.h>

#include "rd_common.cuh"
#include "rd_partial.cuh"

namespace rd {

typedef __nv_bfloat16 bf16;

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }
// four consecutive values as one store (dst aligned to four elements); same roundings as from_f
__device__ __forceinline__ void store4(float* dst, float a, float b, float c, float d) {
    *reinterpret_cast<float4*>(dst) = make_float4(a, b, c, d);
}
__device__ __forceinline__ void store4(bf16* dst, float a, float b, float c, float d) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    uint2 w;
    w.x = *reinterpret_cast<const uint32_t*>(&lo);
    w.y = *reinterpret_cast<const uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(dst) = w;
}

// 16-byte vector load of 16/sizeof(T) elements, widened to float.
template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int N = 4;
    __device__ static __forceinline__ void load(const float* p, float* out) {
        float4 v = *reinterpret_cast<const float4*>(p);
        out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
    }
};
template <> struct Vec16<bf16> {
    static constexpr int N = 8;
    __device__ static __forceinline__ void load(const bf16* p, float* out) {
        uint4 v = *reinterpret_cast<const uint4*>(p);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; i++) {
            out[2 * i] = __uint_as_float(w[i] << 16);
            out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
};

// Sum over the block, same value in every thread; fixed order (xor tree, then warps 0..n-1).
__device__ __forceinline__ float block_sum(float v, float* sm) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    const int w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sm[w] = v;
    __syncthreads();
    float t = 0.f;
    for (int i = 0; i < nw; i++) t += sm[i];
    return t;
}

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11) and the two streams the method draws from.
// Counter = (block, position, sequence, stream); key = the session seed.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
    for (int i = 0; i < 10; i++) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
        c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
        k.x += 0x9E3779B9u;
        k.y += 0xBB67AE85u;
    }
    return c;
}
enum { STREAM_INIT_STATE = 0, STREAM_GUMBEL = 1, STREAM_NOISE = 2 };

// u = ((x >> 9) + 1/2) 2^-23 lies in (0,1) and is exact in float32.
__device__ __forceinline__ float unit_open(uint32_t x) { return ((float)(x >> 9) + 0.5f) * 1.1920928955078125e-07f; }

// Row tables -----------------------------------------------------------------------------------
// A "row" is one position being processed in this pass.  row_pos[i] < 0 marks an unused slot.

// Decode: slot s = b*Wmax + (p mod Wmax) holds position p of sequence b while p is in flight.
__global__ void plan_rows_kernel(const int* __restrict__ n_committed, const int* __restrict__ win_len,
                                 const int* __restrict__ done, int B, int Wmax, int* __restrict__ row_pos,
                                 int* __restrict__ row_seq, int* __restrict__ step_first,
                                 int* __restrict__ step_n) {
    pdl_enter();
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= B * Wmax) return;
    const int b = s / Wmax, j = s % Wmax;
    const int f = n_committed[b] - 1;
    const int w = done[b] ? 0 : win_len[b];
    const int p = f + ((j - f % Wmax + Wmax) % Wmax);
    row_pos[s] = (p < f + w) ? p : -1;
    row_seq[s] = b;
    if (j == 0) { step_first[b] = f; step_n[b] = w; }
}

// Prefill: n consecutive positions of one sequence.
__global__ void fill_rows_kernel(int seq, int start, int n, int n_slots, int* __restrict__ row_pos,
                                 int* __restrict__ row_seq) {
    pdl_enter();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_slots) return;
    row_pos[i] = i < n ? start + i : -1;
    row_seq[i] = seq;
}

// Four N(0, sigma^2) values from one Philox block: two Box-Muller pairs, evaluated in double.
__device__ __forceinline__ void normal4(uint4 x, float sigma, float* out) {
    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int a = 0; a < 4; a += 2) {
        const double u0 = ((double)(w[a] >> 9) + 0.5) * 1.1920928955078125e-07;
        const double u1 = ((double)(w[a + 1] >> 9) + 0.5) * 1.1920928955078125e-07;
        const double rad = sqrt(-2.0 * log(u0));
        double sn, cs;
        sincos(6.283185307179586476925286766559 * u1, &sn, &cs);
        out[a] = (float)((double)sigma * (rad * cs));
        out[a + 1] = (float)((double)sigma * (rad * sn));
    }
}

// Start of a pass over the rows; grid (rows, parts).
// s_0 ~ N(0, sigma^2 I), keyed by (seed, sequence, position): element j is output j%4 of block j/4.
// only_fresh: only rows whose step counter is 0 (rows appended last step) get s_0; the others keep z.
// With z_prev the kernel also takes the snapshot z_prev <- z of every active row (Algorithm 2).
// With beta > 0 it then mixes noise into z (Section 3.4): z <- (1 - b) z + b z_noise, b = beta
// max(0, 1 - t / sched_steps) for a row that has taken t steps, z_noise a fresh N(0, sigma^2 I) draw
// keyed by (seed, sequence, position, t) on its own stream.
__global__ void init_state_kernel(const int* __restrict__ row_pos, const int* __restrict__ row_seq,
                                  const int* __restrict__ row_steps, int only_fresh, int hidden,
                                  float sigma, uint64_t seed, float* __restrict__ z, size_t ldz,
                                  float* __restrict__ z_prev, float beta, int sched_steps) {
    pdl_enter();
    const int r = blockIdx.x;
    const int p = row_pos[r];
    if (p < 0) return;
    const int t = only_fresh ? row_steps[r] : 0;
    const bool fresh = !only_fresh || t == 0;
    const float b = beta > 0.f ? beta * fmaxf(0.f, 1.0f - (float)t / (float)sched_steps) : 0.f;
    const uint2 key = make_uint2((uint32_t)seed, (uint32_t)(seed >> 32));
    const uint32_t seq = (uint32_t)row_seq[r];
    const int nb = (hidden + 3) / 4;
    const bool vec = (hidden & 3) == 0 && (ldz & 3) == 0;       // 16-byte accesses
    for (int blk = blockIdx.y * blockDim.x + threadIdx.x; blk < nb; blk += gridDim.y * blockDim.x) {
        float v[4];
        if (fresh) {
            normal4(philox4x32_10(make_uint4((uint32_t)blk, (uint32_t)p, seq, STREAM_INIT_STATE), key), sigma, v);
        } else if (vec) {
            const float4 q = *reinterpret_cast<const float4*>(z + (size_t)r * ldz + blk * 4);
            v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
        } else {
#pragma unroll
            for (int a = 0; a < 4; a++) v[a] = blk * 4 + a < hidden ? z[(size_t)r * ldz + blk * 4 + a] : 0.f;
        }
        float zn[4] = {v[0], v[1], v[2], v[3]};
        if (b > 0.f) {
            float nz[4];
            normal4(philox4x32_10(make_uint4((uint32_t)blk, (uint32_t)p, seq, STREAM_NOISE | ((uint32_t)t << 8)), key), sigma, nz);
#pragma unroll
            for (int a = 0; a < 4; a++) zn[a] = __fadd_rn(__fmul_rn(1.0f - b, v[a]), __fmul_rn(b, nz[a]));
        }
        if (vec) {
            if (fresh || b > 0.f) *reinterpret_cast<float4*>(z + (size_t)r * ldz + blk * 4) = make_float4(zn[0], zn[1], zn[2], zn[3]);
            if (z_prev) *reinterpret_cast<float4*>(z_prev + (size_t)r * ldz + blk * 4) = make_float4(v[0], v[1], v[2], v[3]);
            continue;
        }
#pragma unroll
        for (int a = 0; a < 4; a++)
            if (blk * 4 + a < hidden) {
                if (fresh || b > 0.f) z[(size_t)r * ldz + blk * 4 + a] = zn[a];
                if (z_prev) z_prev[(size_t)r * ldz + blk * 4 + a] = v[a];
            }
    }
}

// x[row] = emb[token at the row's position]; grid (rows, parts), 16-byte loads.
template <typename T>
__global__ void embed_kernel(const int* __restrict__ row_pos, const int* __restrict__ row_seq,
                             const int* __restrict__ tokens, int tok_stride, const T* __restrict__ emb,
                             int hidden, float* __restrict__ x) {
    pdl_enter();
    constexpr int VEC = Vec16<T>::N;
    const int r = blockIdx.x;
    const int p = row_pos[r];
    if (p < 0) return;
    const int tok = tokens[(size_t)row_seq[r] * tok_stride + p];
    for (int j = (blockIdx.y * blockDim.x + threadIdx.x) * VEC; j < hidden; j += gridDim.y * blockDim.x * VEC) {
        float v[VEC];
        Vec16<T>::load(emb + (size_t)tok * hidden + j, v);
#pragma unroll
        for (int i = 0; i < VEC; i++) x[(size_t)r * hidden + j + i] = v[i];
    }
}

// x[row] = src[row] (+ resid[row]);  out[row] = g * x / sqrt(mean(x^2) + eps).
// One cluster of CL blocks per row, grid (CL, rows): each block takes a run of
// features, keeps its part of x in shared memory, and the blocks exchange their sums of squares
// through distributed shared memory (added in block order).  `src` is a finished array or the
// partial sums of the GEMM before (added here, in k order); with x_store, x is written out as the
// new residual stream (x_store may alias resid).
// CL blocks per row: 8 up to 32 rows in flight (latency), 4 up to 127 rows and 2 from 128 rows on (as
// few waves of blocks as possible, each thread several groups of four).
template <typename TO, int CL>
__global__ void __launch_bounds__(256, CL == 2 ? 4 : 3)
rmsnorm_kernel(const RowSource src, const float* __restrict__ resid, size_t ldr, float* __restrict__ x_store,
               size_t ldx, const float* __restrict__ g, int hidden, float eps, TO* __restrict__ out, size_t ldo,
               const int* __restrict__ row_pos) {
    extern __shared__ __align__(16) float xpart[];
    __shared__ float sm[32];
    __shared__ float ss_all[CL];                       // every block's sum, pushed by its owner
    // the gains are weights: they are fetched before the wait for the predecessor
    pdl_trigger();
    const int chunk = ((hidden / 4 + CL - 1) / CL) * 4;
    const int m0 = blockIdx.x * chunk, m1 = min(hidden, m0 + chunk);
    constexpr int GMAX = 4;                                      // gains kept in registers per thread
    float gr[GMAX];
#pragma unroll
    for (int i = 0; i < GMAX; i++) {
        const int j = m0 + threadIdx.x + i * blockDim.x;
        gr[i] = j < m1 ? g[j] : 0.f;
    }
    const int r = blockIdx.y;
    // where this thread's first group of four sits in the GEMM's scratch: arithmetic only, also before the wait
    constexpr int NQ = 8;      // out- and down-projection tiles are cut into up to 8 segments at 32 rows
    const int m_first = m0 + threadIdx.x * 4;
    RowSlots<NQ> first_slots;
    first_slots.n = NQ + 1;
    // (many rows in flight, CL == 2: the kernel is bound by its instruction count and its registers,
    // not by the latency after the wait; every group goes through row_source_load4)
    if constexpr (CL > 2)
        if (m_first < m1) first_slots = row_source_locate<NQ>(src, r, m_first);
    pdl_wait();
    cooperative_groups::cluster_group cluster = cooperative_groups::this_cluster();
    if (row_pos && row_pos[r] < 0) return;                       // the whole cluster leaves
    // first cluster barrier, split: arrive now, wait before the first access to another block's
    // shared memory (which is only legal once that block runs)
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    float ss = 0.f;
    for (int m = m_first; m < m1; m += blockDim.x * 4) {
        float4 v;
        if constexpr (CL > 2) v = (m == m_first && first_slots.n <= NQ) ? row_source_fetch<NQ>(first_slots) : row_source_load4(src, r, m);
        else v = row_source_load4(src, r, m);
        if (resid) {
            const float4 q = *reinterpret_cast<const float4*>(resid + (size_t)r * ldr + m);
            v.x += q.x; v.y += q.y; v.z += q.z; v.w += q.w;
        }
        if (x_store) *reinterpret_cast<float4*>(x_store + (size_t)r * ldx + m) = v;
        *reinterpret_cast<float4*>(xpart + (m - m0)) = v;
        ss += v.x * v.x;
        ss += v.y * v.y;
        ss += v.z * v.z;
        ss += v.w * v.w;
    }
    ss = block_sum(ss, sm);
    // each block writes its sum into every block's table; after the cluster barrier all tables are
    // complete and nobody touches another block's memory again
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    if (threadIdx.x < CL) *cluster.map_shared_rank(&ss_all[blockIdx.x], threadIdx.x) = ss;
    cluster.sync();
    float tot = 0.f;
    for (int k = 0; k < CL; k++) tot += ss_all[k];
    const float inv = 1.0f / sqrtf(tot / (float)hidden + eps);
#pragma unroll
    for (int i = 0; i < GMAX; i++) {
        const int j = m0 + threadIdx.x + i * blockDim.x;
        if (j < m1) out[(size_t)r * ldo + j] = from_f<TO>(gr[i] * (xpart[j - m0] * inv));
    }
    for (int j = m0 + threadIdx.x + GMAX * blockDim.x; j < m1; j += blockDim.x)
        out[(size_t)r * ldo + j] = from_f<TO>(g[j] * (xpart[j - m0] * inv));
}

// out[row] = src[row] (+ resid[row]) as a plain float32 array (n multiple of 4: vector path).
// With eta > 0 (momentum on the input conditioning, Section 3.4) a row that has already taken a step
// gets out = eta out_old + (1 - eta) (src + resid); a row at its first step has no out_old.
__global__ void reduce_store_kernel(const RowSource src, const float* __restrict__ resid, size_t ldr,
                                    float* __restrict__ out, size_t ldo, int n, int n_rows,
                                    const int* __restrict__ row_pos, const int* __restrict__ row_steps, float eta) {
    pdl_trigger();
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if ((n & 3) == 0) {
        const size_t quads = (size_t)n / 4;
        const bool mine = i < (size_t)n_rows * quads;
        const int r = mine ? (int)(i / quads) : 0, m = mine ? (int)(i % quads) * 4 : 0;
        // slots located before the wait for the GEMM (arithmetic only)
        constexpr int NQ = 8;
        const RowSlots<NQ> sl = row_source_locate<NQ>(src, r, m);
        pdl_wait();
        if (!mine || row_pos[r] < 0) return;
        float4 v = sl.n <= NQ ? row_source_fetch<NQ>(sl) : row_source_load4(src, r, m);
        if (resid) {
            const float4 q = *reinterpret_cast<const float4*>(resid + (size_t)r * ldr + m);
            v.x += q.x; v.y += q.y; v.z += q.z; v.w += q.w;
        }
        float4* dst = reinterpret_cast<float4*>(out + (size_t)r * ldo + m);
        if (eta > 0.f && row_steps[r] > 0) {
            const float4 o = *dst;
            const float k = 1.0f - eta;
            v.x = __fadd_rn(__fmul_rn(eta, o.x), __fmul_rn(k, v.x));
            v.y = __fadd_rn(__fmul_rn(eta, o.y), __fmul_rn(k, v.y));
            v.z = __fadd_rn(__fmul_rn(eta, o.z), __fmul_rn(k, v.z));
            v.w = __fadd_rn(__fmul_rn(eta, o.w), __fmul_rn(k, v.w));
        }
        *dst = v;
    } else {
        pdl_wait();
        const size_t per_row = ((size_t)n + 3) / 4;
        if (i >= (size_t)n_rows * per_row) return;
        const int r = (int)(i / per_row), m0 = (int)(i % per_row) * 4;
        if (row_pos[r] < 0) return;
        const bool mix = eta > 0.f && row_steps[r] > 0;
        for (int m = m0; m < min(m0 + 4, n); m++) {
            float v = row_source_load(src, r, m);
            if (resid) v += resid[(size_t)r * ldr + m];
            float* dst = out + (size_t)r * ldo + m;
            *dst = mix ? __fadd_rn(__fmul_rn(eta, *dst), __fmul_rn(1.0f - eta, v)) : v;
        }
    }
}

// act[row] = [ e[row] ; z[row] ] in the GEMM input type (adapter input, Section 3.2).
template <typename T>
__global__ void concat_kernel(const float* __restrict__ e, size_t lde, const float* __restrict__ z,
                              size_t ldz, int hidden, T* __restrict__ act, size_t lda,
                              const int* __restrict__ row_pos) {
    pdl_enter();
    const int r = blockIdx.x;
    if (row_pos[r] < 0) return;
    for (int j = (blockIdx.y * blockDim.x + threadIdx.x) * 4; j < hidden; j += gridDim.y * blockDim.x * 4) {
        const float4 a = *reinterpret_cast<const float4*>(e + (size_t)r * lde + j);
        const float4 b = *reinterpret_cast<const float4*>(z + (size_t)r * ldz + j);
        T* d0 = act + (size_t)r * lda + j;
        T* d1 = d0 + hidden;
        d0[0] = from_f<T>(a.x); d0[1] = from_f<T>(a.y); d0[2] = from_f<T>(a.z); d0[3] = from_f<T>(a.w);
        d1[0] = from_f<T>(b.x); d1[1] = from_f<T>(b.y); d1[2] = from_f<T>(b.z); d1[3] = from_f<T>(b.w);
    }
}

// Plain GEMM  Y[r, o] = sum_k A[r, k] W[o, k] (+ resid[r, o]);  one warp per output feature,
// RT rows per warp, 16-byte loads, lanes split K, xor-tree reduction.
template <typename T, int RT>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const T* __restrict__ A, size_t lda, const T* __restrict__ W, int K, int n_out,
                 float* __restrict__ Y, size_t ldy, const float* __restrict__ resid, size_t ldr, int n_rows) {
    pdl_enter();
    constexpr int VEC = Vec16<T>::N;
    const int lane = threadIdx.x & 31;
    const int o = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int r0 = blockIdx.y * RT;
    if (o >= n_out) return;
    float acc[RT];
#pragma unroll
    for (int r = 0; r < RT; r++) acc[r] = 0.f;
    const T* wrow = W + (size_t)o * K;
    for (int k = lane * VEC; k < K; k += 32 * VEC) {
        float wf[VEC];
        Vec16<T>::load(wrow + k, wf);
#pragma unroll
        for (int r = 0; r < RT; r++) {
            const int rr = min(r0 + r, n_rows - 1);
            float af[VEC];
            Vec16<T>::load(A + (size_t)rr * lda + k, af);
#pragma unroll
            for (int i = 0; i < VEC; i++) acc[r] = fmaf(af[i], wf[i], acc[r]);
        }
    }
#pragma unroll
    for (int r = 0; r < RT; r++) {
        float v = acc[r];
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
        if (lane == 0 && r0 + r < n_rows) {
            const size_t row = (size_t)(r0 + r);
            Y[row * ldy + o] = resid ? resid[row * ldr + o] + v : v;
        }
    }
}

// Rotary embedding on adjacent pairs of q and k, then: q -> q_t (GEMM/attention input type),
// k, v -> the row's own cache entry (overwrite: KV-cache sharing, Section 3.2).
// src: result of the QKV GEMM, [rows, 3h] (q | k | v).  cos/sin: [max_ctx, d/2] float32.
// LOCATE: the slots of the first group are worked out before the wait for the GEMM (few rows in flight:
// latency); without it every group goes through row_source_load4 (many rows: instruction count).
template <typename T, bool LOCATE>
__global__ void rope_kv_kernel(const RowSource src, const int* __restrict__ row_pos,
                               const int* __restrict__ row_seq, const float* __restrict__ cos_t,
                               const float* __restrict__ sin_t, int hidden, int head_dim, T* __restrict__ q_t,
                               T* __restrict__ Kc, T* __restrict__ Vc, size_t seq_stride, size_t head_stride) {
    pdl_trigger();
    const int r = blockIdx.x;
    const int half = head_dim / 2;
    T* qdst = q_t + (size_t)r * hidden;
    // where the first group's q, k and v sums sit: arithmetic only, done before the wait for the GEMM
    constexpr int NQ = 4;
    const int m_first = (blockIdx.y * blockDim.x + threadIdx.x) * 4;
    RowSlots<NQ> sq, sk, sv;
    sq.n = NQ + 1;
    if constexpr (LOCATE)
        if (m_first < hidden) {
            sq = row_source_locate<NQ>(src, r, m_first);
            sk = row_source_locate<NQ>(src, r, hidden + m_first);
            sv = row_source_locate<NQ>(src, r, 2 * hidden + m_first);
        }
    const bool vec = (head_dim & 3) == 0;      // a group of four stays inside one head: 8- or 16-byte stores
    pdl_wait();
    // four features = two rotary pairs per thread and turn
    for (int m = m_first; m < hidden; m += gridDim.y * blockDim.x * 4) {
        // the sums are requested first; the row's position (and with it the rotary angles) meanwhile
        const bool located = LOCATE && m == m_first && sq.n <= NQ && sk.n <= NQ && sv.n <= NQ;
        const float4 q = located ? row_source_fetch<NQ>(sq) : row_source_load4(src, r, m),
                     k = located ? row_source_fetch<NQ>(sk) : row_source_load4(src, r, hidden + m),
                     v = located ? row_source_fetch<NQ>(sv) : row_source_load4(src, r, 2 * hidden + m);
        const int p = row_pos[r];
        if (p < 0) return;
        // cache layout [sequence][head][position][head_dim]: a head's keys are one contiguous stream
        T* kseq = Kc + (size_t)row_seq[r] * seq_stride + (size_t)p * head_dim;
        T* vseq = Vc + (size_t)row_seq[r] * seq_stride + (size_t)p * head_dim;
        const int i0 = ((m % head_dim) >> 1), i1 = (((m + 2) % head_dim) >> 1);
        const float c0 = cos_t[(size_t)p * half + i0], s0 = sin_t[(size_t)p * half + i0];
        const float c1 = cos_t[(size_t)p * half + i1], s1 = sin_t[(size_t)p * half + i1];
        // the two pairs may lie in different heads when head_dim is not a multiple of 4
        const size_t d0 = (size_t)(m / head_dim) * head_stride + (m % head_dim);
        if (vec) {
            store4(qdst + m, q.x * c0 - q.y * s0, q.x * s0 + q.y * c0, q.z * c1 - q.w * s1, q.z * s1 + q.w * c1);
            store4(kseq + d0, k.x * c0 - k.y * s0, k.x * s0 + k.y * c0, k.z * c1 - k.w * s1, k.z * s1 + k.w * c1);
            store4(vseq + d0, v.x, v.y, v.z, v.w);
            continue;
        }
        qdst[m] = from_f<T>(q.x * c0 - q.y * s0);
        qdst[m + 1] = from_f<T>(q.x * s0 + q.y * c0);
        qdst[m + 2] = from_f<T>(q.z * c1 - q.w * s1);
        qdst[m + 3] = from_f<T>(q.z * s1 + q.w * c1);
        const size_t d1 = (size_t)((m + 2) / head_dim) * head_stride + ((m + 2) % head_dim);
        kseq[d0] = from_f<T>(k.x * c0 - k.y * s0);
        kseq[d0 + 1] = from_f<T>(k.x * s0 + k.y * c0);
        kseq[d1] = from_f<T>(k.z * c1 - k.w * s1);
        kseq[d1 + 1] = from_f<T>(k.z * s1 + k.w * c1);
        vseq[d0] = from_f<T>(v.x);
        vseq[d0 + 1] = from_f<T>(v.y);
        vseq[d1] = from_f<T>(v.z);
        vseq[d1 + 1] = from_f<T>(v.w);
    }
}

// Causal attention, one block (4 warps) per (row, head): the row at position p attends cache
// entries 0..p of its sequence (committed prefix, and in-flight rows <= p as written this pass).
// Warps take keys round-robin with an online softmax; partials merge in warp order.
template <typename T>
__global__ void __launch_bounds__(128)
attn_row_kernel(const T* __restrict__ q_t, const int* __restrict__ row_pos, const int* __restrict__ row_seq,
                const T* __restrict__ Kc, const T* __restrict__ Vc, size_t seq_stride, size_t head_stride,
                int hidden, int head_dim, float scale, T* __restrict__ out) {
    pdl_enter();
    __shared__ float sm_m[4], sm_l[4], sm_o[4][128];
    const int r = blockIdx.x, hd = blockIdx.y;
    const int p = row_pos[r];
    if (p < 0) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const T* kb = Kc + (size_t)row_seq[r] * seq_stride + (size_t)hd * head_stride;
    const T* vb = Vc + (size_t)row_seq[r] * seq_stride + (size_t)hd * head_stride;
    float q[4], o[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int t = 0; t < 4; t++) {
        const int e = lane + 32 * t;
        q[t] = e < head_dim ? to_f(q_t[(size_t)r * hidden + hd * head_dim + e]) : 0.f;
    }
    float m = -INFINITY, l = 0.f;
    for (int j = warp; j <= p; j += 4) {
        float d = 0.f;
#pragma unroll
        for (int t = 0; t < 4; t++) {
            const int e = lane + 32 * t;
            if (e < head_dim) d = fmaf(q[t], to_f(kb[(size_t)j * head_dim + e]), d);
        }
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) d += __shfl_xor_sync(0xffffffffu, d, s);
        d *= scale;
        const float mn = fmaxf(m, d);
        const float corr = expf(m - mn), pj = expf(d - mn);
        l = l * corr + pj;
#pragma unroll
        for (int t = 0; t < 4; t++) {
            const int e = lane + 32 * t;
            if (e < head_dim) o[t] = o[t] * corr + pj * to_f(vb[(size_t)j * head_dim + e]);
        }
        m = mn;
    }
    if (lane == 0) { sm_m[warp] = m; sm_l[warp] = l; }
#pragma unroll
    for (int t = 0; t < 4; t++) sm_o[warp][lane + 32 * t] = o[t];
    __syncthreads();
    if (warp == 0) {
        float mm = sm_m[0];
        for (int w = 1; w < 4; w++) mm = fmaxf(mm, sm_m[w]);
        float ll = 0.f, acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int w = 0; w < 4; w++) {
            if (sm_m[w] == -INFINITY) continue;      // warp saw no key
            const float c = expf(sm_m[w] - mm);
            ll += sm_l[w] * c;
#pragma unroll
            for (int t = 0; t < 4; t++) acc[t] += sm_o[w][lane + 32 * t] * c;
        }
#pragma unroll
        for (int t = 0; t < 4; t++) {
            const int e = lane + 32 * t;
            if (e < head_dim) out[(size_t)r * hidden + hd * head_dim + e] = from_f<T>(acc[t] / ll);
        }
    }
}

// act[r, j..j+3] = silu(gate) * up of the gate/up GEMM's result.  Stacked layout: gate j = acc[r, j],
// up j = acc[r, I + j].  Interleaved layout (models whose gate/up matrix was interleaved at load for
// the fused tensor-core epilogue): gate j = acc[r, 2j], up j = acc[r, 2j + 1].
template <typename T>
__global__ void swiglu_kernel(const RowSource src, int inner, T* __restrict__ act, size_t lda, int n_rows,
                              const int* __restrict__ row_pos, int interleaved) {
    pdl_trigger();
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t quads = (size_t)inner / 4;
    const bool mine = i < (size_t)n_rows * quads;
    const int r = mine ? (int)(i / quads) : 0, j = mine ? (int)(i % quads) * 4 : 0;
    // where the sums sit: arithmetic only, done before the wait for the GEMM
    constexpr int NQ = 2;      // a gate/up tile is cut into at most 2 segments at the model shapes here
    const int ma = interleaved ? 2 * j : j, mb = interleaved ? 2 * j + 4 : inner + j;
    const RowSlots<NQ> sa = row_source_locate<NQ>(src, r, ma), sb = row_source_locate<NQ>(src, r, mb);
    pdl_wait();
    if (!mine) return;
    const bool located = sa.n <= NQ && sb.n <= NQ;
    const float4 a = located ? row_source_fetch<NQ>(sa) : row_source_load4(src, r, ma),
                 b = located ? row_source_fetch<NQ>(sb) : row_source_load4(src, r, mb);
    if (row_pos[r] < 0) return;
    float gv[4], uv[4];
    if (interleaved) {
        gv[0] = a.x; uv[0] = a.y; gv[1] = a.z; uv[1] = a.w;
        gv[2] = b.x; uv[2] = b.y; gv[3] = b.z; uv[3] = b.w;
    } else {
        gv[0] = a.x; gv[1] = a.y; gv[2] = a.z; gv[3] = a.w;
        uv[0] = b.x; uv[1] = b.y; uv[2] = b.z; uv[3] = b.w;
    }
#pragma unroll
    for (int k = 0; k < 4; k++) act[(size_t)r * lda + j + k] = from_f<T>((gv[k] / (1.0f + expf(-gv[k]))) * uv[k]);
}

// dst row 2j = gate row j, dst row 2j + 1 = up row j (rows of `cols` elements, 16-byte chunks).
template <typename T>
__global__ void interleave_rows_kernel(const T* __restrict__ gate, const T* __restrict__ up, T* __restrict__ dst,
                                       size_t inner, size_t cols) {
    constexpr int VEC = 16 / sizeof(T);
    const size_t chunks = cols / VEC, total = 2 * inner * chunks;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const size_t row = i / chunks, c = i % chunks;
        const T* src = (row & 1 ? up : gate) + (row >> 1) * cols + c * VEC;
        *reinterpret_cast<uint4*>(dst + row * cols + c * VEC) = *reinterpret_cast<const uint4*>(src);
    }
}

// Sample(p) of Algorithms 1-2 in two kernels.  Greedy: arg max, lowest index on ties.  Otherwise
// Gumbel-max: arg max of logit / T - log(-log u_v), u_v keyed by (seed, sequence, token position, v).
// The row at position p drafts the token of position p + 1.
//
// First kernel, grid (rows, chunks): block (r, c) takes the logits of row r (result of the LM-head
// GEMM, partial sums added here) for the c-th run of `chunk` vocabulary entries (chunk a multiple
// of 4), optionally stores them, and leaves its best (score, index).
constexpr int SAMPLE_CHUNKS = 16;
__global__ void __launch_bounds__(256)
sample_scan_kernel(const RowSource src, int vocab, int chunk, const int* __restrict__ row_pos,
                   const int* __restrict__ row_seq, float temperature, uint64_t seed,
                   float* __restrict__ logits_store, float* __restrict__ best_val, int* __restrict__ best_idx) {
    __shared__ float sv[8];
    __shared__ int si[8];
    pdl_trigger();
    const int r = blockIdx.x, ck = blockIdx.y;
    const int v0 = ck * chunk, v1 = min(vocab, v0 + chunk);
    // slots of this thread's first four logits, located before the wait for the head GEMM
    constexpr int NQ = 4;
    const int v_first = v0 + threadIdx.x * 4;
    RowSlots<NQ> first_slots;
    first_slots.n = NQ + 1;
    if (v_first + 3 < vocab && (vocab & 3) == 0 && v_first < v1) first_slots = row_source_locate<NQ>(src, r, v_first);
    pdl_wait();
    const int p = row_pos[r];
    if (p < 0) return;
    const uint2 key = make_uint2((uint32_t)seed, (uint32_t)(seed >> 32));
    const uint32_t seq = (uint32_t)row_seq[r];
    float best = -INFINITY;
    int bi = 0x7fffffff;
    for (int v = v0 + threadIdx.x * 4; v < v1; v += blockDim.x * 4) {
        float x[4];
        if (v + 3 < vocab && (vocab & 3) == 0) {
            const float4 q = (v == v_first && first_slots.n <= NQ) ? row_source_fetch<NQ>(first_slots) : row_source_load4(src, r, v);
            x[0] = q.x; x[1] = q.y; x[2] = q.z; x[3] = q.w;
        } else {
#pragma unroll
            for (int a = 0; a < 4; a++) x[a] = v + a < vocab ? row_source_load(src, r, v + a) : -INFINITY;
        }
        if (logits_store) {
#pragma unroll
            for (int a = 0; a < 4; a++)
                if (v + a < vocab) logits_store[(size_t)r * vocab + v + a] = x[a];
        }
        if (temperature > 0.f) {
            const uint4 w4 = philox4x32_10(make_uint4((uint32_t)(v >> 2), (uint32_t)(p + 1), seq, STREAM_GUMBEL), key);
            const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
            for (int a = 0; a < 4; a++) {
                const float g = -logf(-logf(unit_open(w[a])));
                x[a] = __fadd_rn(__fdiv_rn(x[a], temperature), g);
            }
        }
#pragma unroll
        for (int a = 0; a < 4; a++)
            if (v + a < vocab && x[a] > best) { best = x[a]; bi = v + a; }
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, s);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, s);
        if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
    }
    if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = best; si[threadIdx.x >> 5] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); w++)
            if (sv[w] > best || (sv[w] == best && si[w] < bi)) { best = sv[w]; bi = si[w]; }
        best_val[r * SAMPLE_CHUNKS + ck] = best;
        best_idx[r * SAMPLE_CHUNKS + ck] = bi;
    }
}

// Sample(p) with top-p (temperature > 0 and top_p < 1; the evaluation's settings in the paper's
// Appendix are temperature 0.2, top-p 0.95), one kernel.  A cluster of NUC_CLUSTER blocks takes a
// row; every thread keeps NUC_PER logits and their Gumbel-max scores in registers.  With M = max logit, mass_v = exp((l_v - M) / T), Z = sum of masses, the kept set is
//   {v : l_v >= tau}, tau the largest value with mass{l_v >= tau} >= top_p Z
// (the most probable tokens up to the first at which the cumulative probability reaches top_p, equal
// logits at the cut kept together), and v is in it exactly when mass{l_w > l_v} < top_p Z.
// The draft is the arg max of the scores over the kept set.  It is found without tau: take the arg
// max c over the tokens still eligible (all, at first); if mass{l_w > l_c} < top_p Z it is the draft;
// otherwise c and every token with a logit <= l_c are outside the kept set and leave the eligible
// ones.  A try succeeds with the probability of the kept set (>= top_p), so NUC_TRIES tries almost
// always do; the rows they leave undecided compute tau by a search over the order-preserving integer
// image of float32 (NUC_CUTS thresholds per round) and take the arg max over {l_v >= tau}.
// All sums are taken in a fixed order (thread, warp tree, warps of a block, blocks of the cluster by
// rank), so every block takes the same decisions and the result is bit-reproducible.
constexpr int NUC_CLUSTER = 8;
constexpr int NUC_THREADS = 256;
constexpr int NUC_PER = 32;                                   // logits per thread, as 8 quads
constexpr int NUC_MAX_VOCAB = NUC_CLUSTER * NUC_THREADS * NUC_PER;   // 65536
constexpr int NUC_TRIES = 4;
constexpr int NUC_CUTS = 7;                                   // thresholds per round of the search for tau

__device__ __forceinline__ uint32_t float_order_key(float x) {
    const uint32_t b = __float_as_uint(x);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

struct NucShared {
    float warp_f[NUC_THREADS / 32];
    int warp_i[NUC_THREADS / 32];
    uint32_t warp_k[NUC_THREADS / 32];
    float sum_slots[2 * NUC_CLUSTER];                         // double-buffered: one cluster barrier per reduction
    float arg_v[2 * NUC_CLUSTER];
    int arg_i[2 * NUC_CLUSTER];
    uint32_t arg_k[2 * NUC_CLUSTER];
    float cut_part[(NUC_THREADS / 32) * NUC_CUTS];
    float cut_slots[2 * NUC_CLUSTER * NUC_CUTS];
};

// Sum of `v` over the cluster, the same bits in every thread of every block.
__device__ __forceinline__ float nuc_cluster_sum(float v, NucShared& sh, int& phase, cooperative_groups::cluster_group& cluster) {
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
    if ((threadIdx.x & 31) == 0) sh.warp_f[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x < NUC_CLUSTER) {
        float b = 0.f;
        for (int w = 0; w < NUC_THREADS / 32; w++) b += sh.warp_f[w];
        *cluster.map_shared_rank(&sh.sum_slots[phase * NUC_CLUSTER + blockIdx.x], threadIdx.x) = b;   // into every block's table
    }
    cluster.sync();
    float tot = 0.f;
    for (int k = 0; k < NUC_CLUSTER; k++) tot += sh.sum_slots[phase * NUC_CLUSTER + k];
    phase ^= 1;
    return tot;
}

// Arg max (lowest index on ties) over the cluster, with the winner's key; same result everywhere.
__device__ __forceinline__ void nuc_cluster_argmax(float& best, int& bi, uint32_t& bk, NucShared& sh, int& phase,
                                                   cooperative_groups::cluster_group& cluster) {
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, s);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, s);
        const uint32_t ok = __shfl_xor_sync(0xffffffffu, bk, s);
        if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; bk = ok; }
    }
    if ((threadIdx.x & 31) == 0) { sh.warp_f[threadIdx.x >> 5] = best; sh.warp_i[threadIdx.x >> 5] = bi; sh.warp_k[threadIdx.x >> 5] = bk; }
    __syncthreads();
    if (threadIdx.x < NUC_CLUSTER) {
        float v = sh.warp_f[0]; int i = sh.warp_i[0]; uint32_t k = sh.warp_k[0];
        for (int w = 1; w < NUC_THREADS / 32; w++)
            if (sh.warp_f[w] > v || (sh.warp_f[w] == v && sh.warp_i[w] < i)) { v = sh.warp_f[w]; i = sh.warp_i[w]; k = sh.warp_k[w]; }
        const int slot = phase * NUC_CLUSTER + blockIdx.x;
        *cluster.map_shared_rank(&sh.arg_v[slot], threadIdx.x) = v;
        *cluster.map_shared_rank(&sh.arg_i[slot], threadIdx.x) = i;
        *cluster.map_shared_rank(&sh.arg_k[slot], threadIdx.x) = k;
    }
    cluster.sync();
    best = -INFINITY; bi = 0x7fffffff; bk = 0;
    for (int c = 0; c < NUC_CLUSTER; c++) {
        const int slot = phase * NUC_CLUSTER + c;
        if (sh.arg_v[slot] > best || (sh.arg_v[slot] == best && sh.arg_i[slot] < bi)) { best = sh.arg_v[slot]; bi = sh.arg_i[slot]; bk = sh.arg_k[slot]; }
    }
    phase ^= 1;
}

__global__ void __launch_bounds__(NUC_THREADS, 2)
sample_nucleus_kernel(const RowSource src, int vocab, const int* __restrict__ row_pos, const int* __restrict__ row_seq,
                      float temperature, float top_p, uint64_t seed, float* __restrict__ logits_store,
                      int* __restrict__ draft, int* __restrict__ tokens, int tok_stride) {
    __shared__ NucShared sh;
    pdl_enter();
    cooperative_groups::cluster_group cluster = cooperative_groups::this_cluster();
    const int r = blockIdx.y;
    const int p = row_pos[r];
    if (p < 0) return;                                         // the whole cluster leaves
    cluster.sync();                                            // nobody writes into a block's tables before it runs

    // quad q of the row belongs to thread (q mod 2048): consecutive threads read consecutive quads
    float x[NUC_PER];
#pragma unroll
    for (int i = 0; i < NUC_PER / 4; i++) {
        const int v = 4 * (i * (NUC_CLUSTER * NUC_THREADS) + blockIdx.x * NUC_THREADS + threadIdx.x);
        if (v + 3 < vocab && (vocab & 3) == 0) {
            const float4 q = row_source_load4(src, r, v);
            x[4 * i] = q.x; x[4 * i + 1] = q.y; x[4 * i + 2] = q.z; x[4 * i + 3] = q.w;
            if (logits_store) *reinterpret_cast<float4*>(logits_store + (size_t)r * vocab + v) = q;
        } else {
#pragma unroll
            for (int a = 0; a < 4; a++) {
                x[4 * i + a] = v + a < vocab ? row_source_load(src, r, v + a) : -INFINITY;
                if (logits_store && v + a < vocab) logits_store[(size_t)r * vocab + v + a] = x[4 * i + a];
            }
        }
    }
    // Gumbel-max scores (same noise as sample_scan_kernel); -inf beyond the vocabulary
    float sc[NUC_PER];
    {
        const uint2 key = make_uint2((uint32_t)seed, (uint32_t)(seed >> 32));
        const uint32_t seq = (uint32_t)row_seq[r];
#pragma unroll
        for (int i = 0; i < NUC_PER / 4; i++) {
            const int v = 4 * (i * (NUC_CLUSTER * NUC_THREADS) + blockIdx.x * NUC_THREADS + threadIdx.x);
            const uint4 w4 = philox4x32_10(make_uint4((uint32_t)(v >> 2), (uint32_t)(p + 1), seq, STREAM_GUMBEL), key);
            const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
            for (int a = 0; a < 4; a++) {
                const float g = -logf(-logf(unit_open(w[a])));
                sc[4 * i + a] = v + a < vocab ? __fadd_rn(__fdiv_rn(x[4 * i + a], temperature), g) : -INFINITY;
            }
        }
    }
    int phase = 0;
    // M: max over the cluster (exact, so the order does not matter)
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < NUC_PER; j++) mx = fmaxf(mx, x[j]);
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, s));
    if ((threadIdx.x & 31) == 0) sh.warp_f[threadIdx.x >> 5] = mx;
    __syncthreads();
    if (threadIdx.x < NUC_CLUSTER) {
        float b = -INFINITY;
        for (int w = 0; w < NUC_THREADS / 32; w++) b = fmaxf(b, sh.warp_f[w]);
        *cluster.map_shared_rank(&sh.sum_slots[phase * NUC_CLUSTER + blockIdx.x], threadIdx.x) = b;
    }
    cluster.sync();
    float M = -INFINITY;
    for (int k = 0; k < NUC_CLUSTER; k++) M = fmaxf(M, sh.sum_slots[phase * NUC_CLUSTER + k]);
    phase ^= 1;

    int token = 0x7fffffff;
    uint32_t allow = 0;                                        // eligible: keys >= allow
    if (M > -INFINITY && M < INFINITY) {
        const float c = 1.4426950408889634f / temperature;    // exp(d / T) = 2^(d c)
        // masses are recomputed where they are used (the same bits every time): two blocks fit an SM
        auto mass_of = [&](float l) { return l > -INFINITY ? exp2f((l - M) * c) : 0.f; };
        float zs = 0.f;
#pragma unroll
        for (int j = 0; j < NUC_PER; j++) zs += mass_of(x[j]);
        const float Z = nuc_cluster_sum(zs, sh, phase, cluster);
        const float target = top_p * Z;
        bool undecided = true;
        for (int t = 0; t < NUC_TRIES; t++) {
            float best = -INFINITY;
            int bi = 0x7fffffff;
            uint32_t bk = 0;
#pragma unroll
            for (int j = 0; j < NUC_PER; j++) {
                const int v = 4 * ((j >> 2) * (NUC_CLUSTER * NUC_THREADS) + blockIdx.x * NUC_THREADS + threadIdx.x) + (j & 3);
                const uint32_t k = float_order_key(x[j]);
                if (k >= allow && (sc[j] > best || (sc[j] == best && v < bi))) { best = sc[j]; bi = v; bk = k; }
            }
            nuc_cluster_argmax(best, bi, bk, sh, phase, cluster);
            if (bi == 0x7fffffff) break;                       // nothing eligible (a row of NaN)
            float above = 0.f;
#pragma unroll
            for (int j = 0; j < NUC_PER; j++) above += float_order_key(x[j]) > bk ? mass_of(x[j]) : 0.f;
            above = nuc_cluster_sum(above, sh, phase, cluster);
            if (above < target) { token = bi; undecided = false; break; }
            allow = bk + 1;                                    // bk is a finite number's key: no wrap
        }
        if (undecided) {
            // tau: largest key t with mass{key_v >= t} >= target; at t = 0 the mass is Z, above key(M) it is 0.
            // Each round cuts [lo, hi) at up to NUC_CUTS thresholds and sums the mass above each of them.
            uint32_t lo = 0, hi = float_order_key(M);
            if (hi != 0xffffffffu) hi += 1;
            while (hi - lo > 1) {
                const uint32_t span = hi - lo;
                const uint32_t step = (uint32_t)(((uint64_t)span + NUC_CUTS) / (NUC_CUTS + 1));   // ceil(span / (cuts + 1)) >= 1
                // thresholds lo + (i + 1) step below hi; at least one since span >= 2
                const int nt = (int)min((uint64_t)NUC_CUTS, ((uint64_t)span - 1) / step);
                float acc[NUC_CUTS];
                uint32_t cut[NUC_CUTS];                        // unused thresholds: above every key of a number
#pragma unroll
                for (int i = 0; i < NUC_CUTS; i++) {
                    acc[i] = 0.f;
                    cut[i] = i < nt ? lo + (uint32_t)(i + 1) * step : 0xffffffffu;
                }
#pragma unroll
                for (int j = 0; j < NUC_PER; j++) {
                    const uint32_t k = float_order_key(x[j]);
                    const float mj = mass_of(x[j]);
#pragma unroll
                    for (int i = 0; i < NUC_CUTS; i++) acc[i] += k >= cut[i] ? mj : 0.f;
                }
#pragma unroll
                for (int i = 0; i < NUC_CUTS; i++) {
#pragma unroll
                    for (int sft = 16; sft > 0; sft >>= 1) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], sft);
                    if ((threadIdx.x & 31) == 0) sh.cut_part[(threadIdx.x >> 5) * NUC_CUTS + i] = acc[i];
                }
                __syncthreads();
                if (threadIdx.x < NUC_CUTS) {
                    float b = 0.f;
                    for (int w = 0; w < NUC_THREADS / 32; w++) b += sh.cut_part[w * NUC_CUTS + threadIdx.x];
                    for (int k = 0; k < NUC_CLUSTER; k++)      // every block's table gets this block's sums
                        *cluster.map_shared_rank(&sh.cut_slots[(phase * NUC_CLUSTER + blockIdx.x) * NUC_CUTS + threadIdx.x], k) = b;
                }
                cluster.sync();
                int count = 0;                                 // thresholds whose mass still reaches the target
                for (int i = 0; i < nt; i++) {
                    float tot = 0.f;
                    for (int k = 0; k < NUC_CLUSTER; k++) tot += sh.cut_slots[(phase * NUC_CLUSTER + k) * NUC_CUTS + i];
                    if (tot >= target) count = i + 1; else break;
                }
                phase ^= 1;
                const uint32_t new_lo = count ? lo + (uint32_t)count * step : lo;
                if (count < nt) hi = lo + (uint32_t)(count + 1) * step;
                lo = new_lo;
            }
            allow = max(allow, lo);                            // tokens the tries removed are below tau anyway
        }
    }
    if (token == 0x7fffffff) {
        // arg max over the eligible tokens (the kept set after the search; everything for a row of NaN)
        float best = -INFINITY;
        int bi = 0x7fffffff;
        uint32_t bk = 0;
#pragma unroll
        for (int j = 0; j < NUC_PER; j++) {
            const int v = 4 * ((j >> 2) * (NUC_CLUSTER * NUC_THREADS) + blockIdx.x * NUC_THREADS + threadIdx.x) + (j & 3);
            if (float_order_key(x[j]) >= allow && (sc[j] > best || (sc[j] == best && v < bi))) { best = sc[j]; bi = v; bk = 1; }
        }
        nuc_cluster_argmax(best, bi, bk, sh, phase, cluster);
        token = bi == 0x7fffffff ? 0 : bi;                     // all -inf / NaN row: defined result
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        draft[r] = token;
        tokens[(size_t)row_seq[r] * tok_stride + p + 1] = token;
    }
}

// Second kernel, one thread per row: best of the chunks (lowest index on ties) -> draft.
__global__ void sample_pick_kernel(const float* __restrict__ best_val, const int* __restrict__ best_idx, int n_chunks,
                                   int n_rows, const int* __restrict__ row_pos, const int* __restrict__ row_seq,
                                   int* __restrict__ draft, int* __restrict__ tokens, int tok_stride) {
    pdl_enter();
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= n_rows) return;
    const int p = row_pos[r];
    if (p < 0) return;
    float best = -INFINITY;
    int bi = 0x7fffffff;
    for (int c = 0; c < n_chunks; c++) {
        const float v = best_val[r * SAMPLE_CHUNKS + c];
        const int i = best_idx[r * SAMPLE_CHUNKS + c];
        if (v > best || (v == best && i < bi)) { best = v; bi = i; }
    }
    if (bi == 0x7fffffff) bi = 0;                 // all -inf / NaN row: defined result
    draft[r] = bi;
    tokens[(size_t)row_seq[r] * tok_stride + p + 1] = bi;
}

// delta_i = ||z_i - z_prev,i|| / ||z_i||  (Eq. 3); +inf when ||z_i|| = 0.
constexpr int DELTA_THREADS = 1024;              // a 5280-wide row is one 16-byte load per thread and array
__global__ void __launch_bounds__(DELTA_THREADS)
delta_kernel(const float* __restrict__ z, const float* __restrict__ z_prev, int hidden,
             const int* __restrict__ row_pos, float* __restrict__ delta) {
    pdl_enter();
    __shared__ float sm[32];
    const int r = blockIdx.x;
    if (row_pos[r] < 0) return;
    float num = 0.f, den = 0.f;
    if ((hidden & 3) == 0) {
        const float4* a4 = reinterpret_cast<const float4*>(z + (size_t)r * hidden);
        const float4* b4 = reinterpret_cast<const float4*>(z_prev + (size_t)r * hidden);
        for (int j = threadIdx.x; j < hidden / 4; j += blockDim.x) {
            const float4 a = a4[j], b = b4[j];
            const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int k = 0; k < 4; k++) {
                const float d = av[k] - bv[k];
                num += d * d;
                den += av[k] * av[k];
            }
        }
    } else {
        for (int j = threadIdx.x; j < hidden; j += blockDim.x) {
            const float a = z[(size_t)r * hidden + j], d = a - z_prev[(size_t)r * hidden + j];
            num += d * d;
            den += a * a;
        }
    }
    num = block_sum(num, sm);
    den = block_sum(den, sm);
    if (threadIdx.x == 0) delta[r] = den > 0.f ? sqrtf(num) / sqrtf(den) : INFINITY;
}

// End of a step, one thread per sequence: count the step on every in-flight row, find k* (the
// longest finished prefix; Eq. 3 and the freeze step of Algorithm 1), commit, drop, append one fresh row while
// the wavefront is below `window` and the row's draft is still wanted.
struct SeqState {
    int* n_prompt; int* n_committed; int* win_len; int* done;
    int* row_steps; int* row_iters;
    unsigned long long* counters;   // [0] rows through P, [1] R, [2] C, [3] tokens committed,
                                    // [4] cache rows read (context of a sequence, once per layer and pass),
                                    // [5] (row, attended key) pairs summed over layers and passes,
                                    // [8 + k] (step, live sequence) pairs that committed k tokens (k = 15: 15 or more)
};
constexpr int RD_COUNTERS = 32;
constexpr int RD_HIST_AT = 8, RD_HIST_BINS = 16;
// layer_passes: layers a row goes through in this step (prelude + coda + inner_iters * core).
__global__ void advance_kernel(SeqState st, const float* __restrict__ delta, int B, int Wmax, int window,
                               int inner_iters, float exit_threshold, int cap, int max_new, int layer_passes) {
    pdl_enter();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B || st.done[b]) return;
    const int f = st.n_committed[b] - 1;
    int w = st.win_len[b];
    int k = 0;
    bool open = true;
    for (int i = 0; i < w; i++) {
        const int s = b * Wmax + (f + i) % Wmax;
        const int steps = ++st.row_steps[s];
        const int iters = (st.row_iters[s] += inner_iters);
        const bool fin = exit_threshold <= 0.f ? steps >= window : (delta[s] < exit_threshold || iters >= cap);
        if (open && fin) k++; else open = false;
    }
    atomicAdd(&st.counters[0], (unsigned long long)w);
    atomicAdd(&st.counters[1], (unsigned long long)w * inner_iters);
    atomicAdd(&st.counters[2], (unsigned long long)w);
    // rows at positions f .. f+w-1: the cache rows 0 .. f+w-1 are read once for the whole window;
    // the row at position p attends p + 1 keys
    atomicAdd(&st.counters[4], (unsigned long long)(f + w) * layer_passes);
    atomicAdd(&st.counters[5], ((unsigned long long)w * (f + 1) + (unsigned long long)w * (w - 1) / 2) * layer_passes);
    int nc = st.n_committed[b];
    const int np = st.n_prompt[b];
    k = min(k, max_new - (nc - np));
    nc += k;
    w -= k;
    atomicAdd(&st.counters[3], (unsigned long long)k);
    atomicAdd(&st.counters[RD_HIST_AT + min(k, RD_HIST_BINS - 1)], 1ull);
    if (nc - np >= max_new) {
        st.done[b] = 1;
        w = 0;
    } else if (w < window) {
        const int nxt = nc - 1 + w;
        if (nxt <= np + max_new - 2) {
            const int s = b * Wmax + nxt % Wmax;
            st.row_steps[s] = 0;
            st.row_iters[s] = 0;
            w++;
        }
    }
    st.n_committed[b] = nc;
    st.win_len[b] = w;
}

// End of a prefill, on the stream: |y_frozen| = L and one fresh in-flight row at position L-1
// (the initialisation steps of Algorithm 1).
__global__ void seq_start_kernel(SeqState st, int seq, int L, int slot, int is_done) {
    pdl_enter();
    if (blockIdx.x != 0 || threadIdx.x != 0) return;
    st.n_prompt[seq] = L;
    st.n_committed[seq] = L;
    st.win_len[seq] = is_done ? 0 : 1;
    st.done[seq] = is_done;
    st.row_steps[slot] = 0;
    st.row_iters[slot] = 0;
}

// ---------------------------------------------------------------------------------------------
// Pooled latent slots (Appendix, "Larger Batch Sizes": a number of slots for hidden states, an
// occupancy multiple of the maximum wavefront, shared by the sequences; a slot need not belong to a
// contiguous run of positions).  ring[b * Wmax + (p mod Wmax)] names the slot that holds in-flight
// position p of sequence b (-1: none); free_list[0 .. *free_top) are the unused slots.
// ---------------------------------------------------------------------------------------------
struct SlotPool {
    int* ring;        // [B * Wmax]
    int* free_list;   // [n_slots]
    int* free_top;    // [1]
};

// Row tables of a decode step from the ring: row = slot.  One block.  grp_index[b * Wmax + i] = slot of
// the i-th in-flight position of sequence b (-1 beyond its wavefront): the attention kernel's groups.
__global__ void plan_rows_pool_kernel(const int* __restrict__ n_committed, const int* __restrict__ win_len,
                                      const int* __restrict__ done, int B, int Wmax, int n_slots, SlotPool pool,
                                      int* __restrict__ row_pos, int* __restrict__ row_seq, int* __restrict__ grp_index,
                                      int* __restrict__ step_first, int* __restrict__ step_n) {
    pdl_enter();
    for (int s = threadIdx.x; s < n_slots; s += blockDim.x) { row_pos[s] = -1; row_seq[s] = 0; }
    __syncthreads();
    for (int e = threadIdx.x; e < B * Wmax; e += blockDim.x) {
        const int b = e / Wmax, i = e % Wmax;
        const int f = n_committed[b] - 1;
        const int w = done[b] ? 0 : win_len[b];
        int slot = -1;
        if (i < w) {
            slot = pool.ring[b * Wmax + (f + i) % Wmax];
            row_pos[slot] = f + i;
            row_seq[slot] = b;
        }
        grp_index[e] = slot;
        if (i == 0) { step_first[b] = f; step_n[b] = w; }
    }
}

// advance_kernel for pooled slots.  One block, one thread per sequence (B <= blockDim.x) for the
// freeze / commit decisions; then thread 0 returns the slots of the rows that left (sequences in
// index order) and hands free slots to the sequences that want to append a row (index order again):
// a sequence that finds no free slot does not append this step (it stalls, like a full wavefront).
__global__ void advance_pool_kernel(SeqState st, const float* __restrict__ delta, int B, int Wmax, int window,
                                    int inner_iters, float exit_threshold, int cap, int max_new, int layer_passes,
                                    SlotPool pool) {
    extern __shared__ int sh[];                  // [B] rows dropped, [B] their first position, [B] position to append or -1
    int* dropped = sh;
    int* first = sh + B;
    int* want = sh + 2 * B;
    pdl_enter();
    const int b = threadIdx.x;
    if (b < B) { dropped[b] = 0; first[b] = 0; want[b] = -1; }
    if (b < B && !st.done[b]) {
        const int f = st.n_committed[b] - 1;
        int w = st.win_len[b];
        int k = 0;
        bool open = true;
        for (int i = 0; i < w; i++) {
            const int s = pool.ring[b * Wmax + (f + i) % Wmax];
            const int steps = ++st.row_steps[s];
            const int iters = (st.row_iters[s] += inner_iters);
            const bool fin = exit_threshold <= 0.f ? steps >= window : (delta[s] < exit_threshold || iters >= cap);
            if (open && fin) k++; else open = false;
        }
        atomicAdd(&st.counters[0], (unsigned long long)w);
        atomicAdd(&st.counters[1], (unsigned long long)w * inner_iters);
        atomicAdd(&st.counters[2], (unsigned long long)w);
        if (w > 0) {
            atomicAdd(&st.counters[4], (unsigned long long)(f + w) * layer_passes);
            atomicAdd(&st.counters[5], ((unsigned long long)w * (f + 1) + (unsigned long long)w * (w - 1) / 2) * layer_passes);
        }
        int nc = st.n_committed[b];
        const int np = st.n_prompt[b];
        k = min(k, max_new - (nc - np));
        nc += k;
        first[b] = f;                            // the rows that leave are the oldest ones: positions f, f + 1, ...
        atomicAdd(&st.counters[3], (unsigned long long)k);
        atomicAdd(&st.counters[RD_HIST_AT + min(k, RD_HIST_BINS - 1)], 1ull);
        if (nc - np >= max_new) {
            st.done[b] = 1;
            dropped[b] = w;                      // everything this sequence held
            w = 0;
        } else {
            dropped[b] = k;
            w -= k;
            if (w < window) {
                const int nxt = nc - 1 + w;
                if (nxt <= np + max_new - 2) want[b] = nxt;
            }
        }
        st.n_committed[b] = nc;
        st.win_len[b] = w;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int top = *pool.free_top;
        for (int q = 0; q < B; q++)
            for (int i = 0; i < dropped[q]; i++) {
                const int e = q * Wmax + (first[q] + i) % Wmax;
                pool.free_list[top++] = pool.ring[e];
                pool.ring[e] = -1;
            }
        for (int q = 0; q < B; q++) {
            if (want[q] < 0 || top == 0) continue;
            const int s = pool.free_list[--top];
            pool.ring[q * Wmax + want[q] % Wmax] = s;
            st.row_steps[s] = 0;
            st.row_iters[s] = 0;
            st.win_len[q] += 1;
        }
        *pool.free_top = top;
    }
}

// seq_start_kernel for pooled slots: a restarted sequence first returns what it held, then takes one
// slot for position L-1 if one is free (otherwise it starts with an empty wavefront and gets its
// first row from advance_pool_kernel as soon as a slot frees up).
__global__ void seq_start_pool_kernel(SeqState st, int seq, int L, int Wmax, int is_done, SlotPool pool) {
    pdl_enter();
    if (blockIdx.x != 0 || threadIdx.x != 0) return;
    int top = *pool.free_top;
    for (int j = 0; j < Wmax; j++) {
        const int s = pool.ring[seq * Wmax + j];
        if (s >= 0) { pool.free_list[top++] = s; pool.ring[seq * Wmax + j] = -1; }
    }
    int w = 0;
    if (!is_done && top > 0) {
        const int s = pool.free_list[--top];
        pool.ring[seq * Wmax + (L - 1) % Wmax] = s;
        st.row_steps[s] = 0;
        st.row_iters[s] = 0;
        w = 1;
    }
    *pool.free_top = top;
    st.n_prompt[seq] = L;
    st.n_committed[seq] = L;
    st.win_len[seq] = w;
    st.done[seq] = is_done;
}

// float32 -> T copy (weight upload path; bf16 rounds to nearest even once).
template <typename T>
__global__ void convert_kernel(const float* __restrict__ src, T* __restrict__ dst, size_t n) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        dst[i] = from_f<T>(src[i]);
}
// K or V of positions pos0 .. pos0+n-1 of one sequence, gathered from the cache's
// [head][position][head_dim] layout into float32 rows [n, hidden].
template <typename T>
__global__ void kv_gather_kernel(const T* __restrict__ seq_base, size_t head_stride, int head_dim, int hidden, int pos0,
                                 int n, float* __restrict__ dst) {
    const size_t total = (size_t)n * hidden;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const size_t row = i / hidden, m = i % hidden;
        dst[i] = to_f(seq_base[(m / head_dim) * head_stride + (pos0 + row) * head_dim + m % head_dim]);
    }
}

}  // namespace rd
