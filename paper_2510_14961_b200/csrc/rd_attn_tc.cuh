// Causal prefill attention on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// Prefill (Section 3.3: all prompt positions iterate the recurrence together) attends 128 consecutive
// prompt rows of one sequence to the cache entries 0..p of that sequence.  With 128 queries per K/V
// tile the arithmetic (4 * 128 * head_dim FLOPs per key) is past what mma.sync sustains, so here both
// products run as tcgen05.mma with the accumulators in tensor memory:
//   S[128 q, 64 keys] = Q K^T        A = Q (K-major), B = K tile (K-major), M = 128, N = 64
//   O[128 q, D]      += P V          A = P (bf16, written to shared memory by the softmax warps),
//                                    B = V tile as it lies in the cache, [key][d] (MN-major), N = 64 (+ 32)
// One CTA per (group of 128 rows, head), no key splits: a group's keys are walked tile by tile.
//   warp 0 / lane 0   TMA producer: Q once, then K and V tiles through rings of stages (K one tile ahead of V)
//   warp 1 / lane 0   issues the MMAs; tcgen05.commit signals the softmax warps and frees stages
//   warps 2-5         one query row per thread (TMEM lane = row): S from TMEM, causal mask, online
//                     softmax in float32 (log2 domain), P to shared memory in the 128-byte swizzle
// O stays in TMEM and accumulates over the tiles.  A row's running maximum is only moved when a tile's
// maximum exceeds it by more than 2^8 (P = 2^(s - m) then stays below 256, exact enough in bf16 and
// float32, and the final O / l does not depend on which m was used); when it moves, the row's O is
// rescaled in place (tcgen05.ld / st by the row's own thread, before it releases P).
// S is double-buffered in TMEM and K has its own barriers: Q K^T of tile t + 2 is issued as soon as the
// softmax warps have read S(t), so S(t + 1) is ready when they finish tile t and the tensor core works
// under the softmax instead of in turn with it.  Before a softmax thread touches O (rescale) or the P
// buffer for tile t it waits for the commit behind P V of tile t - 1 (the barrier that also frees that V tile).
// Q, K, V sub-tiles are the ones of rd_attn.cuh (64 columns with the 128-byte swizzle, 32 with the
// 64-byte swizzle for the last third of a 96-wide head), written by TMA and described to the MMA by
// shared-memory descriptors.  Every wait is bounded; on time-out the kernel raises the status word,
// lets its copies land, frees its TMEM and returns.
#pragma once
#include "rd_attn.cuh"
#include "rd_gemm_tc.cuh"

namespace rd {

constexpr int ATC_Q = 128;          // queries per CTA (UMMA M)
constexpr int ATC_THREADS = 192;
constexpr int ATC_STAGES = 2;        // 91 KB at head_dim 96: two CTAs per SM (one's MMAs run under the other's softmax)

// K-major tile with rows of 64 bytes (32 bf16), 64-byte swizzle: 8-row groups 512 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_k64(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(512 >> 4) << 32) | (1ull << 46) | (4ull << 61);
}
// MN-major operand ([k][n] in memory, n contiguous): rows of 128 bytes (64 n) with the 128-byte swizzle,
// 8-row (8 k) groups 1024 bytes apart; rows of 64 bytes (32 n) with the 64-byte swizzle, groups 512 apart.
__device__ __forceinline__ uint64_t umma_desc_mn128(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ uint64_t umma_desc_mn64(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(512 >> 4) << 32) | (1ull << 46) | (4ull << 61);
}
// instruction descriptor with B given MN-major (bit 16)
__host__ __device__ constexpr uint32_t umma_idesc_bmn(int bn) { return umma_idesc(bn) | (1u << 16); }

// 2^x, one MUFU instruction (relative error 2^-22; -inf gives 0): P is rounded to bf16 right after
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* v) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
          "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]),
          "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]),
          "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31]) : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

template <int D> struct AtcCfg {
    using T = AttTile<D>;
    static constexpr int NA = T::NA, NB = T::NB;
    static constexpr int QA_BYTES = ATC_Q * 128, QB_BYTES = ATC_Q * 64;       // Q sub-tiles (128 rows)
    static constexpr int Q_BYTES = NA * QA_BYTES + NB * QB_BYTES;
    static constexpr int KV_STAGE = 2 * T::BYTES;                             // K tile, V tile of 64 keys
    static constexpr int P_BYTES = ATC_Q * 128;                               // P: 128 rows x 64 keys bf16
    static constexpr int SMEM = 1024 + Q_BYTES + ATC_STAGES * KV_STAGE + P_BYTES + 256;
    static constexpr int TMEM_COLS = 256;                                     // S 64 | O 64 (+64) | O 32
    static constexpr int O_COL = 64;
    static constexpr int S1_COL = 192;                                        // second S buffer
};

struct AtcMaps {
    CUtensorMap q64, q32;             // boxes of 128 rows x 64 / 32 columns over the query buffer [rows, hidden]
    AttMaps kv;                       // boxes of 64 keys over the K and the V cache of the block
};

template <int D>
__global__ void __launch_bounds__(ATC_THREADS, 2)
attn_prefill_tc_kernel(const __grid_constant__ AtcMaps maps, const int* __restrict__ row_pos, const int* __restrict__ row_seq,
                       int n_rows, int row_base, int n_heads, int max_context, int hidden, float scale_log2,
                       __nv_bfloat16* __restrict__ out, int* __restrict__ status) {
    using C = AtcCfg<D>;
    using T = AttTile<D>;
    constexpr int S = ATC_STAGES;
    extern __shared__ uint8_t atc_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)atc_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* Qs = smem;
    uint8_t* ring = Qs + C::Q_BYTES;
    uint8_t* Ps = ring + S * C::KV_STAGE;
    uint64_t* q_full = (uint64_t*)(Ps + C::P_BYTES);
    uint64_t* k_full = q_full + 1;            // [S]  K tile of a stage landed
    uint64_t* k_empty = k_full + S;           // [S]  ... has been read by its Q K^T
    uint64_t* v_full = k_empty + S;           // [S]
    uint64_t* v_empty = v_full + S;           // [S]  V tile read by its P V (also: that P V has completed)
    uint64_t* s_full = v_empty + S;           // [2]  one per S buffer
    uint64_t* p_full = s_full + 2;
    uint64_t* o_full = p_full + 1;
    uint64_t* o_free = o_full + 1;
    uint32_t* tmem_slot = (uint32_t*)(o_free + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    __shared__ int kv_len_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int hd = blockIdx.x, r0 = blockIdx.y * ATC_Q;
    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int s = 0; s < S; s++) {
            mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1);
            mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1);
        }
        mbar_init(&s_full[0], 1); mbar_init(&s_full[1], 1); mbar_init(p_full, 4); mbar_init(o_full, 1); mbar_init(o_free, ATC_Q);
        *abort_flag = 0;
        kv_len_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(tmem_slot, C::TMEM_COLS);
    pdl_enter();
    // positions of the group's rows (consecutive rows of the row table); kv_len = 1 + the largest
    int my_pos = -1;
    if (warp >= 2) {
        const int r = r0 + (warp & 3) * 32 + lane;
        my_pos = r < n_rows ? row_pos[r] : -1;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp >= 2) {
        const int wmax = __reduce_max_sync(0xffffffffu, my_pos);
        if (lane == 0 && wmax >= 0) atomicMax(&kv_len_s, wmax + 1);
    }
    __syncthreads();
    const int kv_len = kv_len_s;
    const int nt = (kv_len + ATT_KT - 1) / ATT_KT;
    const uint32_t tmem_base = *tmem_slot;
    const int seq = row_seq[min(r0, n_rows - 1)];
    const int head_row0 = row_base + (seq * n_heads + hd) * max_context;

    if (warp == 0) {
        if (lane == 0 && nt > 0) {
            // ---- TMA producer ----
            mbar_expect_tx(q_full, C::Q_BYTES);
#pragma unroll
            for (int a = 0; a < C::NA; a++) tma_load_2d(Qs + a * C::QA_BYTES, &maps.q64, hd * D + a * 64, r0, q_full);
            if (C::NB) tma_load_2d(Qs + C::NA * C::QA_BYTES, &maps.q32, hd * D + C::NA * 64, r0, q_full);
            // K runs one tile ahead of V: the K tile of a stage is free as soon as its Q K^T has been
            // issued and completed, the V tile only after the P V of the same keys
            int issued_k = 0, issued_v = 0;
            auto load_k = [&](int t) {
                const int s = t % S;
                uint8_t* kdst = ring + s * C::KV_STAGE;
                const int y = head_row0 + t * ATT_KT;
                mbar_expect_tx(&k_full[s], T::BYTES);
#pragma unroll
                for (int a = 0; a < T::NA; a++) tma_load_2d(kdst + a * T::A_BYTES, &maps.kv.k64, a * 64, y, &k_full[s]);
                if (T::NB) tma_load_2d(kdst + T::NA * T::A_BYTES, &maps.kv.k32, T::NA * 64, y, &k_full[s]);
                issued_k = t + 1;
            };
            auto load_v = [&](int t) {
                const int s = t % S;
                uint8_t* vdst = ring + s * C::KV_STAGE + T::BYTES;
                const int y = head_row0 + t * ATT_KT;
                mbar_expect_tx(&v_full[s], T::BYTES);
#pragma unroll
                for (int a = 0; a < T::NA; a++) tma_load_2d(vdst + a * T::A_BYTES, &maps.kv.v64, a * 64, y, &v_full[s]);
                if (T::NB) tma_load_2d(vdst + T::NA * T::A_BYTES, &maps.kv.v32, T::NA * 64, y, &v_full[s]);
                issued_v = t + 1;
            };
            load_k(0);
            for (int t = 0; t < nt; t++) {
                if (t + 1 < nt) {
                    if (t + 1 >= S && (*abort_flag || !mbar_wait(&k_empty[(t + 1) % S], (((t + 1) / S) - 1) & 1))) { *abort_flag = 1; break; }
                    load_k(t + 1);
                }
                if (t >= S && (*abort_flag || !mbar_wait(&v_empty[t % S], ((t / S) - 1) & 1))) { *abort_flag = 1; break; }
                load_v(t);
            }
            if (*abort_flag) {
                mbar_wait(q_full, 0);
                for (int t = max(0, issued_k - S); t < issued_k; t++) mbar_wait(&k_full[t % S], (t / S) & 1);
                for (int t = max(0, issued_v - S); t < issued_v; t++) mbar_wait(&v_full[t % S], (t / S) & 1);
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && nt > 0) {
            // ---- MMA issuer ----
            constexpr uint32_t idesc_s = umma_idesc(ATT_KT);            // S: N = 64 keys
            constexpr uint32_t idesc_o64 = umma_idesc_bmn(64);          // O columns of a 64-wide V sub-tile
            constexpr uint32_t idesc_o32 = umma_idesc_bmn(32);
            const uint32_t q0 = smem_u32(Qs), p0 = smem_u32(Ps);
            bool ok = mbar_wait(q_full, 0);
            // S(t) goes to buffer t & 1 (columns 0..63 / S1_COL..): Q K^T of tile t + 2 is issued as soon as
            // the softmax warps have read S(t), so they find S(t + 1) waiting when they are done with tile t
            auto issue_qk = [&](int t) {
                const uint32_t k0 = smem_u32(ring + (t % S) * C::KV_STAGE);
                const uint32_t d = tmem_base + (uint32_t)((t & 1) ? C::S1_COL : 0);
                tc_fence_after();
                int step = 0;
#pragma unroll
                for (int a = 0; a < C::NA; a++)
#pragma unroll
                    for (int k = 0; k < 4; k++, step++)
                        umma_bf16(d, umma_desc_k128(q0 + a * C::QA_BYTES) + (uint64_t)(k * 2),
                                  umma_desc_k128(k0 + a * T::A_BYTES) + (uint64_t)(k * 2), idesc_s, step ? 1u : 0u);
                if (C::NB) {
#pragma unroll
                    for (int k = 0; k < 2; k++, step++)
                        umma_bf16(d, umma_desc_k64(q0 + C::NA * C::QA_BYTES) + (uint64_t)(k * 2),
                                  umma_desc_k64(k0 + T::NA * T::A_BYTES) + (uint64_t)(k * 2), idesc_s, step ? 1u : 0u);
                }
                umma_commit(&k_empty[t % S]);            // the K tile has been read
                umma_commit(&s_full[t & 1]);
            };
            for (int t = 0; t < 2 && t < nt && ok; t++) {
                ok = mbar_wait(&k_full[t % S], (t / S) & 1);
                if (ok) issue_qk(t);
            }
            for (int t = 0; t < nt && ok; t++) {
                const int s = t % S;
                if (*abort_flag || !mbar_wait(p_full, t & 1)) { ok = false; break; }          // P(t) in shared memory, S(t) read
                if (!mbar_wait(&v_full[s], (t / S) & 1)) { ok = false; break; }
                tc_fence_after();
                const uint32_t v0 = smem_u32(ring + s * C::KV_STAGE + T::BYTES);
#pragma unroll
                for (int a = 0; a < T::NA; a++)
#pragma unroll
                    for (int k = 0; k < 4; k++)          // 16 keys per MMA: 16 rows of the V sub-tile further on
                        umma_bf16(tmem_base + (uint32_t)(C::O_COL + a * 64), umma_desc_k128(p0) + (uint64_t)(k * 2),
                                  umma_desc_mn128(v0 + a * T::A_BYTES + k * 2048), idesc_o64, (t | k) ? 1u : 0u);
                if (T::NB) {
#pragma unroll
                    for (int k = 0; k < 4; k++)
                        umma_bf16(tmem_base + (uint32_t)(C::O_COL + T::NA * 64), umma_desc_k128(p0) + (uint64_t)(k * 2),
                                  umma_desc_mn64(v0 + T::NA * T::A_BYTES + k * 1024), idesc_o32, (t | k) ? 1u : 0u);
                }
                umma_commit(&v_empty[s]);                // V of this stage and P have been read, O holds tile t
                if (t + 2 < nt) {
                    if (*abort_flag || !mbar_wait(&k_full[(t + 2) % S], ((t + 2) / S) & 1)) { ok = false; break; }
                    issue_qk(t + 2);
                } else if (t + 1 == nt) {
                    umma_commit(o_full);                 // the last P V: O is complete
                }
            }
            if (!ok) *abort_flag = 1;
        }
    } else {
        // ---- softmax warps: thread = query row ----
        const int quad = warp & 3;
        const int row = quad * 32 + lane;                 // row of the group = TMEM lane
        const uint32_t t_lane = tmem_base + ((uint32_t)(quad * 32) << 16);
        float m = -INFINITY, l = 0.f;                  // m: the maximum the row's P and O are scaled by (log2 domain)
        const int wmin_pos = __reduce_min_sync(0xffffffffu, my_pos);
        bool ok = true;
        for (int t = 0; t < nt && ok; t++) {
            if (*abort_flag || !mbar_wait(&s_full[t & 1], (t >> 1) & 1)) { ok = false; break; }
            tc_fence_after();
            uint32_t sr[64];
            const uint32_t t_s = t_lane + (uint32_t)((t & 1) ? C::S1_COL : 0);
            tmem_ld32(t_s, sr);
            tmem_ld32(t_s + 32, sr + 32);
            const int key0 = t * ATT_KT;
            // causal mask: only tiles that reach past the smallest position of the warp's rows need it
            if (key0 + ATT_KT - 1 > wmin_pos) {
#pragma unroll
                for (int j = 0; j < 64; j++)
                    if (key0 + j > my_pos) sr[j] = 0xff800000u;      // -inf
            }
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < 64; j++) mx = fmaxf(mx, __uint_as_float(sr[j]));
            mx *= scale_log2;                                        // scale > 0: the maximum commutes with it
            // S(t) was computed while the previous tile's softmax ran; its P V may still be in flight: O and
            // the P buffer are at rest once the commit behind that P V has arrived
            if (t > 0 && !mbar_wait(&v_empty[(t - 1) % S], ((t - 1) / S) & 1)) { ok = false; break; }
            tc_fence_after();
            // move the row's maximum only when the tile exceeds it by more than 8 (a factor 256)
            const bool move = mx > m + 8.0f || (m == -INFINITY && mx > -INFINITY);
            if (__any_sync(0xffffffffu, move && t > 0 && l > 0.f)) {
                // rescale O in place (at rest: see the wait above)
                const float corr = move ? exp2f(m - mx) : 1.0f;       // (m = -inf: the row has nothing yet, corr 0 is harmless)
#pragma unroll
                for (int c = 0; c < D; c += 32) {
                    uint32_t orow[32];
                    tmem_ld32(t_lane + (uint32_t)(C::O_COL + c), orow);
#pragma unroll
                    for (int j = 0; j < 32; j++) orow[j] = __float_as_uint(__uint_as_float(orow[j]) * corr);
                    tmem_st32(t_lane + (uint32_t)(C::O_COL + c), orow);
                }
                if (move) l *= corr;
            } else if (move) {
                l *= (m == -INFINITY ? 0.f : exp2f(m - mx));
            }
            if (move) m = mx;
            const float u = m == -INFINITY ? 0.f : m;
            float sum = 0.f;
            // P row: 64 bf16 = 8 chunks of 16 bytes, chunk c at (c ^ (row & 7)) of the row's 128 bytes
            uint8_t* prow = Ps + row * 128;
#pragma unroll
            for (int c = 0; c < 8; c++) {
                uint32_t w[4];
#pragma unroll
                for (int q = 0; q < 4; q++) {
                    const float p0 = ex2_approx(fmaf(__uint_as_float(sr[c * 8 + 2 * q]), scale_log2, -u)),
                                p1 = ex2_approx(fmaf(__uint_as_float(sr[c * 8 + 2 * q + 1]), scale_log2, -u));
                    sum += p0 + p1;
                    w[q] = pack_bf16(p0, p1);
                }
                *reinterpret_cast<uint4*>(prow + ((c ^ (row & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
            }
            l += sum;
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // P visible to the tensor core's reads
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(p_full);                               // one arrival per softmax warp
        }
        float o[D];
        if (ok && nt > 0 && !mbar_wait(o_full, 0)) ok = false;
        if (ok) {
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < D; c += 32) {
                uint32_t orow[32];
                tmem_ld32(t_lane + (uint32_t)(C::O_COL + c), orow);
#pragma unroll
                for (int j = 0; j < 32; j++) o[c + j] = __uint_as_float(orow[j]);
            }
        }
        if (!ok) *abort_flag = 1;
        if (ok && my_pos >= 0) {
            const float inv = l > 0.f ? 1.0f / l : 0.f;
            __nv_bfloat16* dst = out + (size_t)(r0 + row) * hidden + hd * D;
#pragma unroll
            for (int c = 0; c < D; c += 8) {
                uint32_t w[4];
#pragma unroll
                for (int q = 0; q < 4; q++) w[q] = pack_bf16(o[c + 2 * q] * inv, o[c + 2 * q + 1] * inv);
                *reinterpret_cast<uint4*>(dst + c) = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) atomicExch(status, 1);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(*tmem_slot, C::TMEM_COLS);
    }
}

}  // namespace rd
