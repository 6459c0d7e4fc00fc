// Where the consumer of a GEMM finds the GEMM's result.
//
// The tensor-core GEMM (rd_gemm_tc.cuh) cuts the k range of a 128-feature tile between CTAs and
// leaves one slot of fp32 partial sums per (CTA, tile it touched).  The kernel that consumes the
// result adds the slots of a tile in ascending k order while it reads: the order is fixed by the
// shapes alone, so results are bit-reproducible.  The plain GEMM kernel writes finished sums to an
// ordinary [rows, n_out] array instead; RowSource covers both.
#pragma once
#include <cuda_runtime.h>

namespace rd {

// Tile number = (row tile) * n_tiles_m + (feature tile >> mt_shift).  Units (tile, k-block) are numbered tile by
// tile, kb per tile; CTA g owns units [g*per, (g+1)*per).
// The j-th tile CTA g touches went to slot g*max_seg + j, laid out [feature tile][bn rows][128 features].
struct PartialSums {
    const float* scratch;
    int kb, per, n_tiles_m, bn, max_seg;
    int mt_shift;         // a tile covers 1 << mt_shift feature tiles of 128 (slot: [feature tile][bn rows][128])
};

struct RowSource {
    const float* plain;   // non-null: value(r, m) = plain[r * ld + m]
    size_t ld;
    PartialSums part;     // otherwise: sum of the tile's slots
};

// Sum of features m..m+3 (m a multiple of 4) of row r.
__device__ __forceinline__ float4 row_source_load4(const RowSource& s, int r, int m) {
    if (s.plain) return *reinterpret_cast<const float4*>(s.plain + (size_t)r * s.ld + m);
    const PartialSums& d = s.part;
    // (unit numbers stay far below 2^31: 32-bit arithmetic)
    const unsigned ft = (unsigned)(m >> 7);
    const unsigned tile = (unsigned)(r / d.bn) * d.n_tiles_m + (ft >> d.mt_shift);
    const unsigned t_lo = tile * (unsigned)d.kb;
    const int g_lo = (int)(t_lo / (unsigned)d.per), g_hi = (int)((t_lo + d.kb - 1) / (unsigned)d.per);
    const size_t in_slot = ((size_t)(ft & ((1u << d.mt_shift) - 1)) * d.bn + (size_t)(r % d.bn)) * 128 + (m & 127);
    const float* base = d.scratch + in_slot;
    const size_t slot_elems = ((size_t)d.bn * 128) << d.mt_shift;
    if (d.bn >= 128) {
        // Many rows in flight (batched steps, prefill): the readers are bound by their instruction count
        // there, so the slot addresses come from one division.  CTA g_lo may have started in an earlier
        // tile; every later CTA of the tile starts inside it, so its first slot is the tile's.  Same slots,
        // same order of addition as below: the same bits.
        const unsigned first0 = ((unsigned)g_lo * (unsigned)d.per) / (unsigned)d.kb;
        const size_t cta_stride = (size_t)d.max_seg * slot_elems;
        float4 acc = __ldcg(reinterpret_cast<const float4*>(base + (size_t)g_lo * cta_stride + (size_t)(tile - first0) * slot_elems));
        const float* q = base + (size_t)(g_lo + 1) * cta_stride;
        for (int g = g_lo + 1; g <= g_hi; g += 4, q += 4 * cta_stride) {
            float4 v[4];
#pragma unroll
            for (int j = 0; j < 4; j++) {
                v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (g + j <= g_hi) v[j] = __ldcg(reinterpret_cast<const float4*>(q + (size_t)j * cta_stride));
            }
#pragma unroll
            for (int j = 0; j < 4; j++)
                if (g + j <= g_hi) { acc.x += v[j].x; acc.y += v[j].y; acc.z += v[j].z; acc.w += v[j].w; }
        }
        return acc;
    }
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    // up to eight slots are requested together (one round trip to L2), then added in ascending k order
    for (int gb = g_lo; gb <= g_hi; gb += 8) {
        float4 v[8];
#pragma unroll
        for (int q = 0; q < 8; q++) {
            v[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (gb + q <= g_hi) {
                const unsigned g = (unsigned)(gb + q);
                const unsigned first_tile = (g * (unsigned)d.per) / (unsigned)d.kb;
                v[q] = __ldcg(reinterpret_cast<const float4*>(base + ((size_t)g * d.max_seg + (tile - first_tile)) * slot_elems));
            }
        }
#pragma unroll
        for (int q = 0; q < 8; q++)
            if (gb + q <= g_hi) { acc.x += v[q].x; acc.y += v[q].y; acc.z += v[q].z; acc.w += v[q].w; }
    }
    return acc;
}
// The same in two halves, for kernels that can do the index arithmetic before they wait for the GEMM:
// where the (up to MAXQ) slots of features m..m+3 of row r are, then the loads and the ordered sum.
template <int MAXQ>
struct RowSlots {
    const float* p[MAXQ];
    int n;                // slots to add; n > MAXQ: not covered, use row_source_load4
};
template <int MAXQ>
__device__ __forceinline__ RowSlots<MAXQ> row_source_locate(const RowSource& s, int r, int m) {
    RowSlots<MAXQ> o;
    if (s.plain) {
        o.n = 1;
        o.p[0] = s.plain + (size_t)r * s.ld + m;
#pragma unroll
        for (int q = 1; q < MAXQ; q++) o.p[q] = o.p[0];
        return o;
    }
    const PartialSums& d = s.part;
    const unsigned ft = (unsigned)(m >> 7);
    const unsigned tile = (unsigned)(r / d.bn) * d.n_tiles_m + (ft >> d.mt_shift);
    const unsigned t_lo = tile * (unsigned)d.kb;
    const int g_lo = (int)(t_lo / (unsigned)d.per), g_hi = (int)((t_lo + d.kb - 1) / (unsigned)d.per);
    const size_t in_slot = ((size_t)(ft & ((1u << d.mt_shift) - 1)) * d.bn + (size_t)(r % d.bn)) * 128 + (m & 127);
    const float* base = d.scratch + in_slot;
    const size_t slot_elems = ((size_t)d.bn * 128) << d.mt_shift;
    o.n = g_hi - g_lo + 1;
#pragma unroll
    for (int q = 0; q < MAXQ; q++) {
        const unsigned g = (unsigned)(g_lo + min(q, g_hi - g_lo));
        const unsigned first_tile = (g * (unsigned)d.per) / (unsigned)d.kb;
        o.p[q] = base + ((size_t)g * d.max_seg + (tile - first_tile)) * slot_elems;
    }
    return o;
}
template <int MAXQ>
__device__ __forceinline__ float4 row_source_fetch(const RowSlots<MAXQ>& o) {
    float4 v[MAXQ];
#pragma unroll
    for (int q = 0; q < MAXQ; q++) {
        v[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (q < o.n) v[q] = __ldcg(reinterpret_cast<const float4*>(o.p[q]));
    }
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int q = 0; q < MAXQ; q++)
        if (q < o.n) { acc.x += v[q].x; acc.y += v[q].y; acc.z += v[q].z; acc.w += v[q].w; }
    return acc;
}

__device__ __forceinline__ float row_source_load(const RowSource& s, int r, int m) {
    if (s.plain) return s.plain[(size_t)r * s.ld + m];
    const float4 v = row_source_load4(s, r, m & ~3);
    const int k = m & 3;
    return k == 0 ? v.x : k == 1 ? v.y : k == 2 ? v.z : v.w;
}

}  // namespace rd
