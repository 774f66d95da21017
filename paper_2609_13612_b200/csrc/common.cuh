// Shared device-side pieces of the attention kernels: tile geometry, mask classification,
// and the in-shared-memory RoPE rotation of a TMA-loaded (128-byte swizzled) tile.
#pragma once
#include "ptx.cuh"

namespace af {

constexpr int BM = 128;          // query rows per tile (= TMEM lanes, one row per thread)
constexpr int BN = 128;          // key rows per tile
constexpr int BOX_COLS = 64;     // bf16 columns per TMA box (128 bytes: one swizzle row)
constexpr int BOX_BYTES = 128 * 128;  // 128 rows x 128 bytes

struct MaskSpec {
    int S;
    int causal;
    int window;  // < 0: none; host clamps to S
    int skip_rows = 0;  // backward only: query rows below this are computed by the first-rows kernel, so the
                        // MMA kernels drop every pair (i, j) with i < skip_rows
};

// Key-tile range [jlo, jhi] that a query tile starting at row i0 can see (Section 5: fully masked
// tiles are skipped).
__device__ __forceinline__ void tile_range(const MaskSpec& m, int i0, int& jlo, int& jhi) {
    int ilast = min(i0 + BM - 1, m.S - 1);
    int hi_row = m.causal ? ilast : (m.window >= 0 ? min(ilast + m.window, m.S - 1) : m.S - 1);
    int lo_row = m.window >= 0 ? max(0, i0 - m.window) : 0;
    jlo = lo_row / BN;
    jhi = hi_row / BN;
}

// Query-tile range [ilo, ihi] (in tiles of BM rows) that can see the key tile starting at row j0.
__device__ __forceinline__ void qtile_range(const MaskSpec& m, int j0, int& ilo, int& ihi) {
    int jlast = min(j0 + BN - 1, m.S - 1);
    int lo_row = m.causal ? j0 : (m.window >= 0 ? max(0, j0 - m.window) : 0);
    int hi_row = m.window >= 0 ? min(jlast + m.window, m.S - 1) : m.S - 1;
    ilo = lo_row / BM;
    ihi = hi_row / BM;
}

// True if some (i, j) of the tile pair is masked out, so per-element mask logic is needed.
__device__ __forceinline__ bool tile_needs_mask(const MaskSpec& m, int i0, int j0) {
    if (j0 + BN > m.S) return true;
    if (i0 < m.skip_rows) return true;
    if (m.causal && j0 + BN - 1 > i0) return true;
    if (m.window >= 0) {
        if (i0 + BM - 1 - j0 > m.window) return true;
        if (!m.causal && j0 + BN - 1 - i0 > m.window) return true;
    }
    return false;
}

__device__ __forceinline__ bool pair_kept(const MaskSpec& m, int i, int j) {
    if (j >= m.S) return false;
    int d = i - j;
    if (m.causal && d < 0) return false;
    if (m.window >= 0) {
        if (d < 0) d = -d;
        if (d > m.window) return false;
    }
    return true;
}

// For a fixed row of a tile pair the kept columns form one interval (causal, window and the sequence
// end are all half-lines in the column index).  Returns lo and the width n: column e (0..127) is kept
// iff (unsigned)(e - lo) < n.
//   Query-major tiles (lane = query i, column = key j0 + e):     kept_keys_of_query
//   Key-major tiles   (lane = key j,   column = query i0 + e):   kept_queries_of_key
__device__ __forceinline__ void kept_keys_of_query(const MaskSpec& m, int i, int j0, int& lo, uint32_t& n) {
    const int d = i - j0;
    int hi = min(BN - 1, m.S - 1 - j0);
    lo = 0;
    if (m.causal) hi = min(hi, d);
    if (m.window >= 0) {
        lo = max(lo, d - m.window);
        if (!m.causal) hi = min(hi, d + m.window);
    }
    n = (hi >= lo && i >= m.skip_rows) ? static_cast<uint32_t>(hi - lo + 1) : 0u;
}
__device__ __forceinline__ void kept_queries_of_key(const MaskSpec& m, int j, int i0, int& lo, uint32_t& n) {
    const int d = j - i0;
    int hi = BM - 1;
    lo = max(0, m.skip_rows - i0);
    if (m.causal) lo = max(lo, d);
    if (m.window >= 0) {
        hi = min(hi, d + m.window);
        if (!m.causal) lo = max(lo, d - m.window);
    }
    n = (hi >= lo && j < m.S) ? static_cast<uint32_t>(hi - lo + 1) : 0u;
}

// Byte offset of the 16-byte chunk `chunk` (8 bf16 columns) of row `r` inside a tile made of
// D/64 TMA boxes, each [128 rows][64 cols] with the 128-byte swizzle.
__device__ __forceinline__ uint32_t swz_chunk_offset(int r, int chunk) {
    return static_cast<uint32_t>((chunk >> 3) * BOX_BYTES + r * 128 + (((chunk & 7) ^ (r & 7)) << 4));
}

// Rotate one word pair: (a, b) are the bf16x2 words at column pair (d, d + R/2); cs holds
// {cos0, sin0, cos1, sin1} for the two columns of the word.  sgn = +1 forward, -1 transpose.
__device__ __forceinline__ void rotate_word(uint32_t& a, uint32_t& b, float c0, float s0, float c1, float s1) {
    float a0 = bf16lo_to_f32(a), a1 = bf16hi_to_f32(a);
    float b0 = bf16lo_to_f32(b), b1 = bf16hi_to_f32(b);
    float na0 = fmaf(a0, c0, -b0 * s0), nb0 = fmaf(b0, c0, a0 * s0);
    float na1 = fmaf(a1, c1, -b1 * s1), nb1 = fmaf(b1, c1, a1 * s1);
    a = pack_bf16x2(na0, na1);
    b = pack_bf16x2(nb0, nb1);
}

// Section 4.1: rotate, in place, the first R columns of a [128 x D] bf16 tile that TMA left in
// shared memory; row r of the tile sits at table row min(row0 + r, S-1).  Called by `nthreads`
// threads with ids tid = 0..nthreads-1.  Column d pairs with d + R/2 (NeoX half-swap); both
// partners of 8 consecutive columns are one 16-byte chunk each, read and written by the same
// thread, so no shuffle and no second global load is needed.
__device__ __forceinline__ void rotate_tile_smem(uint8_t* tile, int row0, int S, int R, const float2* table,
                                                 int tid, int nthreads) {
    const int CP = R >> 4;  // chunk pairs per row
    const int half = R >> 1;
    for (int idx = tid; idx < 128 * CP; idx += nthreads) {
        int r = idx / CP, cp = idx - r * CP;
        int prow = min(row0 + r, S - 1);
        const float4* tb = reinterpret_cast<const float4*>(table + static_cast<size_t>(prow) * half + cp * 8);
        float4 t0 = __ldg(tb), t1 = __ldg(tb + 1), t2 = __ldg(tb + 2), t3 = __ldg(tb + 3);
        uint4* pl = reinterpret_cast<uint4*>(tile + swz_chunk_offset(r, cp));
        uint4* ph = reinterpret_cast<uint4*>(tile + swz_chunk_offset(r, cp + CP));
        uint4 lo = *pl, hi = *ph;
        rotate_word(lo.x, hi.x, t0.x, t0.y, t0.z, t0.w);
        rotate_word(lo.y, hi.y, t1.x, t1.y, t1.z, t1.w);
        rotate_word(lo.z, hi.z, t2.x, t2.y, t2.z, t2.w);
        rotate_word(lo.w, hi.w, t3.x, t3.y, t3.z, t3.w);
        *pl = lo;
        *ph = hi;
    }
}

// Same rotation for the common case R in {16, 32, 64, 128} (CP = R/16 chunk pairs per row), with
// far fewer table reads: thread (rg, cp) owns chunk pair cp of rows rg, rg + RP, rg + 2 RP, ...
// (RP = 128 / CP).  It reads the table once, for its first row, and walks to the next rows with the
// angle-addition recurrence (cos, sin)(a + d) from (cos, sin)(a) and the constant (cos, sin)(d),
// d = RP * theta_i, which the table carries as a trailer row.  The first-row read is split off
// (rotate_prefetch) so that it can be issued before waiting for the tile to land.  After a tile the
// state has advanced by 128 rows, i.e. to the thread's first row of the next consecutive tile, so a
// run of consecutive tiles needs no table read at all; callers re-read the table every
// kRotResync tiles to keep the accumulated rounding of the recurrence far below bf16 resolution.
constexpr int kRotResync = 16;
// The arithmetic uses the packed fp32 instructions of sm_100 (two lanes per instruction): a bf16x2
// word holds two adjacent columns, i.e. two frequencies, so cos and sin are kept as float2 pairs.
template <int CP>
struct RotState {
    float2 c[4], s[4];   // cos / sin of the 8 frequencies (4 column pairs) at the current row
};
struct RotStep {
    float2 c[4], s[4], ns[4];   // cos, sin, -sin of the row-to-row step angle
};

template <int CP>
__device__ __forceinline__ void rotate_load_step(const float2* table, int S, int R, int tid, RotStep& step) {
    const int cp = tid % CP;
    const float4* tb = reinterpret_cast<const float4*>(table + static_cast<size_t>(S) * (R >> 1) + cp * 8);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const float4 t = __ldg(tb + u);   // {cos0, sin0, cos1, sin1}
        step.c[u] = make_float2(t.x, t.z);
        step.s[u] = make_float2(t.y, t.w);
        step.ns[u] = make_float2(-t.y, -t.w);
    }
}

template <int CP>
__device__ __forceinline__ void rotate_prefetch(RotState<CP>& st, const float2* table, int row0, int S, int R,
                                                int tid) {
    const int rg = tid / CP, cp = tid % CP;
    const int prow = min(row0 + rg, S - 1);
    const float4* tb = reinterpret_cast<const float4*>(table + static_cast<size_t>(prow) * (R >> 1) + cp * 8);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const float4 t = __ldg(tb + u);
        st.c[u] = make_float2(t.x, t.z);
        st.s[u] = make_float2(t.y, t.w);
    }
}

// (a, b): bf16x2 words at column pairs (d, d+1) and (d + R/2, d + R/2 + 1); c, s: their cos / sin.
__device__ __forceinline__ void rotate_word2(uint32_t& a, uint32_t& b, float2 c, float2 s) {
    const float2 A = make_float2(bf16lo_to_f32(a), bf16hi_to_f32(a));
    const float2 B = make_float2(bf16lo_to_f32(b), bf16hi_to_f32(b));
    const float2 ns = make_float2(-s.x, -s.y);
    const float2 na = __ffma2_rn(B, ns, __fmul2_rn(A, c));   // a cos - b sin
    const float2 nb = __ffma2_rn(A, s, __fmul2_rn(B, c));    // b cos + a sin
    a = pack_bf16x2(na.x, na.y);
    b = pack_bf16x2(nb.x, nb.y);
}

template <int CP>
__device__ __forceinline__ void rotate_tile_fast(uint8_t* tile, RotState<CP>& st, const RotStep& step, int tid) {
    constexpr int RP = 128 / CP;
    constexpr int NB = CP < 2 ? CP : 2;  // rows in flight per thread (more would spill at this role's register budget)
    const int rg = tid / CP, cp = tid % CP;
    // (rolled: the unrolled walk was 4 times the code, and the instruction path is a loaded resource of the kernels
    // that rotate on chip - config 2 forward 0.1663 -> 0.1642 ms, config 5 forward 0.197 -> 0.193 ms)
#pragma unroll 1
    for (int k0 = 0; k0 < CP; k0 += NB) {
        uint4 lo[NB], hi[NB];
#pragma unroll
        for (int u = 0; u < NB; ++u) {
            const int r = rg + RP * (k0 + u);
            lo[u] = *reinterpret_cast<const uint4*>(tile + swz_chunk_offset(r, cp));
            hi[u] = *reinterpret_cast<const uint4*>(tile + swz_chunk_offset(r, cp + CP));
        }
#pragma unroll
        for (int u = 0; u < NB; ++u) {
            rotate_word2(lo[u].x, hi[u].x, st.c[0], st.s[0]);
            rotate_word2(lo[u].y, hi[u].y, st.c[1], st.s[1]);
            rotate_word2(lo[u].z, hi[u].z, st.c[2], st.s[2]);
            rotate_word2(lo[u].w, hi[u].w, st.c[3], st.s[3]);
            // after the last row the state sits RP * CP = 128 rows further: the same row of the next tile
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                const float2 nc = __ffma2_rn(st.s[w], step.ns[w], __fmul2_rn(st.c[w], step.c[w]));
                const float2 nsn = __ffma2_rn(st.c[w], step.s[w], __fmul2_rn(st.s[w], step.c[w]));
                st.c[w] = nc;
                st.s[w] = nsn;
            }
        }
#pragma unroll
        for (int u = 0; u < NB; ++u) {
            const int r = rg + RP * (k0 + u);
            *reinterpret_cast<uint4*>(tile + swz_chunk_offset(r, cp)) = lo[u];
            *reinterpret_cast<uint4*>(tile + swz_chunk_offset(r, cp + CP)) = hi[u];
        }
    }
}

// Table-tile variant of the same rotation, an optional mode for the streamed key tiles of the forward kernel:
// the cos/sin values of the tile's 128 positions arrive by TMA from the bf16 copy of the table (row layout
// [R/2 cos | R/2 sin], densely packed, row r at byte 2 R r) and the arithmetic runs on packed bf16 pairs, four
// multiply-adds per pair of words.  It needs about a quarter of the issue slots of rotate_tile_fast, which
// matters because the rotation shares its schedulers with the softmax warps.  The result is rounded to bf16 in
// either variant; here the table entries and the sine product carry one more bf16 rounding each, which makes the
// rounding error of a rotated key about 1.4 times that of the fp32 arithmetic.
__device__ __forceinline__ void rotate_word_bf16(uint32_t& a, uint32_t& b, uint32_t c, uint32_t s) {
    const __nv_bfloat162 A = *reinterpret_cast<const __nv_bfloat162*>(&a), B = *reinterpret_cast<const __nv_bfloat162*>(&b);
    const __nv_bfloat162 C = *reinterpret_cast<const __nv_bfloat162*>(&c), Sn = *reinterpret_cast<const __nv_bfloat162*>(&s);
    const __nv_bfloat162 na = __hfma2(__hneg2(B), Sn, __hmul2(A, C));   // a cos - b sin
    const __nv_bfloat162 nb = __hfma2(A, Sn, __hmul2(B, C));            // b cos + a sin
    a = *reinterpret_cast<const uint32_t*>(&na);
    b = *reinterpret_cast<const uint32_t*>(&nb);
}
template <int CP>
__device__ __forceinline__ void rotate_tile_tab(uint8_t* tile, const uint8_t* tab, int tid) {
    constexpr int RP = 128 / CP;
    constexpr int ROW_BYTES = CP * 32;       // 2 R
    constexpr int NB = CP < 2 ? CP : 2;      // rows in flight per thread
    const int rg = tid / CP, cp = tid % CP;
#pragma unroll 1   // (rolled, like rotate_tile_fast)
    for (int k0 = 0; k0 < CP; k0 += NB) {
        uint4 lo[NB], hi[NB], c[NB], s[NB];
#pragma unroll
        for (int u = 0; u < NB; ++u) {
            const int r = rg + RP * (k0 + u);
            lo[u] = *reinterpret_cast<const uint4*>(tile + swz_chunk_offset(r, cp));
            hi[u] = *reinterpret_cast<const uint4*>(tile + swz_chunk_offset(r, cp + CP));
            c[u] = *reinterpret_cast<const uint4*>(tab + r * ROW_BYTES + cp * 16);
            s[u] = *reinterpret_cast<const uint4*>(tab + r * ROW_BYTES + CP * 16 + cp * 16);
        }
#pragma unroll
        for (int u = 0; u < NB; ++u) {
            rotate_word_bf16(lo[u].x, hi[u].x, c[u].x, s[u].x);
            rotate_word_bf16(lo[u].y, hi[u].y, c[u].y, s[u].y);
            rotate_word_bf16(lo[u].z, hi[u].z, c[u].z, s[u].z);
            rotate_word_bf16(lo[u].w, hi[u].w, c[u].w, s[u].w);
        }
#pragma unroll
        for (int u = 0; u < NB; ++u) {
            const int r = rg + RP * (k0 + u);
            *reinterpret_cast<uint4*>(tile + swz_chunk_offset(r, cp)) = lo[u];
            *reinterpret_cast<uint4*>(tile + swz_chunk_offset(r, cp + CP)) = hi[u];
        }
    }
}

// The same walk restricted to a share of the rows: with PARTS warpgroups working on one tile, part p
// takes the rows rg + RP * k for k in [p * CP / PARTS, (p + 1) * CP / PARTS).  Used where otherwise idle
// warpgroups rotate a stationary tile together.  (CP < PARTS: part 0 does everything.)
template <int CP, int PARTS>
__device__ __forceinline__ void rotate_tile_share(uint8_t* tile, const float2* table, int row0, int S, int R,
                                                  const RotStep& step, int tid, int part) {
    constexpr int RP = 128 / CP;
    constexpr int KC = CP >= PARTS ? CP / PARTS : CP;
    if (CP < PARTS && part != 0) return;
    const int kb = CP >= PARTS ? part * KC : 0;
    const int rg = tid / CP, cp = tid % CP;
    RotState<CP> st;
    {
        const int prow = min(row0 + rg + RP * kb, S - 1);
        const float4* tb = reinterpret_cast<const float4*>(table + static_cast<size_t>(prow) * (R >> 1) + cp * 8);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float4 t = __ldg(tb + u);
            st.c[u] = make_float2(t.x, t.z);
            st.s[u] = make_float2(t.y, t.w);
        }
    }
#pragma unroll
    for (int k = 0; k < KC; ++k) {
        const int r = rg + RP * (kb + k);
        uint4* pl = reinterpret_cast<uint4*>(tile + swz_chunk_offset(r, cp));
        uint4* ph = reinterpret_cast<uint4*>(tile + swz_chunk_offset(r, cp + CP));
        uint4 lo = *pl, hi = *ph;
        rotate_word2(lo.x, hi.x, st.c[0], st.s[0]);
        rotate_word2(lo.y, hi.y, st.c[1], st.s[1]);
        rotate_word2(lo.z, hi.z, st.c[2], st.s[2]);
        rotate_word2(lo.w, hi.w, st.c[3], st.s[3]);
        *pl = lo;
        *ph = hi;
        if (k + 1 < KC) {
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                const float2 nc = __ffma2_rn(st.s[w], step.ns[w], __fmul2_rn(st.c[w], step.c[w]));
                const float2 nsn = __ffma2_rn(st.c[w], step.s[w], __fmul2_rn(st.s[w], step.c[w]));
                st.c[w] = nc;
                st.s[w] = nsn;
            }
        }
    }
}

// Rows of the trailer: the recurrence stride for a given rotary dim (0: no fast path).
__host__ __device__ constexpr int rope_fast_stride(int R) {
    return (R == 16 || R == 32 || R == 64 || R == 128) ? 128 / (R / 16) : 0;
}

}  // namespace af
