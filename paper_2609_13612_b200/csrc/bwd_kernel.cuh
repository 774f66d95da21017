// Backward kernels (Section 4.4, FlashAttention-2 decomposition):
//   1. bwd_delta_kernel      delta_i = sum_d dO_id * O_id             (row-reduced gradients)
//   2. attn_bwd_kernel<DKV>  per key tile: dV += P^T dO, dK' += dS^T Q'   (no atomics: one CTA owns the tile)
//   3. attn_bwd_kernel<DQ>   per query tile: dQ' += dS K'
// Both MMA kernels recompute P from the saved L, recompute the RoPE rotation on chip, and rotate
// the accumulated gradient back (transpose rotation) in the epilogue.
//
// One template covers 2 and 3.  A CTA keeps a stationary pair of tiles (X, Y) and streams pairs
// (A, Bc):      DKV: X = K', Y = V,  A = Q', Bc = dO   (TMEM lane = key row,   column = query row)
//               DQ : X = Q', Y = dO, A = K', Bc = V    (TMEM lane = query row, column = key row)
//   T1 = X A^T  (scores or their transpose),  T2 = Y Bc^T  (dP or its transpose)
//   P = 2^(c2 T1 + bias - L2), dS = P (T2 - delta); P, dS go back to TMEM as bf16 over T1, T2
//   DKV: acc1 += P Bc, acc2 += dS A.      DQ: acc1 += dS A.
// Warp roles (512 threads): warp 0 TMA producer, warp 1 MMA issuer, warps 4-7 rotation, warps 8-11 and
// 12-15 two gradient warpgroups: each owns 64 of the 128 columns of T1/T2 (all 128 lanes).  The MMAs are
// issued per column half (N = 64 for T1/T2, 4 of the 8 K-steps for the accumulators) in the order
//   T(a,n) T(b,n) | acc(a,n) T(a,n+1) | acc(b,n) T(b,n+1) | acc(a,n+1) ...
// so that while one warpgroup turns its half of (S, dP) into (P, dS), the tensor pipe works on the other
// half and on the next streamed tile: nothing in the loop waits for a whole tile.
#pragma once
#include <cuda.h>
#include <type_traits>
#include "common.cuh"

namespace af {

struct BwdParams {
    int B, Hq, Hkv, S, group;
    int R;
    int causal, window;
    float scale, scale_log2;
    const float* slopes;
    const float2* table;
    const float* lse;     // [B,Hq,S]
    const float* delta;   // [B,Hq,S]
    void* out1;           // DKV: dV   DQ: dQ
    void* out2;           // DKV: dK   DQ: unused
    int out_f32;
    int store_x;          // write the rotated X tile through tm_s
    // Block-sparse attention (Section 4.3), BS kernels only: index lists of the active 128 x 128 blocks by
    // stationary block - for the dK/dV role by key block (the query blocks that see it), for the dQ role by
    // query block (its key blocks): ptr [ceil(S/128) + 1], idx [ptr[last]] (device).
    const int* bs_ptr;
    const int* bs_idx;
    const int* bs_order;   // optional launch order of the stationary blocks (longest lists first), or nullptr
    int skip_rows;         // query rows i < skip_rows are left to bwd_first_rows_kernel (0: none)
    float* dq_acc;         // one-pass kernel only: fp32 accumulator of dQ' [B, Hq, S, D], zero on entry
    // Section 3.1 extras (GEN kernels only): additive bias [bias_B, bias_H, S, S] with the element strides of its batch
    // and head extents (0 where broadcast), and the ReLU normaliser, for which `lse` holds n_i, the number of kept
    // pairs of the row (what the forward wrote there), and delta is not used.
    const float* bias;
    long long bias_sb, bias_sh;
    int relu;
};

// delta[row] = <dO[row], O[row]>; one 16-byte chunk per thread, D/8 threads per row.
template <int D>
__global__ void __launch_bounds__(256) bwd_delta_kernel(const uint4* __restrict__ o, const uint4* __restrict__ d_o,
                                                        float* __restrict__ delta, long long rows) {
    constexpr int TPR = D / 8;
    grid_dep_launch();   // the next kernel of the backward sequence may be scheduled while this one runs
    const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
    const long long row = idx / TPR;
    float acc = 0.f;
    if (row < rows) {
        const uint4 a = __ldg(o + idx), b = __ldg(d_o + idx);
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int u = 0; u < 4; ++u)
            acc += bf16lo_to_f32(aw[u]) * bf16lo_to_f32(bw[u]) + bf16hi_to_f32(aw[u]) * bf16hi_to_f32(bw[u]);
    }
#pragma unroll
    for (int off = TPR / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (row < rows && (threadIdx.x % TPR) == 0) delta[row] = acc;
}

template <int D>
struct BwdSmem {
    static constexpr int TILE = 128 * D * 2;
    static constexpr int NST = 2;                 // stream stages
    static constexpr int OFF_X = 0, OFF_Y = TILE;
    static constexpr int OFF_A = 2 * TILE;        // NST tiles
    static constexpr int OFF_B = OFF_A + NST * TILE;
    static constexpr int OFF_STATS = OFF_B + NST * TILE;      // float [2][2][128]: L2 and delta of the streamed tile
    static constexpr int OFF_BAR = OFF_STATS + 2 * 2 * 128 * 4;
    static constexpr int B_XFULL = 0, B_XROT = 1, B_YFULL = 2, B_AFULL = 3, B_AROT = B_AFULL + NST,
                         B_BFULL = B_AROT + NST, B_EMPTY = B_BFULL + NST, B_TFULL = B_EMPTY + NST,
                         B_PDS = B_TFULL + 2, B_DONE = B_PDS + 2, N_BARS = B_DONE + 1;   // TFULL, PDS: one per column half
    static constexpr int OFF_MISC = OFF_BAR + N_BARS * 8;
    static constexpr int BYTES = OFF_MISC + 16 + 1024;
    static constexpr int STG_STRIDE = D + 4;      // floats per staged row (padding keeps 16-byte stores conflict-free)
    static_assert(128 * STG_STRIDE * 4 <= 2 * NST * TILE, "staging buffer must fit in the stream stages");
};

// Named barriers of the gradient warpgroups: id 3 joins both (256 threads), ids 1 and 2 one each.
__device__ __forceinline__ void wg_sync() { asm volatile("bar.sync 3, 256;" ::: "memory"); }
// Barrier that also ANDs a flag, so that a wait that gave up in one thread ends the loop in all of
// them (nobody is left alone at a barrier).  id/count: 3/256 for both warpgroups, 1+hf/128 for one.
__device__ __forceinline__ bool bar_all(bool v, int id, int count) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %1, 0;\n\tbar.red.and.pred q, %2, %3, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"(static_cast<uint32_t>(v)), "r"(id), "r"(count)
        : "memory");
    return r != 0;
}
__device__ __forceinline__ bool wg_all(bool v) { return bar_all(v, 3, 256); }

// Epilogue helper: the 256 threads of the two gradient warpgroups move a [128 x D] fp32 accumulator
// from TMEM (thread gtid reads lane gtid % 128, column half gtid / 128) through shared memory to
// global memory, scaling it and, when R > 0, applying the transpose rotation for positions row0..
// (gradients w.r.t. rotated rows are rotated back).  Global writes are coalesced along D.  (Writing each
// thread's TMEM row straight to global memory - no staging, no barriers, cos/sin read per row - measured
// slower: a warp's store then touches 32 rows, and the store rate is what bounds this epilogue.)
template <int D>
__device__ __forceinline__ void store_acc_rotated(uint32_t t_acc, float* stg, int gtid, float mul, int R,
                                                  const float2* table, int row0, int S, void* out, size_t out_row0,
                                                  int out_f32) {
    constexpr int STRIDE = BwdSmem<D>::STG_STRIDE;
    // (set-up of the second phase first: its table reads are in flight while the first phase runs)
    // Second phase: thread (rsub, d4) writes the four columns 4 d4 .. 4 d4 + 3 of rows rsub, rsub + RPP, ...
    // with 16-byte shared loads and coalesced 16-byte (fp32) or 8-byte (bf16) global stores.  The four
    // frequencies' cos/sin come from the table once (first row, and the next one to get the step angle as
    // a difference of angles) and then walk by the angle-addition recurrence: no table read in the loop.
    constexpr int TPR = D / 4;        // threads per row
    constexpr int RPP = 256 / TPR;    // rows per pass (8 for D = 128, 16 for D = 64)
    const int d = (gtid % TPR) * 4, rsub = gtid / TPR;
    const int half = R >> 1;
    const bool rot = d < R;           // R is a multiple of 8: the four columns are on one side of R and of R / 2
    const bool upper = d >= half;
    const int partner = upper ? d - half : d + half;
    float c[4] = {1.f, 1.f, 1.f, 1.f}, sn[4] = {0.f, 0.f, 0.f, 0.f}, cst[4] = {1.f, 1.f, 1.f, 1.f}, sst[4] = {0.f, 0.f, 0.f, 0.f};
    if (rot) {
        const int fi = upper ? d - half : d;
        const int r0 = min(row0 + rsub, S - 1), r1 = min(row0 + rsub + RPP, S - 1);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float2 t0 = __ldg(table + static_cast<size_t>(r0) * half + fi + u);
            const float2 t1 = __ldg(table + static_cast<size_t>(r1) * half + fi + u);
            c[u] = t0.x;
            sn[u] = upper ? -t0.y : t0.y;                 // transpose rotation: y c + other s below R/2, y c - other s above
            cst[u] = fmaf(t1.x, t0.x, t1.y * t0.y);       // cos(a1 - a0)
            sst[u] = fmaf(t1.y, t0.x, -t1.x * t0.y);      // sin(a1 - a0)
            if (upper) sst[u] = -sst[u];                  // the sign rides along with sn
        }
    }
    const int lane_row = gtid & 127, chalf = gtid >> 7;
#pragma unroll 1
    for (int cc = 0; cc < D / 64; ++cc) {
        const int col = chalf * (D / 2) + cc * 32;
        uint32_t v[32];
        tmem_ld32(t_acc + col, v);
        tmem_wait_ld();
        float4* dst = reinterpret_cast<float4*>(stg + lane_row * STRIDE + col);
#pragma unroll
        for (int e = 0; e < 32; e += 4)
            dst[e >> 2] = make_float4(__uint_as_float(v[e]) * mul, __uint_as_float(v[e + 1]) * mul,
                                      __uint_as_float(v[e + 2]) * mul, __uint_as_float(v[e + 3]) * mul);
    }
    wg_sync();
#pragma unroll 2
    for (int r = rsub; r < 128; r += RPP) {
        if (row0 + r < S) {
            float4 y = *reinterpret_cast<const float4*>(stg + r * STRIDE + d);
            if (rot) {
                const float4 o = *reinterpret_cast<const float4*>(stg + r * STRIDE + partner);
                y.x = fmaf(y.x, c[0], o.x * sn[0]);
                y.y = fmaf(y.y, c[1], o.y * sn[1]);
                y.z = fmaf(y.z, c[2], o.z * sn[2]);
                y.w = fmaf(y.w, c[3], o.w * sn[3]);
            }
            const size_t oi = (out_row0 + r) * D + d;
            if (out_f32) {
                *reinterpret_cast<float4*>(static_cast<float*>(out) + oi) = y;
            } else {
                *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(out) + oi) =
                    make_uint2(pack_bf16x2(y.x, y.y), pack_bf16x2(y.z, y.w));
            }
        }
        if (rot) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                // (c, sn) -> next row; with sn and sst negated together the recurrence keeps its form
                const float nc = fmaf(c[u], cst[u], -sn[u] * sst[u]), ns = fmaf(sn[u], cst[u], c[u] * sst[u]);
                c[u] = nc;
                sn[u] = ns;
            }
        }
    }
    wg_sync();
}

// One 32-column pass of a gradient warpgroup over its lane's row of T1 (scores) and T2 (dP):
//   p = 2^(c2 * s + bias - L2),  ds = p * (dP - delta),  masked entries give 0;
// p (DKV role only) and ds go back to TMEM as bf16 pairs at `out_col` of T1 / T2.
// nl2 / ndl: -L2 and -delta, either per column from shared memory (DKV: the columns are query rows) or
// the thread's own (DQ).  MASKED / ALIBI select straight-line code; arithmetic is packed fp32 (f32x2).
template <bool DKV, bool MASKED, bool ALIBI>
__device__ __forceinline__ void grad_pass32(uint32_t t1, uint32_t t2, int col0, uint32_t out_col, float scale_log2,
                                            float cbias, float sb, const float* s_nl2, const float* s_ndl, float my_nl2,
                                            float my_ndl, int mlo, uint32_t mn) {
    uint32_t s[32], dp[32], pk[16], dk[16];
    tmem_ld32(t1 + col0, s);
    tmem_ld32(t2 + col0, dp);
    tmem_wait_ld();
    const float2 sc2 = make_float2(scale_log2, scale_log2), cb2 = make_float2(cbias, cbias);
#pragma unroll
    for (int e = 0; e < 32; e += 4) {
        float2 nl[2], nd[2];
        if (DKV) {
            const float4 a4 = *reinterpret_cast<const float4*>(s_nl2 + col0 + e);
            const float4 b4 = *reinterpret_cast<const float4*>(s_ndl + col0 + e);
            nl[0] = make_float2(a4.x, a4.y); nl[1] = make_float2(a4.z, a4.w);
            nd[0] = make_float2(b4.x, b4.y); nd[1] = make_float2(b4.z, b4.w);
        } else {
            nl[0] = nl[1] = make_float2(my_nl2, my_nl2);
            nd[0] = nd[1] = make_float2(my_ndl, my_ndl);
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int c = e + 2 * u;
            float2 t = __ffma2_rn(make_float2(__uint_as_float(s[c]), __uint_as_float(s[c + 1])), sc2,
                                  __fadd2_rn(cb2, nl[u]));
            if (ALIBI) {
                t.x = fmaf(sb, static_cast<float>(c), t.x);
                t.y = fmaf(sb, static_cast<float>(c + 1), t.y);
            }
            float2 pe = make_float2(ex2(t.x), ex2(t.y));
            if (MASKED) {
                pe.x = (static_cast<uint32_t>(col0 + c - mlo) < mn) ? pe.x : 0.f;
                pe.y = (static_cast<uint32_t>(col0 + c + 1 - mlo) < mn) ? pe.y : 0.f;
            }
            const float2 ds = __fmul2_rn(pe, __fadd2_rn(make_float2(__uint_as_float(dp[c]), __uint_as_float(dp[c + 1])), nd[u]));
            pk[c >> 1] = pack_bf16x2(pe.x, pe.y);
            dk[c >> 1] = pack_bf16x2(ds.x, ds.y);
        }
    }
    if (DKV) {
        tmem_st16(t1 + out_col, pk);
        tmem_st16(t2 + out_col, dk);
    } else {
        tmem_st16(t1 + out_col, dk);
    }
}

// The same pass for the variants with an additive bias and / or the ReLU normaliser (Section 3.1: additive_bias,
// relu_attention), mask, ALiBi and bias decided at run time:
//   softmax:  p = 2^(c2 s + alibi + log2(e) bias - L2),  ds = p (dP - delta)
//   RELU:     t = c s + alibi + bias (natural units),  p = max(t, 0) / n,  ds = [t > 0] dP / n   (no delta)
// A masked pair and a pair whose bias is -inf give p = ds = 0.  For RELU the per-row statistic passed in the place
// of -L2 is 1 / n.  bias: address of the pair (this lane, column col0), col_stride elements between columns, cols_ok
// valid columns from col0 on (nullptr: no bias, or this lane's row / key lies outside the sequence).
template <bool DKV, bool RELU>
__device__ __forceinline__ void grad_pass32_general(uint32_t t1, uint32_t t2, int col0, uint32_t out_col, float scale_log2,
                                                    float cbias, float sb, const float* s_nl2, const float* s_ndl, float my_nl2,
                                                    float my_ndl, int mlo, uint32_t mn, const float* bias, long long col_stride,
                                                    int cols_ok) {
    constexpr float kLog2e = 1.4426950408889634f, kLn2 = 0.6931471805599453f;
    uint32_t s[32], dp[32], pk[16], dk[16];
    tmem_ld32(t1 + col0, s);
    tmem_ld32(t2 + col0, dp);
    float bv[32];
#pragma unroll
    for (int c = 0; c < 32; ++c) bv[c] = (bias && c < cols_ok) ? __ldg(bias + c * col_stride) : 0.f;
    tmem_wait_ld();
#pragma unroll
    for (int c = 0; c < 32; c += 2) {
        float pe[2], ds[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const float stat = DKV ? s_nl2[col0 + c + u] : my_nl2;
            const float ndl = DKV ? s_ndl[col0 + c + u] : my_ndl;
            const bool kept = static_cast<uint32_t>(col0 + c + u - mlo) < mn && bv[c + u] > -INFINITY;
            // score in the log2 domain without the row statistic
            const float t2v = fmaf(__uint_as_float(s[c + u]), scale_log2, fmaf(sb, static_cast<float>(c + u), cbias)) + bv[c + u] * kLog2e;
            const float g = __uint_as_float(dp[c + u]);
            if (RELU) {
                const float tn = t2v * kLn2;
                pe[u] = kept ? fmaxf(tn, 0.f) * stat : 0.f;
                ds[u] = (kept && tn > 0.f) ? g * stat : 0.f;
            } else {
                pe[u] = kept ? ex2(t2v + stat) : 0.f;
                ds[u] = pe[u] * (g + ndl);
            }
        }
        pk[c >> 1] = pack_bf16x2(pe[0], pe[1]);
        dk[c >> 1] = pack_bf16x2(ds[0], ds[1]);
    }
    if (DKV) {
        tmem_st16(t1 + out_col, pk);
        tmem_st16(t2 + out_col, dk);
    } else {
        tmem_st16(t1 + out_col, dk);
    }
}

// ROT_X / ROT_A: rotate the stationary tile X / every streamed tile A on chip.  With p.store_x the rotated
// stationary tile is also written to a cache in the caller's workspace through tm_s, so that the other
// role can stream rotated rows instead of rotating every streamed tile again for every stationary tile.
// Three set-ups, by the room the workspace has:
//  - both caches: a RoPE pass writes K' first; the dQ role (ROT_X, stores Q') streams K'; the dK/dV role then
//    runs without any on-chip rotation on (K', V) and streamed (Q', dO) - only its epilogue rotates dK' back;
//  - K' cache only: the dK/dV role runs first (ROT_X, ROT_A, stores K'), the dQ role (ROT_X) streams K';
//  - no cache: both roles rotate everything they touch.
// timeline stamps for tuning (compiled out unless AF_TRACE): CTA (0, 0), lane 0 of each warp
#ifdef AF_TRACE
#define AF_BSTAMP(role, it, ph)                                                                          \
    do {                                                                                                 \
        if (g_trace && blockIdx.x == 0 && blockIdx.y == 0 && (threadIdx.x & 31) == 0 && (it) < 64)       \
            g_trace[((role) * 64 + (it)) * 8 + (ph)] = clock64();                                        \
    } while (0)
#else
#define AF_BSTAMP(role, it, ph) do { } while (0)
#endif

// GEN: the instantiation for additive_bias / relu_attention (grad_pass32_general), kept apart from the others.
template <int D, bool DKV, bool ROT_X, bool ROT_A, bool BS = false, bool GEN = false>
__global__ void __launch_bounds__(512, 1)
attn_bwd_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_y,
                const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                const __grid_constant__ CUtensorMap tm_s, const BwdParams p) {
    using L = BwdSmem<D>;
    constexpr int TILE = L::TILE, NST = L::NST;
    constexpr int NBOX = D / BOX_COLS;
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t T1 = 0, T2 = 128, ACC1 = 256, ACC2 = 256 + D;
    constexpr uint32_t IDESC_T = idesc_bf16_f32(128, 128, 0, 0);
    constexpr uint32_t IDESC_ACC = idesc_bf16_f32(128, D, 0, 1);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *sX = smem + L::OFF_X, *sY = smem + L::OFF_Y, *sA = smem + L::OFF_A, *sB = smem + L::OFF_B;
    float* sStats = reinterpret_cast<float*>(smem + L::OFF_STATS);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::OFF_MISC);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + L::OFF_MISC + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const MaskSpec ms{p.S, p.causal, p.window, p.skip_rows};
    // stationary tile: DKV -> key tile of kv head (b, hk); DQ -> query tile of head (b, h)
    const int xh_count = DKV ? p.Hkv : p.Hq;
    const int b = blockIdx.x / xh_count, xh = blockIdx.x - b * xh_count;
    // heaviest tiles first: under a causal mask early key tiles and late query tiles see the most work
    const int x0 = ((BS && p.bs_order) ? __ldg(p.bs_order + blockIdx.y)
                                       : (DKV ? static_cast<int>(blockIdx.y) : static_cast<int>(gridDim.y - 1 - blockIdx.y))) * 128;
    int lo, hi;  // streamed tile range
    if (DKV) qtile_range(ms, x0, lo, hi);
    else tile_range(ms, x0, lo, hi);
    int bs_base = 0;
    if constexpr (BS) {   // block-sparse: positions in the stationary block's list instead of a tile range
        bs_base = __ldg(p.bs_ptr + x0 / 128);
        lo = 0;
        hi = __ldg(p.bs_ptr + x0 / 128 + 1) - bs_base - 1;
    }
    const int per_head = hi - lo + 1;
    const int n_it = DKV ? per_head * p.group : per_head;
    // iteration n -> (streamed head, streamed row0)
    auto stream_head = [&](int n) { return DKV ? xh * p.group + n / per_head : xh / p.group; };
    auto stream_row0 = [&](int n) {
        const int pos = lo + (DKV ? n % per_head : n);
        return (BS ? __ldg(p.bs_idx + bs_base + pos) : pos) * 128;
    };
    // The producer and the gradient warpgroups walk the same sequence with a cursor instead: a division and a modulo
    // per tile are some 350 cycles of dependent integer arithmetic each, on the warpgroups' loop-carried chain.
    struct Cursor {
        int pos, head;
    };
    const Cursor first{0, DKV ? xh * p.group : xh / p.group};
    auto advance = [&](Cursor& c) {
        if (++c.pos == per_head) {
            c.pos = 0;
            ++c.head;
        }
    };
    auto row0_of = [&](const Cursor& c) { return (BS ? __ldg(p.bs_idx + bs_base + lo + c.pos) : lo + c.pos) * 128; };

    if (threadIdx.x == 0) {
        for (int i = 0; i < L::N_BARS; ++i) {
            uint32_t cnt = 1;
            if ((i >= L::B_AROT && i < L::B_AROT + NST) || i == L::B_PDS || i == L::B_PDS + 1) cnt = 4;  // per-warp arrives
            if (i == L::B_XROT) cnt = 8;  // both gradient warpgroups
            if (i == L::B_TFULL || i == L::B_TFULL + 1 || i == L::B_DONE || (i >= L::B_EMPTY && i < L::B_EMPTY + NST))
                cnt = 2;  // one arrival per MMA issuer
            mbar_init(&bars[i], cnt);
        }
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // Programmatic dependent launch: this grid may have been scheduled while its predecessor in the backward
    // sequence (delta, RoPE pass or the other gradient kernel) was still running; from here on it reads what
    // they wrote.  The next kernel of the sequence may in turn be scheduled from now on.
    grid_dep_wait();
    grid_dep_launch();
    AF_BSTAMP(5, 0, 0);

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tmap(&tm_x); prefetch_tmap(&tm_y); prefetch_tmap(&tm_a); prefetch_tmap(&tm_b);
            mbar_arrive_expect_tx(&bars[L::B_XFULL], TILE);
            mbar_arrive_expect_tx(&bars[L::B_YFULL], TILE);
#pragma unroll
            for (int bx = 0; bx < NBOX; ++bx) {
                tma_load_4d(sX + bx * BOX_BYTES, &tm_x, &bars[L::B_XFULL], bx * BOX_COLS, x0, xh, b);
                tma_load_4d(sY + bx * BOX_BYTES, &tm_y, &bars[L::B_YFULL], bx * BOX_COLS, x0, xh, b);
            }
            Cursor cur = first;
            for (int n = 0; n < n_it; ++n) {
                const int st = n % NST, ah = cur.head, a0 = row0_of(cur);
                advance(cur);
                if (!mbar_wait(&bars[L::B_EMPTY + st], ((n / NST) & 1) ^ 1, abort_flag, 21)) break;
                mbar_arrive_expect_tx(&bars[L::B_AFULL + st], TILE);
                mbar_arrive_expect_tx(&bars[L::B_BFULL + st], TILE);
#pragma unroll
                for (int bx = 0; bx < NBOX; ++bx) {
                    tma_load_4d(sA + st * TILE + bx * BOX_BYTES, &tm_a, &bars[L::B_AFULL + st], bx * BOX_COLS, a0, ah, b);
                    tma_load_4d(sB + st * TILE + bx * BOX_BYTES, &tm_b, &bars[L::B_BFULL + st], bx * BOX_COLS, a0, ah, b);
                }
            }
        }
    } else if (warp == 1 || warp == 2) {
        // ------------------------------------------------------------ MMA issuers
        // Two issuing threads on different SM sub-partitions, split by product so that every accumulator has
        // exactly one issuer (the order of its additions stays fixed: deterministic results):
        //   issuer 0: T1 = X A^T and acc1 (DKV: dV += P^T dO;  DQ: dQ' += dS K')
        //   issuer 1: T2 = Y Bc^T and, in the DKV role, acc2 (dK' += dS^T Q')
        // A single thread issuing all 48 MMAs of a tile pair was the bottleneck of this kernel.
        if (lane == 0) {
            constexpr int B_XREADY = ROT_X ? L::B_XROT : L::B_XFULL;
            constexpr int B_AREADY = ROT_A ? L::B_AROT : L::B_AFULL;
            const int who = warp - 1;
            bool ok = true;
            if (who == 0) {
                ok = mbar_wait(&bars[B_XREADY], 0, abort_flag, 22);
                if (ok && ROT_X && p.store_x) {
                    // publish the rotated stationary tile (rows past S are clipped by the tensor map)
#pragma unroll
                    for (int bx = 0; bx < NBOX; ++bx) tma_store_4d(&tm_s, sX + bx * BOX_BYTES, bx * BOX_COLS, x0, xh, b);
                    tma_store_commit();
                }
            } else {
                ok = mbar_wait(&bars[L::B_YFULL], 0, abort_flag, 23);
            }
            const uint32_t xa = smem_u32(sX), ya = smem_u32(sY);
            constexpr uint32_t IDESC_TH = idesc_bf16_f32(128, 64, 0, 0);   // half tile: 64 streamed rows
            const uint32_t dhi = desc_hi(1024);
            const uint32_t s_lo = desc_lo(who == 0 ? xa : ya, 16);          // this issuer's stationary operand
            const uint32_t t_dst = tmem_base + (who == 0 ? T1 : T2);
            // T1 or T2, half hf of streamed tile n: rows [64 hf, 64 hf + 64) of A (or Bc) are the N index
#ifndef AF_BWD_TFULL
#define AF_BWD_TFULL 0
#endif
            constexpr bool kTFull = AF_BWD_TFULL != 0;   // T1/T2 as one N = 128 MMA group per tile instead of two N = 64 halves
            auto issue_T = [&](int n, int hf) {
                const int st = n % NST;
                if (kTFull) {
                    if (hf == 0) return;   // issued once per tile, at the second half's turn
                    const uint32_t r_lo = desc_lo(smem_u32((who == 0 ? sA : sB) + st * TILE), 16);
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t off = ((kk >> 2) * BOX_BYTES + (kk & 3) * 32) >> 4;
                        if (kk == 0) mma_ss_lo<false>(t_dst, s_lo + off, r_lo + off, dhi, IDESC_T);
                        else mma_ss_lo<true>(t_dst, s_lo + off, r_lo + off, dhi, IDESC_T);
                    }
                    mma_commit(&bars[L::B_TFULL + 0]);
                    mma_commit(&bars[L::B_TFULL + 1]);
                    return;
                }
                const uint32_t r_lo = desc_lo(smem_u32((who == 0 ? sA : sB) + st * TILE) + hf * 64 * 128, 16);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = ((kk >> 2) * BOX_BYTES + (kk & 3) * 32) >> 4;
                    if (kk == 0) mma_ss_lo<false>(t_dst + hf * 64, s_lo + off, r_lo + off, dhi, IDESC_TH);
                    else mma_ss_lo<true>(t_dst + hf * 64, s_lo + off, r_lo + off, dhi, IDESC_TH);
                }
                mma_commit(&bars[L::B_TFULL + hf]);   // complete when both issuers' halves are
            };
            auto wait_stream = [&](int n) {
                const int st = n % NST;
                bool r = mbar_wait(&bars[(who == 0 ? B_AREADY : L::B_BFULL) + st], (n / NST) & 1, abort_flag, 24);
                // the accumulator MMAs of issuer 1 (DKV) read A as well, those of issuer 0 (DKV) read Bc
                if (r && DKV) r = mbar_wait(&bars[(who == 0 ? L::B_BFULL : B_AREADY) + st], (n / NST) & 1, abort_flag, 25);
                tc_fence_after_sync();
                return r;
            };
            const bool has_acc = who == 0 || DKV;
            AF_BSTAMP(who, 63, 0);   // stationary operand ready
            if (ok && n_it > 0) ok = wait_stream(0);
            AF_BSTAMP(who, 63, 1);   // first streamed tile ready
            if (ok && n_it > 0) {
                issue_T(0, 0);
                issue_T(0, 1);
            }
            for (int n = 0; ok && n < n_it; ++n) {
                const int st = n % NST;
                // MN-major B operand of this issuer's accumulator MMAs: 16 streamed rows (2 KB) per K step
                const uint32_t m_lo = desc_lo(smem_u32(((who == 0) == DKV ? sB : sA) + st * TILE), BOX_BYTES);
                const uint32_t acc_dst = tmem_base + (who == 0 ? ACC1 : ACC2);
                const bool next = n + 1 < n_it;
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    // this half: 4 K = 16 steps over its 64 streamed rows; the bf16 operands sit at the start of
                    // the half's own columns of T1 (issuer 0) or T2 (issuer 1)
                    AF_BSTAMP(who, n, 3 * hf);
                    ok = mbar_wait(&bars[L::B_PDS + hf], n & 1, abort_flag, 26);
                    AF_BSTAMP(who, n, 3 * hf + 1);
                    if (!ok) break;
                    tc_fence_after_sync();
                    if (has_acc) {
#pragma unroll
                        for (int k4 = 0; k4 < 4; ++k4) {
                            const int kk = hf * 4 + k4;
                            mma_ts_lo(acc_dst, t_dst + hf * 64 + k4 * 8, m_lo + kk * 128, dhi, IDESC_ACC, (n > 0 || kk > 0) ? 1u : 0u);
                        }
                    }
                    if (hf == 1) {
                        // the stage is free once both issuers have consumed both halves
                        if (has_acc) mma_commit(&bars[L::B_EMPTY + st]);
                        else mbar_arrive(&bars[L::B_EMPTY + st]);   // DQ, issuer 1: its T2 MMAs of this stage were complete at TFULL
                    }
                    // the same half of the next streamed tile may overwrite T1/T2 right behind (in-order per issuer)
                    if (next) {
                        if (hf == 0) ok = wait_stream(n + 1);
                        if (!ok) break;
                        issue_T(n + 1, hf);
                    }
                    AF_BSTAMP(who, n, 3 * hf + 2);
                }
                if (!ok) break;
                if (!next) {
                    if (has_acc) mma_commit(&bars[L::B_DONE]);
                    else mbar_arrive(&bars[L::B_DONE]);
                }
            }
            if (who == 0 && ROT_X && p.store_x) tma_store_wait_all();   // the tile must stay in place until it has been read
        }
    } else if (warp >= 4 && warp < 8) {
        // ------------------------------------------------------------ rotation warpgroup: X once, every A tile
        if (ROT_A) {
            const int t = threadIdx.x - 128;
            auto run = [&](auto cp_tag) {
                constexpr int CP = decltype(cp_tag)::value;
                constexpr int CPT = CP > 0 ? CP : 1;
                RotStep step;
                RotState<CPT> st;
                if (CP > 0) rotate_load_step<CPT>(p.table, p.S, p.R, t, step);
                // (the stationary tile X is rotated by the two gradient warpgroups, idle at that point)
                if (!ROT_A) return;
                // streamed tiles are consecutive within a head: the recurrence carries the state along
                for (int n = 0; n < n_it; ++n) {
                    const int sg = n % NST, a0 = stream_row0(n);
                    const int run_pos = DKV ? n % per_head : n;
                    // (listed tiles need not be consecutive: then the cos/sin state is read for every tile)
                    if (CP > 0 && (BS || (run_pos % kRotResync) == 0)) rotate_prefetch(st, p.table, a0, p.S, p.R, t);
                    AF_BSTAMP(4, n, 0);
                    if (!mbar_wait_warp(&bars[L::B_AFULL + sg], (n / NST) & 1, abort_flag, 28)) return;
                    AF_BSTAMP(4, n, 1);
                    if (CP > 0) rotate_tile_fast(sA + sg * TILE, st, step, t);
                    else rotate_tile_smem(sA + sg * TILE, a0, p.S, p.R, p.table, t, 128);
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars[L::B_AROT + sg]);
                    AF_BSTAMP(4, n, 2);
                }
            };
            if (p.R == 128) run(std::integral_constant<int, 8>{});
            else if (p.R == 64) run(std::integral_constant<int, 4>{});
            else if (p.R == 32) run(std::integral_constant<int, 2>{});
            else if (p.R == 16) run(std::integral_constant<int, 1>{});
            else run(std::integral_constant<int, 0>{});
        }
    } else if (warp >= 8) {
        // ------------------------------------------------------------ gradient warpgroups (one TMEM lane per thread)
        const int gtid = threadIdx.x - 256;          // 0..255 over both warpgroups
        const int hf = gtid >> 7;                    // column half owned by this warpgroup
        const int tid = gtid & 127;                  // == TMEM lane
        const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tb = tmem_base + lane_addr;
        const int xrow = x0 + tid;  // DKV: key row j; DQ: query row i
        const bool alibi = p.slopes != nullptr;
        constexpr float kLog2e = 1.4426950408889634f;
        float my_l2 = 0.f, my_delta = 0.f, my_slope2 = 0.f;
        if (!DKV) {
            const size_t r = (static_cast<size_t>(b) * p.Hq + xh) * p.S + xrow;
            if (GEN && p.relu) {   // lse holds n_i; the pass wants 1 / n_i
                const float cnt = xrow < p.S ? p.lse[r] : 0.f;
                my_l2 = cnt > 0.f ? 1.f / cnt : 0.f;
            } else {
                my_l2 = xrow < p.S ? -p.lse[r] * kLog2e : -INFINITY;   // kept negated
                my_delta = xrow < p.S ? -p.delta[r] : 0.f;
            }
            my_slope2 = alibi ? p.slopes[xh] * kLog2e : 0.f;
        }
        bool ok = true;
        if (ROT_X) {
            // the stationary tile is rotated once, by these two warpgroups (half of the rows each): they
            // have nothing else to do until the first scores arrive
            auto rot_x = [&](auto cp_tag) {
                constexpr int CP = decltype(cp_tag)::value;
                ok = wg_all(mbar_wait(&bars[L::B_XFULL], 0, abort_flag, 27));
                if (!ok) return;
                if constexpr (CP > 0) {
                    RotStep step;
                    rotate_load_step<CP>(p.table, p.S, p.R, tid, step);
                    rotate_tile_share<CP, 2>(sX, p.table, x0, p.S, p.R, step, tid, hf);
                } else {
                    rotate_tile_smem(sX, x0, p.S, p.R, p.table, gtid, 256);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars[L::B_XROT]);
            };
            if (p.R == 128) rot_x(std::integral_constant<int, 8>{});
            else if (p.R == 64) rot_x(std::integral_constant<int, 4>{});
            else if (p.R == 32) rot_x(std::integral_constant<int, 2>{});
            else if (p.R == 16) rot_x(std::integral_constant<int, 1>{});
            else rot_x(std::integral_constant<int, 0>{});
        }
        // DKV: per-column statistics of the streamed query tile (each warpgroup stages its own 64 columns).  The
        // global loads for tile n + 1 are issued at the top of iteration n and land in the other buffer after this
        // iteration's passes, so that their latency is off the loop-carried chain of the warpgroup.
        // (Nothing touches the loaded registers before store_stats: arithmetic at the load would make the warp sit out
        // the load's latency in front of its wait for the scores.)
        float nx_l = 0.f, nx_d = 0.f, nx_slope = 0.f;
        bool nx_in = false;
        Cursor cur_stats = first;
        auto load_stats = [&]() {   // of the tile under the cursor, which then moves on
            const int ah = cur_stats.head, a0 = row0_of(cur_stats);
            advance(cur_stats);
            if (tid < 64) {
                const int qi = a0 + hf * 64 + tid;
                const size_t r = (static_cast<size_t>(b) * p.Hq + ah) * p.S + min(qi, p.S - 1);
                nx_in = qi < p.S;
                nx_l = p.lse[r];
                if (!(GEN && p.relu)) nx_d = p.delta[r];
            }
            if (alibi) nx_slope = p.slopes[ah];
        };
        auto store_stats = [&](int n) {
            if (tid < 64) {
                float* dst = sStats + (n & 1) * 256 + hf * 64 + tid;
                if (GEN && p.relu) {
                    dst[0] = (nx_in && nx_l > 0.f) ? 1.f / nx_l : 0.f;   // 1 / n_i
                    dst[128] = 0.f;
                } else {
                    dst[0] = nx_in ? -nx_l * kLog2e : -INFINITY;   // kept negated
                    dst[128] = nx_in ? -nx_d : 0.f;
                }
            }
        };
        if (DKV && ok && n_it > 0) {
            load_stats();
            store_stats(0);
        }
        Cursor cur = first;
        for (int n = 0; ok && n < n_it; ++n) {
            const int ah = cur.head, a0 = row0_of(cur);
            advance(cur);
            float* sL2 = sStats + (n & 1) * 256;
            float* sDl = sL2 + 128;
            if (DKV) {
                my_slope2 = nx_slope * kLog2e;
                if (n + 1 < n_it) load_stats();
            }
            const int i0 = DKV ? a0 : x0, j0 = DKV ? x0 : a0;
            const bool need_mask = tile_needs_mask(ms, i0, j0);
            int mlo = 0;
            uint32_t mn = 128;
            if (need_mask) {
                if (DKV) kept_queries_of_key(ms, xrow, a0, mlo, mn);
                else kept_keys_of_query(ms, xrow, a0, mlo, mn);
            }
            // ALiBi: slope2 * (j - i) = sb * (col + base), sb = +-slope2
            const float sb = DKV ? -my_slope2 : my_slope2;
            const float bias_base = sb * static_cast<float>(a0 - xrow);
            // this warpgroup's half of T1/T2; the barrier also publishes the statistics within the warpgroup
            AF_BSTAMP(2 + hf, n, 0);
            ok = bar_all(mbar_wait(&bars[L::B_TFULL + hf], n & 1, abort_flag, 29), 1 + hf, 128);
            AF_BSTAMP(2 + hf, n, 1);
            if (!ok) break;
            tc_fence_after_sync();
#pragma unroll
            for (int qt = 0; qt < 2; ++qt) {
                const int col0 = hf * 64 + qt * 32;
                const uint32_t out_col = hf * 64 + qt * 16;   // bf16 results: start of this warpgroup's own half
                const float cbias = fmaf(sb, static_cast<float>(col0), bias_base);
                if constexpr (GEN) {
                    // bias of the pair (this lane, first column of the pass): DKV lane = key, columns = queries
                    const float* bp = nullptr;
                    long long cs = 1;
                    int cols_ok = 0;
                    if (p.bias && xrow < p.S) {
                        const int hq = DKV ? ah : xh;
                        const float* bh = p.bias + b * p.bias_sb + hq * p.bias_sh;
                        if (DKV) { bp = bh + static_cast<long long>(a0 + col0) * p.S + xrow; cs = p.S; }
                        else { bp = bh + static_cast<long long>(xrow) * p.S + a0 + col0; cs = 1; }
                        cols_ok = p.S - (a0 + col0);
                        if (cols_ok <= 0) bp = nullptr;
                    }
                    if (p.relu) grad_pass32_general<DKV, true>(tb + T1, tb + T2, col0, out_col, p.scale_log2, cbias, sb, sL2, sDl, my_l2, my_delta, mlo, mn, bp, cs, cols_ok);
                    else grad_pass32_general<DKV, false>(tb + T1, tb + T2, col0, out_col, p.scale_log2, cbias, sb, sL2, sDl, my_l2, my_delta, mlo, mn, bp, cs, cols_ok);
                } else if (alibi) {
                    if (need_mask) grad_pass32<DKV, true, true>(tb + T1, tb + T2, col0, out_col, p.scale_log2, cbias, sb, sL2, sDl, my_l2, my_delta, mlo, mn);
                    else grad_pass32<DKV, false, true>(tb + T1, tb + T2, col0, out_col, p.scale_log2, cbias, sb, sL2, sDl, my_l2, my_delta, mlo, mn);
                } else {
                    if (need_mask) grad_pass32<DKV, true, false>(tb + T1, tb + T2, col0, out_col, p.scale_log2, cbias, sb, sL2, sDl, my_l2, my_delta, mlo, mn);
                    else grad_pass32<DKV, false, false>(tb + T1, tb + T2, col0, out_col, p.scale_log2, cbias, sb, sL2, sDl, my_l2, my_delta, mlo, mn);
                }
            }
            AF_BSTAMP(2 + hf, n, 2);
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars[L::B_PDS + hf]);
            AF_BSTAMP(2 + hf, n, 3);
            if (DKV && n + 1 < n_it) store_stats(n + 1);   // (the named barrier at the top of the next iteration publishes it)
        }
        // epilogue: stage through shared memory (the stream stages are idle now), rotate back, store
        AF_BSTAMP(2 + hf, 63, 0);
        // (every thread of both warpgroups takes this barrier, also after a wait that gave up in one of them:
        // a warpgroup that left its loop early must not leave the other alone at it)
        ok = wg_all(ok && (n_it <= 0 || mbar_wait(&bars[L::B_DONE], 0, abort_flag, 30)));
        AF_BSTAMP(2 + hf, 63, 1);   // accumulators complete
        if (BS && ok && n_it <= 0) {
            // no active block for this stationary block: its gradient rows are zero
            const size_t row0 = (static_cast<size_t>(b) * xh_count + xh) * p.S + x0;
            const int rows = min(128, p.S - x0);
            for (int idx = gtid; idx < rows * (D / 4); idx += 256) {
                const size_t off = (row0 + idx / (D / 4)) * D + (idx % (D / 4)) * 4;
                for (int w2 = 0; w2 < (DKV ? 2 : 1); ++w2) {
                    void* out = w2 == 0 ? p.out1 : p.out2;
                    if (p.out_f32) *reinterpret_cast<float4*>(static_cast<float*>(out) + off) = make_float4(0.f, 0.f, 0.f, 0.f);
                    else *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(out) + off) = make_uint2(0u, 0u);
                }
            }
        }
        if (ok && n_it > 0) {
            tc_fence_after_sync();
            float* stg = reinterpret_cast<float*>(sA);
            const size_t out_row0 = (static_cast<size_t>(b) * xh_count + xh) * p.S + x0;
            if (DKV) {
                store_acc_rotated<D>(tb + ACC1, stg, gtid, 1.f, 0, p.table, x0, p.S, p.out1, out_row0, p.out_f32);
                store_acc_rotated<D>(tb + ACC2, stg, gtid, p.scale, p.R, p.table, x0, p.S, p.out2, out_row0, p.out_f32);
            } else {
                store_acc_rotated<D>(tb + ACC1, stg, gtid, p.scale, p.R, p.table, x0, p.S, p.out1, out_row0, p.out_f32);
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    AF_BSTAMP(5, 0, 1);
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace af
