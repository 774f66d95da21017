// One-pass backward (Section 4.4): dK, dV and dQ from ONE walk over the kept tile pairs - five products per pair
// instead of the seven that the two-kernel sequence of bwd_kernel.cuh executes (it recomputes S and dP in both
// of its roles).  A CTA owns a key tile (K', V stationary), streams the (Q', dO) tiles of the query heads that
// see it, and per streamed tile forms
//     S^T = K' Q'^T,  dP^T = V dO^T,  P^T, dS^T (gradient warpgroups),
//     dV += P^T dO,   dK' += dS^T Q',   dQ'^T(tile) = K'^T dS^T.
// dQ' is a sum over key tiles, i.e. over CTAs: every CTA adds its [D x 64] partials into an fp32 accumulator in
// the caller's workspace with red.global.add.f32 (zeroed beforehand; bwd_dq_finish_kernel then scales, rotates
// back and converts).  The order of those additions depends on how the CTAs are scheduled, so dQ is NOT
// bit-reproducible from run to run (dK and dV are: one CTA, one issuer per accumulator); the two-kernel
// sequence stays available for callers that need reproducible dQ.
//
// No on-chip rotation: K' and Q' come rotated from RoPE passes (or are K and Q themselves without RoPE); only the
// epilogue rotates dK' back.  TMEM (512 columns): T1 = S^T -> P^T, T2 = dP^T -> dQ'^T, dV, dK'.  T1 and T2 are
// worked on in two column halves of 64 streamed rows each, as in bwd_kernel.cuh.  dS^T goes to shared memory
// (bf16, 128-byte rows of 64 query positions per key, 128-byte swizzle), where the same bytes are the K-major A
// operand of dK' += dS^T Q' and the MN-major B operand of dQ'^T = K'^T dS^T; once a gradient warpgroup has read
// its half of dP^T out of T2 that half is free for the dQ'^T partial of the same 64 query rows.
// What bounds it: shared-memory bandwidth.  Every product whose two operands come from shared memory reads
// 128 bytes per clock while it runs, and the N = 64 halves re-read the stationary operand twice per tile:
// 384 KB of operand reads per tile pair (against 256 KB in the dK/dV role of the two-kernel sequence) plus the
// TMA writes and the dS^T stores, about 3.8 k cycles of shared-memory time per tile pair; a timeline shows the
// gradient passes crawling (3.8 k cycles instead of 1.3 k) whenever the tensor pipe is busy.  Measured 6.5 k
// cycles per tile pair against 3.7 k + 3.2 k for the two roles of the two-kernel sequence: ahead where the dQ
// role's CTAs are short (few key tiles per query tile), behind on long rows.  (A variant with ONE dP^T buffer
// handed back as soon as it is in registers and ONE dQ'^T buffer of its own measured slower still, 8.0 k.)
// D = 64: the same kernel; dQ'^T then has M = 64 rows, which tcgen05 keeps in the first 16 lanes of each 32-lane quarter of
// TMEM (row d in lane 32 (d / 16) + d % 16), so half of the reducing lanes carry a row; and the accumulators leave 128
// TMEM columns free, so the partials get two 64-column buffers of their own and T2 never waits for a read-out.
// Shared-memory traffic per tile pair is half that of D = 128; the sequence measured 1.23-1.31 times faster than the
// two-kernel one on every shape tried (0.691 -> 0.546 ms at B = 4, 12 heads, N = 4096).
// Warp roles (512 threads): warp 0 TMA producer; warps 1, 2, 3 MMA issuers (T1 and dV; T2 and dK'; dQ'^T), one
// per SM sub-partition; warps 4-7 read the dQ'^T partials out of TMEM and add them to global memory; warps 8-11
// and 12-15 are the two gradient warpgroups, one per column half.  A gradient warpgroup works in two phases per
// tile (P^T from S^T, then dS^T from dP^T) and announces each on a barrier of its own, so that S^T of the next
// tile is issued while dS^T is still being formed and dP^T of the next tile while the next P^T is.  A timeline of
// the D = 64 kernel (4.4 k cycles per tile pair): phase P 1.5-2.3 k cycles for 64 columns (the exponentials of
// both warpgroups share one special-function unit per sub-partition: 1 k cycles per tile pair is its floor, and
// a microbenchmark of the phase alone gives 0.76 k for one warp per sub-partition, 1.1 k for two), phase dS
// 0.9-1.1 k, the rest waits on the products.  Measured and not kept: both warpgroups on the same half with the
// phases interleaved by half (each phase pays the TMEM load and store latencies again: 5.2 k cycles per pair);
// working out the next tile's mask and addresses between the two phases (the warpgroups fall into step and the
// shared exponential unit stretches phase P: 4.9 k).
#pragma once
#include "bwd_kernel.cuh"

namespace af {

template <int D>
struct BwdFusedSmem {
    static constexpr int TILE = 128 * D * 2;
    static constexpr int NST = 2;
    static constexpr int DS_HALF = 128 * 128;     // dS^T of 64 streamed rows: 128 key rows x 128 bytes
    static constexpr int OFF_X = 0, OFF_Y = TILE;
    static constexpr int OFF_A = 2 * TILE;
    static constexpr int OFF_B = OFF_A + NST * TILE;
    static constexpr int OFF_DS = OFF_B + NST * TILE;
    static constexpr int OFF_STATS = OFF_DS + 2 * DS_HALF;
    static constexpr int OFF_BAR = OFF_STATS + 2 * 2 * 128 * 4;
    static constexpr int B_XFULL = 0, B_YFULL = 1, B_AFULL = 2, B_BFULL = B_AFULL + NST, B_EMPTY = B_BFULL + NST,
                         B_SFULL = B_EMPTY + NST, B_DPFULL = B_SFULL + 2, B_PRDY = B_DPFULL + 2, B_PDS = B_PRDY + 2,
                         B_DQFULL = B_PDS + 2, B_DSFREE = B_DQFULL + 2, B_T2FREE = B_DSFREE + 2, B_DONE = B_T2FREE + 2,
                         N_BARS = B_DONE + 1;
    static constexpr int OFF_MISC = OFF_BAR + N_BARS * 8;
    static constexpr int NEEDED = OFF_MISC + 16;
    // The layout needs 1024-byte alignment (swizzle atoms).  The request leaves what room there is for rounding
    // the base up; the kernel checks that the rounded layout still fits and gives up with a status otherwise.
    static constexpr int BYTES = NEEDED + 1024 <= 232448 ? NEEDED + 1024 : 232448;
    static constexpr int STG_STRIDE = BwdSmem<D>::STG_STRIDE;
    static_assert(NEEDED <= 232448, "shared-memory layout exceeds one CTA's limit");
    static_assert(128 * STG_STRIDE * 4 <= 2 * NST * TILE, "staging buffer must fit in the stream stages");
};

// timeline stamps for tuning (compiled out unless AF_TRACE): as AF_BSTAMP, with the buffer's address read once per
// thread (`trc`) so that a stamp costs a clock read and a store
#ifdef AF_TRACE
#define AF_FSTAMP(role, it, ph)                                                                  \
    do {                                                                                         \
        if (trc && (threadIdx.x & 31) == 0 && (it) < 64) trc[((role) * 64 + (it)) * 8 + (ph)] = clock64(); \
    } while (0)
#else
#define AF_FSTAMP(role, it, ph) do { } while (0)
#endif

constexpr int kFusedLightRegs = 64, kFusedReduceRegs = 96, kFusedGradRegs = 176;
constexpr uint32_t kFusedSmemCode = 0x40;   // status code: dynamic shared memory too misaligned for the layout

// The gradient warpgroups work on a half tile (64 streamed rows) in two phases, so that each of the two products
// that feed them is re-issued for the next tile as soon as its own result has been consumed:
//   phase P:  S^T half -> P^T (bf16 into TMEM for dV; fp32 kept in registers), after which T1's half is free;
//   phase dS: dP^T half -> dS^T = P^T (dP^T - delta) to shared memory (row = this thread's key, 16-byte chunks
//             `chunk0`.. of its 128-byte row, swizzled), after which T2's half is free.
template <bool MASKED, bool ALIBI>
__device__ __forceinline__ void grad_phase_p32(uint32_t t1, int col0, uint32_t out_col, float scale_log2, float cbias, float sb,
                                               const float* s_nl2, int mlo, uint32_t mn, uint32_t* s) {
    // s: 32 columns of S^T already in registers; overwritten in place with the bits of the fp32 probabilities
    uint32_t pk[16];
    const float2 sc2 = make_float2(scale_log2, scale_log2), cb2 = make_float2(cbias, cbias);
#pragma unroll
    for (int e = 0; e < 32; e += 4) {
        const float4 a4 = *reinterpret_cast<const float4*>(s_nl2 + col0 + e);
        const float2 nl[2] = {make_float2(a4.x, a4.y), make_float2(a4.z, a4.w)};
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int c = e + 2 * u;
            // (without ALiBi the row's bias is zero: one packed add per column pair less)
            float2 t = __ffma2_rn(make_float2(__uint_as_float(s[c]), __uint_as_float(s[c + 1])), sc2, ALIBI ? __fadd2_rn(cb2, nl[u]) : nl[u]);
            if (ALIBI) {
                t.x = fmaf(sb, static_cast<float>(c), t.x);
                t.y = fmaf(sb, static_cast<float>(c + 1), t.y);
            }
            float2 pe = make_float2(ex2(t.x), ex2(t.y));
            if (MASKED) {
                pe.x = (static_cast<uint32_t>(col0 + c - mlo) < mn) ? pe.x : 0.f;
                pe.y = (static_cast<uint32_t>(col0 + c + 1 - mlo) < mn) ? pe.y : 0.f;
            }
            s[c] = __float_as_uint(pe.x);
            s[c + 1] = __float_as_uint(pe.y);
            pk[c >> 1] = pack_bf16x2(pe.x, pe.y);
        }
    }
    tmem_st16(t1 + out_col, pk);
}

__device__ __forceinline__ void grad_phase_ds32(const uint32_t* dp, int col0, const float* s_ndl, const uint32_t* pe_keep,
                                                uint32_t ds_row_addr, int row7, int chunk0) {
    uint32_t dk[16];
#pragma unroll
    for (int e = 0; e < 32; e += 4) {
        const float4 b4 = *reinterpret_cast<const float4*>(s_ndl + col0 + e);
        const float2 nd[2] = {make_float2(b4.x, b4.y), make_float2(b4.z, b4.w)};
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int c = e + 2 * u;
            const float2 ds = __fmul2_rn(make_float2(__uint_as_float(pe_keep[c]), __uint_as_float(pe_keep[c + 1])),
                                         __fadd2_rn(make_float2(__uint_as_float(dp[c]), __uint_as_float(dp[c + 1])), nd[u]));
            dk[c >> 1] = pack_bf16x2(ds.x, ds.y);
        }
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const uint32_t a = ds_row_addr + (static_cast<uint32_t>((chunk0 + c) ^ row7) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(dk[4 * c]), "r"(dk[4 * c + 1]), "r"(dk[4 * c + 2]),
                     "r"(dk[4 * c + 3])
                     : "memory");
    }
}

// BS: block-sparse attention (Section 4.3) - the streamed query tiles of a key block come from its list of active
// blocks (p.bs_ptr / p.bs_idx by key block, p.bs_order the launch order) instead of a contiguous range.
template <int D, bool BS = false>
__global__ void __launch_bounds__(512, 1)
attn_bwd_fused_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_y,
                      const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b, const BwdParams p) {
    static_assert(D == 128 || D == 64, "head dimension");
    using L = BwdFusedSmem<D>;
    constexpr int TILE = L::TILE, NST = L::NST;
    constexpr int NBOX = D / BOX_COLS;
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t T1 = 0, T2 = 128, ACC1 = 256, ACC2 = 256 + D;
    // Where the dQ'^T partial of a half lands.  D = 128: TMEM is full, it takes the half of T2 whose dP^T has just been
    // consumed, and the next dP^T of that half waits for its read-out.  D = 64: the accumulators leave 128 columns free,
    // the partials get two 64-column buffers of their own there and T2 never waits for them.
    constexpr bool kOwnDq = D == 64;
    constexpr uint32_t TDQ = kOwnDq ? 384 : T2;
    constexpr uint32_t IDESC_TH = idesc_bf16_f32(128, 64, 0, 0);     // S^T / dP^T half: 64 streamed rows
    constexpr uint32_t IDESC_ACC = idesc_bf16_f32(128, D, 0, 1);     // dV, dK': B MN-major
    constexpr uint32_t IDESC_DQ = idesc_bf16_f32(D, 64, 1, 1);       // dQ'^T half: A = K'^T and B = dS^T both MN-major

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    if (static_cast<int>(smem - smem_raw) + L::NEEDED > L::BYTES) {
        if (threadIdx.x == 0) atomicCAS(&g_device_status, 0u, (kFusedSmemCode << 16) | (blockIdx.x & 0xffffu));
        return;
    }
    uint8_t *sX = smem + L::OFF_X, *sY = smem + L::OFF_Y, *sA = smem + L::OFF_A, *sB = smem + L::OFF_B;
    uint8_t* sDS = smem + L::OFF_DS;
    float* sStats = reinterpret_cast<float*>(smem + L::OFF_STATS);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::OFF_MISC);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + L::OFF_MISC + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const MaskSpec ms{p.S, p.causal, p.window, p.skip_rows};
    const int b = blockIdx.x / p.Hkv, xh = blockIdx.x - b * p.Hkv;
    // heaviest key tiles first under a causal mask; with block lists the caller's order
    const int x0 = ((BS && p.bs_order) ? __ldg(p.bs_order + blockIdx.y) : static_cast<int>(blockIdx.y)) * 128;
    int lo, hi;
    qtile_range(ms, x0, lo, hi);
    int bs_base = 0;
    if constexpr (BS) {   // positions in the key block's list instead of a tile range
        bs_base = __ldg(p.bs_ptr + x0 / 128);
        lo = 0;
        hi = __ldg(p.bs_ptr + x0 / 128 + 1) - bs_base - 1;
    }
    const int per_head = hi - lo + 1;
    const int n_it = per_head > 0 ? per_head * p.group : 0;
    // Streamed tile n = (query head xh * group + n / per_head, position lo + n % per_head): every role walks the
    // sequence with a cursor of its own (a division per tile sat on the gradient warpgroups' loop-carried chain).
    struct Cursor {
        int pos, head;
    };
    const Cursor first{0, xh * p.group};
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
            if (i == L::B_PDS || i == L::B_PDS + 1 || i == L::B_PRDY || i == L::B_PRDY + 1 || i == L::B_T2FREE || i == L::B_T2FREE + 1)
                cnt = 4;   // per-warp arrives
            if (i == L::B_DSFREE || i == L::B_DSFREE + 1 || i == L::B_DONE ||
                (i >= L::B_EMPTY && i < L::B_EMPTY + NST))
                cnt = 2;   // one arrival from each of two MMA issuers
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
#ifdef AF_TRACE
    long long* const trc = (blockIdx.x == 0 && blockIdx.y == 0) ? g_trace : nullptr;
#endif
    grid_dep_wait();     // delta, the RoPE passes and the zeroed accumulator precede this grid in the stream
    grid_dep_launch();
    if (warp == 0) AF_FSTAMP(5, 0, 0);

    // register budgets per role (they sum to the 512 a scheduler's four warps share): the gradient warpgroups
    // keep a half tile of probabilities next to a half tile of dP^T
    if (warp < 4) setmaxnreg_dec<kFusedLightRegs>();
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
                if (!mbar_wait(&bars[L::B_EMPTY + st], ((n / NST) & 1) ^ 1, abort_flag, 41)) break;
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
        // ------------------------------------------------------------ MMA issuers 0 and 1
        //   issuer 0: T1 = K' Q'^T  and dV  += P^T dO    (A from TMEM)
        //   issuer 1: T2 = V dO^T   and dK' += dS^T Q'   (A from shared memory)
        if (lane == 0) {
            const int who = warp - 1;
            bool ok = mbar_wait(&bars[who == 0 ? L::B_XFULL : L::B_YFULL], 0, abort_flag, 42);
            const uint32_t dhi = desc_hi(1024);
            const uint32_t s_lo = desc_lo(smem_u32(who == 0 ? sX : sY), 16);
            const uint32_t t_dst = tmem_base + (who == 0 ? T1 : T2);
            const uint32_t acc_dst = tmem_base + (who == 0 ? ACC1 : ACC2);
            auto issue_T = [&](int n, int hf) {
                const int st = n % NST;
                const uint32_t r_lo = desc_lo(smem_u32((who == 0 ? sA : sB) + st * TILE) + hf * 64 * 128, 16);
#pragma unroll 2   // (partly rolled: loop code against issue slots per MMA)
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = ((kk >> 2) * BOX_BYTES + (kk & 3) * 32) >> 4;
                    mma_ss_lo_rt(t_dst + hf * 64, s_lo + off, r_lo + off, dhi, IDESC_TH, kk > 0 ? 1u : 0u);
                }
                mma_commit(&bars[(who == 0 ? L::B_SFULL : L::B_DPFULL) + hf]);
            };
            auto wait_stream = [&](int n) {
                const int st = n % NST;
                bool r = mbar_wait(&bars[L::B_AFULL + st], (n / NST) & 1, abort_flag, 43);
                if (r) r = mbar_wait(&bars[L::B_BFULL + st], (n / NST) & 1, abort_flag, 44);
                tc_fence_after_sync();
                return r;
            };
            if (ok && n_it > 0) ok = wait_stream(0);
            if (ok && n_it > 0) {
                issue_T(0, 0);
                issue_T(0, 1);
            }
            for (int n = 0; ok && n < n_it; ++n) {
                const int st = n % NST;
                // MN-major B operand of the accumulator MMAs: 16 streamed rows (2 KB) per K step
                const uint32_t m_lo = desc_lo(smem_u32((who == 0 ? sB : sA) + st * TILE), BOX_BYTES);
                const bool next = n + 1 < n_it;
#pragma unroll 1   // (rolled: half the issuer's loop code; the instruction path is the tightest resource of this kernel)
                for (int hf = 0; hf < 2; ++hf) {
                    AF_FSTAMP(who, n, hf * 4);
                    // issuer 0 goes on when P^T of the half is in TMEM, issuer 1 when dS^T is in shared memory
                    ok = mbar_wait(&bars[(who == 0 ? L::B_PRDY : L::B_PDS) + hf], n & 1, abort_flag, 45);
                    if (!ok) break;
                    AF_FSTAMP(who, n, hf * 4 + 1);
                    tc_fence_after_sync();
                    if (who == 0) {
#pragma unroll
                        for (int k4 = 0; k4 < 4; ++k4) {
                            const int kk = hf * 4 + k4;
                            mma_ts_lo(acc_dst, t_dst + hf * 64 + k4 * 8, m_lo + kk * 128, dhi, IDESC_ACC, (n > 0 || kk > 0) ? 1u : 0u);
                        }
                    } else {
                        // A = dS^T half (K-major: 128 key rows of 128 bytes, 32 bytes per K step)
                        const uint32_t a_lo = desc_lo(smem_u32(sDS + hf * L::DS_HALF), 16);
#pragma unroll
                        for (int k4 = 0; k4 < 4; ++k4) {
                            const int kk = hf * 4 + k4;
                            mma_ss_lo_rt(acc_dst, a_lo + k4 * 2, m_lo + kk * 128, dhi, IDESC_ACC, (n > 0 || kk > 0) ? 1u : 0u);
                        }
                        mma_commit(&bars[L::B_DSFREE + hf]);
                    }
                    if (hf == 1) mma_commit(&bars[L::B_EMPTY + st]);
                    if (next) {
                        if (hf == 0) ok = wait_stream(n + 1);
                        // T2's half is free once the dQ'^T partial of the same rows has been read out of it
                        if (ok && who == 1 && !kOwnDq) ok = mbar_wait(&bars[L::B_T2FREE + hf], n & 1, abort_flag, 46);
                        if (!ok) break;
                        tc_fence_after_sync();
                        AF_FSTAMP(who, n, hf * 4 + 2);
                        issue_T(n + 1, hf);
                    }
                    AF_FSTAMP(who, n, hf * 4 + 3);
                }
                if (!ok) break;
                if (!next) mma_commit(&bars[L::B_DONE]);
            }
        }
    } else if (warp == 3) {
        // ------------------------------------------------------------ MMA issuer 2: dQ'^T half = K'^T dS^T half -> T2 half
        if (lane == 0) {
            bool ok = mbar_wait(&bars[L::B_XFULL], 0, abort_flag, 47);
            const uint32_t dhi = desc_hi(1024);
            const uint32_t a_lo = desc_lo(smem_u32(sX), BOX_BYTES);   // MN-major: 16 key rows (2 KB) per K step
            for (int n = 0; ok && n < n_it; ++n) {
#pragma unroll 1   // (rolled: half the issuer's loop code; the instruction path is the tightest resource of this kernel)
                for (int hf = 0; hf < 2; ++hf) {
                    AF_FSTAMP(6, n, hf * 4);
                    ok = mbar_wait(&bars[L::B_PDS + hf], n & 1, abort_flag, 48);
                    AF_FSTAMP(6, n, hf * 4 + 1);
                    // (own buffers: the previous tile's partial of this half must have been read out)
                    if (ok && kOwnDq && n > 0) ok = mbar_wait(&bars[L::B_T2FREE + hf], (n - 1) & 1, abort_flag, 54);
                    if (!ok) break;
                    AF_FSTAMP(6, n, hf * 4 + 2);
                    tc_fence_after_sync();
                    const uint32_t b_lo = desc_lo(smem_u32(sDS + hf * L::DS_HALF), 16);
                    const uint32_t dst = tmem_base + TDQ + hf * 64;
#pragma unroll 2
                    for (int kk = 0; kk < 8; ++kk)
                        mma_ss_lo_rt(dst, a_lo + kk * 128, b_lo + kk * 128, dhi, IDESC_DQ, kk > 0 ? 1u : 0u);
                    mma_commit(&bars[L::B_DQFULL + hf]);
                    mma_commit(&bars[L::B_DSFREE + hf]);
                    AF_FSTAMP(6, n, hf * 4 + 3);
                }
            }
        }
    } else if (warp >= 4 && warp < 8) {
        // ------------------------------------------------------------ dQ'^T partials: TMEM -> fp32 accumulator in global memory
        // TMEM lane = column d of dQ', TMEM column = query row: a warp's 32 lanes add 128 contiguous bytes.
        // D = 128: M = 128, TMEM lane = row d.  D = 64: the product has M = 64 rows, which sit in the first 16 lanes
        // of each 32-lane quarter (row d in lane 32 (d / 16) + d % 16); the other 16 lanes of a warp hold nothing.
        const int d = D == 128 ? (warp & 3) * 32 + lane : (warp & 3) * 16 + (lane & 15);
        const bool has_row = D == 128 || lane < 16;
        setmaxnreg_dec<kFusedReduceRegs>();
        const uint32_t tsrc = tmem_base + TDQ + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        bool ok = true;
        Cursor cur = first;
        for (int n = 0; ok && n < n_it; ++n) {
            const int ah = cur.head, a0 = row0_of(cur);
            advance(cur);
#pragma unroll 1
            for (int hf = 0; hf < 2; ++hf) {
                if (warp == 4) AF_FSTAMP(4, n, hf * 4);
                ok = mbar_wait_warp(&bars[L::B_DQFULL + hf], n & 1, abort_flag, 49);
                if (!ok) break;
                if (warp == 4) AF_FSTAMP(4, n, hf * 4 + 1);
                tc_fence_after_sync();
                uint32_t v[64];
                tmem_ld32(tsrc + hf * 64, v);
                tmem_ld32(tsrc + hf * 64 + 32, v + 32);
                tmem_wait_ld();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars[L::B_T2FREE + hf]);
                if (warp == 4) AF_FSTAMP(4, n, hf * 4 + 2);
                const int q0 = a0 + hf * 64;
                float* dst = p.dq_acc + ((static_cast<size_t>(b) * p.Hq + ah) * p.S + q0) * D + d;
                const int nq = min(64, p.S - q0);
                if (nq == 64) {
#pragma unroll
                    for (int q = 0; q < 64; ++q)
                        if (has_row) asm volatile("red.global.add.f32 [%0], %1;" ::"l"(dst + q * D), "f"(__uint_as_float(v[q])) : "memory");
                } else {
#pragma unroll
                    for (int q = 0; q < 64; ++q)
                        if (has_row && q < nq) asm volatile("red.global.add.f32 [%0], %1;" ::"l"(dst + q * D), "f"(__uint_as_float(v[q])) : "memory");
                }
                if (warp == 4) AF_FSTAMP(4, n, hf * 4 + 3);
            }
        }
    } else if (warp >= 8) {
        // ------------------------------------------------------------ gradient warpgroups (one TMEM lane = key row per thread)
        setmaxnreg_inc<kFusedGradRegs>();
        const int gtid = threadIdx.x - 256;
        const int hf = gtid >> 7;                    // column half (64 streamed rows) owned by this warpgroup
        const int tid = gtid & 127;
        const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tb = tmem_base + lane_addr;
        const int xrow = x0 + tid;                   // key row j
        const bool alibi = p.slopes != nullptr;
        constexpr float kLog2e = 1.4426950408889634f;
        const uint32_t ds_row_addr = smem_u32(sDS + hf * L::DS_HALF) + static_cast<uint32_t>(tid) * 128;
        bool ok = true;
        // per-column statistics of the streamed query tile; the loads for tile n + 1 are issued at the top of
        // iteration n and stored to the other buffer after its passes (off the warpgroup's loop-carried chain).
        // Nothing touches the loaded registers before store_stats: any arithmetic at the load would make the warp
        // sit out the load's latency in front of the wait for S^T (measured: 1.1 k cycles per tile).
        float nx_l = 0.f, nx_d = 0.f, nx_slope = 0.f;
        bool nx_in = false;
        int nx_a0 = 0;
        Cursor cur = first;
        auto load_stats = [&]() {   // of the tile under the cursor, which then moves on
            const int ah = cur.head, a0 = row0_of(cur);
            advance(cur);
            nx_a0 = a0;
            if (tid < 64) {
                const int qi = a0 + hf * 64 + tid;
                const size_t r = (static_cast<size_t>(b) * p.Hq + ah) * p.S + min(qi, p.S - 1);
                nx_in = qi < p.S;
                nx_l = p.lse[r];
                nx_d = p.delta[r];
            }
            if (alibi) nx_slope = p.slopes[ah];
        };
        auto store_stats = [&](int n) {
            if (tid < 64) {
                float* dst = sStats + (n & 1) * 256 + hf * 64 + tid;
                dst[0] = nx_in ? -nx_l * kLog2e : -INFINITY;   // kept negated
                dst[128] = nx_in ? -nx_d : 0.f;
            }
        };
        if (n_it > 0) {
            load_stats();
            store_stats(0);
        }
        for (int n = 0; ok && n < n_it; ++n) {
            const int a0 = nx_a0;
            float* sL2 = sStats + (n & 1) * 256;
            float* sDl = sL2 + 128;
            const float my_slope2 = nx_slope * kLog2e;
            if (n + 1 < n_it) load_stats();
            const bool need_mask = tile_needs_mask(ms, a0, x0);
            int mlo = 0;
            uint32_t mn = 128;
            if (need_mask) kept_queries_of_key(ms, xrow, a0, mlo, mn);
            const float sb = -my_slope2;
            const float bias_base = sb * static_cast<float>(a0 - xrow);
            // the previous tile's dS^T half must have been consumed by both MMAs that read it
            if ((warp & 3) == 0) AF_FSTAMP(2 + hf, n, 0);
            ok = bar_all(ok && mbar_wait(&bars[L::B_SFULL + hf], n & 1, abort_flag, 51), 1 + hf, 128);
            if (!ok) break;
            if ((warp & 3) == 0) AF_FSTAMP(2 + hf, n, 1);
            tc_fence_after_sync();
            // both 32-column chunks are requested up front; the second one lands while the first is worked on
            uint32_t pe_keep[64];
            tmem_ld32(tb + T1 + hf * 64, pe_keep);
            tmem_wait_ld();
            tmem_ld32(tb + T1 + hf * 64 + 32, pe_keep + 32);
#pragma unroll
            for (int qt = 0; qt < 2; ++qt) {
                const int col0 = hf * 64 + qt * 32;
                const uint32_t out_col = hf * 64 + qt * 16;
                const float cbias = fmaf(sb, static_cast<float>(col0), bias_base);
                if (qt == 1) tmem_wait_ld();
                if (alibi) {
                    if (need_mask) grad_phase_p32<true, true>(tb + T1, col0, out_col, p.scale_log2, cbias, sb, sL2, mlo, mn, pe_keep + qt * 32);
                    else grad_phase_p32<false, true>(tb + T1, col0, out_col, p.scale_log2, cbias, sb, sL2, mlo, mn, pe_keep + qt * 32);
                } else {
                    if (need_mask) grad_phase_p32<true, false>(tb + T1, col0, out_col, p.scale_log2, cbias, sb, sL2, mlo, mn, pe_keep + qt * 32);
                    else grad_phase_p32<false, false>(tb + T1, col0, out_col, p.scale_log2, cbias, sb, sL2, mlo, mn, pe_keep + qt * 32);
                }
            }
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars[L::B_PRDY + hf]);
            if ((warp & 3) == 0) AF_FSTAMP(2 + hf, n, 2);
            // the previous tile's dS^T half must have been consumed by both MMAs that read it
            ok = mbar_wait(&bars[L::B_DSFREE + hf], (n & 1) ^ 1, abort_flag, 50);
            // (the vote keeps the warpgroup together: a warp that gave up must not leave the others at the barrier above)
            ok = bar_all(ok && mbar_wait(&bars[L::B_DPFULL + hf], n & 1, abort_flag, 53), 1 + hf, 128);
            if (!ok) break;
            if ((warp & 3) == 0) AF_FSTAMP(2 + hf, n, 3);
            tc_fence_after_sync();
            uint32_t dp[64];
            tmem_ld32(tb + T2 + hf * 64, dp);
            tmem_wait_ld();
            tmem_ld32(tb + T2 + hf * 64 + 32, dp + 32);
            grad_phase_ds32(dp, hf * 64, sDl, pe_keep, ds_row_addr, tid & 7, 0);
            tmem_wait_ld();
            grad_phase_ds32(dp + 32, hf * 64 + 32, sDl, pe_keep + 32, ds_row_addr, tid & 7, 4);
            fence_proxy_async_smem();   // dS^T in shared memory is read by the tensor core's asynchronous proxy
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars[L::B_PDS + hf]);
            if ((warp & 3) == 0) AF_FSTAMP(2 + hf, n, 4);
            if (n + 1 < n_it) store_stats(n + 1);   // (published by the named barrier at the top of the next iteration)
        }
        // (every thread of both warpgroups takes this barrier, also after a wait that gave up in one of them:
        // a warpgroup that left its loop early must not leave the other alone at it)
        ok = wg_all(ok && (n_it <= 0 || mbar_wait(&bars[L::B_DONE], 0, abort_flag, 52)));
        if (ok && n_it <= 0) {
            // no query tile sees this key tile: its gradient rows are zero
            const size_t row0 = (static_cast<size_t>(b) * p.Hkv + xh) * p.S + x0;
            const int rows = min(128, p.S - x0);
            for (int idx = gtid; idx < rows * (D / 4); idx += 256) {
                const size_t off = (row0 + idx / (D / 4)) * D + (idx % (D / 4)) * 4;
                for (int w2 = 0; w2 < 2; ++w2) {
                    void* out = w2 == 0 ? p.out1 : p.out2;
                    if (p.out_f32) *reinterpret_cast<float4*>(static_cast<float*>(out) + off) = make_float4(0.f, 0.f, 0.f, 0.f);
                    else *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(out) + off) = make_uint2(0u, 0u);
                }
            }
        }
        if (ok && n_it > 0) {
            tc_fence_after_sync();
            float* stg = reinterpret_cast<float*>(sA);
            const size_t out_row0 = (static_cast<size_t>(b) * p.Hkv + xh) * p.S + x0;
            store_acc_rotated<D>(tb + ACC1, stg, gtid, 1.f, 0, p.table, x0, p.S, p.out1, out_row0, p.out_f32);
            store_acc_rotated<D>(tb + ACC2, stg, gtid, p.scale, p.R, p.table, x0, p.S, p.out2, out_row0, p.out_f32);
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// dQ = c * R^T(accumulated dQ'): fp32 accumulator [rows][D] -> the caller's dQ (bf16 or fp32), rows = B * Hq * S in
// [B, Hq, S] order.  One thread per four columns below R / 2 together with their partners above (or four
// unrotated columns).  HBM bound: 4 + 2 (or 4) bytes per element.
template <int D>
__global__ void __launch_bounds__(256) bwd_dq_finish_kernel(const float* __restrict__ acc, void* __restrict__ out, int out_f32,
                                                            const float2* __restrict__ table, int S, int R, float scale,
                                                            long long rows) {
    grid_dep_wait();
    grid_dep_launch();
    constexpr int TPR = D / 4;
    const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
    const long long row = idx / TPR;
    if (row >= rows) return;
    const int d = static_cast<int>(idx % TPR) * 4;
    const int half = R >> 1;
    const float4 a = __ldcs(reinterpret_cast<const float4*>(acc + row * D + d));
    float4 y = make_float4(a.x * scale, a.y * scale, a.z * scale, a.w * scale);
    if (d < R) {
        const bool upper = d >= half;
        const int partner = upper ? d - half : d + half, fi = upper ? d - half : d;
        const float4 o = __ldcs(reinterpret_cast<const float4*>(acc + row * D + partner));
        const int pos = static_cast<int>(row % S);
        const float4 t01 = __ldg(reinterpret_cast<const float4*>(table + static_cast<size_t>(pos) * half + fi));
        const float4 t23 = __ldg(reinterpret_cast<const float4*>(table + static_cast<size_t>(pos) * half + fi + 2));
        const float sg = upper ? -scale : scale;   // transpose rotation: y c + other s below R / 2, y c - other s above
        y.x = fmaf(y.x, t01.x, o.x * sg * t01.y);
        y.y = fmaf(y.y, t01.z, o.y * sg * t01.w);
        y.z = fmaf(y.z, t23.x, o.z * sg * t23.y);
        y.w = fmaf(y.w, t23.z, o.w * sg * t23.w);
    }
    const size_t oi = static_cast<size_t>(row) * D + d;
    if (out_f32) *reinterpret_cast<float4*>(static_cast<float*>(out) + oi) = y;
    else *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(out) + oi) = make_uint2(pack_bf16x2(y.x, y.y), pack_bf16x2(y.z, y.w));
}

}  // namespace af
