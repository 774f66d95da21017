// Fused forward kernel, CTA-pair variant (Sections 2 and 4.1) for GQA groups that are a multiple of 4.
//
// Two CTAs of a cluster (two SMs) work on the four query heads of one kv-head quad at the same 128
// query rows: CTA r owns heads 4u + 2r and 4u + 2r + 1 (its two query tiles).  All four tiles see the
// same K/V tiles, so every tcgen05.mma is issued once, by the leader CTA, over M = 256 (cta_group::2):
// each CTA supplies its own 128 rows of Q' (or P) and keeps its own 128 rows of the accumulator, and
// each supplies half of the B operand - 64 of the 128 key rows of K', 64 of the 128 columns of V.
// Per SM this halves the K/V bytes loaded, the K rows rotated (the O(N^2 D / BM) rotation term of
// Section 5.3) and the MMA instructions issued, compared with the one-CTA kernel in fwd_kernel.cuh.
//
// Roles per CTA as in fwd_kernel.cuh (producer warp, MMA warp - idle in the peer -, rotation warpgroup,
// one softmax warpgroup per query tile).  Barriers that the leader's MMA thread waits on collect
// arrivals from both CTAs (remote mbarrier arrive); MMA completion is multicast to both CTAs.
#pragma once
#include <cuda.h>
#include <type_traits>
#include "common.cuh"
#include "fwd_kernel.cuh"

namespace af {

template <int D, int KS, int VS>
struct Fwd2Smem {
    static constexpr int QTILE = 128 * D * 2;       // a query tile
    static constexpr int KHALF = 64 * D * 2;        // 64 key rows x D
    static constexpr int VHALF = 128 * 64 * 2;      // 128 key rows x 64 columns
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = OFF_Q + 2 * QTILE;
    static constexpr int OFF_V = OFF_K + KS * KHALF;
    static constexpr int OFF_BAR = OFF_V + VS * VHALF;
    static constexpr int B_QFULL = 0, B_KFULL = B_QFULL + 2, B_VFULL = B_KFULL + KS, B_KEMPTY = B_VFULL + VS,
                         B_VEMPTY = B_KEMPTY + KS, B_SFULL = B_VEMPTY + VS, B_ODONE = B_SFULL + 4,   // SFULL: two slots per tile (first used)
                         // consumed by the leader's MMA thread, arrivals from both CTAs:
                         B_QREADY = B_ODONE + 2, B_KREADY = B_QREADY + 2, B_VREADY = B_KREADY + KS,
                         B_PREADY = B_VREADY + VS, N_BARS = B_PREADY + 8;   // PREADY: up to four P parts per tile
    static constexpr int OFF_MISC = OFF_BAR + N_BARS * 8;
    static constexpr int BYTES = OFF_MISC + 16 + 1024;
};

// Byte offset of chunk `chunk` of row r in a K half tile: D/64 boxes of [64 rows][64 cols], 8 KB each.
__device__ __forceinline__ uint32_t swz_chunk_offset_khalf(int r, int chunk) {
    return static_cast<uint32_t>((chunk >> 3) * 8192 + r * 128 + (((chunk & 7) ^ (r & 7)) << 4));
}

// Rotate the 64 rows of a K half tile (positions row0 .. row0 + 63): thread (rg, cp) takes rows rg + 16 k, k < 4.
template <int CP>
__device__ __forceinline__ void rotate_khalf(uint8_t* tile, RotState<CP>& st, const RotStep& step, int tid) {
    constexpr int RP = 128 / CP;          // rows between a thread's rows (16 for CP = 8)
    constexpr int KC = 64 / RP;           // its rows in a half tile
    const int rg = tid / CP, cp = tid % CP;   // (st is consumed: the caller re-reads the table per tile)
#pragma unroll
    for (int k = 0; k < KC; ++k) {
        const int r = rg + RP * k;
        uint4* pl = reinterpret_cast<uint4*>(tile + swz_chunk_offset_khalf(r, cp));
        uint4* ph = reinterpret_cast<uint4*>(tile + swz_chunk_offset_khalf(r, cp + CP));
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

template <int D, bool ROPE, int KS, int VS>
__global__ void __launch_bounds__(512, 1)
attn_fwd2_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v, const FwdParams p) {
    static_assert(D == 128, "the CTA-pair kernel is built for head dim 128");
    using L = Fwd2Smem<D, KS, VS>;
    constexpr int NQ = 2;
    constexpr int NBOX = D / BOX_COLS;
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t IDESC_S = idesc_bf16_f32(256, BN, 0, 0);
    constexpr uint32_t IDESC_O = idesc_bf16_f32(256, D, 0, 1);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem + L::OFF_Q;
    uint8_t* sK = smem + L::OFF_K;
    uint8_t* sV = smem + L::OFF_V;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::OFF_MISC);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + L::OFF_MISC + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();     // 0: leader (issues the MMAs)
    const int unit = static_cast<int>(blockIdx.x) >> 1;      // (batch, head quad)
    const int quads = p.Hq / 4;
    const int b = unit / quads, uq = unit - b * quads;
    int hq[NQ];
#pragma unroll
    for (int q = 0; q < NQ; ++q) hq[q] = 4 * uq + 2 * static_cast<int>(rank) + q;
    const int hk = (4 * uq) / p.group;
    const int rb = p.n_row_blocks - 1 - static_cast<int>(blockIdx.y);   // heaviest row blocks first
    const int i0 = rb * BM;
    const MaskSpec ms{p.S, p.causal, p.window};
    int jlo, jhi;
    tile_range(ms, i0, jlo, jhi);
    const int n_it = jhi - jlo + 1;

    if (threadIdx.x == 0) {
        for (int i = 0; i < L::N_BARS; ++i) {
            uint32_t cnt = 1;
            if ((i >= L::B_QREADY && i < L::B_QREADY + 2) || (i >= L::B_KREADY && i < L::B_KREADY + KS) ||
                (i >= L::B_PREADY && i < L::B_PREADY + 8))
                cnt = 8;   // four warps of a warpgroup in each of the two CTAs
            if (i >= L::B_VREADY && i < L::B_VREADY + VS) cnt = 2;   // one relay thread per CTA
            mbar_init(&bars[i], cnt);
        }
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc2(tmem_slot, TMEM_COLS);
        tmem_relinquish2();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();            // both CTAs' barriers are initialised before anyone arrives remotely
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    // Per-warpgroup register budgets: one warp of each warpgroup per SM sub-partition, 64+96+176+176 = 512.
    if (warp < 4) setmaxnreg_dec<64>();
    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (this CTA's halves)
        if (lane == 0) {
            prefetch_tmap(&tm_q);
            prefetch_tmap(&tm_k);
            prefetch_tmap(&tm_v);
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                mbar_arrive_expect_tx(&bars[L::B_QFULL + q], L::QTILE);
#pragma unroll
                for (int bx = 0; bx < NBOX; ++bx)
                    tma_load_4d(sQ + q * L::QTILE + bx * BOX_BYTES, &tm_q, &bars[L::B_QFULL + q], bx * BOX_COLS, i0, hq[q], b);
            }
            for (int it = 0; it < n_it; ++it) {
                const int j0 = (jlo + it) * BN;
                const int ks = it % KS, vs = it % VS;
                if (!mbar_wait(&bars[L::B_KEMPTY + ks], ((it / KS) & 1) ^ 1, abort_flag, 41)) break;
                mbar_arrive_expect_tx(&bars[L::B_KFULL + ks], L::KHALF);
#pragma unroll
                for (int bx = 0; bx < NBOX; ++bx)   // key rows [64 rank, +64) of the tile
                    tma_load_4d(sK + ks * L::KHALF + bx * 8192, &tm_k, &bars[L::B_KFULL + ks], bx * BOX_COLS,
                                j0 + 64 * static_cast<int>(rank), hk, b);
                if (!mbar_wait(&bars[L::B_VEMPTY + vs], ((it / VS) & 1) ^ 1, abort_flag, 42)) break;
                mbar_arrive_expect_tx(&bars[L::B_VFULL + vs], L::VHALF);
                // columns [64 rank, +64) of all 128 key rows
                tma_load_4d(sV + vs * L::VHALF, &tm_v, &bars[L::B_VFULL + vs], 64 * static_cast<int>(rank), j0, hk, b);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only)
        if (lane == 0 && rank == 0) {
            bool ok = true;
            const uint32_t dhi = desc_hi(1024);
            auto issue_S = [&](int q, int ks) {
                const uint32_t q_lo = desc_lo(smem_u32(sQ + q * L::QTILE), 16), k_lo = desc_lo(smem_u32(sK + ks * L::KHALF), 16);
                const uint32_t d = tmem_base + q * BN;
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t qoff = ((kk >> 2) * BOX_BYTES + (kk & 3) * 32) >> 4;
                    const uint32_t koff = ((kk >> 2) * 8192 + (kk & 3) * 32) >> 4;
                    if (kk == 0) mma2_ss_lo<false>(d, q_lo + qoff, k_lo + koff, dhi, IDESC_S);
                    else mma2_ss_lo<true>(d, q_lo + qoff, k_lo + koff, dhi, IDESC_S);
                }
                mma2_commit_both(&bars[L::B_SFULL + 2 * q]);
            };
            auto issue_O_part = [&](int q, int vs, bool acc, int pt) {
                constexpr int KPP = 8 / kPParts;
                const uint32_t v_lo = desc_lo(smem_u32(sV + vs * L::VHALF), BOX_BYTES);
                const uint32_t d = tmem_base + NQ * BN + q * D, a = tmem_base + q * BN + pt * (BN / kPParts);
#pragma unroll
                for (int k = 0; k < KPP; ++k)
                    mma2_ts_lo(d, a + k * 8, v_lo + (pt * KPP + k) * 128, dhi, IDESC_O, (acc || pt > 0 || k > 0) ? 1u : 0u);
            };
            ok = mbar_wait_cluster(&bars[L::B_KREADY + 0], 0, abort_flag, 44);
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                if (ok) ok = mbar_wait_cluster(&bars[L::B_QREADY + q], 0, abort_flag, 43);
                tc_fence_after_sync();
                if (ok) issue_S(q, 0);
            }
            if (ok) mma2_commit_both(&bars[L::B_KEMPTY + 0]);
            for (int it = 0; ok && it < n_it; ++it) {
                const int vs = it % VS, ks1 = (it + 1) % KS;
                const bool next = it + 1 < n_it;
                bool kwaited = false;
                ok = mbar_wait_cluster(&bars[L::B_VREADY + vs], (it / VS) & 1, abort_flag, 45);
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
#pragma unroll
                    for (int pt = 0; pt < kPParts; ++pt) {
                        if (ok) ok = mbar_wait_cluster(&bars[L::B_PREADY + 4 * q + pt], it & 1, abort_flag, 46);
                        if (ok) {
                            tc_fence_after_sync();
                            issue_O_part(q, vs, it > 0, pt);
                        }
                    }
                    if (ok && !next) mma2_commit_both(&bars[L::B_ODONE + q]);
                    if (ok && next) {
                        if (!kwaited) {
                            ok = mbar_wait_cluster(&bars[L::B_KREADY + ks1], ((it + 1) / KS) & 1, abort_flag, 47);
                            tc_fence_after_sync();
                            kwaited = true;
                        }
                        if (ok) issue_S(q, ks1);
                    }
                }
                if (ok) {
                    mma2_commit_both(&bars[L::B_VEMPTY + vs]);
                    if (next) mma2_commit_both(&bars[L::B_KEMPTY + ks1]);
                }
            }
        }
    } else if (warp >= 4 && warp < 8) {
        // ------------------------------------------------------------ rotation warpgroup: this CTA's K halves
        setmaxnreg_dec<96>();
        const int t = threadIdx.x - 128;
        auto run = [&](auto cp_tag) {
            constexpr int CP = decltype(cp_tag)::value;   // chunk pairs per row; the pair kernel needs R in {16,32,64,128}
            constexpr int CPT = CP > 0 ? CP : 1;
            bool ok = true;
            RotStep step;
            RotState<CPT> st, nx;
            const int krow0 = jlo * BN + 64 * static_cast<int>(rank);
            if (ROPE) {
                rotate_load_step<CPT>(p.table, p.S, p.R, t, step);
                rotate_prefetch(st, p.table, krow0, p.S, p.R, t);
            }
            for (int it = 0; ok && it < n_it; ++it) {
                const int ks = it % KS, vs = it % VS;
                // cos/sin of the next tile's first rows are fetched one tile ahead
                if (ROPE && it + 1 < n_it) rotate_prefetch(nx, p.table, krow0 + (it + 1) * BN, p.S, p.R, t);
                ok = mbar_wait_warp(&bars[L::B_KFULL + ks], (it / KS) & 1, abort_flag, 48);
                if (!ok) break;
                if (ROPE) {
                    rotate_khalf<CPT>(sK + ks * L::KHALF, st, step, t);
                    fence_proxy_async_smem();
                    st = nx;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(&bars[L::B_KREADY + ks], 0);
                // relay: this CTA's half of V has landed
                if (warp == 4) {
                    ok = mbar_wait_warp(&bars[L::B_VFULL + vs], (it / VS) & 1, abort_flag, 49);
                    if (ok && lane == 0) mbar_arrive_cluster(&bars[L::B_VREADY + vs], 0);
                }
            }
        };
        if (p.R == 64) run(std::integral_constant<int, 4>{});
        else if (p.R == 32) run(std::integral_constant<int, 2>{});
        else if (p.R == 16) run(std::integral_constant<int, 1>{});
        else run(std::integral_constant<int, 8>{});   // R = 128, or no rotation (ROPE = false)
    } else if (warp >= 8) {
        // ------------------------------------------------------------ softmax warpgroups (one query row per thread)
        setmaxnreg_inc<176>();
        const int q = (warp - 8) >> 2;
        const int row = threadIdx.x - 256 - q * 128;            // == TMEM lane
        const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_base + lane_addr + q * BN;      // S (fp32) and, over it, P (bf16x2)
        const uint32_t tO = tmem_base + lane_addr + NQ * BN + q * D;
        const int i = i0 + row;
        const int bh = b * p.Hq + hq[q];
        const float slope2 = p.slopes ? p.slopes[hq[q]] * 1.4426950408889634f : 0.f;
        const bool alibi = p.slopes != nullptr;
        const float kb = slope2 / p.scale_log2;
        float m_run = -INFINITY, l_run = 0.f;
        bool ok = true;
        {
            // Section 4.1: the query tile is rotated once, before the key loop, by its softmax warpgroup
            auto rot_q = [&](auto cp_tag) {
                constexpr int CP = decltype(cp_tag)::value;
                RotStep step;
                RotState<CP> st;
                if (ROPE) {
                    rotate_load_step<CP>(p.table, p.S, p.R, row, step);
                    rotate_prefetch(st, p.table, i0, p.S, p.R, row);
                }
                ok = mbar_wait_warp(&bars[L::B_QFULL + q], 0, abort_flag, 50);
                if (!ok) return;
                if (ROPE) {
                    rotate_tile_fast(sQ + q * L::QTILE, st, step, row);
                    fence_proxy_async_smem();
                }
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(&bars[L::B_QREADY + q], 0);
            };
            if (p.R == 64) rot_q(std::integral_constant<int, 4>{});
            else if (p.R == 32) rot_q(std::integral_constant<int, 2>{});
            else if (p.R == 16) rot_q(std::integral_constant<int, 1>{});
            else rot_q(std::integral_constant<int, 8>{});
        }
        for (int it = 0; ok && it < n_it; ++it) {
            const int j0 = (jlo + it) * BN;
            const bool need_mask = tile_needs_mask(ms, i0, j0);
            const float bias0 = slope2 * static_cast<float>(j0 - i);
            int mlo = 0;
            uint32_t mn = BN;
            if (need_mask) kept_keys_of_query(ms, i, j0, mlo, mn);
            uint64_t* sf = &bars[L::B_SFULL + 2 * q];
            uint64_t* pr = &bars[L::B_PREADY + 4 * q];
            const int n = it;
            if (alibi) {
                if (need_mask) ok = softmax_tile_halves<D, true, true, true>(tS, tO, n, p.scale_log2, kb, bias0, mlo, mn, sf, pr, n & 1, abort_flag, lane, m_run, l_run);
                else ok = softmax_tile_halves<D, false, true, true>(tS, tO, n, p.scale_log2, kb, bias0, mlo, mn, sf, pr, n & 1, abort_flag, lane, m_run, l_run);
            } else {
                if (need_mask) ok = softmax_tile_halves<D, true, false, true>(tS, tO, n, p.scale_log2, kb, bias0, mlo, mn, sf, pr, n & 1, abort_flag, lane, m_run, l_run);
                else ok = softmax_tile_halves<D, false, false, true>(tS, tO, n, p.scale_log2, kb, bias0, mlo, mn, sf, pr, n & 1, abort_flag, lane, m_run, l_run);
            }
        }
        // epilogue (Section 4.4: save L = m + ln l)
        if (ok) ok = mbar_wait_warp(&bars[L::B_ODONE + q], 0, abort_flag, 52);
        if (ok) {
            tc_fence_after_sync();
            const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
            const size_t orow = (static_cast<size_t>(bh) * p.S + i) * D;
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
                uint32_t v[32];
                tmem_ld32(tO + c * 32, v);
                tmem_wait_ld();
                if (i < p.S) {
                    if (p.o_f32) {
                        float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.o) + orow + c * 32);
#pragma unroll
                        for (int e = 0; e < 32; e += 4)
                            dst[e >> 2] = make_float4(__uint_as_float(v[e]) * inv, __uint_as_float(v[e + 1]) * inv,
                                                      __uint_as_float(v[e + 2]) * inv, __uint_as_float(v[e + 3]) * inv);
                    } else {
                        uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.o) + orow + c * 32);
#pragma unroll
                        for (int e = 0; e < 32; e += 8)
                            dst[e >> 3] = make_uint4(
                                pack_bf16x2(__uint_as_float(v[e]) * inv, __uint_as_float(v[e + 1]) * inv),
                                pack_bf16x2(__uint_as_float(v[e + 2]) * inv, __uint_as_float(v[e + 3]) * inv),
                                pack_bf16x2(__uint_as_float(v[e + 4]) * inv, __uint_as_float(v[e + 5]) * inv),
                                pack_bf16x2(__uint_as_float(v[e + 6]) * inv, __uint_as_float(v[e + 7]) * inv));
                    }
                }
            }
            if (p.lse && i < p.S)
                p.lse[static_cast<size_t>(bh) * p.S + i] =
                    l_run > 0.f ? (m_run + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();   // neither CTA leaves while the other may still touch its shared memory, TMEM or barriers
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc2(tmem_base, TMEM_COLS);
    }
}

}  // namespace af
