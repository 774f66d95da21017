// Forward with 8-bit E4M3 operands (opt-in; the paper's Section 9.1 names fp8 tensor cores as the natural extension).
// Q and K arrive as E4M3 codes [B, H, S, D], V as E4M3 codes in the transposed layout [B, Hkv, D, S] (keys contiguous, so
// that both products read K-major operands), each with one dequantisation scale; no rotation inside (a caller rotates in
// bf16 and quantises afterwards).  S = Q K^T and O = P V run on `tcgen05.mma.kind::f8f6f4` (K = 32 per instruction, fp32
// accumulators in TMEM); the softmax is the fp32 one of the bf16 kernel; P goes back to TMEM as E4M3 (probabilities
// relative to the running reference, at most 2^8 with the lazy rescale, below the format's 448); the row sum adds the
// unrounded fp32 probabilities.  Same CTA layout as attn_fwd_kernel with two query tiles: warp 0 TMA producer, warp 1
// MMA issuer, warps 8-15 two softmax warpgroups (warps 4-7 idle: nothing to rotate).  D = 128, causal / window masks.
#pragma once
#include <cuda.h>
#include "fwd_kernel.cuh"

namespace af {

struct Fp8Params {
    int B, Hq, Hkv, S, group;
    int causal, window;
    float scale_log2;     // softmax scale x scale_q x scale_k x log2(e)
    float out_scale;      // scale_v
    void* o;              // [B, Hq, S, D] bf16 or fp32
    int o_f32;
    float* lse;           // nullable
    int pair_heads, n_row_blocks;
};

struct Fp8Smem {
    static constexpr int TILE = 128 * 128;        // 128 rows of 128 one-byte elements: one TMA box
    static constexpr int NQ = 2, KS = 2, VS = 2;
    static constexpr int OFF_Q = 0, OFF_K = OFF_Q + NQ * TILE, OFF_V = OFF_K + KS * TILE, OFF_BAR = OFF_V + VS * TILE;
    static constexpr int B_QFULL = 0, B_KFULL = B_QFULL + NQ, B_KEMPTY = B_KFULL + KS, B_VFULL = B_KEMPTY + KS,
                         B_VEMPTY = B_VFULL + VS, B_SFULL = B_VEMPTY + VS, B_PREADY = B_SFULL + NQ, B_ODONE = B_PREADY + 2 * NQ,
                         N_BARS = B_ODONE + NQ;
    static constexpr int OFF_MISC = OFF_BAR + N_BARS * 8;
    static constexpr int BYTES = OFF_MISC + 16 + 1024;
};

// Instruction descriptor for kind::f8f6f4 with E4M3 operands (format code 0 for A and B), fp32 accumulation, both
// operands K-major.
__host__ __device__ constexpr uint32_t idesc_e4m3_f32(int M, int N) {
    return (1u << 4) | (static_cast<uint32_t>(N >> 3) << 17) | (static_cast<uint32_t>(M >> 4) << 24);
}
template <bool ACC>
__device__ __forceinline__ void mma_f8_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc) {
    if (ACC)
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
            "setp.eq.b32 p, 0, 0;\n\ttcgen05.mma.cta_group::1.kind::f8f6f4 [%0], da, db, %4, p;\n\t}" ::"r"(d_tmem),
            "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc)
            : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
            "setp.ne.b32 p, 0, 0;\n\ttcgen05.mma.cta_group::1.kind::f8f6f4 [%0], da, db, %4, p;\n\t}" ::"r"(d_tmem),
            "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc)
            : "memory");
}
__device__ __forceinline__ void mma_f8_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\tmov.b64 db, {%2, %3};\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], [%1], db, %4, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t* r) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(taddr), "r"(r[0]), "r"(r[1]),
                 "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}
// four fp32 values -> four E4M3 codes in one word, element 0 in the lowest byte (round to nearest even, saturating)
__device__ __forceinline__ uint32_t pack_e4m3x4(float a, float b, float c, float d) {
    uint16_t lo, hi;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo) : "f"(b), "f"(a));   // first source -> upper byte
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi) : "f"(d), "f"(c));
    return static_cast<uint32_t>(lo) | (static_cast<uint32_t>(hi) << 16);
}

// One key tile of the online softmax for one query row, as softmax_tile_halves of the bf16 kernel (no ALiBi), with P
// written back as E4M3: a half of 64 probabilities takes 16 TMEM columns at the start of the half's own score columns.
template <bool MASKED>
__device__ __forceinline__ bool softmax_tile_fp8(uint32_t tS, uint32_t tO, int n, float scale_log2, int mlo, uint32_t mn,
                                                 uint64_t* s_full, uint64_t* p_ready, uint32_t parity,
                                                 volatile uint32_t* abort_flag, int lane, float& m_run, float& l_run) {
    uint32_t v[BN];
    if (!mbar_wait_warp(s_full, parity, abort_flag, 60)) return false;
    tc_fence_after_sync();
    tmem_ld32(tS, v);
    tmem_ld32(tS + 32, v + 32);
    tmem_ld32(tS + 64, v + 64);
    tmem_ld32(tS + 96, v + 96);
    tmem_wait_ld();
    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
    for (int e = 0; e < BN; e += 2) {
        float sv[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            sv[u] = __uint_as_float(v[e + u]);
            if (MASKED) {
                sv[u] = (static_cast<uint32_t>(e + u - mlo) < mn) ? sv[u] : -INFINITY;
                v[e + u] = __float_as_uint(sv[u]);
            }
        }
        mx4[(e >> 1) & 3] = fmax3(mx4[(e >> 1) & 3], sv[0], sv[1]);
    }
    const float mx = fmax3(fmaxf(mx4[0], mx4[1]), mx4[2], mx4[3]) * scale_log2;
    const bool upd = mx > m_run + kRescaleThreshold;
    float alpha = 1.f;
    if (upd) {
        alpha = ex2(m_run - mx);
        m_run = mx;
    }
    const float sub = -((m_run == -INFINITY) ? 0.f : m_run);
    const float2 sc2 = make_float2(scale_log2, scale_log2), sub2 = make_float2(sub, sub);
    float2 ps2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
    for (int pt = 0; pt < 2; ++pt) {
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            uint32_t pk[8];
            const int col0 = (pt * 2 + c) * 32;
#pragma unroll
            for (int e = 0; e < 32; e += 4) {
                const float2 t0 = __ffma2_rn(make_float2(__uint_as_float(v[col0 + e]), __uint_as_float(v[col0 + e + 1])), sc2, sub2);
                const float2 t1 = __ffma2_rn(make_float2(__uint_as_float(v[col0 + e + 2]), __uint_as_float(v[col0 + e + 3])), sc2, sub2);
                const float2 p0 = make_float2(ex2(t0.x), ex2(t0.y)), p1 = make_float2(ex2(t1.x), ex2(t1.y));
                ps2[0] = __fadd2_rn(ps2[0], p0);
                ps2[1] = __fadd2_rn(ps2[1], p1);
                pk[e >> 2] = pack_e4m3x4(p0.x, p0.y, p1.x, p1.y);
            }
            tmem_st8(tS + pt * 64 + c * 8, pk);
        }
        if (pt == 0 && n > 0 && __any_sync(0xffffffffu, upd)) {
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                uint32_t o[32];
                tmem_ld32(tO + c * 32, o);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                tmem_st32(tO + c * 32, o);
            }
        }
        tmem_wait_st();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_ready[pt]);
    }
    l_run = l_run * alpha + ((ps2[0].x + ps2[0].y) + (ps2[1].x + ps2[1].y));
    return true;
}

__global__ void __launch_bounds__(512, 1)
attn_fwd_fp8_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_vt, const Fp8Params p) {
    using L = Fp8Smem;
    constexpr int D = 128, NQ = L::NQ, KS = L::KS, VS = L::VS, TILE = L::TILE;
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t IDESC = idesc_e4m3_f32(BM, BN);   // S: N = 128 keys; O: N = D = 128

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *sQ = smem + L::OFF_Q, *sK = smem + L::OFF_K, *sV = smem + L::OFF_V;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::OFF_MISC);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + L::OFF_MISC + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int upb = p.pair_heads ? p.Hq / 2 : p.Hq;
    const int b = static_cast<int>(blockIdx.x) / upb, u = static_cast<int>(blockIdx.x) - b * upb;
    int hq[NQ];
#pragma unroll
    for (int q = 0; q < NQ; ++q) hq[q] = p.pair_heads ? 2 * u + q : u;
    const int hk = hq[0] / p.group;
    const int rb = p.n_row_blocks - 1 - static_cast<int>(blockIdx.y);   // heaviest row blocks first
    const MaskSpec ms{p.S, p.causal, p.window};
    int i0[NQ], jlo[NQ], jhi[NQ];
    int jlo_c = 0x7fffffff, jhi_c = -1;
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        i0[q] = p.pair_heads ? rb * BM : (rb * NQ + q) * BM;
        if (i0[q] < p.S) {
            tile_range(ms, i0[q], jlo[q], jhi[q]);
            jlo_c = min(jlo_c, jlo[q]);
            jhi_c = max(jhi_c, jhi[q]);
        } else {
            jlo[q] = 1;
            jhi[q] = 0;
        }
    }
    auto active = [&](int q, int j) { return j >= jlo[q] && j <= jhi[q]; };
    const int n_it = jhi_c - jlo_c + 1;

    if (threadIdx.x == 0) {
        for (int i = 0; i < L::N_BARS; ++i)
            mbar_init(&bars[i], (i >= L::B_PREADY && i < L::B_PREADY + 2 * NQ) ? 4 : 1);   // P: one arrive per warp
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

    if (warp < 8) setmaxnreg_dec<80>();
    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tmap(&tm_q);
            prefetch_tmap(&tm_k);
            prefetch_tmap(&tm_vt);
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                if (jhi[q] < jlo[q]) continue;
                mbar_arrive_expect_tx(&bars[L::B_QFULL + q], TILE);
                tma_load_4d(sQ + q * TILE, &tm_q, &bars[L::B_QFULL + q], 0, i0[q], hq[q], b);
            }
            for (int it = 0; it < n_it; ++it) {
                const int j0 = (jlo_c + it) * BN;
                const int ks = it % KS, vs = it % VS;
                if (!mbar_wait(&bars[L::B_KEMPTY + ks], ((it / KS) & 1) ^ 1, abort_flag, 61)) break;
                mbar_arrive_expect_tx(&bars[L::B_KFULL + ks], TILE);
                tma_load_4d(sK + ks * TILE, &tm_k, &bars[L::B_KFULL + ks], 0, j0, hk, b);
                if (!mbar_wait(&bars[L::B_VEMPTY + vs], ((it / VS) & 1) ^ 1, abort_flag, 62)) break;
                mbar_arrive_expect_tx(&bars[L::B_VFULL + vs], TILE);
                tma_load_4d(sV + vs * TILE, &tm_vt, &bars[L::B_VFULL + vs], j0, 0, hk, b);   // V^T: keys innermost
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int cnt[NQ];
            bool ok = true;
#pragma unroll
            for (int q = 0; q < NQ; ++q) cnt[q] = 0;
            const uint32_t dhi = desc_hi(1024);
            auto issue_S = [&](int q, int ks) {
                const uint32_t q_lo = desc_lo(smem_u32(sQ + q * TILE), 16), k_lo = desc_lo(smem_u32(sK + ks * TILE), 16);
                const uint32_t d = tmem_base + q * BN;
#pragma unroll
                for (int kk = 0; kk < D / 32; ++kk) {   // 32 one-byte elements = 32 bytes of the swizzled row per step
                    if (kk == 0) mma_f8_ss<false>(d, q_lo + kk * 2, k_lo + kk * 2, dhi, IDESC);
                    else mma_f8_ss<true>(d, q_lo + kk * 2, k_lo + kk * 2, dhi, IDESC);
                }
                mma_commit(&bars[L::B_SFULL + q]);
            };
            // half pt of O += P V: keys [64 pt, 64 pt + 64) = two K = 32 steps; P (E4M3) sits in 8 columns per step
            auto issue_O_part = [&](int q, int vs, bool acc, int pt) {
                const uint32_t v_lo = desc_lo(smem_u32(sV + vs * TILE), 16);
                const uint32_t d = tmem_base + NQ * BN + q * D, a = tmem_base + q * BN + pt * 64;
#pragma unroll
                for (int k = 0; k < 2; ++k)
                    mma_f8_ts(d, a + k * 8, v_lo + (pt * 2 + k) * 2, dhi, IDESC, (acc || pt > 0 || k > 0) ? 1u : 0u);
            };
            if (n_it <= 0) ok = false;
            if (ok) ok = mbar_wait(&bars[L::B_KFULL + 0], 0, abort_flag, 63);
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                if (ok && jhi[q] >= jlo[q]) {
                    ok = mbar_wait(&bars[L::B_QFULL + q], 0, abort_flag, 64);
                    tc_fence_after_sync();
                    if (ok && active(q, jlo_c)) issue_S(q, 0);
                }
            }
            if (ok) mma_commit(&bars[L::B_KEMPTY + 0]);
            for (int it = 0; ok && it < n_it; ++it) {
                const int j = jlo_c + it, vs = it % VS, ks1 = (it + 1) % KS;
                const bool next = it + 1 < n_it;
                bool kwaited = false;
                ok = mbar_wait(&bars[L::B_VFULL + vs], (it / VS) & 1, abort_flag, 65);
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    if (ok && active(q, j)) {
#pragma unroll
                        for (int pt = 0; pt < 2; ++pt) {
                            if (ok) ok = mbar_wait(&bars[L::B_PREADY + 2 * q + pt], cnt[q] & 1, abort_flag, 66);
                            if (ok) {
                                tc_fence_after_sync();
                                issue_O_part(q, vs, cnt[q] > 0, pt);
                            }
                        }
                        if (ok) {
                            ++cnt[q];
                            if (j == jhi[q]) mma_commit(&bars[L::B_ODONE + q]);
                        }
                    }
                    if (ok && next && active(q, j + 1)) {
                        if (!kwaited) {
                            ok = mbar_wait(&bars[L::B_KFULL + ks1], ((it + 1) / KS) & 1, abort_flag, 67);
                            tc_fence_after_sync();
                            kwaited = true;
                        }
                        if (ok) issue_S(q, ks1);
                    }
                }
                if (ok) {
                    mma_commit(&bars[L::B_VEMPTY + vs]);
                    if (next) mma_commit(&bars[L::B_KEMPTY + ks1]);
                }
            }
        }
    } else if (warp >= 8) {
        // ------------------------------------------------------------ softmax warpgroups (one query row per thread)
        setmaxnreg_inc<176>();
        const int q = (warp - 8) >> 2;
        const int row = threadIdx.x - 256 - q * 128;
        const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_base + lane_addr + q * BN;
        const uint32_t tO = tmem_base + lane_addr + NQ * BN + q * D;
        const int i = i0[q] + row;
        const int bh = b * p.Hq + hq[q];
        float m_run = -INFINITY, l_run = 0.f;
        bool ok = true;
        int n = 0;
        for (int j = jlo[q]; ok && j <= jhi[q]; ++j) {
            const int j0 = j * BN;
            const bool need_mask = tile_needs_mask(ms, i0[q], j0);
            int mlo = 0;
            uint32_t mn = BN;
            if (need_mask) kept_keys_of_query(ms, i, j0, mlo, mn);
            uint64_t* sf = &bars[L::B_SFULL + q];
            uint64_t* pr = &bars[L::B_PREADY + 2 * q];
            if (need_mask) ok = softmax_tile_fp8<true>(tS, tO, n, p.scale_log2, mlo, mn, sf, pr, n & 1, abort_flag, lane, m_run, l_run);
            else ok = softmax_tile_fp8<false>(tS, tO, n, p.scale_log2, mlo, mn, sf, pr, n & 1, abort_flag, lane, m_run, l_run);
            ++n;
        }
        if (ok && jhi[q] >= jlo[q]) ok = mbar_wait_warp(&bars[L::B_ODONE + q], 0, abort_flag, 68);
        if (ok && jhi[q] >= jlo[q]) {
            tc_fence_after_sync();
            const float inv = l_run > 0.f ? p.out_scale / l_run : 0.f;
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
                            dst[e >> 3] = make_uint4(pack_bf16x2(__uint_as_float(v[e]) * inv, __uint_as_float(v[e + 1]) * inv),
                                                     pack_bf16x2(__uint_as_float(v[e + 2]) * inv, __uint_as_float(v[e + 3]) * inv),
                                                     pack_bf16x2(__uint_as_float(v[e + 4]) * inv, __uint_as_float(v[e + 5]) * inv),
                                                     pack_bf16x2(__uint_as_float(v[e + 6]) * inv, __uint_as_float(v[e + 7]) * inv));
                    }
                }
            }
            if (p.lse && i < p.S)
                p.lse[static_cast<size_t>(bh) * p.S + i] = l_run > 0.f ? (m_run + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace af
