// Fused forward kernel (Sections 2 and 4.1): per CTA, NQ query tiles of 128 rows of one head.
//   TMA -> shared memory (128-byte swizzle) -> RoPE rotation in place -> tcgen05.mma S = Q'K'^T into
//   TMEM -> scale / ALiBi / mask / online softmax in registers (one query row per thread) ->
//   P (bf16) back into TMEM over S -> tcgen05.mma O += P V -> normalise, store O and L.
// Warp roles: warp 0 TMA producer, warp 1 MMA issuer (one elected thread each), warps 4-7 rotate
// Q once and every K tile, warps 8.. are one softmax warpgroup per query tile.
#pragma once
#include <cuda.h>
#include <type_traits>
#include "common.cuh"

namespace af {

struct FwdParams {
    int B, Hq, Hkv, S, group;
    int R;              // rotary dim (0: none)
    int causal, window;
    float scale_log2;   // softmax scale * log2(e)
    const float* slopes;  // Hq ALiBi slopes or nullptr
    const float2* table;  // [S][R/2] {cos, sin}
    void* o;
    int o_f32;
    float* lse;         // nullable
    int n_row_blocks;   // ceil(S / (128 * NQ)), or ceil(S / 128) with pair_heads
    int pair_heads;     // NQ = 2 only: the two query tiles are the same 128 rows of two heads of one kv group
    // Block-sparse attention (Section 4.3), BS kernels only: CSR lists of the active 128 x 128 blocks, row_ptr
    // [ceil(S/128) + 1] and col_idx [row_ptr[last]] (device).  The key loop walks a row block's list instead of
    // a contiguous tile range; the element mask (causal, window) still applies inside the listed tiles.
    const int* bs_row_ptr;
    const int* bs_col_idx;
    const int* bs_order;   // optional launch order of the row blocks (longest lists first), or nullptr
    // bs_rowpair (BS, NQ = 2, not pair_heads): the two query tiles of a CTA are the row blocks 2 rb and 2 rb + 1 of one
    // head, and bs_row_ptr / bs_col_idx / bs_order describe PAIRS of row blocks: the list of pair rb is the sorted union
    // of the two row blocks' lists, each entry = key block | (1 << 28 if row block 2 rb has it) | (1 << 29 if 2 rb + 1).
    int bs_rowpair;
    int keys_bf16;         // host-side choice of the TAB instantiation (packed-bf16 key rotation)
    int rot_k;             // ROPE kernels: 1 = rotate the key tiles on chip; 0 = the keys arrive rotated (hybrid
                           // arm of Section 5.3: K rotated once by a RoPE pass, only Q rotated in the kernel)
    // Section 3.1, additive_bias: fp32 bias[bb, hh, i, j] added to the scaled score (nullptr: none); element strides
    // of its batch and head extents (0 where the extent is 1 and the bias is broadcast), rows of S floats.
    const float* bias;
    long long bias_sb, bias_sh;
    int relu;              // Section 3.1, relu_attention: P = max(s, 0) / (kept pairs of the row) in place of the softmax
    // ALiBi by the tensor core (set by the host when the layout has room for the operand tiles, see FwdSmem::HAS_AX):
    // the term slope (j - i) is linear in the key column, so one more K step of the S product adds it - S += A B^T
    // with A = [kb_hi, kb_lo, 0 ...] in every query row and B = [e, e, 0 ...] in key row e (kb = slope / c split
    // into two bf16 values, e exact in bf16) - and the softmax warps run their plain straight-line code.
    int alibi_mma;
#ifdef AF_TRACE
    long long* trace;
#endif
};

template <int D, int NQ, int KS, int VS, bool TAB = false>
struct FwdSmem {
    static constexpr int TILE = 128 * D * 2;
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = OFF_Q + NQ * TILE;
    static constexpr int OFF_V = OFF_K + KS * TILE;
    // TAB: one stage for the bf16 cos/sin rows of a key tile's 128 positions ([R/2 cos | R/2 sin] per row, R <= D)
    static constexpr int OFF_T = OFF_V + VS * TILE;
    static constexpr int T_BYTES = TAB ? 128 * 2 * D : 0;
    static constexpr int OFF_BAR = OFF_T + T_BYTES;
    // barrier slots
    static constexpr int B_QFULL = 0, B_QROT = B_QFULL + NQ, B_KFULL = B_QROT + NQ, B_KROT = B_KFULL + KS,
                         B_KEMPTY = B_KROT + KS, B_VFULL = B_KEMPTY + KS, B_VEMPTY = B_VFULL + VS,
                         B_SFULL = B_VEMPTY + VS, B_PREADY = B_SFULL + 2 * NQ, B_ODONE = B_PREADY + 4 * NQ,   // SFULL: per column half; PREADY: per P part (up to 4)
                         B_TFULL = B_ODONE + NQ, B_TEMPTY = B_TFULL + 1, N_BARS = B_TEMPTY + 1;
    static constexpr int OFF_MISC = OFF_BAR + N_BARS * 8;
    // operand tiles of the ALiBi K step: [128 rows x 16 columns] bf16, K-major, no swizzle (core matrices of 8 rows x
    // 16 bytes; 128 bytes between the two core matrices of a row group, 256 bytes between row groups): one for the
    // key side, one per query tile.  Left out where they do not fit (the TAB variant's table stage takes the room).
    static constexpr int AX_TILE = 128 * 16 * 2;
    static constexpr int OFF_AX = (OFF_MISC + 16 + 127) / 128 * 128;
    static constexpr bool HAS_AX = OFF_AX + (NQ + 1) * AX_TILE + 1024 <= 232448;
    static constexpr int BYTES = (HAS_AX ? OFF_AX + (NQ + 1) * AX_TILE : OFF_MISC + 16) + 1024;  // + alignment slack
};

// Optional timeline instrumentation for tuning (compiled out unless AF_TRACE is defined): one CTA
// records SM-clock stamps per role, iteration and phase into a caller-provided buffer.
#ifdef AF_TRACE
#define AF_STAMP(role, it, ph)                                                                         \
    do {                                                                                               \
        if (p.trace && blockIdx.x == 0 && blockIdx.y == 0 && (threadIdx.x & 31) == 0 && (it) < 64)     \
            p.trace[((role) * 64 + (it)) * 8 + (ph)] = clock64();                                      \
    } while (0)
// fine-grained stamps inside softmax_tile: slots 3..7 of role 2 (query tile 0, warp 8 lane 0 only)
#define AF_STAMP_SM(ph)                                                                                \
    do {                                                                                               \
        if (g_trace && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 256 && n < 64)             \
            g_trace[(2 * 64 + n) * 8 + (ph)] = clock64();                                              \
    } while (0)
#else
#define AF_STAMP(role, it, ph) do { } while (0)
#define AF_STAMP_SM(ph) do { } while (0)
#endif

#ifdef AF_TRACE
__device__ long long* g_trace = nullptr;
#endif
constexpr float kRescaleThreshold = 8.0f;  // log2 units: O is rescaled only when the row max grows by more

constexpr int kPParts = 2;   // P is handed to the MMA issuer in two column halves (four parts, and an S tile produced as
                             // two N = 64 halves, measured slower)

// One key tile of the online softmax for one query row (this thread's TMEM lane): reads the 128
// raw scores, adds ALiBi and the mask in the raw domain, updates the running max and sum in the
// log2 domain, writes P (bf16) over S and, when the reference max moved, rescales O.
// MASKED / ALIBI select straight-line code: interior tiles carry no mask logic at all.
//   score (log2 domain) t_e = c2 * (S_e + kb * e) + bias0,  kb = slope2 / c2, bias0 = slope2 * (j0 - i)
// The work is handed over in column halves, so that less of it sits on the
// S-MMA -> softmax -> PV-MMA dependency chain of a query tile:
//  - P goes back in two halves, each announced on its own barrier (p_ready[0], p_ready[1]), so that the
//    first four K-steps of O += P V run while the second half of the exponentials is computed.
// P halves sit at the start of their own 64 score columns (bf16 pairs: 32 columns each).
// Returns false if a bounded wait gave up.
template <int D, bool MASKED, bool ALIBI>
__device__ __forceinline__ bool softmax_tile_halves(uint32_t tS, uint32_t tO, int n, float scale_log2, float kb,
                                                    float bias0, int mlo, uint32_t mn, uint64_t* s_full, uint64_t* p_ready,
                                                    uint32_t parity, volatile uint32_t* abort_flag, int lane, float& m_run,
                                                    float& l_run) {
    uint32_t v[BN];
    if (!mbar_wait_warp(&s_full[0], parity, abort_flag, 10)) return false;
    tc_fence_after_sync();
    tmem_ld32(tS, v);
    tmem_ld32(tS + 32, v + 32);
    tmem_ld32(tS + 64, v + 64);
    tmem_ld32(tS + 96, v + 96);
    tmem_wait_ld();
    AF_STAMP_SM(3);
    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
    for (int e = 0; e < BN; e += 2) {
        float sv[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            sv[u] = __uint_as_float(v[e + u]);
            if (ALIBI) sv[u] = fmaf(kb, static_cast<float>(e + u), sv[u]);
            if (MASKED) sv[u] = (static_cast<uint32_t>(e + u - mlo) < mn) ? sv[u] : -INFINITY;
            if (ALIBI || MASKED) v[e + u] = __float_as_uint(sv[u]);
        }
        mx4[(e >> 1) & 3] = fmax3(mx4[(e >> 1) & 3], sv[0], sv[1]);   // two scores per instruction
    }
    // scale > 0, so the max commutes with it
    const float mx = fmaf(fmax3(fmaxf(mx4[0], mx4[1]), mx4[2], mx4[3]), scale_log2, bias0);
    AF_STAMP_SM(4);
    // lazy rescale: keep the old reference max unless it grew by more than the threshold
    const bool upd = mx > m_run + kRescaleThreshold;
    float alpha = 1.f;
    if (upd) {
        alpha = ex2(m_run - mx);  // m_run = -inf -> 0
        m_run = mx;
    }
    const float sub = bias0 - ((m_run == -INFINITY) ? 0.f : m_run);
    const float2 sc2 = make_float2(scale_log2, scale_log2), sub2 = make_float2(sub, sub);
    float2 ps2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
    constexpr int CPP = 4 / kPParts;   // 32-column chunks per part
#pragma unroll
    for (int pt = 0; pt < kPParts; ++pt) {
#pragma unroll
        for (int c = 0; c < CPP; ++c) {
            uint32_t pk[16];
            const int col0 = (pt * CPP + c) * 32;
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
                // packed fp32: one instruction scales and shifts two scores, one adds two probabilities
                const float2 t = __ffma2_rn(make_float2(__uint_as_float(v[col0 + e]), __uint_as_float(v[col0 + e + 1])), sc2, sub2);
                const float2 pe = make_float2(ex2(t.x), ex2(t.y));
                ps2[(e >> 1) & 1] = __fadd2_rn(ps2[(e >> 1) & 1], pe);
                pk[e >> 1] = pack_bf16x2(pe.x, pe.y);
            }
            // a part's bf16 pairs sit at the start of the part's own score columns
            tmem_st16(tS + pt * (BN / kPParts) + c * 16, pk);
        }
        if (pt == 0 && n > 0 && __any_sync(0xffffffffu, upd)) {
            // the accumulator must be rescaled before the first part of P V is added to it
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
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
        if (pt == 0) AF_STAMP_SM(5);
    }
    l_run = l_run * alpha + ((ps2[0].x + ps2[0].y) + (ps2[1].x + ps2[1].y));
    AF_STAMP_SM(6);
    return true;
}

// The same step for the variants with an additive bias and / or the ReLU normaliser (Section 3.1: additive_bias,
// relu_attention): one straight implementation with the mask, ALiBi and the bias decided at run time, so that
// the variants above stay as they are.  Scores are formed in natural units, s = c S + slope (j - i) + bias_ij,
// masked pairs and pairs whose bias is -inf drop out.
//   softmax:  as above (running max and sum in the log2 domain, lazy rescale).
//   RELU:     P = max(s, 0), unnormalised; l_run counts the kept pairs of the row, and the epilogue's division by
//             l_run is the normalisation by the number of kept pairs.  m_run is not used.
// bias_row: this thread's row of the bias at the tile's first column (or nullptr); cols_ok: how many of the 128
// columns lie inside the sequence (loads stop there); vec: the row is 16-byte aligned.
template <int D, bool RELU>
__device__ __forceinline__ bool softmax_tile_general(uint32_t tS, uint32_t tO, int n, float scale_log2, float slope2,
                                                     int j0_minus_i, int mlo, uint32_t mn, const float* bias_row,
                                                     int cols_ok, bool vec, uint64_t* s_full, uint64_t* p_ready,
                                                     uint32_t parity, volatile uint32_t* abort_flag, int lane,
                                                     float& m_run, float& l_run) {
    constexpr float kLog2e = 1.4426950408889634f;
    uint32_t v[BN];
    if (!mbar_wait_warp(&s_full[0], parity, abort_flag, 10)) return false;
    tc_fence_after_sync();
    tmem_ld32(tS, v);
    tmem_ld32(tS + 32, v + 32);
    tmem_ld32(tS + 64, v + 64);
    tmem_ld32(tS + 96, v + 96);
    tmem_wait_ld();
    // scores in the log2 domain: t = c2 S + slope2 (j - i) + log2(e) bias
    float mx = -INFINITY, cnt = 0.f;
#pragma unroll
    for (int e4 = 0; e4 < BN; e4 += 4) {
        float bv[4] = {0.f, 0.f, 0.f, 0.f};
        if (bias_row) {
            if (vec && e4 + 4 <= cols_ok) {
                const float4 b4 = __ldg(reinterpret_cast<const float4*>(bias_row + e4));
                bv[0] = b4.x; bv[1] = b4.y; bv[2] = b4.z; bv[3] = b4.w;
            } else {
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (e4 + u < cols_ok) bv[u] = __ldg(bias_row + e4 + u);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int e = e4 + u;
            float t = fmaf(__uint_as_float(v[e]), scale_log2, slope2 * static_cast<float>(j0_minus_i + e));
            t = fmaf(bv[u], kLog2e, t);
            const bool kept = static_cast<uint32_t>(e - mlo) < mn && t > -INFINITY;
            t = kept ? t : -INFINITY;
            v[e] = __float_as_uint(t);
            mx = fmaxf(mx, t);
            cnt += kept ? 1.f : 0.f;
        }
    }
    float alpha = 1.f;
    bool upd = false;
    if (!RELU) {
        upd = mx > m_run + kRescaleThreshold;
        if (upd) {
            alpha = ex2(m_run - mx);
            m_run = mx;
        }
    }
    const float ref = (m_run == -INFINITY) ? 0.f : m_run;
    float psum = 0.f;
    constexpr int CPP = 4 / kPParts;
#pragma unroll
    for (int pt = 0; pt < kPParts; ++pt) {
#pragma unroll
        for (int c = 0; c < CPP; ++c) {
            uint32_t pk[16];
            const int col0 = (pt * CPP + c) * 32;
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
                const float t0 = __uint_as_float(v[col0 + e]), t1 = __uint_as_float(v[col0 + e + 1]);
                float p0, p1;
                if (RELU) {   // back to natural units; a dropped pair (-inf) gives 0
                    p0 = fmaxf(t0 * 0.6931471805599453f, 0.f);
                    p1 = fmaxf(t1 * 0.6931471805599453f, 0.f);
                } else {
                    p0 = ex2(t0 - ref);
                    p1 = ex2(t1 - ref);
                    psum += p0 + p1;
                }
                pk[e >> 1] = pack_bf16x2(p0, p1);
            }
            tmem_st16(tS + pt * (BN / kPParts) + c * 16, pk);
        }
        if (!RELU && pt == 0 && n > 0 && __any_sync(0xffffffffu, upd)) {
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
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
    l_run = RELU ? l_run + cnt : l_run * alpha + psum;
    return true;
}

// TAB (with ROPE): key tiles are rotated in packed bf16 arithmetic from table tiles that arrive by TMA through
// tm_t (the bf16 copy of the cos/sin table); otherwise in fp32 arithmetic from the fp32 table rows.
// GEN: the instantiation for the variants with an additive bias or the ReLU normaliser (softmax_tile_general); kept
// apart so that the kernels of the other variants carry none of its registers.
template <int D, int NQ, bool ROPE, int KS, int VS, bool BS = false, bool TAB = false, bool GEN = false>
__global__ void __launch_bounds__(128 * (2 + NQ), 1)
attn_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                const __grid_constant__ CUtensorMap tm_t, const FwdParams p) {
    using L = FwdSmem<D, NQ, KS, VS, ROPE && TAB>;
    constexpr int TILE = L::TILE;
    constexpr int NBOX = D / BOX_COLS;
    constexpr uint32_t TMEM_COLS = (NQ * (BN + D) <= 256) ? 256u : 512u;
    constexpr uint32_t IDESC_S = idesc_bf16_f32(BM, BN, 0, 0);
    constexpr uint32_t IDESC_O = idesc_bf16_f32(BM, D, 0, 1);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem + L::OFF_Q;
    uint8_t* sK = smem + L::OFF_K;
    uint8_t* sV = smem + L::OFF_V;
    uint8_t* sT = smem + L::OFF_T;
    constexpr bool tab_tiles = ROPE && TAB;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::OFF_MISC);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + L::OFF_MISC + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // blockIdx.x: a head, or with pair_heads (even GQA group) a pair of adjacent heads that share a kv head.
    // Pairing heads gives both query tiles the same key range, so the two softmax warpgroups stay in
    // step down to the last tile; without it the tiles are rows [256 rb, +128) and [256 rb + 128, +128).
    const int upb = p.pair_heads ? p.Hq / 2 : p.Hq;   // units per batch
    const int b = static_cast<int>(blockIdx.x) / upb, u = static_cast<int>(blockIdx.x) - b * upb;
    int hq[NQ];
#pragma unroll
    for (int q = 0; q < NQ; ++q) hq[q] = p.pair_heads ? 2 * u + q : u;
    const int hk = hq[0] / p.group;
    // heaviest row blocks first: the last ones under a causal mask; with block lists the caller's order
    const int rb = (BS && p.bs_order) ? __ldg(p.bs_order + blockIdx.y) : p.n_row_blocks - 1 - static_cast<int>(blockIdx.y);
    const MaskSpec ms{p.S, p.causal, p.window};

    int i0[NQ], jlo[NQ], jhi[NQ];
    int jlo_c = 0x7fffffff, jhi_c = -1;
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        i0[q] = p.pair_heads ? rb * BM : (rb * NQ + q) * BM;   // (also the row-pair mode of the block lists)
        if (i0[q] < p.S) {
            tile_range(ms, i0[q], jlo[q], jhi[q]);
            jlo_c = min(jlo_c, jlo[q]);
            jhi_c = max(jhi_c, jhi[q]);
        } else {
            jlo[q] = 1;
            jhi[q] = 0;  // empty
        }
    }
    // Block-sparse: the loops below run over positions in the row block's list (jlo = 0, jhi = length - 1, the
    // same for both query tiles, which share the row block); tile_at() gives the key tile of a position.
    int bs_base = 0;
    int last_act[NQ];   // row-pair mode: last list position that is active for query tile q (-1: none)
#pragma unroll
    for (int q = 0; q < NQ; ++q) last_act[q] = -1;
    const bool rowpair = BS && NQ == 2 && p.bs_rowpair;
    if constexpr (BS) {
        bs_base = __ldg(p.bs_row_ptr + rb);
        const int first_row = rowpair ? rb * NQ * BM : rb * BM;
        const int len = (first_row < p.S) ? __ldg(p.bs_row_ptr + rb + 1) - bs_base : 0;
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
            jlo[q] = 0;
            jhi[q] = len - 1;
        }
        jlo_c = 0;
        jhi_c = len - 1;
        if (rowpair) {
            for (int pos = 0; pos < len; ++pos) {
                const int ent = __ldg(p.bs_col_idx + bs_base + pos);
#pragma unroll
                for (int q = 0; q < NQ; ++q)
                    if ((ent >> (28 + q)) & 1) last_act[q] = pos;
            }
#pragma unroll
            for (int q = 0; q < NQ; ++q)
                if (last_act[q] < 0 || i0[q] >= p.S) {   // nothing listed for this row block: treated as empty
                    jlo[q] = 1;
                    jhi[q] = 0;
                }
        }
    }
    auto tile_at = [&](int pos) { return BS ? (__ldg(p.bs_col_idx + bs_base + pos) & 0x0fffffff) : pos; };
    // is list position / key tile j part of query tile q's work?
    auto active = [&](int q, int j) {
        if (rowpair) return jhi[q] >= jlo[q] && ((__ldg(p.bs_col_idx + bs_base + j) >> (28 + q)) & 1) != 0;
        return j >= jlo[q] && j <= jhi[q];
    };
    auto is_last = [&](int q, int j) { return rowpair ? j == last_act[q] : j == jhi[q]; };
    const int n_it = jhi_c - jlo_c + 1;
    AF_STAMP(0, 63, 0);  // kernel entry

    if (threadIdx.x == 0) {
        for (int i = 0; i < L::N_BARS; ++i) {
            uint32_t cnt = 1;
            if ((i >= L::B_QROT && i < L::B_QROT + NQ) || (i >= L::B_KROT && i < L::B_KROT + KS) ||
                (i >= L::B_PREADY && i < L::B_PREADY + 4 * NQ) || i == L::B_TEMPTY)
                cnt = 4;  // one elected arrive per warp of the producing warpgroup
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

    // Register budget: the softmax warpgroups hold a full row of 128 scores; the others need little, but the
    // MMA issuer must not spill (it is the most latency-sensitive thread of the CTA: at 64 registers it spilled
    // and the kernel was 4 % slower), and the rotation warpgroup fits in 80.  80 + 80 + 2 x 176 = 512.
    constexpr int kSoftmaxRegs = NQ == 2 ? 176 : 232;
    constexpr int kIssuerRegs = 80, kRotRegs = 80;

    if (warp < 4) setmaxnreg_dec<kIssuerRegs>();
    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tmap(&tm_q);
            prefetch_tmap(&tm_k);
            prefetch_tmap(&tm_v);
            if (tab_tiles) prefetch_tmap(&tm_t);
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                if (jhi[q] < jlo[q]) continue;
                mbar_arrive_expect_tx(&bars[L::B_QFULL + q], TILE);
#pragma unroll
                for (int bx = 0; bx < NBOX; ++bx)
                    tma_load_4d(sQ + q * TILE + bx * BOX_BYTES, &tm_q, &bars[L::B_QFULL + q], bx * BOX_COLS, i0[q], hq[q], b);
            }
            // hybrid arm: the keys are written by the RoPE pass launched just before this grid, which may still be
            // running (programmatic dependent launch); everything above overlaps with its tail
            if (ROPE && !p.rot_k) grid_dep_wait();
            for (int it = 0; it < n_it; ++it) {
                const int j0 = tile_at(jlo_c + it) * BN;
                const int ks = it % KS, vs = it % VS;
                if (!mbar_wait(&bars[L::B_KEMPTY + ks], ((it / KS) & 1) ^ 1, abort_flag, 1)) break;
                mbar_arrive_expect_tx(&bars[L::B_KFULL + ks], TILE);
#pragma unroll
                for (int bx = 0; bx < NBOX; ++bx)
                    tma_load_4d(sK + ks * TILE + bx * BOX_BYTES, &tm_k, &bars[L::B_KFULL + ks], bx * BOX_COLS, j0, hk, b);
                if (tab_tiles) {
                    // the single table stage is free once the previous tile has been rotated
                    if (!mbar_wait(&bars[L::B_TEMPTY], (it & 1) ^ 1, abort_flag, 12)) break;
                    mbar_arrive_expect_tx(&bars[L::B_TFULL], 256u * p.R);
                    tma_load_2d(sT, &tm_t, &bars[L::B_TFULL], 0, j0);
                }
                if (!mbar_wait(&bars[L::B_VEMPTY + vs], ((it / VS) & 1) ^ 1, abort_flag, 2)) break;
                mbar_arrive_expect_tx(&bars[L::B_VFULL + vs], TILE);
#pragma unroll
                for (int bx = 0; bx < NBOX; ++bx)
                    tma_load_4d(sV + vs * TILE + bx * BOX_BYTES, &tm_v, &bars[L::B_VFULL + vs], bx * BOX_COLS, j0, hk, b);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        const bool alibi_mma = L::HAS_AX && !GEN && p.alibi_mma && p.slopes != nullptr;
        if (alibi_mma) {
            // the operand tiles of the ALiBi K step, written by this warp (its lane 0 issues every MMA that reads them)
            uint8_t* ax = smem + L::OFF_AX;
            for (int c = lane; c < (NQ + 1) * (L::AX_TILE / 16); c += 32) {
                const int tile = c / (L::AX_TILE / 16), cc = c % (L::AX_TILE / 16);
                const int r = (cc >> 4) * 8 + (cc & 7);      // 16-byte chunk cc: row group cc / 16, K half (cc / 8) % 2, row cc % 8
                uint32_t w0 = 0u;
                if (((cc >> 3) & 1) == 0) {
                    if (tile == 0) {
                        w0 = pack_bf16x2(static_cast<float>(r), static_cast<float>(r));
                    } else {
                        const float kb = p.slopes[tile == 1 ? hq[0] : hq[NQ - 1]] * 1.4426950408889634f / p.scale_log2;
                        const float hi = __bfloat162float(__float2bfloat16_rn(kb));
                        w0 = pack_bf16x2(hi, kb - hi);
                    }
                }
                *reinterpret_cast<uint4*>(ax + static_cast<size_t>(c) * 16) = make_uint4(w0, 0u, 0u, 0u);
            }
            fence_proxy_async_smem();
            __syncwarp();
        }
        if (lane == 0) {
            const int B_KREADY = (ROPE && p.rot_k) ? L::B_KROT : L::B_KFULL;
            constexpr int B_QREADY = ROPE ? L::B_QROT : L::B_QFULL;
            int cnt[NQ];
            bool ok = true;
#pragma unroll
            for (int q = 0; q < NQ; ++q) cnt[q] = 0;

            // descriptors differ only in their low word: one add per operand and step
            const uint32_t dhi = desc_hi(1024);
            auto issue_S = [&](int q, int ks) {
                const uint32_t q_lo = desc_lo(smem_u32(sQ + q * TILE), 16), k_lo = desc_lo(smem_u32(sK + ks * TILE), 16);
                const uint32_t d = tmem_base + q * BN;
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = ((kk >> 2) * BOX_BYTES + (kk & 3) * 32) >> 4;
                    if (kk == 0) mma_ss_lo<false>(d, q_lo + off, k_lo + off, dhi, IDESC_S);
                    else mma_ss_lo<true>(d, q_lo + off, k_lo + off, dhi, IDESC_S);
                }
                if (alibi_mma) {
                    const uint32_t ax = smem_u32(smem + L::OFF_AX);
                    mma_ss_lo<true>(d, desc_lo(ax + (1 + q) * L::AX_TILE, 128), desc_lo(ax, 128), desc_hi_noswizzle(256), IDESC_S);
                }
                mma_commit(&bars[L::B_SFULL + 2 * q]);
            };
            // part pt of O += P V: its 8 / kPParts K-steps; that part of P starts at its own score columns
            auto issue_O_part = [&](int q, int vs, bool acc, int pt) {
                constexpr int KPP = 8 / kPParts;
                const uint32_t v_lo = desc_lo(smem_u32(sV + vs * TILE), BOX_BYTES);
                const uint32_t d = tmem_base + NQ * BN + q * D, a = tmem_base + q * BN + pt * (BN / kPParts);
#pragma unroll
                for (int k = 0; k < KPP; ++k)
                    mma_ts_lo(d, a + k * 8, v_lo + (pt * KPP + k) * 128, dhi, IDESC_O, (acc || pt > 0 || k > 0) ? 1u : 0u);
            };

            // prologue: S of the first key tile, each query tile as soon as it is ready (the softmax
            // warpgroups rotate their Q tiles while the rotation warpgroup rotates K tile 0)
            if (BS && n_it <= 0) ok = false;   // a row block without active blocks: nothing to issue
            if (ok) ok = mbar_wait(&bars[B_KREADY + 0], 0, abort_flag, 4);
            AF_STAMP(0, 63, 3);  // first K ready
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                if (ok && jhi[q] >= jlo[q]) {
                    ok = mbar_wait(&bars[B_QREADY + q], 0, abort_flag, 3);
                    tc_fence_after_sync();
                    if (ok && active(q, jlo_c)) issue_S(q, 0);
                }
            }
            AF_STAMP(0, 63, 2);  // Q ready
            if (ok) mma_commit(&bars[L::B_KEMPTY + 0]);
            for (int it = 0; ok && it < n_it; ++it) {
                const int j = jlo_c + it, vs = it % VS, ks1 = (it + 1) % KS;
                const bool next = it + 1 < n_it;
                bool kwaited = false;
                AF_STAMP(0, it, 0);
                ok = mbar_wait(&bars[L::B_VFULL + vs], (it / VS) & 1, abort_flag, 5);
                AF_STAMP(0, it, 1);
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    if (ok && active(q, j)) {
#pragma unroll
                        for (int pt = 0; pt < kPParts; ++pt) {
                            if (ok) ok = mbar_wait(&bars[L::B_PREADY + 4 * q + pt], cnt[q] & 1, abort_flag, 6);
                            if (pt == 0) AF_STAMP(0, it, 2 + 3 * q);
                            if (ok) {
                                tc_fence_after_sync();
                                issue_O_part(q, vs, cnt[q] > 0, pt);
                            }
                        }
                        if (ok) {
                            AF_STAMP(0, it, 3 + 3 * q);
                            ++cnt[q];
                            if (is_last(q, j)) mma_commit(&bars[L::B_ODONE + q]);
                        }
                    }
                    if (ok && next && active(q, j + 1)) {
                        if (!kwaited) {
                            ok = mbar_wait(&bars[B_KREADY + ks1], ((it + 1) / KS) & 1, abort_flag, 7);
                            tc_fence_after_sync();
                            kwaited = true;
                        }
                        if (ok) issue_S(q, ks1);
                        AF_STAMP(0, it, 4 + 3 * q);
                    }
                }
                if (ok) {
                    mma_commit(&bars[L::B_VEMPTY + vs]);
                    if (next) mma_commit(&bars[L::B_KEMPTY + ks1]);
                }
            }
        }
    } else if (warp >= 4 && warp < 8) {
        // ------------------------------------------------------------ rotation warpgroup (Section 4.1)
        setmaxnreg_dec<kRotRegs>();
        if (ROPE && p.rot_k) {
            const int t = threadIdx.x - 128;
            // packed bf16 arithmetic on TMA-fed table tiles (rotary widths with a fast path)
            auto run_tab = [&](auto cp_tag) {
                constexpr int CP = decltype(cp_tag)::value;
                bool ok = true;
                for (int it = 0; ok && it < n_it; ++it) {
                    const int ks = it % KS;
                    AF_STAMP(1, it, 0);
                    ok = mbar_wait_warp(&bars[L::B_KFULL + ks], (it / KS) & 1, abort_flag, 9);
                    if (ok) ok = mbar_wait_warp(&bars[L::B_TFULL], it & 1, abort_flag, 13);
                    AF_STAMP(1, it, 1);
                    if (!ok) break;
                    rotate_tile_tab<CP>(sK + ks * TILE, sT, t);
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(&bars[L::B_KROT + ks]);
                        mbar_arrive(&bars[L::B_TEMPTY]);
                    }
                    AF_STAMP(1, it, 2);
                }
            };
            // fp32 arithmetic from the fp32 table rows
            auto run = [&](auto cp_tag) {
                constexpr int CP = decltype(cp_tag)::value;  // 0: generic path (table read per row)
                bool ok = true;
                RotStep step;
                RotState<(CP > 0 ? CP : 1)> st;
                if (CP > 0) rotate_load_step<(CP > 0 ? CP : 1)>(p.table, p.S, p.R, t, step);
                // (each Q tile is rotated by its own softmax warpgroup, which has nothing else to do yet)
                // K tiles are consecutive: the recurrence carries the cos/sin state from tile to tile
                for (int it = 0; ok && it < n_it; ++it) {
                    const int ks = it % KS;
                    // (listed tiles need not be consecutive: the cos/sin state is read for every tile)
                    if (CP > 0 && (BS || (it % kRotResync) == 0))
                        rotate_prefetch(st, p.table, tile_at(jlo_c + it) * BN, p.S, p.R, t);
                    AF_STAMP(1, it, 0);
                    ok = mbar_wait_warp(&bars[L::B_KFULL + ks], (it / KS) & 1, abort_flag, 9);
                    AF_STAMP(1, it, 1);
                    if (!ok) break;
                    if (CP > 0) rotate_tile_fast(sK + ks * TILE, st, step, t);
                    else rotate_tile_smem(sK + ks * TILE, tile_at(jlo_c + it) * BN, p.S, p.R, p.table, t, 128);
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars[L::B_KROT + ks]);
                    AF_STAMP(1, it, 2);
                }
            };
            if constexpr (tab_tiles) {
                if (p.R == 128) run_tab(std::integral_constant<int, 8>{});
                else if (p.R == 64) run_tab(std::integral_constant<int, 4>{});
                else if (p.R == 32) run_tab(std::integral_constant<int, 2>{});
                else run_tab(std::integral_constant<int, 1>{});
            } else if (p.R == 128) run(std::integral_constant<int, 8>{});
            else if (p.R == 64) run(std::integral_constant<int, 4>{});
            else if (p.R == 32) run(std::integral_constant<int, 2>{});
            else if (p.R == 16) run(std::integral_constant<int, 1>{});
            else run(std::integral_constant<int, 0>{});
        }
    } else if (warp >= 8) {
        // ------------------------------------------------------------ softmax warpgroups (one query row per thread)
        setmaxnreg_inc<kSoftmaxRegs>();
        const int q = (warp - 8) >> 2;
        const int row = threadIdx.x - 256 - q * 128;            // == TMEM lane
        const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_base + lane_addr + q * BN;      // S (fp32) and, over it, P (bf16x2)
        const uint32_t tO = tmem_base + lane_addr + NQ * BN + q * D;
        const int i = i0[q] + row;
        const int bh = b * p.Hq + hq[q];
        const float slope2 = p.slopes ? p.slopes[hq[q]] * 1.4426950408889634f : 0.f;
        // (with the ALiBi K step the scores arrive with the term already in them)
        const bool alibi = p.slopes != nullptr && !(L::HAS_AX && !GEN && p.alibi_mma);
        const float kb = slope2 / p.scale_log2;
        float m_run = -INFINITY, l_run = 0.f;
        bool ok = true;
        int n = 0;
        if (ROPE && jhi[q] >= jlo[q]) {
            // Section 4.1: the query tile is rotated once, before the key loop - by this warpgroup, which
            // would otherwise idle until the first scores arrive (the rotation warpgroup starts on K at once)
            auto rot_q = [&](auto cp_tag) {
                constexpr int CP = decltype(cp_tag)::value;
                constexpr int CPT = CP > 0 ? CP : 1;
                // (fp32 arithmetic: the query tile is rotated once, and every score inherits its rounding)
                RotStep step;
                RotState<CPT> st;
                if (CP > 0) {
                    rotate_load_step<CPT>(p.table, p.S, p.R, row, step);
                    rotate_prefetch(st, p.table, i0[q], p.S, p.R, row);
                }
                ok = mbar_wait_warp(&bars[L::B_QFULL + q], 0, abort_flag, 8);
                if (!ok) return;
                if (CP > 0) rotate_tile_fast(sQ + q * TILE, st, step, row);
                else rotate_tile_smem(sQ + q * TILE, i0[q], p.S, p.R, p.table, row, 128);
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars[L::B_QROT + q]);
            };
            if (p.R == 128) rot_q(std::integral_constant<int, 8>{});
            else if (p.R == 64) rot_q(std::integral_constant<int, 4>{});
            else if (p.R == 32) rot_q(std::integral_constant<int, 2>{});
            else if (p.R == 16) rot_q(std::integral_constant<int, 1>{});
            else rot_q(std::integral_constant<int, 0>{});
        }
        for (int j = jlo[q]; ok && j <= jhi[q]; ++j) {
            if (rowpair && !active(q, j)) continue;   // a listed block of the other row block only
            const int j0 = tile_at(j) * BN;
            AF_STAMP(2 + q, n, 0);
            const bool need_mask = tile_needs_mask(ms, i0[q], j0);
            const float bias0 = slope2 * static_cast<float>(j0 - i);
            int mlo = 0;
            uint32_t mn = BN;
            if (need_mask) kept_keys_of_query(ms, i, j0, mlo, mn);
            uint64_t* sf = &bars[L::B_SFULL + 2 * q];
            uint64_t* pr = &bars[L::B_PREADY + 4 * q];
            if constexpr (GEN) {
                // Section 3.1: additive_bias / relu_attention
                const float* brow = nullptr;
                if (p.bias && i < p.S)
                    brow = p.bias + b * p.bias_sb + hq[q] * p.bias_sh + static_cast<long long>(i) * p.S + j0;
                const int cols_ok = min(BN, p.S - j0);
                const bool vec = (p.S & 3) == 0 && (reinterpret_cast<uintptr_t>(p.bias) & 15u) == 0 &&
                                 (((b * p.bias_sb + hq[q] * p.bias_sh) & 3) == 0);
                if (p.relu) ok = softmax_tile_general<D, true>(tS, tO, n, p.scale_log2, slope2, j0 - i, mlo, mn, brow, cols_ok, vec, sf, pr, n & 1, abort_flag, lane, m_run, l_run);
                else ok = softmax_tile_general<D, false>(tS, tO, n, p.scale_log2, slope2, j0 - i, mlo, mn, brow, cols_ok, vec, sf, pr, n & 1, abort_flag, lane, m_run, l_run);
            } else if (alibi) {
                if (need_mask) ok = softmax_tile_halves<D, true, true>(tS, tO, n, p.scale_log2, kb, bias0, mlo, mn, sf, pr, n & 1, abort_flag, lane, m_run, l_run);
                else ok = softmax_tile_halves<D, false, true>(tS, tO, n, p.scale_log2, kb, bias0, mlo, mn, sf, pr, n & 1, abort_flag, lane, m_run, l_run);
            } else {
                if (need_mask) ok = softmax_tile_halves<D, true, false>(tS, tO, n, p.scale_log2, kb, bias0, mlo, mn, sf, pr, n & 1, abort_flag, lane, m_run, l_run);
                else ok = softmax_tile_halves<D, false, false>(tS, tO, n, p.scale_log2, kb, bias0, mlo, mn, sf, pr, n & 1, abort_flag, lane, m_run, l_run);
            }
            AF_STAMP(2 + q, n, 2);
            ++n;
        }
        // epilogue (Section 4.4: save L = m + ln l)
        if (ok && jhi[q] >= jlo[q]) ok = mbar_wait_warp(&bars[L::B_ODONE + q], 0, abort_flag, 11);
        AF_STAMP(2 + q, 63, 0);  // O complete
        if (ok && jhi[q] >= jlo[q]) {
            tc_fence_after_sync();
            const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
            const size_t orow = (static_cast<size_t>(bh) * p.S + i) * D;
            if (!p.o_f32) {
                // bf16 output: stage the tile in shared memory - in this query tile's own Q buffer, which no MMA
                // reads any more once O is complete, in the layout of the input tiles - and let TMA write it out.
                // (Row-per-thread global stores touch 32 rows per instruction and kept the load/store unit busy
                // for ~4 k cycles per CTA.)  Rows past S are clipped by the tensor map.
                uint8_t* stg = sQ + q * TILE;
#pragma unroll 1
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t v[32];
                    tmem_ld32(tO + c * 32, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; e += 8)
                        *reinterpret_cast<uint4*>(stg + swz_chunk_offset(row, c * 4 + (e >> 3))) = make_uint4(
                            pack_bf16x2(__uint_as_float(v[e]) * inv, __uint_as_float(v[e + 1]) * inv),
                            pack_bf16x2(__uint_as_float(v[e + 2]) * inv, __uint_as_float(v[e + 3]) * inv),
                            pack_bf16x2(__uint_as_float(v[e + 4]) * inv, __uint_as_float(v[e + 5]) * inv),
                            pack_bf16x2(__uint_as_float(v[e + 6]) * inv, __uint_as_float(v[e + 7]) * inv));
                }
                fence_proxy_async_smem();
                asm volatile("bar.sync %0, 128;" ::"r"(4 + q) : "memory");   // this warpgroup only
                if (row == 0) {
#pragma unroll
                    for (int bx = 0; bx < NBOX; ++bx)
                        tma_store_4d(&tm_o, stg + bx * BOX_BYTES, bx * BOX_COLS, i0[q], hq[q], b);
                    tma_store_commit();
                    tma_store_wait_read();   // the buffer must stay in place until it has been read
                }
            }
#pragma unroll 1
            for (int c = 0; p.o_f32 && c < D / 32; ++c) {
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
            if (p.lse && i < p.S) {
                // softmax: L = m + ln l; relu_attention: n_i, the number of kept pairs of the row (its normaliser)
                if (GEN && p.relu) p.lse[static_cast<size_t>(bh) * p.S + i] = l_run;
                else p.lse[static_cast<size_t>(bh) * p.S + i] = l_run > 0.f ? (m_run + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
            }
        }
        if (BS && ok && jhi[q] < jlo[q] && i < p.S) {
            // no active block in this row block: the output row is zero and L = -inf
            const size_t orow = (static_cast<size_t>(bh) * p.S + i) * D;
            if (p.o_f32) {
                float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.o) + orow);
                for (int e = 0; e < D / 4; ++e) dst[e] = make_float4(0.f, 0.f, 0.f, 0.f);
            } else {
                uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.o) + orow);
                for (int e = 0; e < D / 8; ++e) dst[e] = make_uint4(0u, 0u, 0u, 0u);
            }
            if (p.lse) p.lse[static_cast<size_t>(bh) * p.S + i] = -INFINITY;
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    AF_STAMP(0, 63, 1);  // all roles done
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace af
