// Backward pass, the first query rows of every head in fp32 (Section 4.4 algebra, same readings).
//
// Under a causal mask query row i sees i + 1 keys.  For the first few rows a probability is a large number
// that nothing averages, and the bf16 roundings of the tensor-core path (rotated q', k', P, dS, the bf16 O
// behind delta) reach the gradients of those rows and of the first key rows at full size: measured at the
// Llama-3-8B training shape they added up to 0.027 on dK of key row 0 against the fp64 definition, over
// the 2e-2 bound, while every row past the first dozen stays near 0.01.  The pairs (i, j) with
// i < kFirstRows are therefore taken out of the MMA kernels (their mask drops them) and computed here in
// plain fp32 arithmetic, from the bf16 inputs alone: rotation from the fp32 table, scores, max-shifted
// softmax, O and delta recomputed (not read back in bf16), dV, dP, dS, dK', dQ', transpose rotation.
//
// One CTA per (batch, kv head).  The query rows of up to four heads of the group are stacked into one
// [4 * kFirstRows, D] panel, so every product below is a small dense contraction over shared memory and the
// sums over the heads of the group happen in a fixed order: the result is run-to-run deterministic.
// The kernel runs after the two MMA kernels: it overwrites rows i < kFirstRows of dQ (which the dQ kernel
// wrote as zeros) and adds its part to rows j < kFirstRows of dK and dV.
#pragma once
#include "common.cuh"

namespace af {

constexpr int kFirstRows = 16;        // query rows per head computed here
constexpr int kFirstHeads = 4;        // heads of a group per panel

struct FirstRowsParams {
    int B, Hq, Hkv, S, group;
    int R, window, rows;               // rows = min(kFirstRows, S)
    float scale;
    const float* slopes;               // Hq ALiBi slopes or nullptr
    const float2* table;               // [S][R/2] {cos, sin}
    const __nv_bfloat16 *q, *k, *v, *d_o;
    long long qb, qh, qs, kb, kh, ks;  // element strides of q and of k / v (d_o is contiguous)
    void *dq, *dk, *dv;
    int dq_f32, dkv_f32;
};

template <int D>
struct FirstRowsSmem {
    static constexpr int PANEL = kFirstHeads * kFirstRows;                   // 64 stacked query rows
    static constexpr int LDK = D + 1;                                        // padded row of K' and V (bank spread)
    static constexpr int FLOATS = 2 * kFirstRows * LDK + 2 * kFirstRows * D + 3 * PANEL * D + 3 * PANEL * kFirstRows + PANEL +
                                  kFirstRows * D;   // ... + {cos, sin} of the first positions, [kFirstRows][R/2] float2
    static constexpr int BYTES = FLOATS * 4;
};

// y = R(pos)^(sign) x for one row held in shared memory (in place): columns d < R/2 pair with d + R/2.
// table: the {cos, sin} rows of the first positions, staged in shared memory.
__device__ __forceinline__ void first_rows_rotate(float* row, int R, const float2* table, int pos, float sign, int lane) {
    const int half = R >> 1;
    for (int i = lane; i < half; i += 32) {
        const float2 cs = table[pos * half + i];
        const float a = row[i], b = row[i + half], s = cs.y * sign;
        row[i] = a * cs.x - b * s;
        row[i + half] = b * cs.x + a * s;
    }
}

template <int D>
__global__ void __launch_bounds__(256) bwd_first_rows_kernel(const FirstRowsParams p) {
    using L = FirstRowsSmem<D>;
    constexpr int NR = kFirstRows, PANEL = L::PANEL, LDK = L::LDK;
    extern __shared__ float fr_smem[];
    float* Kp = fr_smem;                  // [NR][LDK] rotated keys
    float* Vs = Kp + NR * LDK;            // [NR][LDK]
    float* dKp = Vs + NR * LDK;           // [NR][D] gradient w.r.t. rotated keys
    float* dVs = dKp + NR * D;            // [NR][D]
    float* Qp = dVs + NR * D;             // [PANEL][D] rotated queries of the panel
    float* dOs = Qp + PANEL * D;          // [PANEL][D]
    float* dQp = dOs + PANEL * D;         // [PANEL][D] gradient w.r.t. rotated queries
    float* Ps = dQp + PANEL * D;          // [PANEL][NR] probabilities
    float* dPs = Ps + PANEL * NR;         // [PANEL][NR] dO . v
    float* dSs = dPs + PANEL * NR;        // [PANEL][NR]
    float* dl = dSs + PANEL * NR;         // [PANEL] delta
    float2* cs = reinterpret_cast<float2*>(dl + PANEL);   // [NR][R/2] {cos, sin} of positions 0 .. NR - 1

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int b = blockIdx.x / p.Hkv, hk = blockIdx.x % p.Hkv;
    const int rows = p.rows;              // query rows per head here = key rows they can see
    const __nv_bfloat16* kbase = p.k + b * p.kb + hk * p.kh;
    const __nv_bfloat16* vbase = p.v + b * p.kb + hk * p.kh;

    grid_dep_launch();
    // Every global read below is a 16-byte load issued in a batch before its first use: with one CTA per
    // (batch, kv head) the kernel is a chain of memory latencies, not of arithmetic.
    // {cos, sin} of the first positions (the table rows of positions 0 .. rows - 1 are contiguous)
    if (p.R > 0) {
        const int n4 = rows * (p.R >> 1) / 2;   // float4 = two {cos, sin} pairs; R / 2 is a multiple of 8
        for (int idx = tid; idx < n4; idx += 256)
            reinterpret_cast<float4*>(cs)[idx] = __ldg(reinterpret_cast<const float4*>(p.table) + idx);
    }
    // keys and values of the first rows (8 bf16 per load); gradients start at zero
    static_assert(NR * D / 8 == 256 || NR * D / 8 == 128, "one 16-byte chunk of K and of V per thread");
    if (tid < NR * D / 8) {
        const int j = tid / (D / 8), d = (tid % (D / 8)) * 8;
        uint4 kw = make_uint4(0u, 0u, 0u, 0u), vw = kw;
        if (j < rows) {
            kw = __ldg(reinterpret_cast<const uint4*>(kbase + j * p.ks + d));
            vw = __ldg(reinterpret_cast<const uint4*>(vbase + j * p.ks + d));
        }
        const uint32_t ka[4] = {kw.x, kw.y, kw.z, kw.w}, va[4] = {vw.x, vw.y, vw.z, vw.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            Kp[j * LDK + d + 2 * u] = bf16lo_to_f32(ka[u]);
            Kp[j * LDK + d + 2 * u + 1] = bf16hi_to_f32(ka[u]);
            Vs[j * LDK + d + 2 * u] = bf16lo_to_f32(va[u]);
            Vs[j * LDK + d + 2 * u + 1] = bf16hi_to_f32(va[u]);
        }
    }
    for (int idx = tid; idx < NR * D; idx += 256) {
        dKp[idx] = 0.f;
        dVs[idx] = 0.f;
    }
    __syncthreads();
    if (p.R > 0)
        for (int j = warp; j < rows; j += 8) first_rows_rotate(Kp + j * LDK, p.R, cs, j, 1.f, lane);
    __syncthreads();

    for (int h0 = 0; h0 < p.group; h0 += kFirstHeads) {
        const int nh = min(kFirstHeads, p.group - h0);
        const int prow = nh * NR;          // panel rows in use: r = hh * NR + i
        // 1. queries (rotated) and upstream gradients of the panel
        {
            constexpr int CH = PANEL * D / 8 / 256;   // 16-byte chunks per thread and array
            uint4 qw[CH], gw[CH];
#pragma unroll
            for (int c = 0; c < CH; ++c) {
                const int idx = (tid + c * 256) * 8;
                const int r = idx / D, d = idx - r * D, hh = r / NR, i = r - hh * NR;
                const int h = hk * p.group + h0 + hh;
                qw[c] = make_uint4(0u, 0u, 0u, 0u);
                gw[c] = qw[c];
                if (hh < nh && i < rows) {
                    qw[c] = __ldg(reinterpret_cast<const uint4*>(p.q + b * p.qb + h * p.qh + i * p.qs + d));
                    gw[c] = __ldg(reinterpret_cast<const uint4*>(p.d_o + ((static_cast<size_t>(b) * p.Hq + h) * p.S + i) * D + d));
                }
            }
#pragma unroll
            for (int c = 0; c < CH; ++c) {
                const int idx = (tid + c * 256) * 8;
                const uint32_t qa[4] = {qw[c].x, qw[c].y, qw[c].z, qw[c].w}, ga[4] = {gw[c].x, gw[c].y, gw[c].z, gw[c].w};
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    Qp[idx + 2 * u] = bf16lo_to_f32(qa[u]);
                    Qp[idx + 2 * u + 1] = bf16hi_to_f32(qa[u]);
                    dOs[idx + 2 * u] = bf16lo_to_f32(ga[u]);
                    dOs[idx + 2 * u + 1] = bf16hi_to_f32(ga[u]);
                }
            }
        }
        __syncthreads();
        if (p.R > 0)
            for (int r = warp; r < prow; r += 8)
                if (r % NR < rows) first_rows_rotate(Qp + r * D, p.R, cs, r % NR, 1.f, lane);
        __syncthreads();
        // 2. scores s_rj = c <q'_r, k'_j> + slope (j - i) for the kept pairs (j <= i, i - j <= window), and dP_rj = <dO_r, v_j>
        for (int idx = tid; idx < PANEL * NR; idx += 256) {
            const int r = idx / NR, j = idx - r * NR, hh = r / NR, i = r - hh * NR;
            float s = -INFINITY, dp = 0.f;
            if (hh < nh && i < rows && j <= i && (p.window < 0 || i - j <= p.window)) {
                float acc = 0.f;
                for (int d = 0; d < D; ++d) {
                    acc = fmaf(Qp[r * D + d], Kp[j * LDK + d], acc);
                    dp = fmaf(dOs[r * D + d], Vs[j * LDK + d], dp);
                }
                s = acc * p.scale;
                if (p.slopes) s += p.slopes[hk * p.group + h0 + hh] * static_cast<float>(j - i);
            }
            Ps[idx] = s;
            dPs[idx] = dp;
        }
        __syncthreads();
        // 3. max-shifted softmax per panel row (at most NR kept keys)
        if (tid < PANEL) {
            const int r = tid;
            float m = -INFINITY;
            for (int j = 0; j < NR; ++j) m = fmaxf(m, Ps[r * NR + j]);
            float l = 0.f;
            for (int j = 0; j < NR; ++j) {
                const float e = m == -INFINITY ? 0.f : expf(Ps[r * NR + j] - m);
                Ps[r * NR + j] = e;
                l += e;
            }
            const float inv = l > 0.f ? 1.f / l : 0.f;
            for (int j = 0; j < NR; ++j) Ps[r * NR + j] *= inv;
        }
        __syncthreads();
        // 4. delta_r = <dO_r, O_r> with O_r = sum_j P_rj v_j recomputed here; one warp per row
        for (int r = warp; r < PANEL; r += 8) {
            float part = 0.f;
            for (int d = lane; d < D; d += 32) {
                float o = 0.f;
                for (int j = 0; j < NR; ++j) o = fmaf(Ps[r * NR + j], Vs[j * LDK + d], o);
                part = fmaf(dOs[r * D + d], o, part);
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
            if (lane == 0) dl[r] = part;
        }
        __syncthreads();
        // 5. dS_rj = P_rj (dP_rj - delta_r)
        for (int idx = tid; idx < PANEL * NR; idx += 256) dSs[idx] = Ps[idx] * (dPs[idx] - dl[idx / NR]);
        __syncthreads();
        // 6. dV_j += sum_r P_rj dO_r,  dK'_j += c sum_r dS_rj q'_r   (panel rows in order: fixed summation order)
        for (int idx = tid; idx < NR * D; idx += 256) {
            const int j = idx / D, d = idx - j * D;
            float av = 0.f, ak = 0.f;
            for (int r = 0; r < prow; ++r) {
                av = fmaf(Ps[r * NR + j], dOs[r * D + d], av);
                ak = fmaf(dSs[r * NR + j], Qp[r * D + d], ak);
            }
            dVs[idx] += av;
            dKp[idx] += ak * p.scale;
        }
        //    dQ'_r = c sum_j dS_rj k'_j
        for (int idx = tid; idx < PANEL * D; idx += 256) {
            const int r = idx / D, d = idx - r * D;
            float a = 0.f;
            for (int j = 0; j < NR; ++j) a = fmaf(dSs[r * NR + j], Kp[j * LDK + d], a);
            dQp[idx] = a * p.scale;
        }
        __syncthreads();
        // 7. dQ_r = R(i)^T dQ'_r, written over the zeros the dQ kernel left in these rows
        if (p.R > 0)
            for (int r = warp; r < prow; r += 8)
                if (r % NR < rows) first_rows_rotate(dQp + r * D, p.R, cs, r % NR, -1.f, lane);
        __syncthreads();
        grid_dep_wait();   // (first use of an output: the MMA kernels before this one in the stream are complete)
        for (int idx = tid * 4; idx < PANEL * D; idx += 256 * 4) {
            const int r = idx / D, d = idx - r * D, hh = r / NR, i = r - hh * NR;
            if (hh < nh && i < rows) {
                const size_t off = ((static_cast<size_t>(b) * p.Hq + hk * p.group + h0 + hh) * p.S + i) * D + d;
                const float4 y = *reinterpret_cast<const float4*>(dQp + idx);
                if (p.dq_f32) *reinterpret_cast<float4*>(static_cast<float*>(p.dq) + off) = y;
                else *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(p.dq) + off) = make_uint2(pack_bf16x2(y.x, y.y), pack_bf16x2(y.z, y.w));
            }
        }
        __syncthreads();
    }
    // dK_j = R(j)^T dK'_j; both gradients are added to what the dK/dV kernel wrote for the later query rows
    if (p.R > 0)
        for (int j = warp; j < rows; j += 8) first_rows_rotate(dKp + j * D, p.R, cs, j, -1.f, lane);
    __syncthreads();
    grid_dep_wait();
    // four columns per thread and pass; both passes' loads are issued before the first add
    constexpr int PASSES = NR * D / 4 / 256;
    const size_t out_base = (static_cast<size_t>(b) * p.Hkv + hk) * p.S * D;   // rows j of this kv head are contiguous
    if (p.dkv_f32) {
        float4 ok[PASSES], ov[PASSES];
#pragma unroll
        for (int c = 0; c < PASSES; ++c) {
            const int idx = (tid + c * 256) * 4;
            if (idx / D < rows) {
                ok[c] = *reinterpret_cast<const float4*>(static_cast<float*>(p.dk) + out_base + idx);
                ov[c] = *reinterpret_cast<const float4*>(static_cast<float*>(p.dv) + out_base + idx);
            }
        }
#pragma unroll
        for (int c = 0; c < PASSES; ++c) {
            const int idx = (tid + c * 256) * 4;
            if (idx / D < rows) {
                const float4 a = *reinterpret_cast<const float4*>(dKp + idx), g = *reinterpret_cast<const float4*>(dVs + idx);
                *reinterpret_cast<float4*>(static_cast<float*>(p.dk) + out_base + idx) =
                    make_float4(ok[c].x + a.x, ok[c].y + a.y, ok[c].z + a.z, ok[c].w + a.w);
                *reinterpret_cast<float4*>(static_cast<float*>(p.dv) + out_base + idx) =
                    make_float4(ov[c].x + g.x, ov[c].y + g.y, ov[c].z + g.z, ov[c].w + g.w);
            }
        }
    } else {
        uint2 ok[PASSES], ov[PASSES];
#pragma unroll
        for (int c = 0; c < PASSES; ++c) {
            const int idx = (tid + c * 256) * 4;
            if (idx / D < rows) {
                ok[c] = *reinterpret_cast<const uint2*>(static_cast<__nv_bfloat16*>(p.dk) + out_base + idx);
                ov[c] = *reinterpret_cast<const uint2*>(static_cast<__nv_bfloat16*>(p.dv) + out_base + idx);
            }
        }
#pragma unroll
        for (int c = 0; c < PASSES; ++c) {
            const int idx = (tid + c * 256) * 4;
            if (idx / D < rows) {
                const float4 a = *reinterpret_cast<const float4*>(dKp + idx), g = *reinterpret_cast<const float4*>(dVs + idx);
                *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(p.dk) + out_base + idx) =
                    make_uint2(pack_bf16x2(bf16lo_to_f32(ok[c].x) + a.x, bf16hi_to_f32(ok[c].x) + a.y),
                               pack_bf16x2(bf16lo_to_f32(ok[c].y) + a.z, bf16hi_to_f32(ok[c].y) + a.w));
                *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(p.dv) + out_base + idx) =
                    make_uint2(pack_bf16x2(bf16lo_to_f32(ov[c].x) + g.x, bf16hi_to_f32(ov[c].x) + g.y),
                               pack_bf16x2(bf16lo_to_f32(ov[c].y) + g.z, bf16hi_to_f32(ov[c].y) + g.w));
            }
        }
    }
}

}  // namespace af
