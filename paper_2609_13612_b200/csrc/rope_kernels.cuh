// Bandwidth-class kernels: the cos/sin table (set-up of Section 4.1) and the separate RoPE pass
// (the pre-rotation arm of Section 5.3).
#pragma once
#include "common.cuh"

namespace af {

// table[s][i] = {cos, sin}((p0 + s) * theta^(-2i/R)); the angle is formed in fp64 so that large
// positions do not lose the fraction of a turn, then rounded to fp32.  One trailer row [S][i] holds
// {cos, sin}(stride * theta^(-2i/R)), the constant the fused kernels use to walk from row to row.
__global__ void rope_table_kernel(float2* __restrict__ table, __nv_bfloat16* __restrict__ table_bf16, int S, int R,
                                  double theta, int p0) {
    const int half = R >> 1;
    const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
    if (idx >= static_cast<long long>(S + 1) * half) return;
    const int s = static_cast<int>(idx / half), i = static_cast<int>(idx - static_cast<long long>(s) * half);
    const double freq = pow(theta, -2.0 * static_cast<double>(i) / static_cast<double>(R));
    const double pos = s < S ? static_cast<double>(p0 + s) : static_cast<double>(rope_fast_stride(R));
    double sn, cs;
    sincos(pos * freq, &sn, &cs);
    table[idx] = make_float2(static_cast<float>(cs), static_cast<float>(sn));
    if (s < S) {   // bf16 copy, row layout [R/2 cos | R/2 sin]
        table_bf16[static_cast<size_t>(s) * R + i] = __float2bfloat16_rn(static_cast<float>(cs));
        table_bf16[static_cast<size_t>(s) * R + half + i] = __float2bfloat16_rn(static_cast<float>(sn));
    }
}

// x [B, H, S, D] (element strides xb, xh, xs; D contiguous) -> y [B*H, S, D] contiguous, rows rotated by their position; NH = B * H.  One thread owns the 16-byte chunk pair
// (columns 8cp.., R/2+8cp..) of sequence row s for HPT consecutive heads, so the table entry is
// read once and reused; consecutive threads touch consecutive 16-byte chunks (coalesced).
// Chunks past R are copied when y != x.  sgn = -1 applies the transpose rotation.
template <int HPT>
__global__ void __launch_bounds__(256)
rope_apply_kernel(const uint4* x, uint4* y, const float2* __restrict__ table, int NH, int H, int S,
                  int D, int R, float sgn, long long xb, long long xh, long long xs) {
    // programmatic dependent launch, both ways: as a dependent (inside the backward sequence) wait for the
    // predecessor before touching memory; as a predecessor (of the hybrid forward or of a gradient kernel) let
    // the next grid be scheduled and run its set-up while this pass runs
    grid_dep_wait();
    grid_dep_launch();
    const int CP = R >> 4;                 // rotated chunk pairs per row
    const int PT = (D - R) >> 3;           // pass-through chunks per row
    const int per_row = CP + PT;
    const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
    if (idx >= static_cast<long long>(S) * per_row) return;
    const int s = static_cast<int>(idx / per_row), c = static_cast<int>(idx - static_cast<long long>(s) * per_row);
    const int h0 = blockIdx.y * HPT;
    const int row_chunks = D >> 3;
    // 16-byte chunk index of row s of flattened head h in the (possibly strided) input
    auto in_base = [&](int h) {
        return static_cast<size_t>(((h / H) * xb + (h % H) * xh + static_cast<long long>(s) * xs) >> 3);
    };
    if (c < CP) {
        const float4* tb = reinterpret_cast<const float4*>(table + static_cast<size_t>(s) * (R >> 1) + c * 8);
        float4 t0 = __ldg(tb), t1 = __ldg(tb + 1), t2 = __ldg(tb + 2), t3 = __ldg(tb + 3);
        t0.y *= sgn; t0.w *= sgn; t1.y *= sgn; t1.w *= sgn;
        t2.y *= sgn; t2.w *= sgn; t3.y *= sgn; t3.w *= sgn;
        uint4 lo[HPT], hi[HPT];
#pragma unroll
        for (int u = 0; u < HPT; ++u) {
            if (h0 + u < NH) {
                const size_t base = in_base(h0 + u);
                lo[u] = __ldcs(x + base + c);
                hi[u] = __ldcs(x + base + c + CP);
            }
        }
#pragma unroll
        for (int u = 0; u < HPT; ++u) {
            if (h0 + u < NH) {
                const size_t base = (static_cast<size_t>(h0 + u) * S + s) * row_chunks;
                rotate_word(lo[u].x, hi[u].x, t0.x, t0.y, t0.z, t0.w);
                rotate_word(lo[u].y, hi[u].y, t1.x, t1.y, t1.z, t1.w);
                rotate_word(lo[u].z, hi[u].z, t2.x, t2.y, t2.z, t2.w);
                rotate_word(lo[u].w, hi[u].w, t3.x, t3.y, t3.z, t3.w);
                y[base + c] = lo[u];
                y[base + c + CP] = hi[u];
            }
        }
    } else if (x != y) {
        const int cc = 2 * CP + (c - CP);
#pragma unroll
        for (int u = 0; u < HPT; ++u) {
            if (h0 + u < NH) {
                const size_t base = (static_cast<size_t>(h0 + u) * S + s) * row_chunks;
                y[base + cc] = __ldcs(x + in_base(h0 + u) + cc);
            }
        }
    }
}

}  // namespace af
