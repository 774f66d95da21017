// Flash Decoding (Section 4.2 of the paper): one query position per head against a long KV cache.
//
// Phase 1 (decode_split_kernel): the cache is cut into splits; a CTA takes one split of one kv head
// and computes, for the g query heads of that kv head, a partial (m, l, acc) triple with the online
// softmax.  The g heads are the rows of a 16-row MMA tile (padded by cyclic replication, as the paper
// does), so K and V are read exactly once per CTA.  Phase 2 merges the partials with a log-sum-exp; it runs in
// the same launch, in the CTA that finishes last for its kv head (a ticket counter tells which).
//
// The path is bound by HBM (every K and V byte is read once and used for 4 g flops), so the kernel is
// built around the memory system: each of the 4 warps of a CTA streams its own 32-key tiles through
// its own ring of shared-memory stages with TMA (128-byte swizzle, an mbarrier per stage, no
// CTA-wide synchronisation in the loop), 128 KB in flight per SM.  The two small contractions per
// tile run on the warp-level tensor-core path (mma.sync m16n8k16 with ldmatrix fragments): at M = 16
// rows a tcgen05 tile of 128 rows would be 7/8 padding, and the arithmetic is far from the bound.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace af {

struct DecodeParams {
    int B, Hq, Hkv, N, group;   // N: keys in the cache; the query sits at position N - 1
    int window;                 // < 0: none; else keys j >= N - 1 - window are kept
    float scale_log2;           // softmax scale * log2(e)
    const float* slopes;        // Hq ALiBi slopes (bias m_h (j - (N - 1))) or nullptr
    const __nv_bfloat16* q;     // [B, Hq, D]
    float* part_o;              // [B * Hq, n_splits, D]   unnormalised partial outputs
    float* part_ml;             // [B * Hq, n_splits, 2]   running max (log2 units) and sum of each partial
    int n_splits;               // CTAs per (batch, kv head); the kept 32-key tiles are dealt out evenly among them
    // Merge in the same launch: one counter per (batch, kv head), zero before the launch.  The CTA that finishes
    // last for its kv head (it draws the last ticket) merges the partials of the g query heads, in split order,
    // writes o / lse and sets the counter back to zero.
    unsigned int* tickets;
    __nv_bfloat16* o;           // [B, Hq, D]
    float* lse;                 // [B, Hq] or nullptr
};

constexpr int kCombineThreads = 128;
constexpr int kCombineMaxSplits = 1024;
constexpr int kDecTile = 32;    // keys per warp tile
constexpr int kDecWarps = 4;
#ifndef AF_DEC_STAGES
#define AF_DEC_STAGES 3
#endif
constexpr int kDecStages = AF_DEC_STAGES;   // tiles in flight per warp

template <int D>
struct DecodeSmem {
    static constexpr int TILE_BYTES = kDecTile * D * 2;                      // one K or V tile
    static constexpr int WARP_BYTES = kDecStages * 2 * TILE_BYTES;           // [stage][K | V]
    static constexpr int OFF_BAR = kDecWarps * WARP_BYTES;
    static constexpr int OFF_MISC = OFF_BAR + kDecWarps * kDecStages * 8;
    static constexpr int BYTES = OFF_MISC + 16 + 1024;
    static constexpr int MERGE_STRIDE = D + 4;                               // floats per merged row
    static_assert(kDecWarps * 16 * (MERGE_STRIDE + 2) * 4 <= OFF_BAR, "merge buffer must fit in the stages");
    static_assert((16 * kCombineMaxSplits + 32) * 4 <= OFF_BAR, "combine weights (up to 16 heads) must fit in the stages");
};

// 16-byte chunk `chunk` of key row r in a tile of D/64 boxes [32 rows][64 cols], 128-byte swizzle
__device__ __forceinline__ uint32_t dec_chunk_offset(int r, int chunk) {
    return static_cast<uint32_t>((chunk >> 3) * (kDecTile * 128) + r * 128 + (((chunk & 7) ^ (r & 7)) << 4));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t* r) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t* r) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col)
__device__ __forceinline__ void mma_16816(float* d, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

template <int D>
__global__ void __launch_bounds__(kDecWarps * 32)
decode_split_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                    const DecodeParams p) {
    using L = DecodeSmem<D>;
    constexpr int TILE_BYTES = L::TILE_BYTES;
    constexpr int NBOX = D / 64, KSTEPS = D / 16, DT = D / 8;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + L::OFF_MISC);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int split = blockIdx.x;
    const int b = static_cast<int>(blockIdx.y) / p.Hkv, hk = static_cast<int>(blockIdx.y) - b * p.Hkv;
    const int qpos = p.N - 1;
    const int jmin = p.window >= 0 ? max(0, qpos - p.window) : 0;   // first kept key
    // tiles wholly before the window are skipped; the others are dealt out evenly (to within one tile)
    const int tile0 = jmin / kDecTile, tiles_all = (p.N + kDecTile - 1) / kDecTile - tile0;
    const int t_lo = static_cast<int>(static_cast<long long>(split) * tiles_all / p.n_splits);
    const int t_hi = static_cast<int>(static_cast<long long>(split + 1) * tiles_all / p.n_splits);
    const int k_lo = (tile0 + t_lo) * kDecTile;
    const int n_tiles = t_hi - t_lo;
    const int nt = n_tiles > warp ? (n_tiles - warp + kDecWarps - 1) / kDecWarps : 0;   // this warp's tiles

    if (threadIdx.x == 0) {
        for (int i = 0; i < kDecWarps * kDecStages; ++i) mbar_init(&bars[i], 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();

    uint8_t* wbase = smem + warp * L::WARP_BYTES;
    uint64_t* wbar = bars + warp * kDecStages;
    auto issue = [&](int i) {   // the i-th tile of this warp into stage i % kDecStages
        if (lane == 0) {
            const int st = i % kDecStages;
            const int key0 = k_lo + kDecTile * (warp + kDecWarps * i);
            uint8_t* dk = wbase + st * 2 * TILE_BYTES;
            mbar_arrive_expect_tx(&wbar[st], 2 * TILE_BYTES);
#pragma unroll
            for (int bx = 0; bx < NBOX; ++bx) {
                tma_load_4d(dk + bx * (kDecTile * 128), &tm_k, &wbar[st], bx * 64, key0, hk, b);
                tma_load_4d(dk + TILE_BYTES + bx * (kDecTile * 128), &tm_v, &wbar[st], bx * 64, key0, hk, b);
            }
        }
    };
    if (lane == 0 && nt > 0) {
        prefetch_tmap(&tm_k);
        prefetch_tmap(&tm_v);
    }
#pragma unroll
    for (int i = 0; i < kDecStages; ++i)
        if (nt > i) issue(i);

    // the g query heads of this kv head as the 16 rows of the A operand (row r <-> head r mod g)
    const int r0 = lane >> 2, r1 = r0 + 8;
    const int h0 = hk * p.group + r0 % p.group, h1 = hk * p.group + r1 % p.group;
    uint32_t qa[KSTEPS][4];
    {
        const uint32_t* q0 = reinterpret_cast<const uint32_t*>(p.q + (static_cast<size_t>(b) * p.Hq + h0) * D);
        const uint32_t* q1 = reinterpret_cast<const uint32_t*>(p.q + (static_cast<size_t>(b) * p.Hq + h1) * D);
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
            const int w = ks * 8 + (lane & 3);   // 32-bit word index: columns 16 ks + 2 (lane % 4)
            qa[ks][0] = __ldg(q0 + w);
            qa[ks][1] = __ldg(q1 + w);
            qa[ks][2] = __ldg(q0 + w + 4);
            qa[ks][3] = __ldg(q1 + w + 4);
        }
    }
    const float sl0 = p.slopes ? p.slopes[h0] * 1.4426950408889634f : 0.f;
    const float sl1 = p.slopes ? p.slopes[h1] * 1.4426950408889634f : 0.f;

    float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
    float o[DT][4];
#pragma unroll
    for (int i = 0; i < DT; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;

    bool ok = true;
    for (int i = 0; i < nt; ++i) {
        const int st = i % kDecStages;
        const int key0 = k_lo + kDecTile * (warp + kDecWarps * i);
        ok = mbar_wait_warp(&wbar[st], (i / kDecStages) & 1, abort_flag, 40);
        if (!ok) break;
        const uint32_t sk = smem_u32(wbase + st * 2 * TILE_BYTES), sv = sk + TILE_BYTES;

        // scores S[16 heads][32 keys] = Q K^T.  The fragment loads of the next step are issued before the
        // MMAs of the current one (the asm statements keep their order, so the overlap is written out).
        float s[4][4];
#pragma unroll
        for (int n8 = 0; n8 < 4; ++n8) s[n8][0] = s[n8][1] = s[n8][2] = s[n8][3] = 0.f;
        uint32_t kf[2][4][4];
        auto load_k = [&](int k2, uint32_t (*dst)[4]) {
            // per 8-key tile four 8x8 matrices: keys 8 n8 .. +7 (rows) x 32 head dims (four 16-byte chunks)
#pragma unroll
            for (int n8 = 0; n8 < 4; ++n8)
                ldmatrix_x4(sk + dec_chunk_offset(n8 * 8 + (lane & 7), k2 * 4 + (lane >> 3)), dst[n8]);
        };
        load_k(0, kf[0]);
#pragma unroll
        for (int k2 = 0; k2 < KSTEPS / 2; ++k2) {
            if (k2 + 1 < KSTEPS / 2) load_k(k2 + 1, kf[(k2 + 1) & 1]);
#pragma unroll
            for (int n8 = 0; n8 < 4; ++n8) {
                mma_16816(s[n8], qa[2 * k2], kf[k2 & 1][n8][0], kf[k2 & 1][n8][1]);
                mma_16816(s[n8], qa[2 * k2 + 1], kf[k2 & 1][n8][2], kf[k2 & 1][n8][3]);
            }
        }
        // log2-domain scores with bias and mask; thread holds rows r0 (e = 0, 1) and r1 (e = 2, 3)
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int n8 = 0; n8 < 4; ++n8) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int j = key0 + n8 * 8 + 2 * (lane & 3) + (e & 1);
                const float rel = static_cast<float>(j - qpos);
                float t = fmaf(s[n8][e], p.scale_log2, (e < 2 ? sl0 : sl1) * rel);
                t = (j < p.N && j >= jmin) ? t : -INFINITY;
                s[n8][e] = t;
                if (e < 2) mx0 = fmaxf(mx0, t);
                else mx1 = fmaxf(mx1, t);
            }
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        const float mn0 = fmaxf(m[0], mx0), mn1 = fmaxf(m[1], mx1);
        const float ms0 = mn0 == -INFINITY ? 0.f : mn0, ms1 = mn1 == -INFINITY ? 0.f : mn1;
        const float a0 = ex2(m[0] - ms0), a1 = ex2(m[1] - ms1);   // m = -inf -> 0
        m[0] = mn0;
        m[1] = mn1;
        float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
        for (int n8 = 0; n8 < 4; ++n8) {
            s[n8][0] = ex2(s[n8][0] - ms0);
            s[n8][1] = ex2(s[n8][1] - ms0);
            s[n8][2] = ex2(s[n8][2] - ms1);
            s[n8][3] = ex2(s[n8][3] - ms1);
            ps0 += s[n8][0] + s[n8][1];
            ps1 += s[n8][2] + s[n8][3];
        }
        l[0] = l[0] * a0 + ps0;   // per-thread partial sums; reduced over the quad at the end
        l[1] = l[1] * a1 + ps1;
#pragma unroll
        for (int i2 = 0; i2 < DT; ++i2) {
            o[i2][0] *= a0;
            o[i2][1] *= a0;
            o[i2][2] *= a1;
            o[i2][3] *= a1;
        }
        // O += P V: the score fragments of two adjacent 8-key tiles form the A operand of a 16-key step
        uint32_t pa[2][4];
#pragma unroll
        for (int kb = 0; kb < 2; ++kb) {
            pa[kb][0] = pack_bf16x2(s[2 * kb][0], s[2 * kb][1]);
            pa[kb][1] = pack_bf16x2(s[2 * kb][2], s[2 * kb][3]);
            pa[kb][2] = pack_bf16x2(s[2 * kb + 1][0], s[2 * kb + 1][1]);
            pa[kb][3] = pack_bf16x2(s[2 * kb + 1][2], s[2 * kb + 1][3]);
        }
        // V fragments in groups of four loads (group gi: 16-key step gi / NG, head dims 64 (gi % NG) .. +63),
        // again one group ahead of the MMAs
        constexpr int NG = DT / 8;          // groups per 16-key step
        uint32_t vf[2][4][4];
        auto load_v = [&](int gi, uint32_t (*dst)[4]) {
            const int kb = gi / NG, dp0 = (gi % NG) * 4, mi = lane >> 3;
            // transposed 8x8 matrices: keys 16 kb + {0..7, 8..15} (rows) x head dims 16 dp + {0..7, 8..15}
#pragma unroll
            for (int u = 0; u < 4; ++u)
                ldmatrix_x4_trans(sv + dec_chunk_offset(kb * 16 + (mi & 1) * 8 + (lane & 7), (dp0 + u) * 2 + (mi >> 1)), dst[u]);
        };
        load_v(0, vf[0]);
#pragma unroll
        for (int gi = 0; gi < 2 * NG; ++gi) {
            if (gi + 1 < 2 * NG) load_v(gi + 1, vf[(gi + 1) & 1]);
            const int kb = gi / NG, dp0 = (gi % NG) * 4;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                mma_16816(o[2 * (dp0 + u)], pa[kb], vf[gi & 1][u][0], vf[gi & 1][u][1]);
                mma_16816(o[2 * (dp0 + u) + 1], pa[kb], vf[gi & 1][u][2], vf[gi & 1][u][3]);
            }
        }
        __syncwarp();
        if (i + kDecStages < nt) {
            fence_proxy_async_smem();   // the stage was read through the generic proxy; TMA writes it next
            issue(i + kDecStages);
        }
    }

    // merge the four warps' partials in shared memory (the stages are idle now) and write one partial per head
    l[0] += __shfl_xor_sync(0xffffffffu, l[0], 1);
    l[0] += __shfl_xor_sync(0xffffffffu, l[0], 2);
    l[1] += __shfl_xor_sync(0xffffffffu, l[1], 1);
    l[1] += __shfl_xor_sync(0xffffffffu, l[1], 2);
    __syncthreads();
    float* mo = reinterpret_cast<float*>(smem);                                  // [warp][16][MERGE_STRIDE]
    float* mml = mo + kDecWarps * 16 * L::MERGE_STRIDE;                          // [warp][16][2]
    {
        float* w0 = mo + (warp * 16 + r0) * L::MERGE_STRIDE + 2 * (lane & 3);
        float* w1 = mo + (warp * 16 + r1) * L::MERGE_STRIDE + 2 * (lane & 3);
#pragma unroll
        for (int i2 = 0; i2 < DT; ++i2) {
            *reinterpret_cast<float2*>(w0 + i2 * 8) = make_float2(o[i2][0], o[i2][1]);
            *reinterpret_cast<float2*>(w1 + i2 * 8) = make_float2(o[i2][2], o[i2][3]);
        }
        if ((lane & 3) == 0) {
            mml[(warp * 16 + r0) * 2] = m[0];
            mml[(warp * 16 + r0) * 2 + 1] = l[0];
            mml[(warp * 16 + r1) * 2] = m[1];
            mml[(warp * 16 + r1) * 2 + 1] = l[1];
        }
    }
    __syncthreads();
    if (*abort_flag) return;
    for (int idx = threadIdx.x; idx < p.group * D; idx += kDecWarps * 32) {
        const int h = idx / D, d = idx - h * D;
        float mw[kDecWarps], M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kDecWarps; ++w) {
            mw[w] = mml[(w * 16 + h) * 2];
            M = fmaxf(M, mw[w]);
        }
        float acc = 0.f, lsum = 0.f;
        if (M != -INFINITY) {
#pragma unroll
            for (int w = 0; w < kDecWarps; ++w) {
                const float f = ex2(mw[w] - M);
                acc = fmaf(mo[(w * 16 + h) * L::MERGE_STRIDE + d], f, acc);
                lsum = fmaf(mml[(w * 16 + h) * 2 + 1], f, lsum);
            }
        }
        const size_t row = (static_cast<size_t>(b) * p.Hq + hk * p.group + h) * p.n_splits + split;
        p.part_o[row * D + d] = acc;
        if (d == 0) {
            p.part_ml[row * 2] = M;
            p.part_ml[row * 2 + 1] = lsum;
        }
    }

    // ---- phase 2 in the same launch (Section 4.2: log-sum-exp combine of the partials).  Every CTA publishes its
    // partials (fence), then draws a ticket; the CTA with the last ticket of its kv head sees all of them.  The sums
    // run over the splits in index order whichever CTA is last, so the result is run-to-run deterministic.
    __shared__ int s_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned int t = atomicAdd(p.tickets + blockIdx.y, 1u);
        s_last = (t == static_cast<unsigned int>(p.n_splits) - 1u) ? 1 : 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // weights 2^(m_s - M) of every head and split (the stages are idle): one warp per head, lanes over the splits
    float* wgt = reinterpret_cast<float*>(smem);          // [group][n_splits]
    float* stat = wgt + 16 * kCombineMaxSplits;            // [group][2]: M, L
    const int tid = threadIdx.x, n = p.n_splits;
    const size_t bh0 = static_cast<size_t>(b) * p.Hq + hk * p.group;
    for (int h = warp; h < p.group; h += kDecWarps) {
        const float* ml = p.part_ml + (bh0 + h) * n * 2;
        float mloc = -INFINITY;
        for (int sidx = lane; sidx < n; sidx += 32) mloc = fmaxf(mloc, __ldcg(ml + sidx * 2));
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) mloc = fmaxf(mloc, __shfl_xor_sync(0xffffffffu, mloc, off));
        float lloc = 0.f;
        for (int sidx = lane; sidx < n; sidx += 32) {
            const float2 v2 = __ldcg(reinterpret_cast<const float2*>(ml + sidx * 2));
            const float f = mloc == -INFINITY ? 0.f : ex2(v2.x - mloc);
            wgt[h * n + sidx] = f;
            lloc = fmaf(v2.y, f, lloc);
        }
        // (fixed tree: the sum does not depend on which CTA runs this)
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) lloc += __shfl_xor_sync(0xffffffffu, lloc, off);
        if (lane == 0) {
            stat[2 * h] = mloc;
            stat[2 * h + 1] = lloc;
        }
    }
    __syncthreads();
    // weighted sums: one thread per (head, four head dims), the splits in index order, 16-byte loads several in flight
    constexpr int D4 = D / 4;
    for (int idx = tid; idx < p.group * D4; idx += kDecWarps * 32) {
        const int h = idx / D4, d4 = idx - h * D4;
        const float4* po = reinterpret_cast<const float4*>(p.part_o + (bh0 + h) * n * D) + d4;
        const float* wh = wgt + h * n;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
        for (int sidx = 0; sidx < n; ++sidx) {
            const float4 v4 = __ldcg(po + static_cast<size_t>(sidx) * D4);
            const float f = wh[sidx];
            acc.x = fmaf(v4.x, f, acc.x);
            acc.y = fmaf(v4.y, f, acc.y);
            acc.z = fmaf(v4.z, f, acc.z);
            acc.w = fmaf(v4.w, f, acc.w);
        }
        const float Lsum = stat[2 * h + 1];
        const float inv = Lsum > 0.f ? 1.f / Lsum : 0.f;
        *reinterpret_cast<uint2*>(p.o + (bh0 + h) * D + d4 * 4) =
            make_uint2(pack_bf16x2(acc.x * inv, acc.y * inv), pack_bf16x2(acc.z * inv, acc.w * inv));
    }
    if (p.lse && tid < p.group) {
        const float M = stat[2 * tid], Lsum = stat[2 * tid + 1];
        p.lse[bh0 + tid] = Lsum > 0.f ? (M + log2f(Lsum)) * 0.6931471805599453f : -INFINITY;
    }
    if (tid == 0) p.tickets[blockIdx.y] = 0u;   // ready for the next call on this workspace
}

}  // namespace af
