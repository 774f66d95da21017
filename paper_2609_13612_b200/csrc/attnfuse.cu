// Host side of the C-ABI declared in include/attnfuse.h: argument validation, tensor-map
// encoding, variant selection and launches.  All arithmetic of the path runs in the kernels.
#include <cuda.h>
#include <algorithm>
#include <atomic>
#include <utility>
#include <cuda_runtime.h>
#include <math.h>
#include <mutex>
#include <stdlib.h>
#include <string.h>

#include "../../include/attnfuse.h"
#include "fwd_kernel.cuh"
#include "bwd_kernel.cuh"
#include "bwd_first_rows.cuh"
#include "bwd_fused_kernel.cuh"
#include "fwd_fp8_kernel.cuh"
#include "decode_kernels.cuh"
#include "rope_kernels.cuh"

namespace {

using namespace af;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// Tensor map over a bf16 tensor [B, H, S, D] (D contiguous) with a box of [rows x 64 columns],
// 128-byte swizzle, zero fill outside the tensor.
// Encoding a tensor map costs a driver call of a few microseconds, several per entry point; a map depends only
// on the pointer, the extents, the strides and the box, so each host thread keeps the last few it built.
struct TmapKey {
    const void* ptr;
    int B, H, S, D, rows;
    int64_t sb, sh, ss;
    bool operator==(const TmapKey& o) const {
        return ptr == o.ptr && B == o.B && H == o.H && S == o.S && D == o.D && rows == o.rows && sb == o.sb && sh == o.sh &&
               ss == o.ss;
    }
};
struct TmapSlot {
    TmapKey key;
    CUtensorMap map;
    bool valid;
};
constexpr int kTmapSlots = 32;
thread_local TmapSlot t_tmap_cache[kTmapSlots];

af_status make_tmap_uncached(CUtensorMap* tm, const void* ptr, int B, int H, int S, int D, const af_strides& st, int rows);

af_status make_tmap(CUtensorMap* tm, const void* ptr, int B, int H, int S, int D, const af_strides& st, int rows) {
    const TmapKey key{ptr, B, H, S, D, rows, st.b, st.h, st.s};
    uint64_t hsh = reinterpret_cast<uintptr_t>(ptr) >> 4;
    hsh ^= (static_cast<uint64_t>(S) * 0x9E3779B97F4A7C15ull) ^ (static_cast<uint64_t>(H) << 20) ^ (static_cast<uint64_t>(rows) << 7) ^
           static_cast<uint64_t>(st.s);
    TmapSlot& slot = t_tmap_cache[(hsh ^ (hsh >> 17)) % kTmapSlots];
    if (slot.valid && slot.key == key) {
        *tm = slot.map;
        return AF_OK;
    }
    const af_status r = make_tmap_uncached(tm, ptr, B, H, S, D, st, rows);
    if (r == AF_OK) {
        slot.key = key;
        slot.map = *tm;
        slot.valid = true;
    }
    return r;
}

af_status make_tmap_uncached(CUtensorMap* tm, const void* ptr, int B, int H, int S, int D, const af_strides& st, int rows) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return AF_ERR_CUDA;
    cuuint64_t dims[4] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(S), static_cast<cuuint64_t>(H),
                          static_cast<cuuint64_t>(B)};
    cuuint64_t strides[3] = {static_cast<cuuint64_t>(st.s) * 2, static_cast<cuuint64_t>(st.h) * 2,
                             static_cast<cuuint64_t>(st.b) * 2};
    cuuint32_t box[4] = {static_cast<cuuint32_t>(BOX_COLS), static_cast<cuuint32_t>(rows), 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? AF_OK : AF_ERR_CUDA;
}

// Tensor map over one-byte elements [B, H, rows, cols] (contiguous), box of 128 x 128, 128-byte swizzle, zero fill:
// the E4M3 operands of the fp8 forward (cols = D for Q and K; for the transposed V rows = D and cols = S).
af_status make_tmap_u8(CUtensorMap* tm, const void* ptr, int B, int H, int rows, int cols) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return AF_ERR_CUDA;
    cuuint64_t dims[4] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows), static_cast<cuuint64_t>(H),
                          static_cast<cuuint64_t>(B)};
    cuuint64_t strides[3] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(cols) * rows,
                             static_cast<cuuint64_t>(cols) * rows * H};
    cuuint32_t box[4] = {128, 128, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(ptr), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? AF_OK : AF_ERR_CUDA;
}

// Byte offset of the bf16 copy of the cos/sin table inside the table buffer: after the fp32 rows (S positions
// and the trailer), rounded up to 256 bytes.  Its rows are [R/2 cos | R/2 sin] in bf16, 2 R bytes each.
size_t table_bf16_offset(int S, int R) {
    const size_t f32 = static_cast<size_t>(S + 1) * (R / 2) * sizeof(float2);
    return (f32 + 255) & ~static_cast<size_t>(255);
}

// Tensor map over that copy: [S rows][R columns] bf16, box of 128 rows x R columns, no swizzle, zero fill.
af_status make_tmap_table(CUtensorMap* tm, const void* table, int S, int R) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return AF_ERR_CUDA;
    cuuint64_t dims[2] = {static_cast<cuuint64_t>(R), static_cast<cuuint64_t>(S)};
    cuuint64_t strides[1] = {static_cast<cuuint64_t>(R) * 2};
    cuuint32_t box[2] = {static_cast<cuuint32_t>(R), 128};
    cuuint32_t estr[2] = {1, 1};
    void* base = const_cast<uint8_t*>(static_cast<const uint8_t*>(table) + table_bf16_offset(S, R));
    CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? AF_OK : AF_ERR_CUDA;
}

// Tuning options (attnfuse_set_option / attnfuse_get_option): a process-wide table of atomics.  Each entry
// takes its initial value from the environment variable of the same name once, when the table is first
// touched; launches read the table, never the environment.
struct OptionDef { const char* env; int dflt; };
constexpr OptionDef kOptionDefs[AF_OPT_COUNT_] = {
    {"AF_FWD_NQ", 2},           // AF_OPT_FWD_QTILES
    {"AF_FWD_PAIR", 1},         // AF_OPT_FWD_PAIR_HEADS
    {"AF_FWD_KEYS_BF16", 0},    // AF_OPT_FWD_KEYS_BF16
    {"AF_BS_ROWPAIR", 1},       // AF_OPT_BS_ROWPAIR
    {"AF_BWD_ONEPASS", 1},      // AF_OPT_BWD_ONEPASS
    {"AF_FWD_ALIBI_MMA", 1},    // AF_OPT_FWD_ALIBI_MMA
};
std::atomic<int> g_options[AF_OPT_COUNT_];
std::once_flag g_options_once;
void init_options() {
    std::call_once(g_options_once, [] {
        for (int i = 0; i < AF_OPT_COUNT_; ++i) {
            const char* v = getenv(kOptionDefs[i].env);
            g_options[i].store(v ? atoi(v) : kOptionDefs[i].dflt, std::memory_order_relaxed);
        }
    });
}
int opt(af_option o) {
    init_options();
    return g_options[o].load(std::memory_order_relaxed);
}

// AF_OPT_FWD_KEYS_BF16 (forward only, rotary widths 16, 32, 64, 128): key tiles are rotated in packed bf16
// arithmetic from the table's bf16 copy instead of fp32 arithmetic from the fp32 rows.  Faster (the rotation
// competes with the softmax for issue slots), but a rotated key then carries about three bf16 roundings instead
// of one; the backward pass always rotates in fp32, so a log-sum-exp produced in this mode is slightly
// inconsistent with the scores the backward pass recomputes.  Off by default.
bool keys_rotate_in_bf16(int R) {
    return (R == 16 || R == 32 || R == 64 || R == 128) && opt(AF_OPT_FWD_KEYS_BF16);
}

// Number of SMs of the current device (cached per device ordinal).
int sm_count() {
    static std::atomic<int> cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    int n = cached[dev & 63].load(std::memory_order_relaxed);
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return 0;
        cached[dev & 63].store(n, std::memory_order_relaxed);
    }
    return n;
}

// Opt a kernel in to its dynamic shared-memory size once per device (the attribute is per device and per
// function; `done` is the call site's own bit mask over device ordinals).
template <typename Kernel>
af_status allow_dynamic_smem(Kernel kern, int bytes, std::atomic<unsigned long long>& done) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return AF_ERR_CUDA;
    const unsigned long long bit = 1ull << (dev & 63);
    if (!(done.load(std::memory_order_acquire) & bit)) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess)
            return AF_ERR_CUDA;
        done.fetch_or(bit, std::memory_order_release);
    }
    return AF_OK;
}

// Launch as a programmatic dependent of the kernel that precedes it in the stream: the grid may be scheduled
// while that kernel drains and runs its set-up, then waits (griddepcontrol.wait in the kernel) for the
// predecessor's completion before it touches global memory.  dependent = false: a plain launch.
template <typename... KArgs, typename... Args>
af_status launch_kernel(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, bool dependent,
                        Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...) == cudaSuccess ? AF_OK : AF_ERR_CUDA;
}

// Internal streams and events of attnfuse_fwd_host, per device, created on first use and kept.
struct HostPipe {
    static constexpr int kEvents = 64;
    cudaStream_t compute = nullptr, d2h = nullptr;
    cudaEvent_t ev[kEvents] = {};
    int next = 0;
    bool ready = false;
};
std::mutex g_pipe_mutex;
HostPipe g_pipes[64];
// (caller holds g_pipe_mutex)
HostPipe* get_pipe() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    HostPipe* p = &g_pipes[dev & 63];
    if (!p->ready) {
        if (cudaStreamCreateWithFlags(&p->compute, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        if (cudaStreamCreateWithFlags(&p->d2h, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        for (int i = 0; i < HostPipe::kEvents; ++i)
            if (cudaEventCreateWithFlags(&p->ev[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
        p->ready = true;
    }
    return p;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

af_status check_arch() {
    static std::atomic<int> cached[64];   // per device ordinal: 0 = not asked yet, else major + 1
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return AF_ERR_CUDA;
    int major1 = cached[dev & 63].load(std::memory_order_relaxed);
    if (major1 == 0) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return AF_ERR_CUDA;
        major1 = major + 1;
        cached[dev & 63].store(major1, std::memory_order_relaxed);
    }
    return major1 == 11 ? AF_OK : AF_ERR_ARCH;
}

af_status check_common(const af_shape* sh, const af_rope* rope, const void* table, const af_mask* mask, int group) {
    if (!sh || !rope || !mask) return AF_ERR_NULL;
    if (sh->B < 1 || sh->Hq < 1 || sh->Hkv < 1 || sh->S < 1) return AF_ERR_SHAPE;
    if (sh->D != 64 && sh->D != 128) return AF_ERR_SHAPE;
    if (group < 1 || sh->Hkv * group != sh->Hq) return AF_ERR_SHAPE;
    if (rope->rotary_dim < 0 || rope->rotary_dim > sh->D || (rope->rotary_dim % 16) != 0) return AF_ERR_SPEC;
    if (rope->rotary_dim > 0 && !(rope->theta > 0.f)) return AF_ERR_SPEC;
    if (rope->rotary_dim > 0 && !table) return AF_ERR_NULL;
    if (table && !aligned16(table)) return AF_ERR_ALIGN;
    return AF_OK;
}

af_status resolve_strides(const af_strides* in, int H, int S, int D, af_strides* out) {
    if (in) {
        *out = *in;
    } else {
        out->s = D;
        out->h = static_cast<int64_t>(S) * D;
        out->b = static_cast<int64_t>(H) * S * D;
    }
    if (out->s < D || out->h < 1 || out->b < 1) return AF_ERR_SHAPE;
    if ((out->s % 8) || (out->h % 8) || (out->b % 8)) return AF_ERR_ALIGN;
    return AF_OK;
}

template <int D, int NQ, bool ROPE, int KS, int VS, bool TAB = false, bool GEN = false>
af_status launch_fwd_variant(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to, const CUtensorMap& tt,
                             FwdParams p, cudaStream_t stream) {
    using L = FwdSmem<D, NQ, KS, VS, ROPE && TAB>;
    auto kern = attn_fwd_kernel<D, NQ, ROPE, KS, VS, false, TAB, GEN>;
    static std::atomic<unsigned long long> configured{0};
    if (allow_dynamic_smem(kern, L::BYTES, configured) != AF_OK) return AF_ERR_CUDA;
    // an even GQA group lets the two query tiles of a CTA be two heads of one kv head (same key range)
    p.pair_heads = (NQ == 2 && (p.group % 2) == 0 && opt(AF_OPT_FWD_PAIR_HEADS)) ? 1 : 0;
    // (measured: +5 % at config 3 with the rotation warps at work, -1 % without them; option value 2 takes it there too)
    p.alibi_mma = (L::HAS_AX && !GEN && p.slopes && (opt(AF_OPT_FWD_ALIBI_MMA) >= 2 || (ROPE && opt(AF_OPT_FWD_ALIBI_MMA) == 1))) ? 1 : 0;
    const int rows_per_cta = p.pair_heads ? BM : BM * NQ;
    p.n_row_blocks = (p.S + rows_per_cta - 1) / rows_per_cta;
    dim3 grid(p.pair_heads ? p.B * p.Hq / 2 : p.B * p.Hq, p.n_row_blocks, 1);
    if (ROPE && !p.rot_k) {
        // hybrid arm: launched as a programmatic dependent of the RoPE pass on K that precedes it in the stream;
        // the kernel waits for that pass only before its first key-tile load
        return launch_kernel(kern, grid, dim3(128 * (2 + NQ), 1, 1), L::BYTES, stream, true, tq, tk, tv, to, tt, p);
    }
    kern<<<grid, 128 * (2 + NQ), L::BYTES, stream>>>(tq, tk, tv, to, tt, p);
    return cudaGetLastError() == cudaSuccess ? AF_OK : AF_ERR_CUDA;
}

// Block-sparse variant (Section 4.3): the grid is (heads or head pairs, 128-row blocks); every CTA walks the
// list of active key blocks of its row block.  An even GQA group pairs two heads per CTA, otherwise one head.
template <int D, int NQ, bool ROPE, bool GEN = false>
af_status launch_fwd_blocks_variant(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                                    const CUtensorMap& to, const CUtensorMap& tt, FwdParams p, cudaStream_t stream) {
    using L = FwdSmem<D, NQ, 2, 2>;
    auto kern = attn_fwd_kernel<D, NQ, ROPE, 2, 2, true, false, GEN>;
    static std::atomic<unsigned long long> configured{0};
    if (allow_dynamic_smem(kern, L::BYTES, configured) != AF_OK) return AF_ERR_CUDA;
    // NQ = 2: two heads of one kv head on the same row block (even GQA group), or - with pair lists - the row
    // blocks 2 rb and 2 rb + 1 of one head
    p.pair_heads = (NQ == 2 && !p.bs_rowpair) ? 1 : 0;
    // (measured: +5 % at config 3 with the rotation warps at work, -1 % without them; option value 2 takes it there too)
    p.alibi_mma = (L::HAS_AX && !GEN && p.slopes && (opt(AF_OPT_FWD_ALIBI_MMA) >= 2 || (ROPE && opt(AF_OPT_FWD_ALIBI_MMA) == 1))) ? 1 : 0;
    p.n_row_blocks = (p.S + BM - 1) / BM;
    if (p.bs_rowpair) p.n_row_blocks = (p.n_row_blocks + 1) / 2;
    dim3 grid(p.pair_heads ? p.B * p.Hq / 2 : p.B * p.Hq, p.n_row_blocks, 1);
    kern<<<grid, 128 * (2 + NQ), L::BYTES, stream>>>(tq, tk, tv, to, tt, p);
    return cudaGetLastError() == cudaSuccess ? AF_OK : AF_ERR_CUDA;
}
template <int D>
af_status launch_fwd_blocks(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to, const CUtensorMap& tt,
                            const FwdParams& p, cudaStream_t stream) {
    // (p.bs_rowpair is set only for an odd GQA group, when the caller supplied the lists of row-block pairs)
    const bool two_tiles = (p.group % 2) == 0 || p.bs_rowpair;
    if (p.bias || p.relu) {   // Section 3.1 extras: built for CTAs of two query tiles only
        if (!two_tiles) return AF_ERR_SPEC;
        return p.R > 0 ? launch_fwd_blocks_variant<D, 2, true, true>(tq, tk, tv, to, tt, p, stream)
                       : launch_fwd_blocks_variant<D, 2, false, true>(tq, tk, tv, to, tt, p, stream);
    }
    if (two_tiles)
        return p.R > 0 ? launch_fwd_blocks_variant<D, 2, true>(tq, tk, tv, to, tt, p, stream)
                       : launch_fwd_blocks_variant<D, 2, false>(tq, tk, tv, to, tt, p, stream);
    return p.R > 0 ? launch_fwd_blocks_variant<D, 1, true>(tq, tk, tv, to, tt, p, stream)
                   : launch_fwd_blocks_variant<D, 1, false>(tq, tk, tv, to, tt, p, stream);
}

template <int D>
af_status launch_fwd(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to, const CUtensorMap& tt, const FwdParams& p,
                     cudaStream_t stream) {
    if (p.bias || p.relu)   // Section 3.1 extras (additive_bias, relu_attention): their own instantiation
        return p.R > 0 ? launch_fwd_variant<D, 2, true, 2, 2, false, true>(tq, tk, tv, to, tt, p, stream)
                       : launch_fwd_variant<D, 2, false, 2, 2, false, true>(tq, tk, tv, to, tt, p, stream);
    const int nq = opt(AF_OPT_FWD_QTILES);
    if (nq == 1) {
        return p.R > 0 ? launch_fwd_variant<D, 1, true, 2, 2>(tq, tk, tv, to, tt, p, stream)
                       : launch_fwd_variant<D, 1, false, 2, 2>(tq, tk, tv, to, tt, p, stream);
    }
    if (p.R > 0 && p.keys_bf16) return launch_fwd_variant<D, 2, true, 2, 2, true>(tq, tk, tv, to, tt, p, stream);
    return p.R > 0 ? launch_fwd_variant<D, 2, true, 2, 2>(tq, tk, tv, to, tt, p, stream)
                   : launch_fwd_variant<D, 2, false, 2, 2>(tq, tk, tv, to, tt, p, stream);
}

template <int D, bool DKV, bool ROT_X, bool ROT_A, bool BS>
af_status launch_bwd_variant_bs(const CUtensorMap& tx, const CUtensorMap& ty, const CUtensorMap& ta, const CUtensorMap& tb,
                                const CUtensorMap& ts, const BwdParams& p, dim3 grid, cudaStream_t stream) {
    using L = BwdSmem<D>;
    auto kern = attn_bwd_kernel<D, DKV, ROT_X, ROT_A, BS>;
    static std::atomic<unsigned long long> configured{0};
    if (allow_dynamic_smem(kern, L::BYTES, configured) != AF_OK) return AF_ERR_CUDA;
    // every gradient kernel follows the delta kernel or another kernel of the backward sequence in the stream
    return launch_kernel(kern, grid, dim3(512, 1, 1), L::BYTES, stream, true, tx, ty, ta, tb, ts, p);
}
// dense or, when the parameters carry block lists, block-sparse instantiation
template <int D, bool DKV, bool ROT_X, bool ROT_A>
af_status launch_bwd_variant(const CUtensorMap& tx, const CUtensorMap& ty, const CUtensorMap& ta, const CUtensorMap& tb,
                             const CUtensorMap& ts, const BwdParams& p, dim3 grid, cudaStream_t stream) {
    return p.bs_ptr ? launch_bwd_variant_bs<D, DKV, ROT_X, ROT_A, true>(tx, ty, ta, tb, ts, p, grid, stream)
                    : launch_bwd_variant_bs<D, DKV, ROT_X, ROT_A, false>(tx, ty, ta, tb, ts, p, grid, stream);
}

// Section 3.1 extras in the backward (additive_bias, relu_attention): the GEN instantiations, dense only.
template <int D, bool DKV, bool ROT_X>
af_status launch_bwd_gen(const CUtensorMap& tx, const CUtensorMap& ty, const CUtensorMap& ta, const CUtensorMap& tb,
                         const CUtensorMap& ts, const BwdParams& p, dim3 grid, cudaStream_t stream) {
    using L = BwdSmem<D>;
    auto kern = attn_bwd_kernel<D, DKV, ROT_X, false, false, true>;
    static std::atomic<unsigned long long> configured{0};
    if (allow_dynamic_smem(kern, L::BYTES, configured) != AF_OK) return AF_ERR_CUDA;
    return launch_kernel(kern, grid, dim3(512, 1, 1), L::BYTES, stream, true, tx, ty, ta, tb, ts, p);
}

// RoPE pass x [B, H, S, D] (strided) -> x_out (contiguous); R > 0.
// dependent: launch as a programmatic dependent of the preceding kernel (only inside this library's own sequences).
af_status launch_rope(const void* x_in, const af_strides& st, void* x_out, int B, int H, int S, int D, int R,
                      const void* rope_table, int inverse, cudaStream_t stream, bool dependent = false) {
    constexpr int HPT = 4;
    const long long NH = static_cast<long long>(B) * H;
    const int per_row = (R >> 4) + ((D - R) >> 3);
    const long long items = static_cast<long long>(S) * per_row;
    dim3 grid(static_cast<unsigned>((items + 255) / 256), static_cast<unsigned>((NH + HPT - 1) / HPT), 1);
    if (grid.y > 65535) return AF_ERR_SHAPE;
    return launch_kernel(rope_apply_kernel<HPT>, grid, dim3(256, 1, 1), 0, stream, dependent,
                         static_cast<const uint4*>(x_in), static_cast<uint4*>(x_out),
                         static_cast<const float2*>(rope_table), static_cast<int>(NH), H, S, D, R, inverse ? -1.f : 1.f,
                         static_cast<long long>(st.b), static_cast<long long>(st.h), static_cast<long long>(st.s));
}

// delta, then the two gradient kernels.  tkp / tqp: tensor maps over the rotated-K and rotated-Q caches in
// the workspace, or nullptr when the workspace has no room for them (see bwd_kernel.cuh for the three set-ups).
// k / stkv / kcache: the caller's K, its strides and the K' cache, for the RoPE pass of the two-cache set-up.
// The first query rows of every head in fp32, after the MMA kernels of the sequence (see bwd_first_rows.cuh).
template <int D>
af_status launch_first_rows(const FirstRowsParams& fp, cudaStream_t stream) {
    using L = FirstRowsSmem<D>;
    auto kern = bwd_first_rows_kernel<D>;
    static std::atomic<unsigned long long> configured{0};
    if (allow_dynamic_smem(kern, L::BYTES, configured) != AF_OK) return AF_ERR_CUDA;
    return launch_kernel(kern, dim3(fp.B * fp.Hkv, 1, 1), dim3(256, 1, 1), L::BYTES, stream, true, fp);
}

template <int D>
af_status launch_bwd_mma(const af_shape* sh, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                         const CUtensorMap& tdo, const CUtensorMap* tkp, const CUtensorMap* tqp, const void* k,
                         const af_strides& stkv, void* kcache, const void* o, const void* d_o, BwdParams p, void* dq,
                         int dq_f32, void* dk, void* dv, int dkv_f32, float* delta, const af_blocks* blocks,
                         cudaStream_t stream);

struct OnePassArgs;
template <int D>
af_status launch_bwd_onepass(const af_shape* sh, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                             const CUtensorMap& tdo, const CUtensorMap& tkp, const CUtensorMap& tqp, const void* k,
                             const af_strides& stkv, void* kcache, const void* o, const void* d_o, BwdParams p, void* dq,
                             int dq_f32, void* dk, void* dv, int dkv_f32, float* delta, const OnePassArgs& a,
                             cudaStream_t stream);

template <int D>
af_status launch_bwd(const af_shape* sh, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                     const CUtensorMap& tdo, const CUtensorMap* tkp, const CUtensorMap* tqp, const void* k,
                     const af_strides& stkv, void* kcache, const void* o, const void* d_o, BwdParams p, void* dq,
                     int dq_f32, void* dk, void* dv, int dkv_f32, float* delta, const af_blocks* blocks,
                     cudaStream_t stream, const FirstRowsParams& fp, const OnePassArgs* onepass) {
    p.skip_rows = fp.rows;
    af_status st;
    st = onepass ? launch_bwd_onepass<D>(sh, tq, tk, tv, tdo, tkp ? *tkp : tk, tqp ? *tqp : tq, k, stkv, kcache, o, d_o, p, dq, dq_f32,
                                         dk, dv, dkv_f32, delta, *onepass, stream)
                 : launch_bwd_mma<D>(sh, tq, tk, tv, tdo, tkp, tqp, k, stkv, kcache, o, d_o, p, dq, dq_f32, dk, dv,
                                     dkv_f32, delta, blocks, stream);
    if (st != AF_OK || fp.rows == 0) return st;
    return launch_first_rows<D>(fp, stream);
}

// One-pass sequence (bwd_fused_kernel.cuh): zero the fp32 dQ' accumulator, delta, RoPE passes on K and Q into the
// caches, the one-pass kernel (dK, dV, dQ' partials), then scale / rotate back / convert dQ.
struct OnePassArgs {
    const void* q;
    af_strides stq;
    void* qcache;
    float* dq_acc;
    size_t dq_acc_bytes;
    const af_blocks* blocks;   // block-sparse lists or nullptr
};
template <int D>
af_status launch_bwd_onepass(const af_shape* sh, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                             const CUtensorMap& tdo, const CUtensorMap& tkp, const CUtensorMap& tqp, const void* k,
                             const af_strides& stkv, void* kcache, const void* o, const void* d_o, BwdParams p, void* dq,
                             int dq_f32, void* dk, void* dv, int dkv_f32, float* delta, const OnePassArgs& a,
                             cudaStream_t stream) {
    using L = BwdFusedSmem<D>;
    if (cudaMemsetAsync(a.dq_acc, 0, a.dq_acc_bytes, stream) != cudaSuccess) return AF_ERR_CUDA;
    const long long rows = static_cast<long long>(sh->B) * sh->Hq * sh->S;
    const long long threads = rows * (D / 8);
    bwd_delta_kernel<D><<<static_cast<unsigned>((threads + 255) / 256), 256, 0, stream>>>(
        static_cast<const uint4*>(o), static_cast<const uint4*>(d_o), delta, rows);
    if (cudaGetLastError() != cudaSuccess) return AF_ERR_CUDA;
    af_status st;
    if (p.R > 0) {
        if ((st = launch_rope(k, stkv, kcache, sh->B, sh->Hkv, sh->S, D, p.R, p.table, 0, stream, true)) != AF_OK) return st;
        if ((st = launch_rope(a.q, a.stq, a.qcache, sh->B, sh->Hq, sh->S, D, p.R, p.table, 0, stream, true)) != AF_OK) return st;
    }
    p.delta = delta;
    p.out1 = dv; p.out2 = dk; p.out_f32 = dkv_f32; p.store_x = 0;
    p.dq_acc = a.dq_acc;
    // block lists by key block (the stationary block of this kernel)
    p.bs_ptr = a.blocks ? a.blocks->col_ptr : nullptr;
    p.bs_idx = a.blocks ? a.blocks->row_idx : nullptr;
    p.bs_order = a.blocks ? a.blocks->col_order : nullptr;
    auto kern = a.blocks ? attn_bwd_fused_kernel<D, true> : attn_bwd_fused_kernel<D, false>;
    static std::atomic<unsigned long long> configured[2];
    if (allow_dynamic_smem(kern, L::BYTES, configured[a.blocks ? 1 : 0]) != AF_OK) return AF_ERR_CUDA;
    const unsigned tiles = static_cast<unsigned>((sh->S + 127) / 128);
    dim3 grid(sh->B * sh->Hkv, tiles, 1);
    st = p.R > 0 ? launch_kernel(kern, grid, dim3(512, 1, 1), L::BYTES, stream, true, tkp, tv, tqp, tdo, p)
                 : launch_kernel(kern, grid, dim3(512, 1, 1), L::BYTES, stream, true, tk, tv, tq, tdo, p);
    if (st != AF_OK) return st;
    const long long fthreads = rows * (D / 4);
    return launch_kernel(bwd_dq_finish_kernel<D>, dim3(static_cast<unsigned>((fthreads + 255) / 256), 1, 1), dim3(256, 1, 1), 0,
                         stream, true, static_cast<const float*>(a.dq_acc), dq, dq_f32, p.table, sh->S, p.R, p.scale, rows);
}

template <int D>
af_status launch_bwd_mma(const af_shape* sh, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                         const CUtensorMap& tdo, const CUtensorMap* tkp, const CUtensorMap* tqp, const void* k,
                         const af_strides& stkv, void* kcache, const void* o, const void* d_o, BwdParams p, void* dq,
                         int dq_f32, void* dk, void* dv, int dkv_f32, float* delta, const af_blocks* blocks,
                         cudaStream_t stream) {
    // block lists by stationary block: by key block for the dK/dV role, by query block for the dQ role
    auto role_lists = [&](bool dkv_role) {
        p.bs_ptr = blocks ? (dkv_role ? blocks->col_ptr : blocks->row_ptr) : nullptr;
        p.bs_idx = blocks ? (dkv_role ? blocks->row_idx : blocks->col_idx) : nullptr;
        p.bs_order = blocks ? (dkv_role ? blocks->col_order : blocks->row_order) : nullptr;
    };
    const long long rows = static_cast<long long>(sh->B) * sh->Hq * sh->S;
    const long long threads = rows * (D / 8);
    bwd_delta_kernel<D><<<static_cast<unsigned>((threads + 255) / 256), 256, 0, stream>>>(
        static_cast<const uint4*>(o), static_cast<const uint4*>(d_o), delta, rows);
    if (cudaGetLastError() != cudaSuccess) return AF_ERR_CUDA;
    p.delta = delta;
    const unsigned tiles = static_cast<unsigned>((sh->S + 127) / 128);
    af_status st;
#ifdef AF_TRACE
    // tracing builds only: 1 = dK/dV kernel only, 2 = dQ kernel only (the skipped outputs stay unwritten)
    const int only = getenv("AF_BWD_ONLY") ? atoi(getenv("AF_BWD_ONLY")) : 0;
#else
    constexpr int only = 0;
#endif
    dim3 gkv(sh->B * sh->Hkv, tiles, 1), gq(sh->B * sh->Hq, tiles, 1);
    if (p.bias || p.relu) {
        // additive_bias / relu_attention: the both-caches set-up with rotation, the plain one without
        if (p.R > 0) {
            if (!tkp || !tqp) return AF_ERR_WORKSPACE;
            if ((st = launch_rope(k, stkv, kcache, sh->B, sh->Hkv, sh->S, D, p.R, p.table, 0, stream, true)) != AF_OK) return st;
            p.out1 = dq; p.out2 = nullptr; p.out_f32 = dq_f32; p.store_x = 1;
            if ((st = launch_bwd_gen<D, false, true>(tq, tdo, *tkp, tv, *tqp, p, gq, stream)) != AF_OK) return st;
            p.out1 = dv; p.out2 = dk; p.out_f32 = dkv_f32; p.store_x = 0;
            return launch_bwd_gen<D, true, false>(*tkp, tv, *tqp, tdo, tk, p, gkv, stream);
        }
        p.out1 = dq; p.out2 = nullptr; p.out_f32 = dq_f32; p.store_x = 0;
        if ((st = launch_bwd_gen<D, false, false>(tq, tdo, tk, tv, tk, p, gq, stream)) != AF_OK) return st;
        p.out1 = dv; p.out2 = dk; p.out_f32 = dkv_f32; p.store_x = 0;
        return launch_bwd_gen<D, true, false>(tk, tv, tq, tdo, tk, p, gkv, stream);
    }
    if (p.R > 0 && tkp && tqp && only == 0) {
        // both caches: K' by the RoPE pass, Q' by the dQ kernel, no on-chip rotation in the dK/dV loop
        if ((st = launch_rope(k, stkv, kcache, sh->B, sh->Hkv, sh->S, D, p.R, p.table, 0, stream, true)) != AF_OK) return st;
        p.out1 = dq; p.out2 = nullptr; p.out_f32 = dq_f32; p.store_x = 1;
        role_lists(false);
        if ((st = launch_bwd_variant<D, false, true, false>(tq, tdo, *tkp, tv, *tqp, p, gq, stream)) != AF_OK) return st;
        p.out1 = dv; p.out2 = dk; p.out_f32 = dkv_f32; p.store_x = 0;
        role_lists(true);
        return launch_bwd_variant<D, true, false, false>(*tkp, tv, *tqp, tdo, tk, p, gkv, stream);
    }
    const bool cache = p.R > 0 && tkp != nullptr && only != 2;
    p.out1 = dv; p.out2 = dk; p.out_f32 = dkv_f32; p.store_x = cache ? 1 : 0;
    role_lists(true);
    st = only == 2 ? AF_OK
         : p.R > 0 ? launch_bwd_variant<D, true, true, true>(tk, tv, tq, tdo, cache ? *tkp : tk, p, gkv, stream)
                   : launch_bwd_variant<D, true, false, false>(tk, tv, tq, tdo, tk, p, gkv, stream);
    if (st != AF_OK || only == 1) return st;
    p.out1 = dq; p.out2 = nullptr; p.out_f32 = dq_f32; p.store_x = 0;
    role_lists(false);
    if (p.R == 0) return launch_bwd_variant<D, false, false, false>(tq, tdo, tk, tv, tk, p, gq, stream);
    return cache ? launch_bwd_variant<D, false, true, false>(tq, tdo, *tkp, tv, tk, p, gq, stream)
                 : launch_bwd_variant<D, false, true, true>(tq, tdo, tk, tv, tk, p, gq, stream);
}

size_t bwd_delta_bytes(const af_shape* sh) {
    return (static_cast<size_t>(sh->B) * sh->Hq * sh->S * sizeof(float) + 255) / 256 * 256;
}
size_t bwd_kcache_bytes(const af_shape* sh) {
    return static_cast<size_t>(sh->B) * sh->Hkv * sh->S * sh->D * 2;
}
size_t bwd_qcache_bytes(const af_shape* sh) {
    return static_cast<size_t>(sh->B) * sh->Hq * sh->S * sh->D * 2;
}
size_t bwd_dqacc_bytes(const af_shape* sh) {
    return static_cast<size_t>(sh->B) * sh->Hq * sh->S * sh->D * sizeof(float);
}

}  // namespace

extern "C" {

int attnfuse_version(void) { return 110; }

const char* attnfuse_strerror(af_status st) {
    switch (st) {
        case AF_OK: return "ok";
        case AF_ERR_NULL: return "required pointer is NULL";
        case AF_ERR_SHAPE: return "unsupported or inconsistent shape";
        case AF_ERR_DTYPE: return "unsupported dtype";
        case AF_ERR_ALIGN: return "pointer or stride misaligned";
        case AF_ERR_SPEC: return "bad RoPE or mask specification";
        case AF_ERR_WORKSPACE: return "workspace missing or too small";
        case AF_ERR_ARCH: return "device is not compute capability 10.x";
        case AF_ERR_CUDA: return "CUDA call failed";
        case AF_ERR_DEVICE_TIMEOUT: return "bounded device-side wait ran out";
        case AF_ERR_STATIC_LIMIT:
            return "attnfuse_bwd_static: B*Hq*S exceeds AF_BWD_STATIC_MAX_ROWS (use attnfuse_bwd with a workspace)";
    }
    return "unknown status";
}

af_status attnfuse_set_option(af_option option, int value) {
    if (option < 0 || option >= AF_OPT_COUNT_) return AF_ERR_SPEC;
    init_options();
    g_options[option].store(value, std::memory_order_relaxed);
    return AF_OK;
}

int attnfuse_get_option(af_option option) {
    if (option < 0 || option >= AF_OPT_COUNT_) return -1;
    return opt(option);
}

af_status attnfuse_stream_status(void* cuda_stream, unsigned int* detail) {
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    unsigned int w = 0, zero = 0;
    void* addr = nullptr;
    if (cudaGetSymbolAddress(&addr, af::g_device_status) != cudaSuccess) return AF_ERR_CUDA;
    if (cudaMemcpyAsync(&w, addr, sizeof(w), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return AF_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return AF_ERR_CUDA;
    if (w) {
        if (cudaMemcpyAsync(addr, &zero, sizeof(zero), cudaMemcpyHostToDevice, stream) != cudaSuccess) return AF_ERR_CUDA;
        if (cudaStreamSynchronize(stream) != cudaSuccess) return AF_ERR_CUDA;
    }
    if (detail) *detail = w;
    return w ? AF_ERR_DEVICE_TIMEOUT : AF_OK;
}

af_status attnfuse_device_status(unsigned int* detail) {
    unsigned int w = 0, zero = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return AF_ERR_CUDA;
    if (cudaMemcpyFromSymbol(&w, af::g_device_status, sizeof(w)) != cudaSuccess) return AF_ERR_CUDA;
    if (w && cudaMemcpyToSymbol(af::g_device_status, &zero, sizeof(zero)) != cudaSuccess) return AF_ERR_CUDA;
    if (detail) *detail = w;
    return w ? AF_ERR_DEVICE_TIMEOUT : AF_OK;
}

af_status attnfuse_selftest_wait_timeout(unsigned int limit_cycles, void* cuda_stream) {
    if (limit_cycles < 1000u || limit_cycles > 100000000u) return AF_ERR_SPEC;
    af_status st = check_arch();
    if (st != AF_OK) return st;
    wait_timeout_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(cuda_stream)>>>(static_cast<long long>(limit_cycles));
    return cudaGetLastError() == cudaSuccess ? AF_OK : AF_ERR_CUDA;
}

size_t attnfuse_rope_table_bytes(int S, int rotary_dim) {
    if (S < 1 || rotary_dim < 1) return 0;
    // fp32 rows (+ one trailer row), then the bf16 copy the forward kernel streams by TMA
    return table_bf16_offset(S, rotary_dim) + static_cast<size_t>(S) * rotary_dim * 2;
}

af_status attnfuse_rope_table(const af_rope* rope, int S, void* table, void* cuda_stream) {
    if (!rope) return AF_ERR_NULL;
    if (S < 1) return AF_ERR_SHAPE;
    if (rope->rotary_dim < 0 || (rope->rotary_dim % 16) != 0 || rope->rotary_dim > 128) return AF_ERR_SPEC;
    if (rope->rotary_dim == 0) return AF_OK;
    if (!(rope->theta > 0.f)) return AF_ERR_SPEC;
    if (!table) return AF_ERR_NULL;
    if (!aligned16(table)) return AF_ERR_ALIGN;
    const long long n = static_cast<long long>(S + 1) * (rope->rotary_dim / 2);
    const int threads = 256;
    const unsigned blocks = static_cast<unsigned>((n + threads - 1) / threads);
    rope_table_kernel<<<blocks, threads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        static_cast<float2*>(table),
        reinterpret_cast<__nv_bfloat16*>(static_cast<uint8_t*>(table) + table_bf16_offset(S, rope->rotary_dim)), S,
        rope->rotary_dim, static_cast<double>(rope->theta), rope->pos_offset);
    return cudaGetLastError() == cudaSuccess ? AF_OK : AF_ERR_CUDA;
}

af_status attnfuse_rope(const af_shape* shape, int n_heads, const void* x_in, void* x_out, const af_rope* rope,
                        const void* rope_table, int inverse, void* cuda_stream) {
    if (!shape || !rope || !x_in || !x_out) return AF_ERR_NULL;
    if (shape->B < 1 || n_heads < 1 || shape->S < 1 || shape->D < 16 || (shape->D % 8) != 0) return AF_ERR_SHAPE;
    const int R = rope->rotary_dim, D = shape->D;
    if (R < 0 || R > D || (R % 16) != 0) return AF_ERR_SPEC;
    if (R > 0 && !rope_table) return AF_ERR_NULL;
    if (!aligned16(x_in) || !aligned16(x_out) || (rope_table && !aligned16(rope_table))) return AF_ERR_ALIGN;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const long long NH = static_cast<long long>(shape->B) * n_heads;
    if (R == 0) {
        if (x_in != x_out &&
            cudaMemcpyAsync(x_out, x_in, static_cast<size_t>(NH) * shape->S * D * 2, cudaMemcpyDeviceToDevice, stream) !=
                cudaSuccess)
            return AF_ERR_CUDA;
        return AF_OK;
    }
    af_strides st;
    st.b = static_cast<int64_t>(n_heads) * shape->S * D; st.h = static_cast<int64_t>(shape->S) * D; st.s = D;
    return launch_rope(x_in, st, x_out, shape->B, n_heads, shape->S, D, R, rope_table, inverse, stream);
}

}  // extern "C"

namespace {
// Forward, dense (bs_row_ptr == nullptr) or over CSR lists of active 128 x 128 blocks.
af_status fwd_impl(const af_shape* shape, const void* q, const void* k, const void* v, const af_strides* sq,
                   const af_strides* skv, const af_rope* rope, const void* rope_table, const af_mask* mask,
                   int gqa_group, float softmax_scale, const int* bs_row_ptr, const int* bs_col_idx,
                   const int* bs_order, void* o, af_dtype o_dtype, float* lse, bool k_prerotated, void* cuda_stream,
                   const af_blocks* blocks = nullptr, const float* bias = nullptr, int bias_B = 1, int bias_H = 1,
                   int relu = 0) {
    af_status st = check_common(shape, rope, rope_table, mask, gqa_group);
    if (st != AF_OK) return st;
    if (!q || !k || !v || !o) return AF_ERR_NULL;
    if (o_dtype != AF_BF16 && o_dtype != AF_F32) return AF_ERR_DTYPE;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return AF_ERR_ALIGN;
    if (!(softmax_scale > 0.f) || !isfinite(softmax_scale)) return AF_ERR_SPEC;
    if (bias) {
        if ((bias_B != 1 && bias_B != shape->B) || (bias_H != 1 && bias_H != shape->Hq)) return AF_ERR_SHAPE;
        if ((reinterpret_cast<uintptr_t>(bias) & 3u) != 0) return AF_ERR_ALIGN;
    }
    if (relu && bs_row_ptr) return AF_ERR_SPEC;   // the ReLU normaliser is not built over block lists
    af_strides stq, stkv;
    if ((st = resolve_strides(sq, shape->Hq, shape->S, shape->D, &stq)) != AF_OK) return st;
    if ((st = resolve_strides(skv, shape->Hkv, shape->S, shape->D, &stkv)) != AF_OK) return st;
    if ((st = check_arch()) != AF_OK) return st;

    CUtensorMap tq, tk, tv, to;
    if ((st = make_tmap(&tq, q, shape->B, shape->Hq, shape->S, shape->D, stq, BM)) != AF_OK) return st;
    af_strides stk = stkv;
    if (k_prerotated) resolve_strides(nullptr, shape->Hkv, shape->S, shape->D, &stk);   // K' is contiguous
    if ((st = make_tmap(&tk, k, shape->B, shape->Hkv, shape->S, shape->D, stk, BN)) != AF_OK) return st;
    if ((st = make_tmap(&tv, v, shape->B, shape->Hkv, shape->S, shape->D, stkv, BN)) != AF_OK) return st;
    // bf16 output goes out through TMA (contiguous [B,Hq,S,D]); with fp32 output the map is not used
    to = tq;
    if (o_dtype == AF_BF16) {
        af_strides sto;
        resolve_strides(nullptr, shape->Hq, shape->S, shape->D, &sto);
        if ((st = make_tmap(&to, o, shape->B, shape->Hq, shape->S, shape->D, sto, BM)) != AF_OK) return st;
    }

    // (optional mode) key tiles receive the 128 rows of the table's bf16 copy that belong to them by TMA
    const int Rr = rope->rotary_dim;
    CUtensorMap tt = tq;
    const bool keys_bf16 = !k_prerotated && !bias && !relu && keys_rotate_in_bf16(Rr);
    if (keys_bf16 && (st = make_tmap_table(&tt, rope_table, shape->S, Rr)) != AF_OK) return st;

    FwdParams p;
    p.B = shape->B; p.Hq = shape->Hq; p.Hkv = shape->Hkv; p.S = shape->S; p.group = gqa_group;
    p.R = rope->rotary_dim;
    p.causal = mask->causal ? 1 : 0;
    p.window = mask->window < 0 ? -1 : (mask->window > shape->S ? shape->S : mask->window);
    p.scale_log2 = softmax_scale * 1.4426950408889634f;
    p.slopes = mask->alibi_slopes;
    p.table = static_cast<const float2*>(rope_table);
    p.o = o; p.o_f32 = (o_dtype == AF_F32); p.lse = lse;
    p.n_row_blocks = 0;
    p.pair_heads = 0;
    p.bs_row_ptr = bs_row_ptr;
    p.bs_col_idx = bs_col_idx;
    p.bs_order = bs_order;
    p.bs_rowpair = 0;
    if (blocks && (gqa_group % 2) == 1 && blocks->pair_ptr && blocks->pair_idx && opt(AF_OPT_BS_ROWPAIR)) {
        // odd GQA group: no two heads share K and V, so a CTA takes two row blocks of one head instead
        p.bs_row_ptr = blocks->pair_ptr;
        p.bs_col_idx = blocks->pair_idx;
        p.bs_order = blocks->pair_order;
        p.bs_rowpair = 1;
    }
    p.rot_k = k_prerotated ? 0 : 1;
    p.keys_bf16 = keys_bf16 ? 1 : 0;
    p.bias = bias;
    p.bias_sh = (bias && bias_H > 1) ? static_cast<long long>(shape->S) * shape->S : 0;
    p.bias_sb = (bias && bias_B > 1) ? static_cast<long long>(bias_H) * shape->S * shape->S : 0;
    p.relu = relu ? 1 : 0;
#ifdef AF_TRACE
    p.trace = reinterpret_cast<long long*>(getenv("AF_TRACE_PTR") ? strtoull(getenv("AF_TRACE_PTR"), nullptr, 0) : 0ull);
    cudaMemcpyToSymbol(af::g_trace, &p.trace, sizeof(p.trace));
#endif
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (bs_row_ptr)
        return shape->D == 128 ? launch_fwd_blocks<128>(tq, tk, tv, to, tt, p, stream) : launch_fwd_blocks<64>(tq, tk, tv, to, tt, p, stream);
    return shape->D == 128 ? launch_fwd<128>(tq, tk, tv, to, tt, p, stream) : launch_fwd<64>(tq, tk, tv, to, tt, p, stream);
}
}  // namespace

extern "C" {

af_status attnfuse_fwd(const af_shape* shape, const void* q, const void* k, const void* v, const af_strides* sq,
                       const af_strides* skv, const af_rope* rope, const void* rope_table, const af_mask* mask,
                       int gqa_group, float softmax_scale, void* o, af_dtype o_dtype, float* lse, void* cuda_stream) {
    return fwd_impl(shape, q, k, v, sq, skv, rope, rope_table, mask, gqa_group, softmax_scale, nullptr, nullptr, nullptr,
                    o, o_dtype, lse, false, cuda_stream);
}

af_status attnfuse_fwd_variant(const af_shape* shape, const void* q, const void* k, const void* v, const af_strides* sq,
                               const af_strides* skv, const af_variant* variant, int gqa_group, float softmax_scale,
                               void* o, af_dtype o_dtype, float* lse, void* cuda_stream) {
    if (!variant) return AF_ERR_NULL;
    if (variant->normaliser != AF_NORM_SOFTMAX && variant->normaliser != AF_NORM_RELU) return AF_ERR_SPEC;
    const af_blocks* bl = variant->blocks;
    if (bl) {
        if (!bl->row_ptr || !bl->col_idx) return AF_ERR_NULL;
        if (bl->block != 128) return AF_ERR_SPEC;
    }
    return fwd_impl(shape, q, k, v, sq, skv, &variant->rope, variant->rope_table, &variant->mask, gqa_group, softmax_scale,
                    bl ? bl->row_ptr : nullptr, bl ? bl->col_idx : nullptr, bl ? bl->row_order : nullptr, o, o_dtype, lse,
                    false, cuda_stream, bl, variant->bias, variant->bias_B, variant->bias_H,
                    variant->normaliser == AF_NORM_RELU);
}

af_status attnfuse_fwd_fp8(const af_shape* shape, const void* q8, const void* k8, const void* vt8, const af_mask* mask,
                           int gqa_group, float softmax_scale, float scale_q, float scale_k, float scale_v, void* o,
                           af_dtype o_dtype, float* lse, void* cuda_stream) {
    if (!shape || !mask || !q8 || !k8 || !vt8 || !o) return AF_ERR_NULL;
    if (shape->B < 1 || shape->Hq < 1 || shape->Hkv < 1 || shape->S < 1) return AF_ERR_SHAPE;
    if (shape->D != 128 || (shape->S % 16) != 0) return AF_ERR_SHAPE;   // the transposed V has rows of S bytes: 16-byte strides
    if (gqa_group < 1 || shape->Hkv * gqa_group != shape->Hq) return AF_ERR_SHAPE;
    if (mask->alibi_slopes) return AF_ERR_SPEC;
    if (o_dtype != AF_BF16 && o_dtype != AF_F32) return AF_ERR_DTYPE;
    if (!aligned16(q8) || !aligned16(k8) || !aligned16(vt8) || !aligned16(o)) return AF_ERR_ALIGN;
    if (!(softmax_scale > 0.f) || !isfinite(softmax_scale) || !(scale_q > 0.f) || !(scale_k > 0.f) || !(scale_v > 0.f) ||
        !isfinite(scale_q) || !isfinite(scale_k) || !isfinite(scale_v))
        return AF_ERR_SPEC;
    af_status st = check_arch();
    if (st != AF_OK) return st;
    CUtensorMap tq, tk, tv;
    if ((st = make_tmap_u8(&tq, q8, shape->B, shape->Hq, shape->S, shape->D)) != AF_OK) return st;
    if ((st = make_tmap_u8(&tk, k8, shape->B, shape->Hkv, shape->S, shape->D)) != AF_OK) return st;
    if ((st = make_tmap_u8(&tv, vt8, shape->B, shape->Hkv, shape->D, shape->S)) != AF_OK) return st;
    Fp8Params p;
    p.B = shape->B; p.Hq = shape->Hq; p.Hkv = shape->Hkv; p.S = shape->S; p.group = gqa_group;
    p.causal = mask->causal ? 1 : 0;
    p.window = mask->window < 0 ? -1 : (mask->window > shape->S ? shape->S : mask->window);
    p.scale_log2 = softmax_scale * scale_q * scale_k * 1.4426950408889634f;
    p.out_scale = scale_v;
    p.o = o; p.o_f32 = o_dtype == AF_F32; p.lse = lse;
    p.pair_heads = (gqa_group % 2) == 0 ? 1 : 0;
    const int rows_per_cta = p.pair_heads ? BM : 2 * BM;
    p.n_row_blocks = (shape->S + rows_per_cta - 1) / rows_per_cta;
    static std::atomic<unsigned long long> configured{0};
    if (allow_dynamic_smem(attn_fwd_fp8_kernel, Fp8Smem::BYTES, configured) != AF_OK) return AF_ERR_CUDA;
    dim3 grid(p.pair_heads ? p.B * p.Hq / 2 : p.B * p.Hq, p.n_row_blocks, 1);
    attn_fwd_fp8_kernel<<<grid, 512, Fp8Smem::BYTES, static_cast<cudaStream_t>(cuda_stream)>>>(tq, tk, tv, p);
    return cudaGetLastError() == cudaSuccess ? AF_OK : AF_ERR_CUDA;
}

size_t attnfuse_fwd_hybrid_workspace_bytes(const af_shape* shape) {
    if (!shape || shape->B < 1 || shape->Hkv < 1 || shape->S < 1 || shape->D < 1) return 0;
    return static_cast<size_t>(shape->B) * shape->Hkv * shape->S * shape->D * 2;
}

af_status attnfuse_fwd_hybrid(const af_shape* shape, const void* q, const void* k, const void* v, const af_strides* sq,
                              const af_strides* skv, const af_rope* rope, const void* rope_table, const af_mask* mask,
                              int gqa_group, float softmax_scale, void* o, af_dtype o_dtype, float* lse,
                              void* workspace, size_t workspace_bytes, void* cuda_stream) {
    af_status st = check_common(shape, rope, rope_table, mask, gqa_group);
    if (st != AF_OK) return st;
    if (rope->rotary_dim == 0)   // nothing to rotate: the plain kernel
        return fwd_impl(shape, q, k, v, sq, skv, rope, rope_table, mask, gqa_group, softmax_scale, nullptr, nullptr,
                        nullptr, o, o_dtype, lse, false, cuda_stream);
    if (!k || !workspace) return AF_ERR_NULL;
    if (workspace_bytes < attnfuse_fwd_hybrid_workspace_bytes(shape)) return AF_ERR_WORKSPACE;
    if (!aligned16(k) || !aligned16(workspace)) return AF_ERR_ALIGN;
    af_strides stkv;
    if ((st = resolve_strides(skv, shape->Hkv, shape->S, shape->D, &stkv)) != AF_OK) return st;
    if ((st = check_arch()) != AF_OK) return st;
    // K' = RoPE(K) once, contiguous, into the workspace; the kernel then rotates only its Q tiles
    if ((st = launch_rope(k, stkv, workspace, shape->B, shape->Hkv, shape->S, shape->D, rope->rotary_dim, rope_table, 0,
                          static_cast<cudaStream_t>(cuda_stream))) != AF_OK)
        return st;
    return fwd_impl(shape, q, workspace, v, sq, skv, rope, rope_table, mask, gqa_group, softmax_scale, nullptr, nullptr,
                    nullptr, o, o_dtype, lse, true, cuda_stream);
}

af_status attnfuse_fwd_blocks(const af_shape* shape, const void* q, const void* k, const void* v, const af_strides* sq,
                              const af_strides* skv, const af_rope* rope, const void* rope_table, const af_mask* mask,
                              int gqa_group, float softmax_scale, const af_blocks* blocks, void* o, af_dtype o_dtype,
                              float* lse, void* cuda_stream) {
    if (!blocks || !blocks->row_ptr || !blocks->col_idx) return AF_ERR_NULL;
    if (blocks->block != 128) return AF_ERR_SPEC;
    return fwd_impl(shape, q, k, v, sq, skv, rope, rope_table, mask, gqa_group, softmax_scale, blocks->row_ptr,
                    blocks->col_idx, blocks->row_order, o, o_dtype, lse, false, cuda_stream, blocks);
}

size_t attnfuse_fwd_host_staging_bytes(const af_shape* shape) {
    if (!shape) return 0;
    const size_t qn = static_cast<size_t>(shape->B) * shape->Hq * shape->S * shape->D * 2;
    const size_t kn = static_cast<size_t>(shape->B) * shape->Hkv * shape->S * shape->D * 2;
    const size_t ln = static_cast<size_t>(shape->B) * shape->Hq * shape->S * 4;
    return 2 * qn + 2 * kn + ln + 1024;
}

af_status attnfuse_fwd_host(const af_shape* shape, const void* q_host, const void* k_host, const void* v_host,
                            const af_rope* rope, const void* rope_table, const af_mask* mask, int gqa_group,
                            float softmax_scale, void* o_host, float* lse_host, void* staging, size_t staging_bytes,
                            void* cuda_stream) {
    if (!shape || !q_host || !k_host || !v_host || !o_host || !staging) return AF_ERR_NULL;
    af_status st = check_common(shape, rope, rope_table, mask, gqa_group);
    if (st != AF_OK) return st;
    if (staging_bytes < attnfuse_fwd_host_staging_bytes(shape)) return AF_ERR_WORKSPACE;
    if (!aligned16(staging)) return AF_ERR_ALIGN;
    const size_t row = static_cast<size_t>(shape->S) * shape->D * 2;   // bytes of one head of Q, K, V or O
    const size_t qn = static_cast<size_t>(shape->B) * shape->Hq * row;
    const size_t kn = static_cast<size_t>(shape->B) * shape->Hkv * row;
    uint8_t* base = static_cast<uint8_t*>(staging);
    uint8_t *dq = base, *dk = dq + qn, *dv = dk + kn, *dob = dv + kn, *dl = dob + qn;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    // Work units (batch element, kv head with its query heads) are independent and contiguous in every tensor, so
    // the call is cut into chunks of consecutive units and pipelined: the host-to-device copies of chunk c + 1 (on
    // the caller's stream), the kernel of chunk c (internal stream) and the device-to-host copies of chunk c - 1
    // (second internal stream) run at the same time; the two copy directions use different DMA engines.
    // Chunking: whole batch elements when there are at least 8 of them, else groups of kv heads per batch element.
    int nb = 1, nh = shape->Hkv;   // a chunk = nb batch elements x nh kv heads
    if (shape->B >= 8) {
        nb = (shape->B + 7) / 8;
    } else {
        int per_batch = (8 + shape->B - 1) / shape->B;
        if (per_batch > shape->Hkv) per_batch = shape->Hkv;
        while (shape->Hkv % per_batch) --per_batch;
        nh = shape->Hkv / per_batch;
    }
    const int chunks_b = (shape->B + nb - 1) / nb, chunks_h = shape->Hkv / nh;
    std::lock_guard<std::mutex> lock(g_pipe_mutex);
    HostPipe* pipe = get_pipe();
    if (!pipe) return AF_ERR_CUDA;
    // Whatever happens below, work may already sit on the internal streams when the call returns: on every exit
    // path the caller's stream is made to wait for it, so that reusing `staging` or the host buffers afterwards
    // (in stream order) cannot race with copies or kernels still in flight.
    struct JoinOnExit {
        HostPipe* pipe;
        cudaStream_t stream;
        bool done = false;
        af_status join() {
            done = true;
            cudaEvent_t a = pipe->ev[pipe->next];
            pipe->next = (pipe->next + 1) % HostPipe::kEvents;
            cudaEvent_t b = pipe->ev[pipe->next];
            pipe->next = (pipe->next + 1) % HostPipe::kEvents;
            bool ok = cudaEventRecord(a, pipe->compute) == cudaSuccess && cudaStreamWaitEvent(stream, a, 0) == cudaSuccess;
            ok = cudaEventRecord(b, pipe->d2h) == cudaSuccess && cudaStreamWaitEvent(stream, b, 0) == cudaSuccess && ok;
            return ok ? AF_OK : AF_ERR_CUDA;
        }
        ~JoinOnExit() { if (!done) join(); }
    } joiner{pipe, stream};
    auto next_event = [&]() {
        cudaEvent_t e = pipe->ev[pipe->next];
        pipe->next = (pipe->next + 1) % HostPipe::kEvents;
        return e;
    };
    // the internal streams start after whatever the caller's stream holds so far (e.g. the table build)
    cudaEvent_t e0 = next_event();
    if (cudaEventRecord(e0, stream) != cudaSuccess || cudaStreamWaitEvent(pipe->compute, e0, 0) != cudaSuccess ||
        cudaStreamWaitEvent(pipe->d2h, e0, 0) != cudaSuccess)
        return AF_ERR_CUDA;
    // K and V go first, each as one copy, then one copy of Q per chunk: several small host-to-device copies per
    // chunk interleaved with the device-to-host copies of earlier chunks overlapped poorly (1.42 ms against 1.07 ms
    // for the same bytes at config 2)
    if (cudaMemcpyAsync(dk, k_host, kn, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaMemcpyAsync(dv, v_host, kn, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return AF_ERR_CUDA;
    for (int cb = 0; cb < chunks_b; ++cb) {
        const int b0 = cb * nb, bn = (b0 + nb <= shape->B) ? nb : shape->B - b0;
        for (int ch = 0; ch < chunks_h; ++ch) {
            const int hk0 = ch * nh, hq0 = hk0 * gqa_group;
            // with nh < Hkv a chunk lies inside one batch element (bn = 1), so it is contiguous in every tensor
            const size_t q_off = (static_cast<size_t>(b0) * shape->Hq + hq0) * row;
            const size_t k_off = (static_cast<size_t>(b0) * shape->Hkv + hk0) * row;
            const size_t q_bytes = static_cast<size_t>(bn) * nh * gqa_group * row;
            const size_t l_off = (static_cast<size_t>(b0) * shape->Hq + hq0) * shape->S * 4;
            const uint8_t* qh = static_cast<const uint8_t*>(q_host);
            if (cudaMemcpyAsync(dq + q_off, qh + q_off, q_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess)
                return AF_ERR_CUDA;
            cudaEvent_t e_in = next_event(), e_k = next_event();
            if (cudaEventRecord(e_in, stream) != cudaSuccess || cudaStreamWaitEvent(pipe->compute, e_in, 0) != cudaSuccess)
                return AF_ERR_CUDA;
            af_shape cs = {bn, nh * gqa_group, nh, shape->S, shape->D};
            af_mask cm = *mask;
            if (cm.alibi_slopes) cm.alibi_slopes += hq0;
            // strides of the full tensors: a chunk of kv heads inside a batch element keeps the batch stride
            af_strides sq, skv;
            sq.s = skv.s = shape->D;
            sq.h = skv.h = static_cast<int64_t>(shape->S) * shape->D;
            sq.b = static_cast<int64_t>(shape->Hq) * shape->S * shape->D;
            skv.b = static_cast<int64_t>(shape->Hkv) * shape->S * shape->D;
            // the output of a chunk is contiguous [bn, heads, S, D] only if the chunk covers whole batch elements or
            // a single one; both hold here (bn = 1 when nh < Hkv)
            st = attnfuse_fwd(&cs, dq + q_off, dk + k_off, dv + k_off, &sq, &skv, rope, rope_table, &cm, gqa_group,
                              softmax_scale, dob + q_off, AF_BF16, lse_host ? reinterpret_cast<float*>(dl + l_off) : nullptr,
                              pipe->compute);
            if (st != AF_OK) return st;
            if (cudaEventRecord(e_k, pipe->compute) != cudaSuccess || cudaStreamWaitEvent(pipe->d2h, e_k, 0) != cudaSuccess)
                return AF_ERR_CUDA;
            if (cudaMemcpyAsync(static_cast<uint8_t*>(o_host) + q_off, dob + q_off, q_bytes, cudaMemcpyDeviceToHost,
                                pipe->d2h) != cudaSuccess)
                return AF_ERR_CUDA;
        }
    }
    // L in one copy at the end (small copies between the large ones cost overlap, as above)
    const size_t ln = static_cast<size_t>(shape->B) * shape->Hq * shape->S * 4;
    if (lse_host && cudaMemcpyAsync(lse_host, dl, ln, cudaMemcpyDeviceToHost, pipe->d2h) != cudaSuccess) return AF_ERR_CUDA;
    // the caller's stream continues once the last results are on the host
    return joiner.join();
}

int attnfuse_decode_splits(const af_shape* shape) {
    if (!shape || shape->B < 1 || shape->Hkv < 1 || shape->S < 1) return 0;
    // one CTA per SM fits (its stages take most of the shared memory): as many splits as give at most one
    // CTA per SM of the current device in a single wave, at least 128 keys (one tile per warp) per split
    const int ctas_per_split = shape->B * shape->Hkv;
    int sms = sm_count();
    if (sms < 1) sms = 148;   // no device to ask (host-only callers sizing a workspace): the B200 count
    const int want = sms / ctas_per_split;
    const int most = (shape->S + 127) / 128;
    return want < 1 ? 1 : (want > most ? most : want);
}

// bytes of the ticket counters at the head of the decode workspace (one per (batch, kv head), rounded up to 256)
static size_t decode_ticket_bytes(const af_shape* shape) {
    return (static_cast<size_t>(shape->B) * shape->Hkv * sizeof(unsigned int) + 255) / 256 * 256;
}

size_t attnfuse_decode_workspace_bytes(const af_shape* shape, int n_splits) {
    if (!shape) return 0;
    if (n_splits <= 0) n_splits = attnfuse_decode_splits(shape);
    return decode_ticket_bytes(shape) + static_cast<size_t>(shape->B) * shape->Hq * n_splits * (shape->D + 2) * sizeof(float);
}

af_status attnfuse_decode_workspace_init(void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!workspace) return AF_ERR_NULL;
    if (!aligned16(workspace)) return AF_ERR_ALIGN;
    return cudaMemsetAsync(workspace, 0, workspace_bytes, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? AF_OK
                                                                                                              : AF_ERR_CUDA;
}

af_status attnfuse_decode(const af_shape* shape, const void* q, const void* k, const void* v, const af_strides* skv,
                          const af_mask* mask, int gqa_group, float softmax_scale, void* o, float* lse, int n_splits,
                          void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!shape || !mask || !q || !k || !v || !o || !workspace) return AF_ERR_NULL;
    if (shape->B < 1 || shape->Hq < 1 || shape->Hkv < 1 || shape->S < 1) return AF_ERR_SHAPE;
    if (shape->D != 64 && shape->D != 128) return AF_ERR_SHAPE;
    if (gqa_group < 1 || gqa_group > 16 || shape->Hkv * gqa_group != shape->Hq) return AF_ERR_SHAPE;
    if (static_cast<long long>(shape->B) * shape->Hkv > 65535) return AF_ERR_SHAPE;
    if (!(softmax_scale > 0.f) || !isfinite(softmax_scale)) return AF_ERR_SPEC;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(workspace)) return AF_ERR_ALIGN;
    if (n_splits <= 0) n_splits = attnfuse_decode_splits(shape);
    if (n_splits > (shape->S + 127) / 128) n_splits = (shape->S + 127) / 128;
    if (n_splits > kCombineMaxSplits) n_splits = kCombineMaxSplits;
    if (workspace_bytes < attnfuse_decode_workspace_bytes(shape, n_splits)) return AF_ERR_WORKSPACE;
    af_status st;
    af_strides stkv;
    if ((st = resolve_strides(skv, shape->Hkv, shape->S, shape->D, &stkv)) != AF_OK) return st;
    if ((st = check_arch()) != AF_OK) return st;
    CUtensorMap tk, tv;
    if ((st = make_tmap(&tk, k, shape->B, shape->Hkv, shape->S, shape->D, stkv, kDecTile)) != AF_OK) return st;
    if ((st = make_tmap(&tv, v, shape->B, shape->Hkv, shape->S, shape->D, stkv, kDecTile)) != AF_OK) return st;
    DecodeParams p;
    p.B = shape->B; p.Hq = shape->Hq; p.Hkv = shape->Hkv; p.N = shape->S; p.group = gqa_group;
    p.window = mask->window < 0 ? -1 : mask->window;
    p.scale_log2 = softmax_scale * 1.4426950408889634f;
    p.slopes = mask->alibi_slopes;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.n_splits = n_splits;
    p.tickets = static_cast<unsigned int*>(workspace);
    p.part_o = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + decode_ticket_bytes(shape));
    p.part_ml = p.part_o + static_cast<size_t>(shape->B) * shape->Hq * n_splits * shape->D;
    p.o = static_cast<__nv_bfloat16*>(o);
    p.lse = lse;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    dim3 grid(n_splits, shape->B * shape->Hkv, 1);
    if (shape->D == 128) {
        static std::atomic<unsigned long long> configured{0};
        if (allow_dynamic_smem(decode_split_kernel<128>, DecodeSmem<128>::BYTES, configured) != AF_OK) return AF_ERR_CUDA;
        decode_split_kernel<128><<<grid, kDecWarps * 32, DecodeSmem<128>::BYTES, stream>>>(tk, tv, p);
    } else {
        static std::atomic<unsigned long long> configured{0};
        if (allow_dynamic_smem(decode_split_kernel<64>, DecodeSmem<64>::BYTES, configured) != AF_OK) return AF_ERR_CUDA;
        decode_split_kernel<64><<<grid, kDecWarps * 32, DecodeSmem<64>::BYTES, stream>>>(tk, tv, p);
    }
    return cudaGetLastError() == cudaSuccess ? AF_OK : AF_ERR_CUDA;
}

size_t attnfuse_bwd_workspace_bytes(const af_shape* shape) {
    if (!shape) return 0;
    return bwd_delta_bytes(shape) + bwd_kcache_bytes(shape) + bwd_qcache_bytes(shape);   // delta + rotated-K and -Q caches
}

size_t attnfuse_bwd_onepass_workspace_bytes(const af_shape* shape) {
    if (!shape) return 0;
    return attnfuse_bwd_workspace_bytes(shape) + bwd_dqacc_bytes(shape);   // ... + the fp32 accumulator of dQ'
}

}  // extern "C"

namespace {
// Backward, dense (blocks == nullptr) or over the index lists of active 128 x 128 blocks.
af_status bwd_impl(const af_shape* shape, const void* q, const void* k, const void* v, const void* o,
                   const float* lse, const void* d_o, const af_strides* sq, const af_strides* skv,
                   const af_rope* rope, const void* rope_table, const af_mask* mask, int gqa_group,
                   float softmax_scale, const af_blocks* blocks, void* dq, af_dtype dq_dtype, void* dk, void* dv,
                   af_dtype dkv_dtype, void* workspace, size_t workspace_bytes, void* cuda_stream,
                   const float* bias = nullptr, int bias_B = 1, int bias_H = 1, int relu = 0) {
    af_status st = check_common(shape, rope, rope_table, mask, gqa_group);
    if (st != AF_OK) return st;
    if (!q || !k || !v || !o || !lse || !d_o || !dq || !dk || !dv) return AF_ERR_NULL;
    const bool gen = bias != nullptr || relu != 0;
    if (bias) {
        if ((bias_B != 1 && bias_B != shape->B) || (bias_H != 1 && bias_H != shape->Hq)) return AF_ERR_SHAPE;
        if ((reinterpret_cast<uintptr_t>(bias) & 3u) != 0) return AF_ERR_ALIGN;
    }
    if (gen && blocks) return AF_ERR_SPEC;   // the extras are not built over block lists
    if ((dq_dtype != AF_BF16 && dq_dtype != AF_F32) || (dkv_dtype != AF_BF16 && dkv_dtype != AF_F32))
        return AF_ERR_DTYPE;
    if (!workspace || workspace_bytes < bwd_delta_bytes(shape)) return AF_ERR_WORKSPACE;   // the cache is optional
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(d_o) || !aligned16(dq) ||
        !aligned16(dk) || !aligned16(dv) || !aligned16(workspace) || !aligned16(lse))
        return AF_ERR_ALIGN;
    if (!(softmax_scale > 0.f) || !isfinite(softmax_scale)) return AF_ERR_SPEC;
    af_strides stq, stkv, stc;
    if ((st = resolve_strides(sq, shape->Hq, shape->S, shape->D, &stq)) != AF_OK) return st;
    if ((st = resolve_strides(skv, shape->Hkv, shape->S, shape->D, &stkv)) != AF_OK) return st;
    resolve_strides(nullptr, shape->Hq, shape->S, shape->D, &stc);
    if ((st = check_arch()) != AF_OK) return st;
    CUtensorMap tq, tk, tv, tdo;
    if ((st = make_tmap(&tq, q, shape->B, shape->Hq, shape->S, shape->D, stq, 128)) != AF_OK) return st;
    if ((st = make_tmap(&tk, k, shape->B, shape->Hkv, shape->S, shape->D, stkv, 128)) != AF_OK) return st;
    if ((st = make_tmap(&tv, v, shape->B, shape->Hkv, shape->S, shape->D, stkv, 128)) != AF_OK) return st;
    if ((st = make_tmap(&tdo, d_o, shape->B, shape->Hq, shape->S, shape->D, stc, 128)) != AF_OK) return st;
    BwdParams p;
    p.B = shape->B; p.Hq = shape->Hq; p.Hkv = shape->Hkv; p.S = shape->S; p.group = gqa_group;
    p.R = rope->rotary_dim;
    p.causal = mask->causal ? 1 : 0;
    p.window = mask->window < 0 ? -1 : (mask->window > shape->S ? shape->S : mask->window);
    p.scale = softmax_scale;
    p.scale_log2 = softmax_scale * 1.4426950408889634f;
    p.slopes = mask->alibi_slopes;
    p.table = static_cast<const float2*>(rope_table);
    p.lse = lse;
    p.delta = nullptr; p.out1 = nullptr; p.out2 = nullptr; p.out_f32 = 0; p.store_x = 0;
    p.bs_ptr = nullptr; p.bs_idx = nullptr; p.bs_order = nullptr; p.skip_rows = 0;
    p.bias = bias;
    p.bias_sb = (bias && bias_B > 1) ? static_cast<long long>(bias_H) * shape->S * shape->S : 0;
    p.bias_sh = (bias && bias_H > 1) ? static_cast<long long>(shape->S) * shape->S : 0;
    p.relu = relu ? 1 : 0;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    float* delta = static_cast<float*>(workspace);
    // rotated-K and rotated-Q caches: used when there is a rotation and the workspace has room behind delta
    CUtensorMap tkp, tqp;
    const size_t off_k = bwd_delta_bytes(shape), off_q = off_k + bwd_kcache_bytes(shape);
    const size_t off_acc = off_q + bwd_qcache_bytes(shape);
    // One-pass sequence: dense, room for both caches and the fp32 dQ' accumulator, and not switched off.
    // Left to itself (option value 1) the choice goes by the average number of kept key tiles per query tile: the
    // one-pass kernel costs more per tile pair than the two roles of the two-kernel sequence together, but the dQ
    // role pays a fixed set-up and epilogue per query tile, which dominates while rows are short (measured: ahead at
    // 8.5 and 9.5 tiles per query tile, behind at 16.5).
    const int mode = opt(AF_OPT_BWD_ONEPASS);
    const double n_tiles = (shape->S + 127) / 128;
    double avg_tiles = p.causal ? 0.5 * (n_tiles + 1) : n_tiles;
    if (p.window >= 0) avg_tiles = std::min(avg_tiles, (p.causal ? 1.0 : 2.0) * p.window / 128.0 + 1.5);
    // At D = 64 the one-pass sequence measured 1.2-1.3 times faster on every shape tried (short and long rows,
    // grouped queries, window, no causal mask): shared-memory traffic per tile pair is half that of D = 128.
    // Over block lists (short lists are the rule there) it is taken at D = 64 and, at D = 128, only on request.
    const bool onepass = !gen && workspace_bytes >= off_acc + bwd_dqacc_bytes(shape) &&
                         (mode >= 2 || (mode == 1 && (shape->D == 64 || (!blocks && avg_tiles <= 12.0))));
    const bool have_k = p.R > 0 && workspace_bytes >= off_q;
    const bool have_q = have_k && workspace_bytes >= off_acc;
    void* kc = static_cast<uint8_t*>(workspace) + off_k;
    void* qc = static_cast<uint8_t*>(workspace) + off_q;
    if (have_k) {
        af_strides stk;
        resolve_strides(nullptr, shape->Hkv, shape->S, shape->D, &stk);
        if ((st = make_tmap(&tkp, kc, shape->B, shape->Hkv, shape->S, shape->D, stk, 128)) != AF_OK) return st;
    }
    if (have_q) {
        if ((st = make_tmap(&tqp, qc, shape->B, shape->Hq, shape->S, shape->D, stc, 128)) != AF_OK) return st;
    }
    // Under a causal mask (dense, not over block lists) the first query rows of every head are computed in fp32 by a
    // small kernel of their own and dropped from the MMA kernels: see bwd_first_rows.cuh.
    FirstRowsParams fp = {};
    fp.B = shape->B; fp.Hq = shape->Hq; fp.Hkv = shape->Hkv; fp.S = shape->S; fp.group = gqa_group;
    fp.R = p.R; fp.window = p.window;
    // (not with additive_bias / relu_attention either: the fp32 kernel knows neither)
    fp.rows = (p.causal && !blocks && !gen) ? (shape->S < kFirstRows ? shape->S : kFirstRows) : 0;
    fp.scale = softmax_scale;
    fp.slopes = p.slopes; fp.table = p.table;
    fp.q = static_cast<const __nv_bfloat16*>(q); fp.k = static_cast<const __nv_bfloat16*>(k);
    fp.v = static_cast<const __nv_bfloat16*>(v); fp.d_o = static_cast<const __nv_bfloat16*>(d_o);
    fp.qb = stq.b; fp.qh = stq.h; fp.qs = stq.s; fp.kb = stkv.b; fp.kh = stkv.h; fp.ks = stkv.s;
    fp.dq = dq; fp.dk = dk; fp.dv = dv;
    fp.dq_f32 = dq_dtype == AF_F32; fp.dkv_f32 = dkv_dtype == AF_F32;
    OnePassArgs op = {};
    op.q = q; op.stq = stq; op.qcache = qc;
    op.dq_acc = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + off_acc);
    op.dq_acc_bytes = bwd_dqacc_bytes(shape);
    op.blocks = blocks;
    p.dq_acc = nullptr;
    return shape->D == 128
               ? launch_bwd<128>(shape, tq, tk, tv, tdo, have_k ? &tkp : nullptr, have_q ? &tqp : nullptr, k, stkv, kc, o,
                                 d_o, p, dq, dq_dtype == AF_F32, dk, dv, dkv_dtype == AF_F32, delta, blocks, stream, fp,
                                 onepass ? &op : nullptr)
               : launch_bwd<64>(shape, tq, tk, tv, tdo, have_k ? &tkp : nullptr, have_q ? &tqp : nullptr, k, stkv, kc, o,
                                d_o, p, dq, dq_dtype == AF_F32, dk, dv, dkv_dtype == AF_F32, delta, blocks, stream, fp,
                                onepass ? &op : nullptr);
}
}  // namespace

extern "C" {

af_status attnfuse_bwd(const af_shape* shape, const void* q, const void* k, const void* v, const void* o,
                       const float* lse, const void* d_o, const af_strides* sq, const af_strides* skv,
                       const af_rope* rope, const void* rope_table, const af_mask* mask, int gqa_group,
                       float softmax_scale, void* dq, af_dtype dq_dtype, void* dk, void* dv, af_dtype dkv_dtype,
                       void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return bwd_impl(shape, q, k, v, o, lse, d_o, sq, skv, rope, rope_table, mask, gqa_group, softmax_scale, nullptr, dq,
                    dq_dtype, dk, dv, dkv_dtype, workspace, workspace_bytes, cuda_stream);
}

af_status attnfuse_bwd_variant(const af_shape* shape, const void* q, const void* k, const void* v, const void* o,
                               const float* lse, const void* d_o, const af_strides* sq, const af_strides* skv,
                               const af_variant* variant, int gqa_group, float softmax_scale, void* dq, af_dtype dq_dtype,
                               void* dk, void* dv, af_dtype dkv_dtype, void* workspace, size_t workspace_bytes,
                               void* cuda_stream) {
    if (!variant) return AF_ERR_NULL;
    if (variant->normaliser != AF_NORM_SOFTMAX && variant->normaliser != AF_NORM_RELU) return AF_ERR_SPEC;
    const af_blocks* bl = variant->blocks;
    if (bl) {
        if (!bl->row_ptr || !bl->col_idx || !bl->col_ptr || !bl->row_idx) return AF_ERR_NULL;
        if (bl->block != 128) return AF_ERR_SPEC;
    }
    return bwd_impl(shape, q, k, v, o, lse, d_o, sq, skv, &variant->rope, variant->rope_table, &variant->mask, gqa_group,
                    softmax_scale, bl, dq, dq_dtype, dk, dv, dkv_dtype, workspace, workspace_bytes, cuda_stream, variant->bias,
                    variant->bias_B, variant->bias_H, variant->normaliser == AF_NORM_RELU);
}

af_status attnfuse_bwd_blocks(const af_shape* shape, const void* q, const void* k, const void* v, const void* o,
                              const float* lse, const void* d_o, const af_strides* sq, const af_strides* skv,
                              const af_rope* rope, const void* rope_table, const af_mask* mask, int gqa_group,
                              float softmax_scale, const af_blocks* blocks, void* dq, af_dtype dq_dtype, void* dk,
                              void* dv, af_dtype dkv_dtype, void* workspace, size_t workspace_bytes,
                              void* cuda_stream) {
    if (!blocks || !blocks->row_ptr || !blocks->col_idx || !blocks->col_ptr || !blocks->row_idx) return AF_ERR_NULL;
    if (blocks->block != 128) return AF_ERR_SPEC;
    return bwd_impl(shape, q, k, v, o, lse, d_o, sq, skv, rope, rope_table, mask, gqa_group, softmax_scale, blocks, dq,
                    dq_dtype, dk, dv, dkv_dtype, workspace, workspace_bytes, cuda_stream);
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------------
// Backward for callers that cannot obtain device memory when they call: the scratch (delta) lives in
// a fixed device array of this library.  In host code the array's name is only a stand-in for the
// symbol, not a device address, so its address is looked up once per device and passed on as a
// pointer.  Every call on a device shares the array; see the header for the rules.
static __device__ __align__(256) unsigned char g_bwd_static_scratch[AF_BWD_STATIC_MAX_ROWS * sizeof(float) + 256];   // delta only

namespace {
constexpr int kMaxDevices = 64;
void* g_bwd_static_ptr[kMaxDevices] = {};
std::mutex g_bwd_static_mutex;
}  // namespace

extern "C" af_status attnfuse_bwd_static(const af_shape* shape, const void* q, const void* k, const void* v,
                                         const void* o, const float* lse, const void* d_o, const af_strides* sq,
                                         const af_strides* skv, const af_rope* rope, const void* rope_table,
                                         const af_mask* mask, int gqa_group, float softmax_scale, void* dq,
                                         af_dtype dq_dtype, void* dk, void* dv, af_dtype dkv_dtype,
                                         void* cuda_stream) {
    if (!shape) return AF_ERR_NULL;
    if (shape->B < 1 || shape->Hq < 1 || shape->S < 1) return AF_ERR_SHAPE;
    const long long rows = static_cast<long long>(shape->B) * shape->Hq * shape->S;
    if (rows > AF_BWD_STATIC_MAX_ROWS) return AF_ERR_STATIC_LIMIT;
    static_assert(sizeof(g_bwd_static_scratch) >= AF_BWD_STATIC_MAX_ROWS * sizeof(float) + 256, "scratch holds delta");
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return AF_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return AF_ERR_CUDA;
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_bwd_static_mutex);
        if (!g_bwd_static_ptr[dev]) {
            // once per device, with that device current
            void* ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_bwd_static_scratch) != cudaSuccess || !ptr) return AF_ERR_CUDA;
            g_bwd_static_ptr[dev] = ptr;
        }
        scratch = g_bwd_static_ptr[dev];
    }
    // the size passed is delta's alone, so that the call always takes the delta-only set-up whatever the problem
    // size (with more room attnfuse_bwd would also place its rotated-K / rotated-Q caches in the array)
    return attnfuse_bwd(shape, q, k, v, o, lse, d_o, sq, skv, rope, rope_table, mask, gqa_group, softmax_scale, dq,
                        dq_dtype, dk, dv, dkv_dtype, scratch, bwd_delta_bytes(shape), cuda_stream);
}
