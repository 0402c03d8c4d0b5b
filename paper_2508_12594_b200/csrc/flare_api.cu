// Host side of libflare: argument checks, launch plans, kernel launches.  See include/flare.h for the contract.
#include "../../include/flare.h"

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>

#include <cstdlib>

#include "flare_common.cuh"
#include "flare_simt.cuh"
#include "flare_bwd.cuh"
#include "flare_tc.cuh"
#include "flare_bwd_tc.cuh"
#include "flare_spectral.cuh"
#include "flare_micro.cuh"

using namespace flare;

namespace {

thread_local char g_cuda_error[256] = "";

int cuda_fail(cudaError_t e, const char *what) {
    snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", what, cudaGetErrorString(e));
    return FLARE_ERR_CUDA;
}

#define FLARE_CUDA(call)                                      \
    do {                                                      \
        cudaError_t e__ = (call);                             \
        if (e__ != cudaSuccess) return cuda_fail(e__, #call); \
    } while (0)

struct DeviceInfo {
    std::atomic<int> checked{0};  // 0 = not yet, 1 = ok, -1 = wrong arch, -2 = no device
    std::atomic<int> sms{148};
};
DeviceInfo g_dev[64];

// Properties of the current device (cached per ordinal; concurrent first calls write the same values).  Without
// a device the plan falls back to 148 SMs so that size queries still answer.
struct DeviceView {
    int checked, sms;
};
DeviceView device_info(int *ordinal_out = nullptr) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return DeviceView{-2, 148};
    }
    if (ordinal_out) *ordinal_out = dev;
    DeviceInfo &d = g_dev[dev];
    int checked = d.checked.load(std::memory_order_acquire);
    if (checked == 0) {
        int major = 0, sms = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            cudaGetLastError();
            return DeviceView{-2, 148};
        }
        d.sms.store(sms > 0 ? sms : 148, std::memory_order_relaxed);
        checked = (major == 10) ? 1 : -1;
        d.checked.store(checked, std::memory_order_release);
    }
    return DeviceView{checked, d.sms.load(std::memory_order_relaxed)};
}

// The opt-in to more than 48 KB of dynamic shared memory is a property of (kernel, device): one bit per device
// ordinal in a mask per kernel instantiation.  Setting it twice is harmless, so a race between host threads
// only repeats the call.
template <typename Kernel>
int ensure_big_smem(Kernel kernel, std::atomic<uint64_t> &done, int bytes = 227 * 1024) {
    int dev = 0;
    FLARE_CUDA(cudaGetDevice(&dev));
    const uint64_t bit = 1ull << (dev & 63);
    if (done.load(std::memory_order_acquire) & bit) return FLARE_OK;
    FLARE_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    done.fetch_or(bit, std::memory_order_release);
    return FLARE_OK;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_desc(const flare_desc_t *d) {
    if (d == nullptr) return FLARE_ERR_INVALID_ARG;
    if (d->B <= 0 || d->H <= 0 || d->N <= 0 || d->M <= 0 || d->D <= 0) return FLARE_ERR_INVALID_ARG;
    if (!std::isfinite(d->scale)) return FLARE_ERR_INVALID_ARG;
    if (d->dtype != FLARE_DTYPE_F32 && d->dtype != FLARE_DTYPE_BF16 && d->dtype != FLARE_DTYPE_F16) return FLARE_ERR_UNSUPPORTED;
    if (d->D != 4 && d->D != 8 && d->D != 16 && d->D != 32 && d->D != 64) return FLARE_ERR_UNSUPPORTED;
    if (d->dtype == FLARE_DTYPE_BF16 && (d->M % 16 != 0 || d->M < 16 || d->M > 2048)) return FLARE_ERR_UNSUPPORTED;
    if ((long)d->B * d->N > (1L << 31) - 1 || d->H > 65535 || d->B > 65535) return FLARE_ERR_UNSUPPORTED;
    return FLARE_OK;
}

// Launch plan of the CUDA-core encode: LM latents x G token groups per block, `splits` blocks along N.
struct SimtPlan {
    int LM, G, splits, chunk, P;
};

SimtPlan simt_plan(const flare_desc_t *d, int sms) {
    SimtPlan p;
    p.LM = 1;
    while (p.LM < d->M && p.LM < kSimtThreads) p.LM *= 2;
    p.G = kSimtThreads / p.LM;
    long bh = (long)d->B * d->H;
    long want = (4L * sms + bh - 1) / bh;                  // about four blocks per SM in total
    long most = (d->N + 255) / 256;                        // at least 256 tokens per block
    long s = want < most ? want : most;
    if (s < 1) s = 1;
    p.chunk = (int)((d->N + s - 1) / s);
    p.chunk = (p.chunk + kSimtTileN - 1) / kSimtTileN * kSimtTileN;
    p.splits = (d->N + p.chunk - 1) / p.chunk;
    p.P = p.splits * p.G;
    return p;
}

// The tensor-core kernels take bfloat16 with D in {16, 32, 64} and a positive scale, and D = 8 or 4 as the narrow
// forms of the D = 16 kernels: a token tile of 16 feature columns then spans two or four heads, so the tensor must
// be at least 16 columns wide, and (TMA) its rows a multiple of 16 bytes.  Everything else (float32, non-positive
// scale, narrower tensors) runs on the CUDA-core kernels.  FLARE_DEBUG_PATH=simt forces the latter.
bool use_tc(const flare_desc_t *d) {
    static const bool forced_simt = [] {
        const char *e = std::getenv("FLARE_DEBUG_PATH");
        return e != nullptr && std::strcmp(e, "simt") == 0;
    }();
    // (a scale so small that scale * kMaskedScore no longer dwarfs every real score would let padded tokens through the
    // form that puts padding into the scores: such calls run on the CUDA cores too)
    return !forced_simt && d->dtype == FLARE_DTYPE_BF16 && d->scale > 1e-20f &&
           (d->D == 16 || d->D == 32 || d->D == 64 || (d->D == 8 && d->H >= 2) || (d->D == 4 && d->H >= 4 && d->H % 2 == 0));
}

// Which form of the tensor-core forward kernels runs (flare_set_path).
std::atomic<int> g_path{FLARE_PATH_AUTO};

// The fast forms (no running maximum, see kFastMaxLog2 in flare_tc.cuh) are followed by a launch of the exact
// form that exits at once unless it is needed: two more launches per forward, which pay off from a few tens of
// microseconds of work.
enum FastStage { kFastEncode, kFastDecode };
bool use_fast(const flare_desc_t *d, FastStage stage) {
    if (!use_tc(d)) return false;
    if (stage == kFastDecode && d->D > 32) return false;           // the streaming decode has no form for head width 64
    const int path = g_path.load(std::memory_order_relaxed);
    if (path == FLARE_PATH_EXACT) return false;
    if (path == FLARE_PATH_FAST) return true;
    // Measured (forward stage times, fast against exact form): encode wins from 128 latents (3-5 % there, 15 % at 256),
    // is equal or loses at 32 and 64 latents of width 32; the streaming decode
    // wins from 64 latents (16 % at 64 and 128) and loses at 32; below some tens of microseconds of work the two extra
    // launches cost more than the forms gain.
    // The head-pair form of encode (M <= 64, H even) wins at D = 16 since its K/V ring is deep (0.077 -> 0.062 ms on the
    // 2-D mesh: its rows are short scans, in which the exact form rescales its accumulator on most units) and is equal
    // at D = 32, where it has no room for the ones column and sums the weights in registers.
    const bool pair16 = d->M <= 64 && d->H % 2 == 0 && d->D == 16;
    const bool big_enough = stage == kFastEncode ? (d->M >= 128 || pair16) : d->M >= 64;
    return big_enough && (double)d->B * d->H * d->N * d->M >= 3.0e7;
}

// Launch plan of the tensor-core encode: `pairs` CTAs per head along the latents (two 128-latent blocks each),
// `splits` CTAs along N, about one CTA per SM in total.
struct TcEncodePlan {
    int tiles, pairs, splits, per_split, P;
};

// With at most 64 latents a CTA encodes two adjacent heads at once (see encode_tc_kernel).
bool encode_head_pairs(const flare_desc_t *d) { return d->M <= 64 && d->H % 2 == 0 && d->D >= 16 && d->D <= 32; }

TcEncodePlan tc_encode_plan(const flare_desc_t *d, int sms) {
    TcEncodePlan p;
    p.tiles = (d->N + kTile - 1) / kTile;
    const int mb = (d->M + kTile - 1) / kTile;
    p.pairs = (mb + 1) / 2;
    long groups = (long)d->B * (encode_head_pairs(d) ? d->H / 2 : d->H) * p.pairs;
    long s = sms / groups;
    if (s < 1) s = 1;
    if (s > p.tiles) s = p.tiles;
    p.splits = (int)s;
    p.per_split = (mb == 1) ? 4 : 2;
    p.P = p.splits * p.per_split;
    return p;
}

int partials_for(const flare_desc_t *d, int sms) { return use_tc(d) ? tc_encode_plan(d, sms).P : simt_plan(d, sms).P; }

// ---- TMA descriptors (the driver entry point is looked up at run time; the library does not link libcuda)
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

CUtensorMapSwizzle swizzle_for(int D) {
    return D == 16 ? CU_TENSOR_MAP_SWIZZLE_32B : D == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B;
}

// [B, N, H*D] bf16 viewed as a 3-D tensor (innermost H*D); box = `cols` columns (one head's D, or two adjacent
// heads' 2D) x `rows` tokens.
int make_token_map(CUtensorMap *m, const void *base, const flare_desc_t *d, int rows, int cols = 0) {
    if (cols == 0) cols = d->D;
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) {
        snprintf(g_cuda_error, sizeof(g_cuda_error), "cuTensorMapEncodeTiled not available");
        return FLARE_ERR_CUDA;
    }
    const cuuint64_t C = (cuuint64_t)d->H * d->D;
    cuuint64_t dims[3] = {C, (cuuint64_t)d->N, (cuuint64_t)d->B};
    cuuint64_t strides[2] = {C * 2, C * 2 * (cuuint64_t)d->N};
    cuuint32_t box[3] = {(cuuint32_t)cols, (cuuint32_t)rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(cols), CU_TENSOR_MAP_L2_PROMOTION_NONE,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(g_cuda_error, sizeof(g_cuda_error), "cuTensorMapEncodeTiled(tokens) failed: %d", (int)r);
        return FLARE_ERR_CUDA;
    }
    return FLARE_OK;
}

// Q_lat [H*M, D] bf16 as a 2-D tensor; box = 16 latent rows.
int make_latent_map(CUtensorMap *m, const void *base, const flare_desc_t *d) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) {
        snprintf(g_cuda_error, sizeof(g_cuda_error), "cuTensorMapEncodeTiled not available");
        return FLARE_ERR_CUDA;
    }
    cuuint64_t dims[2] = {(cuuint64_t)d->D, (cuuint64_t)d->H * d->M};
    cuuint64_t strides[1] = {(cuuint64_t)d->D * 2};
    cuuint32_t box[2] = {(cuuint32_t)d->D, 16};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(d->D), CU_TENSOR_MAP_L2_PROMOTION_NONE,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(g_cuda_error, sizeof(g_cuda_error), "cuTensorMapEncodeTiled(latents) failed: %d", (int)r);
        return FLARE_ERR_CUDA;
    }
    return FLARE_OK;
}

constexpr float kLog2e = 1.4426950408889634f;

// kDz: the backward's dZ form of the kernel (V is then dY, lse_dec the decode log-sum-exp rows, pm and pl unused).
// Header words of a workspace beyond the error flag: set by the fast form of encode / decode when its inputs are
// outside the range it is valid for; the exact form that follows runs only then.
constexpr int kRedoEncodeWord = 2, kRedoDecodeWord = 3;

// kAlt: one latent block (M <= 128), the CTA's two slots take alternate tiles: a form of its own with a deeper K/V ring
template <int D, bool kPair, bool kDz, int DRT, bool kHiLo, bool kMaskBody, bool kFast, bool kAlt>
int launch_encode_tc_a(const flare_desc_t *d, const TcEncodePlan &p, const void *Q, const void *K, const void *V,
                       const uint8_t *mask, float *pm, float *pl, float *pacc, uint32_t *status, cudaStream_t st,
                       const float *lse_dec, bool fallback) {
    constexpr int DG = kPair ? 2 * D : D;
    CUtensorMap tmK, tmV, tmQ;
    int rc;
    if ((rc = make_token_map(&tmK, K, d, kTile, DG)) != FLARE_OK) return rc;
    if ((rc = make_token_map(&tmV, V, d, kTile, DG)) != FLARE_OK) return rc;
    if (DRT != 0) tmQ = tmK;   // unused: the narrow forms stage Q with their threads
    else if ((rc = make_latent_map(&tmQ, Q, d)) != FLARE_OK) return rc;
    const size_t smem = EncodeSmem<DG, kAlt>::total();
    static std::atomic<uint64_t> smem_opt_in{0};
    if (int rc_attr = ensure_big_smem(encode_tc_kernel<D, kPair, kDz, DRT, kHiLo, kMaskBody, kFast, kAlt>, smem_opt_in, 227 * 1024)) return rc_attr;
    EncodeTcArgs a;
    a.Q = static_cast<const __nv_bfloat16 *>(Q);
    a.lse_dec = lse_dec;
    a.key_mask = mask; a.part_m = pm; a.part_l = pl; a.part_acc = pacc; a.status = status;
    a.run_if = fallback ? status + kRedoEncodeWord : nullptr;
    a.redo = status + kRedoEncodeWord;
    a.B = d->B; a.H = d->H; a.N = d->N; a.M = d->M;
    a.scale = d->scale; a.sl2 = d->scale * kLog2e;
    a.tiles = p.tiles; a.splits = p.splits; a.pairs = p.pairs; a.partials_per_split = p.per_split;
    dim3 grid(p.splits, (kPair ? d->H / 2 : d->H) * p.pairs, d->B);
    encode_tc_kernel<D, kPair, kDz, DRT, kHiLo, kMaskBody, kFast, kAlt><<<grid, kFast ? kTcThreadsGuarded : kTcThreads, smem, st>>>(tmK, tmV, tmQ, a);
    FLARE_CUDA(cudaGetLastError());
    return FLARE_OK;
}

template <int D, bool kPair, bool kDz = false, int DRT = 0, bool kHiLo = false, bool kMaskBody = false, bool kFast = false>
int launch_encode_tc(const flare_desc_t *d, const TcEncodePlan &p, const void *Q, const void *K, const void *V,
                     const uint8_t *mask, float *pm, float *pl, float *pacc, uint32_t *status, cudaStream_t st,
                     const float *lse_dec = nullptr, bool fallback = false) {
    if constexpr (kPair) {
        return launch_encode_tc_a<D, kPair, kDz, DRT, kHiLo, kMaskBody, kFast, true>(d, p, Q, K, V, mask, pm, pl, pacc, status, st, lse_dec, fallback);
    } else {
        if (d->M <= kTile)
            return launch_encode_tc_a<D, kPair, kDz, DRT, kHiLo, kMaskBody, kFast, true>(d, p, Q, K, V, mask, pm, pl, pacc, status, st, lse_dec, fallback);
        return launch_encode_tc_a<D, kPair, kDz, DRT, kHiLo, kMaskBody, kFast, false>(d, p, Q, K, V, mask, pm, pl, pacc, status, st, lse_dec, fallback);
    }
}

template <int D, int DRT, bool kPadded, bool kAlt>
int launch_bwd_dq_tc_a(const flare_desc_t *d, const TcEncodePlan &p, const void *Q, const void *K, const void *V, const void *dY,
                     const uint8_t *mask, const float *Z, const float *dZ, const float *lse_enc, const float *de,
                     const float *lse_dec, const float *dd, float *part, uint32_t *status, cudaStream_t st) {
    CUtensorMap tmK, tmV, tmG, tmQ;
    int rc;
    if ((rc = make_token_map(&tmK, K, d, kTile, D)) != FLARE_OK) return rc;
    if ((rc = make_token_map(&tmV, V, d, kTile, D)) != FLARE_OK) return rc;
    if ((rc = make_token_map(&tmG, dY, d, kTile, D)) != FLARE_OK) return rc;
    if (DRT != 0) tmQ = tmK;   // unused: the narrow forms stage Q with their threads
    else if ((rc = make_latent_map(&tmQ, Q, d)) != FLARE_OK) return rc;
    const size_t smem = BwdDqSmem<D, kAlt>::total();
    static std::atomic<uint64_t> smem_opt_in{0};
    if (int rc_attr = ensure_big_smem(bwd_dq_tc_kernel<D, DRT, kPadded, kAlt>, smem_opt_in, 227 * 1024)) return rc_attr;
    BwdDqTcArgs a;
    a.Q = static_cast<const __nv_bfloat16 *>(Q);
    a.Z = Z; a.dZ = dZ; a.lse_enc = lse_enc; a.de = de; a.lse_dec = lse_dec; a.dd = dd;
    a.key_mask = mask; a.part = part; a.status = status;
    a.B = d->B; a.H = d->H; a.N = d->N; a.M = d->M;
    a.sl2 = d->scale * kLog2e;
    a.tiles = p.tiles; a.splits = p.splits; a.pairs = p.pairs; a.partials_per_split = p.per_split;
    dim3 grid(p.splits, d->H * p.pairs, d->B);
    bwd_dq_tc_kernel<D, DRT, kPadded, kAlt><<<grid, kTcThreads, smem, st>>>(tmK, tmV, tmG, tmQ, a);
    FLARE_CUDA(cudaGetLastError());
    return FLARE_OK;
}

// (one latent block, M <= 128: the form whose slots take alternate tiles, with a deeper tile ring)
template <int D, int DRT, bool kPadded>
int launch_bwd_dq_tc_p(const flare_desc_t *d, const TcEncodePlan &p, const void *Q, const void *K, const void *V, const void *dY,
                     const uint8_t *mask, const float *Z, const float *dZ, const float *lse_enc, const float *de,
                     const float *lse_dec, const float *dd, float *part, uint32_t *status, cudaStream_t st) {
    if (d->M <= kTile)
        return launch_bwd_dq_tc_a<D, DRT, kPadded, true>(d, p, Q, K, V, dY, mask, Z, dZ, lse_enc, de, lse_dec, dd, part, status, st);
    return launch_bwd_dq_tc_a<D, DRT, kPadded, false>(d, p, Q, K, V, dY, mask, Z, dZ, lse_enc, de, lse_dec, dd, part, status, st);
}

template <int D, int DRT = 0>
int launch_bwd_dq_tc(const flare_desc_t *d, const TcEncodePlan &p, const void *Q, const void *K, const void *V, const void *dY,
                     const uint8_t *mask, const float *Z, const float *dZ, const float *lse_enc, const float *de,
                     const float *lse_dec, const float *dd, float *part, uint32_t *status, cudaStream_t st) {
    // padded tokens: a key mask, or a last partial tile
    if (mask != nullptr || d->N % kTile != 0)
        return launch_bwd_dq_tc_p<D, DRT, true>(d, p, Q, K, V, dY, mask, Z, dZ, lse_enc, de, lse_dec, dd, part, status, st);
    return launch_bwd_dq_tc_p<D, DRT, false>(d, p, Q, K, V, dY, mask, Z, dZ, lse_enc, de, lse_dec, dd, part, status, st);
}

template <int D, int DRT, int kMode, int kM, bool kPadded>
int launch_bwd_token_tc_m(const flare_desc_t *d, int sms, const void *Q, const void *K, const void *V, const void *dY,
                        const uint8_t *mask, const float *Z, const float *dZ, const float *lse_enc, const float *de,
                        const float *lse_dec, void *dK, void *dV, float *dd, uint32_t *status, cudaStream_t st,
                        int m0, int mc, float *kvacc) {
    CUtensorMap tmK, tmV, tmG, tmQ;
    int rc;
    if ((rc = make_token_map(&tmK, K, d, kTile, D)) != FLARE_OK) return rc;
    if ((rc = make_token_map(&tmV, V, d, kTile, D)) != FLARE_OK) return rc;
    if ((rc = make_token_map(&tmG, dY, d, kTile, D)) != FLARE_OK) return rc;
    if (DRT != 0) tmQ = tmK;   // unused: the narrow forms stage Q with their threads
    else if ((rc = make_latent_map(&tmQ, Q, d)) != FLARE_OK) return rc;
    BwdTokTcArgs a;
    a.stages = BwdTokSmem<D>::stages(mc);
    if (a.stages < 1) return FLARE_ERR_UNSUPPORTED;
    const size_t smem = BwdTokSmem<D>::total(a.stages, mc);
    static std::atomic<uint64_t> smem_opt_in{0};
    if (int rc_attr = ensure_big_smem(bwd_token_tc_kernel<D, DRT, kMode, kM, kPadded>, smem_opt_in, 227 * 1024)) return rc_attr;
    a.Q = static_cast<const __nv_bfloat16 *>(Q);
    a.Z = Z; a.dZ = dZ; a.lse_enc = lse_enc; a.de = de; a.lse_dec = lse_dec; a.key_mask = mask;
    a.dK = (__nv_bfloat16 *)dK; a.dV = (__nv_bfloat16 *)dV; a.dd = dd; a.status = status;
    a.B = d->B; a.H = d->H; a.N = d->N; a.M = mc;
    a.mtot = d->M; a.m0 = m0; a.first = m0 == 0; a.last = m0 + mc >= d->M; a.kvacc = kvacc;
    a.scale = d->scale; a.sl2 = d->scale * kLog2e;
    a.tiles = (d->N + kTile - 1) / kTile;
    long per_head = sms / ((long)d->B * d->H);
    if (per_head < 1) per_head = 1;
    if (per_head > a.tiles) per_head = a.tiles;
    bwd_token_tc_kernel<D, DRT, kMode, kM, kPadded><<<dim3((unsigned)per_head, d->H, d->B), kTcThreads, smem, st>>>(tmK, tmV, tmG, tmQ, a);
    FLARE_CUDA(cudaGetLastError());
    return FLARE_OK;
}

// The launch's range of latents is [m0, m0 + mc) (mc = 0: all of them); common sizes have forms of the kernel with
// the number of latents as a compile-time constant.
template <int D, int DRT = 0, int kMode = 0>
int launch_bwd_token_tc(const flare_desc_t *d, int sms, const void *Q, const void *K, const void *V, const void *dY,
                        const uint8_t *mask, const float *Z, const float *dZ, const float *lse_enc, const float *de,
                        const float *lse_dec, void *dK, void *dV, float *dd, uint32_t *status, cudaStream_t st,
                        int m0 = 0, int mc = 0, float *kvacc = nullptr) {
    if (mc == 0) mc = d->M;
    const bool padded = mask != nullptr || d->N % kTile != 0;   // a key mask, or a last partial tile
#define FLARE_TOK(MM)                                                                                                     \
    (padded ? launch_bwd_token_tc_m<D, DRT, kMode, MM, true>(d, sms, Q, K, V, dY, mask, Z, dZ, lse_enc, de, lse_dec, dK, dV, dd, \
                                                            status, st, m0, mc, kvacc)                                   \
            : launch_bwd_token_tc_m<D, DRT, kMode, MM, false>(d, sms, Q, K, V, dY, mask, Z, dZ, lse_enc, de, lse_dec, dK, dV, dd, \
                                                             status, st, m0, mc, kvacc))
    if (mc == 256) return FLARE_TOK(256);
    if (mc == 128) return FLARE_TOK(128);
    if (mc == 64) return FLARE_TOK(64);
    if (mc == 512) return FLARE_TOK(512);
    return FLARE_TOK(0);
#undef FLARE_TOK
}

template <int D, int DRT, bool kPart, int kM>
int launch_decode_tc_m(const flare_desc_t *d, int sms, const void *Q, const void *K, const float *Z, void *Y,
                     float *lse_dec, uint32_t *status, cudaStream_t st, int m0, int mc, float *Ypart, bool fallback = false) {
    CUtensorMap tmK, tmQ;
    int rc;
    if ((rc = make_token_map(&tmK, K, d, kTile, D)) != FLARE_OK) return rc;
    if (DRT != 0) tmQ = tmK;   // unused: the narrow forms stage Q with their threads
    else if ((rc = make_latent_map(&tmQ, Q, d)) != FLARE_OK) return rc;
    const size_t smem = DecodeSmem<D>::total(mc);
    static std::atomic<uint64_t> smem_opt_in{0};
    if (int rc_attr = ensure_big_smem(decode_tc_kernel<D, DRT, kPart, kM>, smem_opt_in, 227 * 1024)) return rc_attr;
    DecodeTcArgs a;
    a.Q = static_cast<const __nv_bfloat16 *>(Q);
    a.Z = Z; a.Y = (__nv_bfloat16 *)Y; a.lse_dec = lse_dec; a.status = status;
    a.run_if = (fallback && status != nullptr) ? status + kRedoDecodeWord : nullptr;
    a.redo = status != nullptr ? status + kRedoDecodeWord : nullptr;
    a.B = d->B; a.H = d->H; a.N = d->N; a.M = mc;
    a.mtot = d->M; a.m0 = m0; a.Ypart = Ypart;
    a.sl2 = d->scale * kLog2e;
    a.tiles = (d->N + kTile - 1) / kTile;
    a.plan = make_decode_plan(mc, D);
    if (a.plan.cs == 0) return FLARE_ERR_UNSUPPORTED;
    long per_head = sms / ((long)d->B * d->H);
    if (per_head < 1) per_head = 1;
    if (per_head > a.tiles) per_head = a.tiles;
    dim3 grid((unsigned)per_head, d->H, d->B);
    decode_tc_kernel<D, DRT, kPart, kM><<<grid, kTcThreads, smem, st>>>(tmK, tmQ, a);
    FLARE_CUDA(cudaGetLastError());
    return FLARE_OK;
}

// The streaming (fast) form of decode: head widths 16 (and narrower) and 32, as many latents as fit shared memory.
template <int D>
bool decode_stream_fits(int mc) { return (D == 16 || D == 32) && DecodeStreamSmem<(D == 16 || D == 32) ? D : 16>::fits(mc); }

template <int D, int DRT, bool kPart, int kM, bool kLse>
int launch_decode_stream_l(const flare_desc_t *d, int sms, const void *Q, const void *K, const float *Z, void *Y,
                           float *lse_dec, uint32_t *status, cudaStream_t st, int m0, int mc, float *Ypart) {
    if constexpr (D == 16 || D == 32) {
        CUtensorMap tmK, tmQ;
        int rc;
        if ((rc = make_token_map(&tmK, K, d, kTile, D)) != FLARE_OK) return rc;
        if (DRT != 0) tmQ = tmK;   // unused: the narrow forms stage Q with their threads
        else if ((rc = make_latent_map(&tmQ, Q, d)) != FLARE_OK) return rc;
        const size_t smem = DecodeStreamSmem<D>::total(mc);
        static std::atomic<uint64_t> smem_opt_in{0};
        if (int rc_attr = ensure_big_smem(decode_stream_kernel<D, DRT, kPart, kM, kLse>, smem_opt_in, 227 * 1024)) return rc_attr;
        DecodeTcArgs a;
        a.Q = static_cast<const __nv_bfloat16 *>(Q);
        a.Z = Z; a.Y = (__nv_bfloat16 *)Y; a.lse_dec = lse_dec; a.status = status;
        a.run_if = nullptr;
        a.redo = status + kRedoDecodeWord;
        a.B = d->B; a.H = d->H; a.N = d->N; a.M = mc;
        a.mtot = d->M; a.m0 = m0; a.Ypart = Ypart;
        a.sl2 = d->scale * kLog2e;
        a.tiles = (d->N + kTile - 1) / kTile;
        a.plan = DecodePlan{};
        long per_head = sms / ((long)d->B * d->H);
        const long four = (a.tiles + 3) / 4;                    // a CTA works on four tiles at a time
        if (per_head > four) per_head = four;
        if (per_head < 1) per_head = 1;
        decode_stream_kernel<D, DRT, kPart, kM, kLse><<<dim3((unsigned)per_head, d->H, d->B), kTcThreadsGuarded, smem, st>>>(tmK, tmQ, a);
        FLARE_CUDA(cudaGetLastError());
        return FLARE_OK;
    } else {
        return FLARE_ERR_UNSUPPORTED;
    }
}

template <int D, int DRT, bool kPart, int kM>
int launch_decode_stream_m(const flare_desc_t *d, int sms, const void *Q, const void *K, const float *Z, void *Y,
                           float *lse_dec, uint32_t *status, cudaStream_t st, int m0, int mc, float *Ypart) {
    if (lse_dec != nullptr) return launch_decode_stream_l<D, DRT, kPart, kM, true>(d, sms, Q, K, Z, Y, lse_dec, status, st, m0, mc, Ypart);
    if constexpr (kPart) return FLARE_ERR_INVALID_ARG;          // a range of the latents always leaves its log-sum-exp
    else return launch_decode_stream_l<D, DRT, kPart, kM, false>(d, sms, Q, K, Z, Y, lse_dec, status, st, m0, mc, Ypart);
}

// (the common latent counts as compile-time constants of the kernel)
template <int D, int DRT, bool kPart>
int launch_decode_stream(const flare_desc_t *d, int sms, const void *Q, const void *K, const float *Z, void *Y,
                         float *lse_dec, uint32_t *status, cudaStream_t st, int m0, int mc, float *Ypart) {
    if (mc == 256) return launch_decode_stream_m<D, DRT, kPart, 256>(d, sms, Q, K, Z, Y, lse_dec, status, st, m0, mc, Ypart);
    if (mc == 128) return launch_decode_stream_m<D, DRT, kPart, 128>(d, sms, Q, K, Z, Y, lse_dec, status, st, m0, mc, Ypart);
    if (mc == 64) return launch_decode_stream_m<D, DRT, kPart, 64>(d, sms, Q, K, Z, Y, lse_dec, status, st, m0, mc, Ypart);
    if (mc == 512) return launch_decode_stream_m<D, DRT, kPart, 512>(d, sms, Q, K, Z, Y, lse_dec, status, st, m0, mc, Ypart);
    return launch_decode_stream_m<D, DRT, kPart, 0>(d, sms, Q, K, Z, Y, lse_dec, status, st, m0, mc, Ypart);
}

// The launch's range of latents is [m0, m0 + mc) (mc = 0: all of them).  The sizes that the workloads use most have
// forms of the kernel with the number of latents as a compile-time constant.  fast: the form without a row maximum
// first, then the exact form, which exits at once unless the first one found its inputs out of range (this needs
// the flag word in a workspace header: status != null).
template <int D, int DRT, bool kPart>
int launch_decode_tc_f(const flare_desc_t *d, int sms, const void *Q, const void *K, const float *Z, void *Y,
                       float *lse_dec, uint32_t *status, cudaStream_t st, int m0, int mc, float *Ypart, bool fallback) {
    if (mc == 256) return launch_decode_tc_m<D, DRT, kPart, 256>(d, sms, Q, K, Z, Y, lse_dec, status, st, m0, mc, Ypart, fallback);
    if (mc == 128) return launch_decode_tc_m<D, DRT, kPart, 128>(d, sms, Q, K, Z, Y, lse_dec, status, st, m0, mc, Ypart, fallback);
    if (mc == 64) return launch_decode_tc_m<D, DRT, kPart, 64>(d, sms, Q, K, Z, Y, lse_dec, status, st, m0, mc, Ypart, fallback);
    if (mc == 32) return launch_decode_tc_m<D, DRT, kPart, 32>(d, sms, Q, K, Z, Y, lse_dec, status, st, m0, mc, Ypart, fallback);
    if (mc == 512) return launch_decode_tc_m<D, DRT, kPart, 512>(d, sms, Q, K, Z, Y, lse_dec, status, st, m0, mc, Ypart, fallback);
    return launch_decode_tc_m<D, DRT, kPart, 0>(d, sms, Q, K, Z, Y, lse_dec, status, st, m0, mc, Ypart, fallback);
}

template <int D, int DRT = 0, bool kPart = false>
int launch_decode_tc(const flare_desc_t *d, int sms, const void *Q, const void *K, const float *Z, void *Y,
                     float *lse_dec, uint32_t *status, cudaStream_t st, int m0 = 0, int mc = 0, float *Ypart = nullptr,
                     bool fast = false) {
    if (mc == 0) mc = d->M;
    fast = fast && status != nullptr && decode_stream_fits<D>(mc);
    if (fast) {
        const int rc = launch_decode_stream<D, DRT, kPart>(d, sms, Q, K, Z, Y, lse_dec, status, st, m0, mc, Ypart);
        if (rc != FLARE_OK) return rc;
    }
    return launch_decode_tc_f<D, DRT, kPart>(d, sms, Q, K, Z, Y, lse_dec, status, st, m0, mc, Ypart, fast);
}

template <typename T>
int launch_encode_simt(const flare_desc_t *d, const SimtPlan &p, const void *Q, const void *K, const void *V,
                       const uint8_t *mask, float *pm, float *pl, float *pacc, cudaStream_t st) {
    dim3 grid(p.splits, d->H, d->B), block(kSimtThreads);
#define FLARE_CASE(DD)                                                                                          \
    case DD:                                                                                                    \
        encode_simt_kernel<T, DD><<<grid, block, 0, st>>>((const T *)Q, (const T *)K, (const T *)V, mask, pm, pl, \
                                                          pacc, d->B, d->H, d->N, d->M, p.LM, p.chunk, d->scale); \
        break;
    switch (d->D) {
        FLARE_CASE(4) FLARE_CASE(8) FLARE_CASE(16) FLARE_CASE(32) FLARE_CASE(64)
        default: return FLARE_ERR_UNSUPPORTED;
    }
#undef FLARE_CASE
    FLARE_CUDA(cudaGetLastError());
    return FLARE_OK;
}

template <typename T>
int launch_decode_simt(const flare_desc_t *d, const void *Q, const void *K, const float *Z, void *Y, float *lse_dec,
                       cudaStream_t st) {
    dim3 grid((d->N + kDecodeSimtThreads - 1) / kDecodeSimtThreads, d->H, d->B), block(kDecodeSimtThreads);
#define FLARE_CASE(DD)                                                                                            \
    case DD:                                                                                                      \
        decode_simt_kernel<T, DD><<<grid, block, 0, st>>>((const T *)Q, (const T *)K, Z, (T *)Y, lse_dec, d->B, d->H, \
                                                          d->N, d->M, d->scale);                                  \
        break;
    switch (d->D) {
        FLARE_CASE(4) FLARE_CASE(8) FLARE_CASE(16) FLARE_CASE(32) FLARE_CASE(64)
        default: return FLARE_ERR_UNSUPPORTED;
    }
#undef FLARE_CASE
    FLARE_CUDA(cudaGetLastError());
    return FLARE_OK;
}

// Launch plans of the CUDA-core backward: pass A (dZ) reuses the encode plan; the dQ pass keeps three latent
// rows per thread in shared memory and therefore caps its latent block at 64.
// Pass A (dZ) runs as the dZ form of the tensor-core encode kernel wherever that kernel runs.
bool bwd_dz_on_tensor_cores(const flare_desc_t *d) { return use_tc(d); }

// Pass B for dQ runs on the tensor cores for narrow heads (S, A, C and the partial dQ of a group share its 128
// TMEM columns: 3 * 32 + D).
bool bwd_dq_on_tensor_cores(const flare_desc_t *d) { return use_tc(d) && d->D <= 32; }

// Plan of the tensor-core dQ kernel: the encode plan without head pairing.
TcEncodePlan tc_dq_plan(const flare_desc_t *d, int sms) {
    TcEncodePlan p;
    const int mb = (d->M + kTile - 1) / kTile;
    p.tiles = (d->N + kTile - 1) / kTile;
    p.pairs = (mb + 1) / 2;
    long s = sms / ((long)d->B * d->H * p.pairs);
    if (s < 1) s = 1;
    if (s > p.tiles) s = p.tiles;
    p.splits = (int)s;
    p.per_split = (mb == 1) ? 4 : 2;
    p.P = p.splits * p.per_split;
    return p;
}

SimtPlan bwd_dq_plan(const flare_desc_t *d, int sms) {
    SimtPlan p = simt_plan(d, sms);
    if (p.LM > 64) p.LM = 64;
    p.G = kBwdThreads / p.LM;
    p.P = p.splits * p.G;
    return p;
}

struct BwdLayout {
    size_t part, dz, de, dd, kvacc, total;
    int P;
};

// Latents one launch of the tensor-core token kernel keeps in shared memory (five operands of D-wide bf16 rows,
// beside at least five tile stages); more are worked off in ranges of this many.
int token_range(const flare_desc_t *d) { return d->D == 32 ? 256 : 512; }
bool token_in_ranges(const flare_desc_t *d) { return bwd_dq_on_tensor_cores(d) && d->M > token_range(d); }

BwdLayout bwd_layout(const flare_desc_t *d, int sms) {
    BwdLayout w;
    const long rows = (long)d->B * d->H * d->M;
    const int pa = simt_plan(d, sms).P, pb = bwd_dq_plan(d, sms).P;
    w.P = pa > pb ? pa : pb;
    if (bwd_dz_on_tensor_cores(d) && tc_encode_plan(d, sms).P > w.P) w.P = tc_encode_plan(d, sms).P;
    if (bwd_dq_on_tensor_cores(d) && tc_dq_plan(d, sms).P > w.P) w.P = tc_dq_plan(d, sms).P;
    size_t off = kHeaderBytes;
    w.part = off; off += align_up(sizeof(float) * (size_t)w.P * rows * d->D);
    w.dz = off;   off += align_up(sizeof(float) * (size_t)rows * d->D);
    w.de = off;   off += align_up(sizeof(float) * (size_t)rows);
    w.dd = off;   off += align_up(sizeof(float) * (size_t)d->B * d->N * d->H);
    w.kvacc = off;                                             // float32 sums of the rows of dK and dV over latent ranges
    if (token_in_ranges(d)) off += align_up(sizeof(float) * 2 * (size_t)d->B * d->N * d->H * d->D);
    w.total = off;
    return w;
}

template <typename T, int D>
int launch_backward_simt(const flare_desc_t *d, int sms, const void *Q, const void *K, const void *V,
                         const uint8_t *mask, const void *Y, const void *dY, const float *Z, const float *lse_enc,
                         const float *lse_dec, float *dQ, void *dK, void *dV, char *ws, cudaStream_t st,
                         bool skip_pass_a = false) {
    // skip_pass_a: dZ and de are already in the workspace (the second of the two runs of the separate-queries variant)
    const BwdLayout w = bwd_layout(d, sms);
    float *part = reinterpret_cast<float *>(ws + w.part);
    float *dZ = reinterpret_cast<float *>(ws + w.dz);
    float *de = reinterpret_cast<float *>(ws + w.de);
    float *dd = reinterpret_cast<float *>(ws + w.dd);
    (void)Y;  // dY_n . Y_n is rebuilt from float32 quantities instead of the rounded stored Y
    const long rows = (long)d->B * d->H * d->M;
    const SimtPlan pa = simt_plan(d, sms), pb = bwd_dq_plan(d, sms);
    FLARE_CUDA(cudaMemsetAsync(ws, 0, kHeaderBytes, st));
    int dz_parts = pa.P;
    bool dz_on_tc = skip_pass_a;
    if constexpr (std::is_same<T, __nv_bfloat16>::value) {
        if (!skip_pass_a && bwd_dz_on_tensor_cores(d)) {
            const TcEncodePlan tp = tc_encode_plan(d, sms);
            uint32_t *status = reinterpret_cast<uint32_t *>(ws);
            int rc;
            if constexpr (D < 16) {
                rc = launch_encode_tc<16, false, true, D>(d, tp, Q, K, dY, nullptr, nullptr, nullptr, part, status, st, lse_dec);
            } else if constexpr (D <= 32) {
                rc = encode_head_pairs(d)
                         ? launch_encode_tc<D, true, true>(d, tp, Q, K, dY, nullptr, nullptr, nullptr, part, status, st, lse_dec)
                         : launch_encode_tc<D, false, true>(d, tp, Q, K, dY, nullptr, nullptr, nullptr, part, status, st, lse_dec);
            } else {
                rc = launch_encode_tc<D, false, true>(d, tp, Q, K, dY, nullptr, nullptr, nullptr, part, status, st, lse_dec);
            }
            if (rc != FLARE_OK) return rc;
            dz_parts = tp.P;
            dz_on_tc = true;
        }
    }
    if (!dz_on_tc) {
        bwd_dz_simt_kernel<T, D><<<dim3(pa.splits, d->H, d->B), kBwdThreads, 0, st>>>(
            (const T *)Q, (const T *)K, (const T *)dY, lse_dec, part, d->B, d->H, d->N, d->M, pa.LM, pa.chunk, d->scale);
        FLARE_CUDA(cudaGetLastError());
    }
    if (!skip_pass_a) {
        bwd_dz_reduce_kernel<<<(unsigned)((rows * d->D + 255) / 256), 256, 0, st>>>(part, dZ, dz_parts, rows, d->D);
        FLARE_CUDA(cudaGetLastError());
        bwd_de_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(dZ, Z, de, rows, d->D);
        FLARE_CUDA(cudaGetLastError());
    }
    bool tok_on_tc = false;
    if constexpr (std::is_same<T, __nv_bfloat16>::value && D <= 32) {
        constexpr int DK = D < 16 ? 16 : D;                     // width the kernels multiply (D < 16: narrow forms)
        constexpr int DRT = D < 16 ? D : 0;
        uint32_t *status = reinterpret_cast<uint32_t *>(ws);
        if (bwd_dq_on_tensor_cores(d) && !token_in_ranges(d) && BwdTokSmem<DK>::stages(d->M) >= 1) {
            const int rc = launch_bwd_token_tc<DK, DRT>(d, sms, Q, K, V, dY, mask, Z, dZ, lse_enc, de, lse_dec, dK, dV, dd,
                                                        status, st);
            if (rc != FLARE_OK) return rc;
            tok_on_tc = true;
        } else if (token_in_ranges(d)) {
            // two series of launches over the latent ranges: dd[n] first, then the rows of dK and dV
            float *kvacc = reinterpret_cast<float *>(ws + w.kvacc);
            const int R = token_range(d);
            for (int mode = 1; mode <= 2; ++mode)
                for (int m0 = 0; m0 < d->M; m0 += R) {
                    const int mc = d->M - m0 < R ? d->M - m0 : R;
                    const int rc = mode == 1 ? launch_bwd_token_tc<DK, DRT, 1>(d, sms, Q, K, V, dY, mask, Z, dZ, lse_enc, de, lse_dec,
                                                                              dK, dV, dd, status, st, m0, mc, kvacc)
                                             : launch_bwd_token_tc<DK, DRT, 2>(d, sms, Q, K, V, dY, mask, Z, dZ, lse_enc, de, lse_dec,
                                                                              dK, dV, dd, status, st, m0, mc, kvacc);
                    if (rc != FLARE_OK) return rc;
                }
            tok_on_tc = true;
        }
    }
    if (!tok_on_tc) {
        bwd_token_simt_kernel<T, D><<<dim3((d->N + 127) / 128, d->H, d->B), 128, 0, st>>>(
            (const T *)Q, (const T *)K, (const T *)V, mask, (const T *)dY, Z, dZ, de, lse_enc, lse_dec, (T *)dK, (T *)dV, dd,
            d->B, d->H, d->N, d->M, d->scale);
        FLARE_CUDA(cudaGetLastError());
    }
    int dq_parts = pb.P;
    bool dq_on_tc = false;
    if constexpr (std::is_same<T, __nv_bfloat16>::value && D <= 32) {
        if (bwd_dq_on_tensor_cores(d)) {
            const int rc = launch_bwd_dq_tc<(D < 16 ? 16 : D), (D < 16 ? D : 0)>(d, tc_dq_plan(d, sms), Q, K, V, dY, mask, Z, dZ, lse_enc, de, lse_dec, dd, part,
                                               reinterpret_cast<uint32_t *>(ws), st);
            if (rc != FLARE_OK) return rc;
            dq_parts = tc_dq_plan(d, sms).P;
            dq_on_tc = true;
        }
    }
    if (!dq_on_tc) {
        const size_t dyn = sizeof(float) * 3 * (size_t)pb.LM * (D + 1);
        static std::atomic<uint64_t> smem_opt_in{0};
        if (int rc_attr = ensure_big_smem(bwd_dq_simt_kernel<T, D>, smem_opt_in, (int)(sizeof(float) * 3 * 64 * (D + 1)))) return rc_attr;
        bwd_dq_simt_kernel<T, D><<<dim3(pb.splits, d->H, d->B), kBwdThreads, dyn, st>>>(
            (const T *)Q, (const T *)K, (const T *)V, mask, (const T *)dY, Z, dZ, de, dd, lse_enc, lse_dec, part, d->B, d->H,
            d->N, d->M, pb.LM, pb.chunk, d->scale);
        FLARE_CUDA(cudaGetLastError());
    }
    bwd_dq_reduce_kernel<<<(unsigned)((long)d->H * d->M), kDqReduceThreads, 0, st>>>(part, dQ, dq_parts, d->B, d->H, d->M,
                                                                                     d->D, d->scale);
    FLARE_CUDA(cudaGetLastError());
    return FLARE_OK;
}

template <typename T>
int backward_simt(const flare_desc_t *d, int sms, const void *Q, const void *K, const void *V, const uint8_t *mask,
                  const void *Y, const void *dY, const float *Z, const float *lse_enc, const float *lse_dec, float *dQ,
                  void *dK, void *dV, char *ws, cudaStream_t st, bool skip_pass_a = false) {
    switch (d->D) {
        case 4: return launch_backward_simt<T, 4>(d, sms, Q, K, V, mask, Y, dY, Z, lse_enc, lse_dec, dQ, dK, dV, ws, st, skip_pass_a);
        case 8: return launch_backward_simt<T, 8>(d, sms, Q, K, V, mask, Y, dY, Z, lse_enc, lse_dec, dQ, dK, dV, ws, st, skip_pass_a);
        case 16: return launch_backward_simt<T, 16>(d, sms, Q, K, V, mask, Y, dY, Z, lse_enc, lse_dec, dQ, dK, dV, ws, st, skip_pass_a);
        case 32: return launch_backward_simt<T, 32>(d, sms, Q, K, V, mask, Y, dY, Z, lse_enc, lse_dec, dQ, dK, dV, ws, st, skip_pass_a);
        case 64: return launch_backward_simt<T, 64>(d, sms, Q, K, V, mask, Y, dY, Z, lse_enc, lse_dec, dQ, dK, dV, ws, st, skip_pass_a);
        default: return FLARE_ERR_UNSUPPORTED;
    }
}

int require_device() {
    const DeviceView di = device_info();
    if (di.checked == -2) {
        snprintf(g_cuda_error, sizeof(g_cuda_error), "no CUDA device");
        return FLARE_ERR_CUDA;
    }
    if (di.checked != 1) return FLARE_ERR_ARCH;
    return FLARE_OK;
}

// The fast form first (if wanted), then the exact form, which exits at once unless the fast one raised its flag.
template <int D, bool kPair, int DRT, bool kHiLo, bool kMaskBody>
int encode_tc_forms(const flare_desc_t *d, const TcEncodePlan &p, const void *Q, const void *K, const void *V,
                    const uint8_t *mask, float *pm, float *pl, float *pacc, uint32_t *status, cudaStream_t st, bool fast) {
    if (fast) {
        const int rc = launch_encode_tc<D, kPair, false, DRT, kHiLo, kMaskBody, true>(d, p, Q, K, V, mask, pm, pl, pacc, status, st);
        if (rc != FLARE_OK) return rc;
    }
    return launch_encode_tc<D, kPair, false, DRT, kHiLo, kMaskBody, false>(d, p, Q, K, V, mask, pm, pl, pacc, status, st, nullptr, fast);
}

int encode_impl(const flare_desc_t *d, const void *Q, const void *K, const void *V, const uint8_t *mask, float *Z,
                float *lse_enc, void *ws, cudaStream_t st) {
    const DeviceView di = device_info();
    const long rows = (long)d->B * d->H * d->M;
    const int P = partials_for(d, di.sms);
    WorkspaceLayout w = make_layout(P, rows, d->D, false);
    char *base = static_cast<char *>(ws);
    float *pm = reinterpret_cast<float *>(base + w.part_m);
    float *pl = reinterpret_cast<float *>(base + w.part_l);
    float *pacc = reinterpret_cast<float *>(base + w.part_acc);
    FLARE_CUDA(cudaMemsetAsync(base, 0, kHeaderBytes, st));
    int rc;
    if (use_tc(d)) {
        TcEncodePlan p = tc_encode_plan(d, di.sms);
        uint32_t *status = reinterpret_cast<uint32_t *>(base);
        // a caller that asks for lse_enc is saving Z for the backward: weights as two bf16 halves (see exp_chunk_hilo)
        const bool fast = use_fast(d, kFastEncode);
#define FLARE_ENC3(DD, PAIR, DRT, MB, HL) encode_tc_forms<DD, PAIR, DRT, HL, MB>(d, p, Q, K, V, mask, pm, pl, pacc, status, st, fast)
#define FLARE_ENC2(DD, PAIR, DRT, MB) (lse_enc != nullptr ? FLARE_ENC3(DD, PAIR, DRT, MB, true) : FLARE_ENC3(DD, PAIR, DRT, MB, false))
        // A call with a key mask has padding in every tile and takes the form that tests every element (see
        // encode_tc_kernel).  Without a mask only a last partial tile has padding and either form serves; which one
        // is faster was measured (B200): the form without the element tests where a CTA holds two latent blocks
        // (M > 128: 0.80 -> 0.68 ms on the million-point shape, 223 -> 201 us at N = 131072, M = 512), the other
        // where two slots share one block (M <= 128: 4-5 % apart).
        const bool mask_body = mask != nullptr || d->M <= kTile;
#define FLARE_ENC(DD, PAIR, DRT) (mask_body ? FLARE_ENC2(DD, PAIR, DRT, true) : FLARE_ENC2(DD, PAIR, DRT, false))
        if (encode_head_pairs(d))
            rc = d->D == 16 ? FLARE_ENC(16, true, 0) : FLARE_ENC(32, true, 0);
        else
            rc = d->D == 4    ? FLARE_ENC(16, false, 4)
                 : d->D == 8  ? FLARE_ENC(16, false, 8)
                 : d->D == 16 ? FLARE_ENC(16, false, 0)
                 : d->D == 32 ? FLARE_ENC(32, false, 0)
                              : FLARE_ENC(64, false, 0);
#undef FLARE_ENC
#undef FLARE_ENC2
#undef FLARE_ENC3
    } else {
        SimtPlan p = simt_plan(d, di.sms);
        rc = (d->dtype == FLARE_DTYPE_F32)   ? launch_encode_simt<float>(d, p, Q, K, V, mask, pm, pl, pacc, st)
             : (d->dtype == FLARE_DTYPE_F16) ? launch_encode_simt<__half>(d, p, Q, K, V, mask, pm, pl, pacc, st)
                                             : launch_encode_simt<__nv_bfloat16>(d, p, Q, K, V, mask, pm, pl, pacc, st);
    }
    if (rc != FLARE_OK) return rc;
    if (P > 8)   // many partials (small problems spread over all SMs): a block per row shares the loads
        merge_kernel<<<(unsigned)rows, kMergeThreads, 0, st>>>(pm, pl, pacc, Z, lse_enc, P, rows, d->D);
    else
        merge_serial_kernel<<<(unsigned)((rows * d->D + 255) / 256), 256, 0, st>>>(pm, pl, pacc, Z, lse_enc, P, rows, d->D);
    FLARE_CUDA(cudaGetLastError());
    return FLARE_OK;
}

// One decode launch holds all M score columns of a token tile in tensor memory (512 columns) and Q_h, Z_h in shared
// memory: up to kDecodeMaxM latents.
constexpr int kDecodeMaxM = 512;

// Ranges of latents a decode over more than kDecodeMaxM latents is cut into, and the scratch their partial results
// take after the encode layout of the forward workspace: float32 rows [C][B*N*H][D] and log-sum-exps [C][B*N*H].
constexpr int kDecodeRange = 256;   // latents per launch when a decode is cut into ranges
int decode_ranges(const flare_desc_t *d) { return (d->M + kDecodeRange - 1) / kDecodeRange; }
bool decode_in_ranges(const flare_desc_t *d) { return use_tc(d) && d->M > kDecodeMaxM; }
size_t decode_range_bytes(const flare_desc_t *d) {
    if (!decode_in_ranges(d)) return 0;
    const size_t rows = (size_t)d->B * d->N * d->H;
    return align_up(sizeof(float) * decode_ranges(d) * rows * d->D) + align_up(sizeof(float) * decode_ranges(d) * rows);
}

template <int D, int DRT>
int decode_tc_any(const flare_desc_t *d, int sms, const void *Q, const void *K, const float *Z, void *Y, float *lse_dec,
                  uint32_t *status, char *range_scratch, cudaStream_t st) {
    const bool fast = use_fast(d, kFastDecode) && status != nullptr;
    if (d->M <= kDecodeMaxM) return launch_decode_tc<D, DRT>(d, sms, Q, K, Z, Y, lse_dec, status, st, 0, 0, nullptr, fast);
    constexpr int DR = DRT ? DRT : D;
    const int C = decode_ranges(d);
    const size_t rows = (size_t)d->B * d->N * d->H;
    float *Ypart = reinterpret_cast<float *>(range_scratch);
    float *lpart = reinterpret_cast<float *>(range_scratch + align_up(sizeof(float) * C * rows * d->D));
    for (int c = 0; c < C; ++c) {
        const int m0 = c * kDecodeRange, mc = d->M - m0 < kDecodeRange ? d->M - m0 : kDecodeRange;
        const int rc = launch_decode_tc<D, DRT, true>(d, sms, Q, K, Z, nullptr, lpart + (size_t)c * rows, status, st, m0, mc,
                                                Ypart + (size_t)c * rows * DR, fast);
        if (rc != FLARE_OK) return rc;
    }
    decode_combine_kernel<DR><<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(Ypart, lpart, C, (long)rows,
                                                                             (__nv_bfloat16 *)Y, lse_dec);
    FLARE_CUDA(cudaGetLastError());
    return FLARE_OK;
}

// range_scratch: decode_range_bytes(d) bytes, or null (then more than kDecodeMaxM latents take the CUDA-core kernel)
int decode_impl(const flare_desc_t *d, const void *Q, const void *K, const float *Z, void *Y, float *lse_dec,
                uint32_t *status, cudaStream_t st, char *range_scratch = nullptr) {
    if (use_tc(d) && (d->M <= kDecodeMaxM || range_scratch != nullptr)) {
        const int sms = device_info().sms;
        switch (d->D) {
            case 4: return decode_tc_any<16, 4>(d, sms, Q, K, Z, Y, lse_dec, status, range_scratch, st);
            case 8: return decode_tc_any<16, 8>(d, sms, Q, K, Z, Y, lse_dec, status, range_scratch, st);
            case 16: return decode_tc_any<16, 0>(d, sms, Q, K, Z, Y, lse_dec, status, range_scratch, st);
            case 32: return decode_tc_any<32, 0>(d, sms, Q, K, Z, Y, lse_dec, status, range_scratch, st);
            default: return decode_tc_any<64, 0>(d, sms, Q, K, Z, Y, lse_dec, status, range_scratch, st);
        }
    }
    return (d->dtype == FLARE_DTYPE_F32)   ? launch_decode_simt<float>(d, Q, K, Z, Y, lse_dec, st)
           : (d->dtype == FLARE_DTYPE_F16) ? launch_decode_simt<__half>(d, Q, K, Z, Y, lse_dec, st)
                                           : launch_decode_simt<__nv_bfloat16>(d, Q, K, Z, Y, lse_dec, st);
}

// Scratch of flare_encode_static_scratch: part of the device image, shared by every call on the device.
// In host code this name is only a handle for cudaGetSymbolAddress; kernels must be given the looked-up address.
static __device__ __align__(256) unsigned char g_static_scratch[FLARE_STATIC_SCRATCH_BYTES];
std::atomic<void *> g_static_scratch_addr[64];

// Device address of g_static_scratch on the current device (looked up once per device, then cached).
int static_scratch_address(void **out) {
    int dev = -1;
    FLARE_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return FLARE_ERR_UNSUPPORTED;
    void *p = g_static_scratch_addr[dev].load(std::memory_order_acquire);
    if (p == nullptr) {
        FLARE_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
        if (p == nullptr) {
            snprintf(g_cuda_error, sizeof(g_cuda_error), "cudaGetSymbolAddress returned a null address");
            return FLARE_ERR_CUDA;
        }
        g_static_scratch_addr[dev].store(p, std::memory_order_release);
    }
    *out = p;
    return FLARE_OK;
}

// Kernels one call of `op` launches (the memset of the workspace header is not a kernel).
int launches_for(const flare_desc_t *d, int op, int sms) {
    // a fast form is followed by the exact form (which may exit at once)
    const int fe = use_fast(d, kFastEncode) ? 2 : 1, f = use_fast(d, kFastDecode) ? 2 : 1;
    const int enc = fe + 1;                                     // encode, merge
    const int dec = decode_in_ranges(d) ? f * decode_ranges(d) + 1 : f;   // ranges of latents and their combination
    switch (op) {
        case FLARE_OP_ENCODE: return enc;
        case FLARE_OP_DECODE: return dec;                       // (given a workspace)
        case FLARE_OP_FORWARD: return enc + dec;
        case FLARE_OP_BACKWARD: {
            (void)sms;
            const int tok = token_in_ranges(d) ? 2 * ((d->M + token_range(d) - 1) / token_range(d)) : 1;
            return 3 + tok + 2;                                 // dZ, its reduction, de; token kernel(s); dQ, its reduction
        }
        default: return 0;
    }
}

// ---- spectral analysis (Algorithm 1 of the paper's spectral appendix)
bool spectral_on_tensor_cores(const flare_desc_t *d) {
    return d->dtype == FLARE_DTYPE_BF16 && d->scale > 0.f && (d->D == 16 || d->D == 32) && d->M <= kTile && d->M % 16 == 0;
}
int spectral_splits(const flare_desc_t *d, int sms) {
    const int tiles = (d->N + kTile - 1) / kTile;
    long s = sms / ((long)d->B * d->H);
    if (s < 1) s = 1;
    if (s > tiles) s = tiles;
    return (int)s;
}
// More than 128 latents (a multiple of 64, bfloat16): the tensor-core kernel holds one block of 128 latents, so G is
// assembled from runs over pairs of 64-latent blocks (i, j): the pair's rows of Q_lat and lse_enc are gathered into a
// 128-latent problem, whose G holds the blocks G_ii, G_ij, G_ji, G_jj.  nb (nb - 1) / 2 runs, each one pass over the
// tokens: 1.5 times the arithmetic of one pass over all latents, two orders of magnitude below the CUDA-core kernel.
bool spectral_by_block_pairs(const flare_desc_t *d) {
    return d->dtype == FLARE_DTYPE_BF16 && d->scale > 0.f && (d->D == 16 || d->D == 32) && d->M > kTile && d->M % 64 == 0 &&
           d->M <= 1024;
}
struct SpectralPairLayout {
    size_t part, qp, lep, gp, total;
};
SpectralPairLayout spectral_pair_layout(const flare_desc_t *d, int sms) {
    SpectralPairLayout w{};
    size_t off = kHeaderBytes;
    w.part = off; off += align_up(sizeof(float) * (size_t)spectral_splits(d, sms) * kSpectralGroups * d->B * d->H * kTile * kTile);
    w.qp = off;   off += align_up((size_t)d->H * kTile * d->D * 2);
    w.lep = off;  off += align_up(sizeof(float) * (size_t)d->B * d->H * kTile);
    w.gp = off;   off += align_up(sizeof(float) * (size_t)d->B * d->H * kTile * kTile);
    w.total = off;
    return w;
}
size_t spectral_bytes(const flare_desc_t *d, int sms) {
    if (spectral_by_block_pairs(d) && use_tc(d)) return spectral_pair_layout(d, sms).total;
    if (!spectral_on_tensor_cores(d)) return kHeaderBytes;
    return kHeaderBytes + align_up(sizeof(float) * (size_t)spectral_splits(d, sms) * kSpectralGroups * d->B * d->H * kTile * kTile);
}

template <int D>
int launch_spectral_gram_tc(const flare_desc_t *d, int sms, const void *Q, const void *K, const float *lse_enc,
                            const float *lse_dec, float *G, char *ws, cudaStream_t st) {
    CUtensorMap tmK, tmQ;
    int rc;
    if ((rc = make_token_map(&tmK, K, d, kTile, D)) != FLARE_OK) return rc;
    if ((rc = make_latent_map(&tmQ, Q, d)) != FLARE_OK) return rc;
    static std::atomic<uint64_t> smem_opt_in{0};
    if (int rc_attr = ensure_big_smem(spectral_gram_tc_kernel<D>, smem_opt_in, 227 * 1024)) return rc_attr;
    SpectralArgs a;
    a.Q = static_cast<const __nv_bfloat16 *>(Q);
    a.lse_enc = lse_enc; a.lse_dec = lse_dec;
    a.part = reinterpret_cast<float *>(ws + kHeaderBytes);
    a.status = reinterpret_cast<uint32_t *>(ws);
    a.B = d->B; a.H = d->H; a.N = d->N; a.M = d->M;
    a.sl2 = d->scale * kLog2e;
    a.tiles = (d->N + kTile - 1) / kTile;
    a.splits = spectral_splits(d, sms);
    spectral_gram_tc_kernel<D><<<dim3(a.splits, d->H, d->B), kTcThreads, SpectralSmem<D>::total, st>>>(tmK, tmQ, a);
    FLARE_CUDA(cudaGetLastError());
    const long n = (long)d->B * d->H * d->M * d->M;
    spectral_gram_reduce_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(a.part, G, a.splits * kSpectralGroups, (long)d->B * d->H, d->M);
    FLARE_CUDA(cudaGetLastError());
    return FLARE_OK;
}

// rows [64 i, 64 i + 64) and [64 j, 64 j + 64) of every head's Q_lat and lse_enc -> a 128-latent problem
__global__ void spectral_gather_pair_kernel(const __nv_bfloat16 *__restrict__ Q, const float *__restrict__ lse_enc,
                                            __nv_bfloat16 *__restrict__ Qp, float *__restrict__ lep, int B, int H, int M, int D,
                                            int bi, int bj) {
    const long t = (long)blockIdx.x * blockDim.x + threadIdx.x;
    const long nq = (long)H * kTile * D, nl = (long)B * H * kTile;
    if (t < nq) {
        const int dcol = (int)(t % D), r = (int)((t / D) % kTile), h = (int)(t / ((long)D * kTile));
        const int m = 64 * (r < 64 ? bi : bj) + (r & 63);
        Qp[t] = Q[((size_t)h * M + m) * D + dcol];
    }
    if (t < nl) {
        const int r = (int)(t % kTile);
        const long bh = t / kTile;
        lep[t] = lse_enc[bh * M + 64 * (r < 64 ? bi : bj) + (r & 63)];
    }
}
// the pair's [128, 128] result -> the blocks (i, j), (j, i) of G, and the diagonal blocks this pair is responsible for
__global__ void spectral_scatter_pair_kernel(const float *__restrict__ Gp, float *__restrict__ G, long BH, int M, int bi, int bj,
                                             int write_ii, int write_jj) {
    const long t = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= BH * kTile * kTile) return;
    const int c = (int)(t % kTile), r = (int)((t / kTile) % kTile);
    const long bh = t / ((long)kTile * kTile);
    const bool rj = r >= 64, cj = c >= 64;
    if (!rj && !cj && !write_ii) return;
    if (rj && cj && !write_jj) return;
    G[(bh * M + 64 * (rj ? bj : bi) + (r & 63)) * M + 64 * (cj ? bj : bi) + (c & 63)] = Gp[t];
}

template <int D>
int spectral_gram_block_pairs(const flare_desc_t *d, int sms, const void *Q, const void *K, const float *lse_enc,
                              const float *lse_dec, float *G, char *ws, cudaStream_t st) {
    const SpectralPairLayout w = spectral_pair_layout(d, sms);
    __nv_bfloat16 *Qp = reinterpret_cast<__nv_bfloat16 *>(ws + w.qp);
    float *lep = reinterpret_cast<float *>(ws + w.lep), *Gp = reinterpret_cast<float *>(ws + w.gp);
    flare_desc_t dp = *d;
    dp.M = kTile;
    const int nb = d->M / 64;
    const long BH = (long)d->B * d->H;
    const long ngather = std::max((long)d->H * kTile * d->D, BH * kTile), nscatter = BH * kTile * kTile;
    for (int i = 0; i < nb; ++i)
        for (int j = i + 1; j < nb; ++j) {
            spectral_gather_pair_kernel<<<(unsigned)((ngather + 255) / 256), 256, 0, st>>>(
                static_cast<const __nv_bfloat16 *>(Q), lse_enc, Qp, lep, d->B, d->H, d->M, d->D, i, j);
            FLARE_CUDA(cudaGetLastError());
            const int rc = launch_spectral_gram_tc<D>(&dp, sms, Qp, K, lep, lse_dec, Gp, ws, st);
            if (rc != FLARE_OK) return rc;
            // every diagonal block is written once: G_ii by the pair (i, i + 1), the last one by the last pair
            spectral_scatter_pair_kernel<<<(unsigned)((nscatter + 255) / 256), 256, 0, st>>>(
                Gp, G, BH, d->M, i, j, j == i + 1, (i == nb - 2 && j == nb - 1) ? 1 : 0);
            FLARE_CUDA(cudaGetLastError());
        }
    return FLARE_OK;
}

template <typename T>
int launch_spectral_gram_simt(const flare_desc_t *d, const void *Q, const void *K, const float *lse_enc, const float *lse_dec,
                              float *G, cudaStream_t st) {
    const int tm = (d->M + 15) / 16;
    dim3 grid(tm * tm, d->H, d->B);
#define FLARE_CASE(DD)                                                                                                   \
    case DD:                                                                                                             \
        spectral_gram_simt_kernel<T, DD><<<grid, 256, 0, st>>>((const T *)Q, (const T *)K, lse_enc, lse_dec, G, d->B, d->H, \
                                                              d->N, d->M, d->scale);                                     \
        break;
    switch (d->D) {
        FLARE_CASE(4) FLARE_CASE(8) FLARE_CASE(16) FLARE_CASE(32) FLARE_CASE(64)
        default: return FLARE_ERR_UNSUPPORTED;
    }
#undef FLARE_CASE
    FLARE_CUDA(cudaGetLastError());
    return FLARE_OK;
}

// ---- variants of the mixer: one latent sequence shared by all heads; separate latent queries for decode

template <typename T>
__global__ void expand_heads_kernel(const T *__restrict__ src, T *__restrict__ dst, long per_head, int H) {
    const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= per_head * H) return;
    dst[i] = src[i % per_head];
}
__global__ void sum_heads_kernel(const float *__restrict__ src, float *__restrict__ dst, long per_head, int H) {
    const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= per_head) return;
    float s = 0.f;
    for (int h = 0; h < H; ++h) s += src[(size_t)h * per_head + i];
    dst[i] = s;
}
__global__ void fill_kernel(float *__restrict__ dst, long n, float v) {
    const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) dst[i] = v;
}
template <typename T>
__global__ void add_into_kernel(T *__restrict__ dst, const T *__restrict__ other, long n) {
    const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    T out;
    from_f32(out, to_f32(dst[i]) + to_f32(other[i]));
    dst[i] = out;
}

struct VariantLayout {
    size_t qe, qd, dq_full, dq2_full, inf_enc, inf_dec, dk2, total;   // offsets behind the operation's own workspace
};
// Scratch of the variant entry points, behind the workspace of the plain operation (base bytes).
VariantLayout variant_layout(const flare_desc_t *d, int op, int shared, int separate, size_t base) {
    VariantLayout v{};
    const size_t e = d->dtype == FLARE_DTYPE_F32 ? 4 : 2;
    const size_t q = align_up((size_t)d->H * d->M * d->D * e), qf = align_up((size_t)d->H * d->M * d->D * 4);
    size_t off = align_up(base);
    v.qe = off; if (shared) off += q;
    v.qd = off; if (shared && separate) off += q;
    if (op == FLARE_OP_BACKWARD) {
        v.dq_full = off; if (shared) off += qf;
        v.dq2_full = off; if (shared && separate) off += qf;
        v.inf_enc = off; if (separate) off += align_up(sizeof(float) * (size_t)d->B * d->H * d->M);
        v.inf_dec = off; if (separate) off += align_up(sizeof(float) * (size_t)d->B * d->N * d->H);
        v.dk2 = off; if (separate) off += align_up((size_t)d->B * d->N * d->H * d->D * e);
    }
    v.total = off;
    return v;
}

int expand_heads(const flare_desc_t *d, const void *src, void *dst, cudaStream_t st) {
    const long per = (long)d->M * d->D, n = per * d->H;
    if (d->dtype == FLARE_DTYPE_F32)
        expand_heads_kernel<float><<<(unsigned)((n + 255) / 256), 256, 0, st>>>((const float *)src, (float *)dst, per, d->H);
    else if (d->dtype == FLARE_DTYPE_F16)
        expand_heads_kernel<__half><<<(unsigned)((n + 255) / 256), 256, 0, st>>>((const __half *)src, (__half *)dst, per, d->H);
    else
        expand_heads_kernel<__nv_bfloat16><<<(unsigned)((n + 255) / 256), 256, 0, st>>>((const __nv_bfloat16 *)src, (__nv_bfloat16 *)dst, per, d->H);
    FLARE_CUDA(cudaGetLastError());
    return FLARE_OK;
}

}  // namespace

extern "C" {

int flare_version(void) { return 100; }

const char *flare_status_string(int status) {
    switch (status) {
        case FLARE_OK: return "ok";
        case FLARE_ERR_INVALID_ARG: return "invalid argument";
        case FLARE_ERR_UNSUPPORTED: return "unsupported shape or dtype";
        case FLARE_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case FLARE_ERR_ARCH: return "device is not compute capability 10.x";
        case FLARE_ERR_CUDA: return "CUDA error";
        case FLARE_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        default: return "unknown status";
    }
}

const char *flare_last_cuda_error(void) { return g_cuda_error; }

int flare_encode_partials(const flare_desc_t *desc) {
    if (check_desc(desc) != FLARE_OK) return 0;
    return partials_for(desc, device_info().sms);
}

int flare_launch_count(const flare_desc_t *desc, int op) {
    if (check_desc(desc) != FLARE_OK) return 0;
    return launches_for(desc, op, device_info().sms);
}

size_t flare_workspace_bytes(const flare_desc_t *desc, int op) {
    if (check_desc(desc) != FLARE_OK) return 0;
    const long rows = (long)desc->B * desc->H * desc->M;
    switch (op) {
        case FLARE_OP_ENCODE: return make_layout(partials_for(desc, device_info().sms), rows, desc->D, false).total;
        case FLARE_OP_DECODE: return kHeaderBytes + decode_range_bytes(desc);
        case FLARE_OP_FORWARD:
            return make_layout(partials_for(desc, device_info().sms), rows, desc->D, true).total + decode_range_bytes(desc);
        case FLARE_OP_BACKWARD: return bwd_layout(desc, device_info().sms).total;
        case FLARE_OP_SPECTRAL: return spectral_bytes(desc, device_info().sms);
        default: return 0;
    }
}

int flare_encode(const flare_desc_t *desc, const void *Q_lat, const void *K, const void *V, const uint8_t *key_mask,
                 float *Z, float *lse_enc, void *workspace, size_t workspace_bytes, flare_stream_t stream) {
    int rc = check_desc(desc);
    if (rc != FLARE_OK) return rc;
    if (!Q_lat || !K || !V || !Z || !workspace) return FLARE_ERR_INVALID_ARG;
    if (!aligned16(Q_lat) || !aligned16(K) || !aligned16(V) || !aligned16(Z) || !aligned16(workspace) ||
        (lse_enc && !aligned16(lse_enc)))
        return FLARE_ERR_INVALID_ARG;
    if ((rc = require_device()) != FLARE_OK) return rc;
    if (workspace_bytes < flare_workspace_bytes(desc, FLARE_OP_ENCODE)) return FLARE_ERR_WORKSPACE_TOO_SMALL;
    return encode_impl(desc, Q_lat, K, V, key_mask, Z, lse_enc, workspace, (cudaStream_t)stream);
}

int flare_encode_static_scratch(const flare_desc_t *desc, const void *Q_lat, const void *K, const void *V,
                                const uint8_t *key_mask, float *Z, float *lse_enc, flare_stream_t stream) {
    int rc = check_desc(desc);
    if (rc != FLARE_OK) return rc;
    if (!Q_lat || !K || !V || !Z) return FLARE_ERR_INVALID_ARG;
    if (!aligned16(Q_lat) || !aligned16(K) || !aligned16(V) || !aligned16(Z) || (lse_enc && !aligned16(lse_enc)))
        return FLARE_ERR_INVALID_ARG;
    if ((rc = require_device()) != FLARE_OK) return rc;
    const size_t need = flare_workspace_bytes(desc, FLARE_OP_ENCODE);
    if (need > (size_t)FLARE_STATIC_SCRATCH_BYTES) {
        snprintf(g_cuda_error, sizeof(g_cuda_error), "problem needs %zu bytes of scratch, the built-in array has %zu",
                 need, (size_t)FLARE_STATIC_SCRATCH_BYTES);
        return FLARE_ERR_WORKSPACE_TOO_SMALL;
    }
    void *scratch = nullptr;
    if ((rc = static_scratch_address(&scratch)) != FLARE_OK) return rc;
    // encode_impl zeroes the header words that must start at zero; every partial it later reads it first writes
    return encode_impl(desc, Q_lat, K, V, key_mask, Z, lse_enc, scratch, (cudaStream_t)stream);
}

int flare_decode(const flare_desc_t *desc, const void *Q_lat, const void *K, const float *Z, void *Y, float *lse_dec,
                 void *workspace, size_t workspace_bytes, flare_stream_t stream) {
    int rc = check_desc(desc);
    if (rc != FLARE_OK) return rc;
    if (!Q_lat || !K || !Z || !Y) return FLARE_ERR_INVALID_ARG;
    if (!aligned16(Q_lat) || !aligned16(K) || !aligned16(Z) || !aligned16(Y) || (lse_dec && !aligned16(lse_dec)) ||
        (workspace && !aligned16(workspace)))
        return FLARE_ERR_INVALID_ARG;
    if ((rc = require_device()) != FLARE_OK) return rc;
    if (workspace == nullptr) return decode_impl(desc, Q_lat, K, Z, Y, lse_dec, nullptr, (cudaStream_t)stream);
    if (workspace_bytes < flare_workspace_bytes(desc, FLARE_OP_DECODE)) return FLARE_ERR_WORKSPACE_TOO_SMALL;
    FLARE_CUDA(cudaMemsetAsync(workspace, 0, kHeaderBytes, (cudaStream_t)stream));
    char *range_scratch = decode_in_ranges(desc) ? static_cast<char *>(workspace) + kHeaderBytes : nullptr;
    return decode_impl(desc, Q_lat, K, Z, Y, lse_dec, static_cast<uint32_t *>(workspace), (cudaStream_t)stream,
                       range_scratch);
}

int flare_set_path(int path) {
    if (path != FLARE_PATH_AUTO && path != FLARE_PATH_EXACT && path != FLARE_PATH_FAST) return FLARE_ERR_INVALID_ARG;
    g_path.store(path, std::memory_order_relaxed);
    return FLARE_OK;
}

int flare_forward(const flare_desc_t *desc, const void *Q_lat, const void *K, const void *V, const uint8_t *key_mask,
                  void *Y, float *Z, float *lse_enc, float *lse_dec, void *workspace, size_t workspace_bytes,
                  flare_stream_t stream) {
    int rc = check_desc(desc);
    if (rc != FLARE_OK) return rc;
    if (!Q_lat || !K || !V || !Y || !workspace) return FLARE_ERR_INVALID_ARG;
    if (!aligned16(Q_lat) || !aligned16(K) || !aligned16(V) || !aligned16(Y) || !aligned16(workspace) ||
        (Z && !aligned16(Z)) || (lse_enc && !aligned16(lse_enc)) || (lse_dec && !aligned16(lse_dec)))
        return FLARE_ERR_INVALID_ARG;
    if ((rc = require_device()) != FLARE_OK) return rc;
    if (workspace_bytes < flare_workspace_bytes(desc, FLARE_OP_FORWARD)) return FLARE_ERR_WORKSPACE_TOO_SMALL;
    const WorkspaceLayout w = make_layout(partials_for(desc, device_info().sms), (long)desc->B * desc->H * desc->M, desc->D, true);
    if (Z == nullptr) Z = reinterpret_cast<float *>(static_cast<char *>(workspace) + w.z);
    rc = encode_impl(desc, Q_lat, K, V, key_mask, Z, lse_enc, workspace, (cudaStream_t)stream);
    if (rc != FLARE_OK) return rc;
    char *range_scratch = decode_in_ranges(desc) ? static_cast<char *>(workspace) + w.total : nullptr;
    return decode_impl(desc, Q_lat, K, Z, Y, lse_dec, reinterpret_cast<uint32_t *>(workspace), (cudaStream_t)stream,
                       range_scratch);
}

int flare_backward(const flare_desc_t *desc, const void *Q_lat, const void *K, const void *V, const uint8_t *key_mask,
                   const void *Y, const void *dY, const float *Z, const float *lse_enc, const float *lse_dec,
                   float *dQ_lat, void *dK, void *dV, void *workspace, size_t workspace_bytes,
                   flare_stream_t stream) {
    int rc = check_desc(desc);
    if (rc != FLARE_OK) return rc;
    const void *ptrs[] = {Q_lat, K, V, Y, dY, Z, lse_enc, lse_dec, dQ_lat, dK, dV, workspace};
    for (const void *p : ptrs)
        if (p == nullptr || !aligned16(p)) return FLARE_ERR_INVALID_ARG;
    if ((rc = require_device()) != FLARE_OK) return rc;
    if (workspace_bytes < flare_workspace_bytes(desc, FLARE_OP_BACKWARD)) return FLARE_ERR_WORKSPACE_TOO_SMALL;
    const int sms = device_info().sms;
    char *ws = static_cast<char *>(workspace);
    cudaStream_t st = (cudaStream_t)stream;
    return desc->dtype == FLARE_DTYPE_F32
               ? backward_simt<float>(desc, sms, Q_lat, K, V, key_mask, Y, dY, Z, lse_enc, lse_dec, dQ_lat, dK, dV, ws, st)
           : desc->dtype == FLARE_DTYPE_F16
               ? backward_simt<__half>(desc, sms, Q_lat, K, V, key_mask, Y, dY, Z, lse_enc, lse_dec, dQ_lat, dK, dV, ws, st)
               : backward_simt<__nv_bfloat16>(desc, sms, Q_lat, K, V, key_mask, Y, dY, Z, lse_enc, lse_dec, dQ_lat, dK,
                                              dV, ws, st);
}

int flare_forward_host(const flare_desc_t *desc, const void *hQ_lat, const void *hK, const void *hV,
                       const uint8_t *hmask, void *hY, void *dQ_lat, void *dK, void *dV, uint8_t *dmask, void *dY,
                       void *workspace, size_t workspace_bytes, flare_stream_t stream) {
    int rc = check_desc(desc);
    if (rc != FLARE_OK) return rc;
    if (!hQ_lat || !hK || !hV || !hY || !dQ_lat || !dK || !dV || !dY || (hmask && !dmask)) return FLARE_ERR_INVALID_ARG;
    if ((rc = require_device()) != FLARE_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t e = desc->dtype == FLARE_DTYPE_F32 ? 4 : 2;
    const size_t qb = (size_t)desc->H * desc->M * desc->D * e;
    const size_t tb = (size_t)desc->B * desc->N * desc->H * desc->D * e;
    FLARE_CUDA(cudaMemcpyAsync(dQ_lat, hQ_lat, qb, cudaMemcpyHostToDevice, st));
    FLARE_CUDA(cudaMemcpyAsync(dK, hK, tb, cudaMemcpyHostToDevice, st));
    FLARE_CUDA(cudaMemcpyAsync(dV, hV, tb, cudaMemcpyHostToDevice, st));
    if (hmask) FLARE_CUDA(cudaMemcpyAsync(dmask, hmask, (size_t)desc->B * desc->N, cudaMemcpyHostToDevice, st));
    rc = flare_forward(desc, dQ_lat, dK, dV, hmask ? dmask : nullptr, dY, nullptr, nullptr, nullptr, workspace,
                       workspace_bytes, stream);
    if (rc != FLARE_OK) return rc;
    FLARE_CUDA(cudaMemcpyAsync(hY, dY, tb, cudaMemcpyDeviceToHost, st));
    return FLARE_OK;
}

size_t flare_variant_workspace_bytes(const flare_desc_t *desc, int op, int shared_latents, int separate_decode_queries) {
    if (op != FLARE_OP_FORWARD && op != FLARE_OP_BACKWARD) return 0;
    const size_t base = flare_workspace_bytes(desc, op);
    if (base == 0) return 0;
    return variant_layout(desc, op, shared_latents, separate_decode_queries, base).total;
}

int flare_forward_variant(const flare_desc_t *desc, int shared_latents, const void *Q_enc, const void *Q_dec, const void *K,
                          const void *V, const uint8_t *key_mask, void *Y, float *Z, float *lse_enc, float *lse_dec,
                          void *workspace, size_t workspace_bytes, flare_stream_t stream) {
    int rc = check_desc(desc);
    if (rc != FLARE_OK) return rc;
    if (!Q_enc || !K || !V || !Y || !workspace) return FLARE_ERR_INVALID_ARG;
    const void *ptrs[] = {Q_enc, Q_dec, K, V, Y, Z, lse_enc, lse_dec, workspace};
    for (const void *p : ptrs)
        if (p != nullptr && !aligned16(p)) return FLARE_ERR_INVALID_ARG;
    if ((rc = require_device()) != FLARE_OK) return rc;
    const size_t base = flare_workspace_bytes(desc, FLARE_OP_FORWARD);
    const VariantLayout v = variant_layout(desc, FLARE_OP_FORWARD, shared_latents, Q_dec != nullptr, base);
    if (workspace_bytes < v.total) return FLARE_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)stream;
    char *ws = static_cast<char *>(workspace);
    const void *qe = Q_enc, *qd = Q_dec ? Q_dec : Q_enc;
    if (shared_latents) {
        if ((rc = expand_heads(desc, Q_enc, ws + v.qe, st)) != FLARE_OK) return rc;
        qe = ws + v.qe;
        qd = qe;
        if (Q_dec) {
            if ((rc = expand_heads(desc, Q_dec, ws + v.qd, st)) != FLARE_OK) return rc;
            qd = ws + v.qd;
        }
    }
    const WorkspaceLayout w = make_layout(partials_for(desc, device_info().sms), (long)desc->B * desc->H * desc->M, desc->D, true);
    if (Z == nullptr) Z = reinterpret_cast<float *>(ws + w.z);
    if ((rc = encode_impl(desc, qe, K, V, key_mask, Z, lse_enc, workspace, st)) != FLARE_OK) return rc;
    char *range_scratch = decode_in_ranges(desc) ? ws + w.total : nullptr;
    return decode_impl(desc, qd, K, Z, Y, lse_dec, reinterpret_cast<uint32_t *>(workspace), st, range_scratch);
}

int flare_backward_variant(const flare_desc_t *desc, int shared_latents, const void *Q_enc, const void *Q_dec, const void *K,
                           const void *V, const uint8_t *key_mask, const void *Y, const void *dY, const float *Z,
                           const float *lse_enc, const float *lse_dec, float *dQ_enc, float *dQ_dec, void *dK, void *dV,
                           void *workspace, size_t workspace_bytes, flare_stream_t stream) {
    int rc = check_desc(desc);
    if (rc != FLARE_OK) return rc;
    const void *need[] = {Q_enc, K, V, Y, dY, Z, lse_enc, lse_dec, dQ_enc, dK, dV, workspace};
    for (const void *p : need)
        if (p == nullptr || !aligned16(p)) return FLARE_ERR_INVALID_ARG;
    if ((Q_dec == nullptr) != (dQ_dec == nullptr)) return FLARE_ERR_INVALID_ARG;
    if ((Q_dec && !aligned16(Q_dec)) || (dQ_dec && !aligned16(dQ_dec))) return FLARE_ERR_INVALID_ARG;
    if ((rc = require_device()) != FLARE_OK) return rc;
    const size_t base = flare_workspace_bytes(desc, FLARE_OP_BACKWARD);
    const bool separate = Q_dec != nullptr;
    const VariantLayout v = variant_layout(desc, FLARE_OP_BACKWARD, shared_latents, separate, base);
    if (workspace_bytes < v.total) return FLARE_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)stream;
    char *ws = static_cast<char *>(workspace);
    const int sms = device_info().sms;
    const void *qe = Q_enc, *qd = Q_dec;
    float *dqe = dQ_enc, *dqd = dQ_dec;
    const long per = (long)desc->M * desc->D;
    if (shared_latents) {
        if ((rc = expand_heads(desc, Q_enc, ws + v.qe, st)) != FLARE_OK) return rc;
        qe = ws + v.qe;
        dqe = reinterpret_cast<float *>(ws + v.dq_full);
        if (separate) {
            if ((rc = expand_heads(desc, Q_dec, ws + v.qd, st)) != FLARE_OK) return rc;
            qd = ws + v.qd;
            dqd = reinterpret_cast<float *>(ws + v.dq2_full);
        }
    }
    auto run = [&](const void *q, const float *le, const float *ld, float *dq, void *dk, bool skip_a) {
        return desc->dtype == FLARE_DTYPE_F32
                   ? backward_simt<float>(desc, sms, q, K, V, key_mask, Y, dY, Z, le, ld, dq, dk, dV, ws, st, skip_a)
               : desc->dtype == FLARE_DTYPE_F16
                   ? backward_simt<__half>(desc, sms, q, K, V, key_mask, Y, dY, Z, le, ld, dq, dk, dV, ws, st, skip_a)
                   : backward_simt<__nv_bfloat16>(desc, sms, q, K, V, key_mask, Y, dY, Z, le, ld, dq, dk, dV, ws, st, skip_a);
    };
    if (!separate) {
        if ((rc = run(qe, lse_enc, lse_dec, dqe, dK, false)) != FLARE_OK) return rc;
    } else {
        // Two runs of the backward over the same workspace.  With lse_enc = +inf every encode weight exp(S - lse_enc) is 0,
        // so the first run (decode queries) leaves dZ, the decode term of dK and dQ_dec; with lse_dec = +inf the second
        // (encode queries; dZ kept from the first) leaves the encode term of dK, dV and dQ_enc.
        float *inf_enc = reinterpret_cast<float *>(ws + v.inf_enc), *inf_dec = reinterpret_cast<float *>(ws + v.inf_dec);
        const long ne = (long)desc->B * desc->H * desc->M, nd = (long)desc->B * desc->N * desc->H;
        fill_kernel<<<(unsigned)((ne + 255) / 256), 256, 0, st>>>(inf_enc, ne, INFINITY);
        fill_kernel<<<(unsigned)((nd + 255) / 256), 256, 0, st>>>(inf_dec, nd, INFINITY);
        FLARE_CUDA(cudaGetLastError());
        void *dk2 = ws + v.dk2;
        if ((rc = run(qd, inf_enc, lse_dec, dqd, dk2, false)) != FLARE_OK) return rc;
        if ((rc = run(qe, lse_enc, inf_dec, dqe, dK, true)) != FLARE_OK) return rc;
        const long nk = (long)desc->B * desc->N * desc->H * desc->D;
        if (desc->dtype == FLARE_DTYPE_F32)
            add_into_kernel<float><<<(unsigned)((nk + 255) / 256), 256, 0, st>>>((float *)dK, (const float *)dk2, nk);
        else if (desc->dtype == FLARE_DTYPE_F16)
            add_into_kernel<__half><<<(unsigned)((nk + 255) / 256), 256, 0, st>>>((__half *)dK, (const __half *)dk2, nk);
        else
            add_into_kernel<__nv_bfloat16><<<(unsigned)((nk + 255) / 256), 256, 0, st>>>((__nv_bfloat16 *)dK, (const __nv_bfloat16 *)dk2, nk);
        FLARE_CUDA(cudaGetLastError());
    }
    if (shared_latents) {
        sum_heads_kernel<<<(unsigned)((per + 255) / 256), 256, 0, st>>>(dqe, dQ_enc, per, desc->H);
        if (separate) sum_heads_kernel<<<(unsigned)((per + 255) / 256), 256, 0, st>>>(dqd, dQ_dec, per, desc->H);
        FLARE_CUDA(cudaGetLastError());
    }
    return FLARE_OK;
}

int flare_spectral_gram(const flare_desc_t *desc, const void *Q_lat, const void *K, const float *lse_enc,
                        const float *lse_dec, float *G, void *workspace, size_t workspace_bytes, flare_stream_t stream) {
    int rc = check_desc(desc);
    if (rc != FLARE_OK) return rc;
    const void *ptrs[] = {Q_lat, K, lse_enc, lse_dec, G, workspace};
    for (const void *p : ptrs)
        if (p == nullptr || !aligned16(p)) return FLARE_ERR_INVALID_ARG;
    if ((rc = require_device()) != FLARE_OK) return rc;
    const int sms = device_info().sms;
    if (workspace_bytes < spectral_bytes(desc, sms)) return FLARE_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)stream;
    FLARE_CUDA(cudaMemsetAsync(workspace, 0, kHeaderBytes, st));
    if (spectral_by_block_pairs(desc) && use_tc(desc)) {
        char *ws = static_cast<char *>(workspace);
        return desc->D == 16 ? spectral_gram_block_pairs<16>(desc, sms, Q_lat, K, lse_enc, lse_dec, G, ws, st)
                             : spectral_gram_block_pairs<32>(desc, sms, Q_lat, K, lse_enc, lse_dec, G, ws, st);
    }
    if (spectral_on_tensor_cores(desc) && use_tc(desc)) {
        char *ws = static_cast<char *>(workspace);
        return desc->D == 16 ? launch_spectral_gram_tc<16>(desc, sms, Q_lat, K, lse_enc, lse_dec, G, ws, st)
                             : launch_spectral_gram_tc<32>(desc, sms, Q_lat, K, lse_enc, lse_dec, G, ws, st);
    }
    return desc->dtype == FLARE_DTYPE_F32   ? launch_spectral_gram_simt<float>(desc, Q_lat, K, lse_enc, lse_dec, G, st)
           : desc->dtype == FLARE_DTYPE_F16 ? launch_spectral_gram_simt<__half>(desc, Q_lat, K, lse_enc, lse_dec, G, st)
                                            : launch_spectral_gram_simt<__nv_bfloat16>(desc, Q_lat, K, lse_enc, lse_dec, G, st);
}

int flare_spectral_eig(int32_t matrices, int32_t M, float *G, float *eigenvalues, float *U, int32_t sweeps, flare_stream_t stream) {
    if (matrices <= 0 || M <= 0 || M > 1024 || !G || !eigenvalues) return FLARE_ERR_INVALID_ARG;
    if (!aligned16(G) || !aligned16(eigenvalues) || (U && !aligned16(U))) return FLARE_ERR_INVALID_ARG;
    int rc = require_device();
    if (rc != FLARE_OK) return rc;
    if (sweeps <= 0) sweeps = 12;
    const int pairs = ((M + 1) & ~1) / 2;
    const size_t shmem = sizeof(float) * (4 * (size_t)pairs + M);
    // a step's rotations touch pairs * M elements: one thread each up to the largest block (the steps are latency-bound)
    const int threads = M >= 128 ? 1024 : M >= 64 ? 512 : 256;
    spectral_jacobi_kernel<<<(unsigned)matrices, threads, shmem, (cudaStream_t)stream>>>(G, eigenvalues, U, M, sweeps);
    FLARE_CUDA(cudaGetLastError());
    return FLARE_OK;
}

int flare_microbench(int which, int iters, void *scratch, size_t scratch_bytes, double *result, flare_stream_t stream) {
    if (!scratch || !result || !aligned16(scratch) || scratch_bytes < 4096 || which < 0 || which > 4) return FLARE_ERR_INVALID_ARG;
    int rc = require_device();
    if (rc != FLARE_OK) return rc;
    if (iters < 1) iters = 1;
    if (iters > 1000000) iters = 1000000;
    cudaStream_t st = (cudaStream_t)stream;
    const int sms = device_info().sms > 512 ? 512 : device_info().sms;
    unsigned long long *out = static_cast<unsigned long long *>(scratch);
    FLARE_CUDA(cudaMemsetAsync(scratch, 0, 4096, st));
    unsigned long long host[512];
    if (which <= 2) {
        if (which == 0) micro_softmax_kernel<0><<<sms, kTcThreads, 0, st>>>(iters, kLog2e, out);
        if (which == 1) micro_softmax_kernel<1><<<sms, kTcThreads, 0, st>>>(iters, kLog2e, out);
        if (which == 2) micro_softmax_kernel<2><<<sms, kTcThreads, 0, st>>>(iters, kLog2e, out);
        FLARE_CUDA(cudaGetLastError());
        FLARE_CUDA(cudaMemcpyAsync(host, out, sizeof(unsigned long long) * sms, cudaMemcpyDeviceToHost, st));
        FLARE_CUDA(cudaStreamSynchronize(st));
        double cycles = 0.0;
        for (int i = 0; i < sms; ++i) cycles += (double)host[i];
        cycles /= sms;
        *result = cycles > 0.0 ? 512.0 * 32.0 * iters / cycles : 0.0;     // 512 threads x 32 columns per round
    } else {
        static std::atomic<uint64_t> smem_opt_in{0};
        if (int rc_attr = ensure_big_smem(micro_mma_kernel, smem_opt_in, 64 * 1024)) return rc_attr;
        micro_mma_kernel<<<1, 64, 24576 + 1024, st>>>(iters, out);
        FLARE_CUDA(cudaGetLastError());
        FLARE_CUDA(cudaMemcpyAsync(host, out, sizeof(unsigned long long) * 2, cudaMemcpyDeviceToHost, st));
        FLARE_CUDA(cudaStreamSynchronize(st));
        *result = (double)host[which - 3];
    }
    return FLARE_OK;
}

int flare_check(const void *workspace, flare_stream_t stream) {
    void *builtin = nullptr;
    if (!workspace) {                                           // the built-in scratch of flare_encode_static_scratch
        const int rc = static_scratch_address(&builtin);
        if (rc != FLARE_OK) return rc;
        workspace = builtin;
    }
    uint32_t words[2] = {0, 0};
    FLARE_CUDA(cudaMemcpyAsync(words, workspace, sizeof(words), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    FLARE_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    return words[0] == 0 ? FLARE_OK : FLARE_ERR_TIMEOUT;
}

int flare_selftest_wait(void *workspace, uint64_t budget_ns, flare_stream_t stream) {
    if (!workspace || !aligned16(workspace)) return FLARE_ERR_INVALID_ARG;
    int rc = require_device();
    if (rc != FLARE_OK) return rc;
    if (budget_ns < 1000) budget_ns = 1000;
    if (budget_ns > 100000000ull) budget_ns = 100000000ull;     // never more than a tenth of a second
    cudaStream_t st = (cudaStream_t)stream;
    FLARE_CUDA(cudaMemsetAsync(workspace, 0, kHeaderBytes, st));
    selftest_wait_kernel<<<1, 32, 0, st>>>(static_cast<uint32_t *>(workspace), (unsigned long long)budget_ns);
    FLARE_CUDA(cudaGetLastError());
    return FLARE_OK;
}

}  // extern "C"
