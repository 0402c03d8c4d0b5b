// Tensor-core (tcgen05 + TMEM + TMA) kernels of the FLARE mixer for bfloat16 inputs on sm_100a.
//
// Both stages are two small dense contractions around a row softmax (paper Section 3.2):
//   encode  S = Q_h K_tile^T   (latents on the 128 TMEM lanes, tokens on columns)   acc += P V_tile
//   decode  S = K_tile Q_h^T   (tokens on the 128 TMEM lanes, latents on columns)   Y    = P Z_h
// Scores land in tensor memory; one thread owns one lane (one latent in encode, one token in decode), so row
// maxima and sums need no shuffles.  The bf16 weights P are written back over the scores in tensor memory and
// feed the second contraction as its A operand.  Warp roles: warp 0 issues TMA loads, warp 1 issues the MMAs
// and owns the TMEM allocation, warps 4-7 and 8-11 are two softmax groups that alternate on two TMEM buffers
// so that one group's exponentials overlap the other's MMAs.
#pragma once

#include "flare_common.cuh"
#include "flare_ptx.cuh"

namespace flare {

constexpr int kTcThreads = 384;
constexpr int kTile = 128;       // tokens per tile (decode: TMEM lanes; encode: score columns)
constexpr int kDecStages = 4;    // K tiles in flight (decode)
constexpr int kEncStages = 3;    // K+V tile pairs in flight (encode)
constexpr size_t kTcMinSmem = 120 * 1024;  // request at least this much so that one CTA owns an SM (and its TMEM)

// Error codes left in the workspace header by a wait that gave up.
enum : uint32_t { kErrDecode = 0x100, kErrEncode = 0x200 };

// Bounded wait whose outcome is the same for every lane of the warp, so that the warp-collective tensor-memory
// instructions that follow are executed by all lanes or by none.
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag, uint32_t code) {
    const bool ok = ptx::mbar_wait(bar, parity, abort_flag, code);
    return __all_sync(0xffffffffu, ok);
}

template <int D>
struct TileGeom {
    static constexpr int RB = D * 2;                                   // bytes per row of a [rows, D] bf16 tile
    static constexpr uint32_t SWZ = RB == 32 ? 6u : RB == 64 ? 4u : 2u;  // descriptor swizzle mode
    static constexpr int TILE_BYTES = kTile * RB;
    static constexpr int SBO = 8 * RB;                                 // stride between 8-row groups
    // 16-byte chunk permutation of the TMA / UMMA swizzle for row r
    __device__ static __forceinline__ int swz(int r) { return RB == 32 ? ((r >> 2) & 1) : RB == 64 ? ((r >> 1) & 3) : (r & 7); }
};

struct DecodeTcArgs {
    const float *Z;      // [B,H,M,D]
    __nv_bfloat16 *Y;    // [B,N,H,D]
    float *lse_dec;      // [B,N,H] or null
    uint32_t *status;    // workspace header or null
    int B, H, N, M;
    float sl2;           // scale * log2(e)
    int tiles;           // ceil(N / 128)
};

// Shared-memory carve-up of the decode kernel.
template <int D>
struct DecodeSmem {
    using G = TileGeom<D>;
    static constexpr size_t k_off = 0;
    // K tiles in flight: kDecStages, or 2 when Q_h and the two halves of Z_bh leave no room for more
    __host__ __device__ static int stages(int M) {
        return ((size_t)kDecStages * G::TILE_BYTES + (size_t)3 * M * G::RB + 2304 <= 227 * 1024) ? kDecStages : 2;
    }
    __host__ __device__ static size_t q_off(int M) { return (size_t)stages(M) * G::TILE_BYTES; }
    __host__ __device__ static size_t z_off(int M) { return q_off(M) + (size_t)M * G::RB; }  // [hi | lo], M rows each
    __host__ __device__ static size_t bar_off(int M) { return align_up(z_off(M) + (size_t)2 * M * G::RB, 1024); }
    __host__ __device__ static size_t total(int M) {
        size_t t = bar_off(M) + 256 + 1024;  // barriers and flags, plus slack to align the base to 1024
        return t < kTcMinSmem ? kTcMinSmem : t;
    }
};

// Decode.  grid = (ctas_per_head, H, B); each CTA walks a contiguous range of 128-token tiles of one (b, h)
// with Q_h and Z_bh resident in shared memory.
template <int D>
__global__ void __launch_bounds__(kTcThreads, 1)
decode_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ, DecodeTcArgs a) {
    using G = TileGeom<D>;
    using SM = DecodeSmem<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int M = a.M;
    uint8_t *sK = smem + SM::k_off;
    uint8_t *sQ = smem + SM::q_off(M);
    uint8_t *sZ = smem + SM::z_off(M);
    const int nstages = SM::stages(M);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + SM::bar_off(M));
    // barrier indices
    enum { K_FULL = 0, K_EMPTY = K_FULL + kDecStages, S_FULL = K_EMPTY + kDecStages, P_FULL = S_FULL + 2,
           Y_FULL = P_FULL + 2, BUF_EMPTY = Y_FULL + 2, Q_FULL = BUF_EMPTY + 2, NBARS };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + NBARS);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = blockIdx.y, b = blockIdx.z;
    const int t_begin = (int)((long)a.tiles * blockIdx.x / gridDim.x);
    const int t_end = (int)((long)a.tiles * (blockIdx.x + 1) / gridDim.x);
    const int ntiles = t_end - t_begin;

    // TMEM plan: per buffer S occupies M columns, P (bf16 pairs) overlays columns [0, M/2), Y sits after P
    // when that still fits inside the S columns, otherwise after S.
    const int nbuf = (M <= 256) ? 2 : 1;
    const int p_end = (M / 2 + 15) & ~15;
    const int y_off = (p_end + D <= M) ? p_end : M;
    const int cb = (((y_off + D > M) ? y_off + D : M) + 31) & ~31;  // columns per buffer
    uint32_t ncols = 32;
    while ((int)ncols < nbuf * cb) ncols *= 2;

    auto bar = [&](int i) { return ptx::smem_u32(bars + i); };

    if (threadIdx.x == 0) {
        for (int i = 0; i < NBARS; ++i) {
            uint32_t count = (i >= P_FULL && i < P_FULL + 2) || (i >= BUF_EMPTY && i < BUF_EMPTY + 2) ? 128u : 1u;
            ptx::mbar_init(bar(i), count);
        }
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmK);
        ptx::prefetch_tensormap(&tmQ);
    }
    if (warp == 1) ptx::tmem_alloc(ptx::smem_u32(tmem_slot), ncols);
    // Z_bh -> two bf16 halves (hi = round(z), lo = round(z - hi)) so that the latent sequence enters the second
    // contraction with about 16 mantissa bits; rows of RB bytes in the swizzled layout the MMA's B operand
    // expects (latent-major rows).
    {
        const float *Zg = a.Z + ((size_t)b * a.H + h) * M * D;
        for (int i = threadIdx.x; i < M * (D / 8); i += kTcThreads) {
            const int m = i / (D / 8), c = i % (D / 8);
            const float4 lo = *reinterpret_cast<const float4 *>(Zg + (size_t)m * D + c * 8);
            const float4 hi = *reinterpret_cast<const float4 *>(Zg + (size_t)m * D + c * 8 + 4);
            const float z[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
            uint32_t vh[4], vl[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                vh[k] = ptx::pack_bf16(z[2 * k], z[2 * k + 1]);
                const float r0 = z[2 * k] - __uint_as_float(vh[k] << 16);
                const float r1 = z[2 * k + 1] - __uint_as_float(vh[k] & 0xffff0000u);
                vl[k] = ptx::pack_bf16(r0, r1);
            }
            uint8_t *dst = sZ + (size_t)m * G::RB + ((c ^ G::swz(m)) << 4);
            *reinterpret_cast<uint4 *>(dst) = make_uint4(vh[0], vh[1], vh[2], vh[3]);
            *reinterpret_cast<uint4 *>(dst + (size_t)M * G::RB) = make_uint4(vl[0], vl[1], vl[2], vl[3]);
        }
        ptx::fence_proxy_async_smem();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tm = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            // Q_h: M/16 boxes of 16 rows
            ptx::mbar_arrive_expect_tx(bar(Q_FULL), (uint32_t)(M * G::RB));
            for (int r = 0; r < M; r += 16)
                ptx::tma_load_2d(ptx::smem_u32(sQ + (size_t)r * G::RB), &tmQ, bar(Q_FULL), 0, h * M + r);
            for (int i = 0; i < ntiles; ++i) {
                const int s = i % nstages;
                if (!ptx::mbar_wait(bar(K_EMPTY + s), ((i / nstages) & 1) ^ 1, abort_flag, kErrDecode | 1)) break;
                ptx::mbar_arrive_expect_tx(bar(K_FULL + s), G::TILE_BYTES);
                ptx::tma_load_3d(ptx::smem_u32(sK + (size_t)s * G::TILE_BYTES), &tmK, bar(K_FULL + s), h * D,
                                 (t_begin + i) * kTile, b);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const int nsplit = (M + 255) / 256;                 // score MMAs per k-step (N <= 256 each)
            const uint32_t idescS0 = ptx::instr_desc_bf16(128, M < 256 ? M : 256, 0, 0);
            const uint32_t idescS1 = ptx::instr_desc_bf16(128, M > 256 ? M - 256 : 16, 0, 0);
            const uint32_t idescY = ptx::instr_desc_bf16(128, D, 0, 1);
            const uint32_t qaddr = ptx::smem_u32(sQ), zaddr = ptx::smem_u32(sZ);
            bool ok = ptx::mbar_wait(bar(Q_FULL), 0, abort_flag, kErrDecode | 2);
            auto issue_scores = [&](int i) -> bool {
                const int s = i % nstages, j = i % nbuf, u = i / nbuf;
                if (!ptx::mbar_wait(bar(K_FULL + s), (i / nstages) & 1, abort_flag, kErrDecode | 3)) return false;
                if (!ptx::mbar_wait(bar(BUF_EMPTY + j), (u & 1) ^ 1, abort_flag, kErrDecode | 4)) return false;
                ptx::tc_fence_after();
                const uint32_t kaddr = ptx::smem_u32(sK + (size_t)s * G::TILE_BYTES);
                for (int ns = 0; ns < nsplit; ++ns)
                    for (int k = 0; k < D / 16; ++k)
                        ptx::mma_ss(tm + j * cb + ns * 256, ptx::smem_desc(kaddr + k * 32, 16, G::SBO, G::SWZ),
                                    ptx::smem_desc(qaddr + ns * 256 * G::RB + k * 32, 16, G::SBO, G::SWZ),
                                    ns == 0 ? idescS0 : idescS1, k > 0);
                ptx::mma_commit(bar(S_FULL + j));
                ptx::mma_commit(bar(K_EMPTY + s));
                return true;
            };
            auto issue_values = [&](int i) -> bool {
                const int j = i % nbuf, u = i / nbuf;
                if (!ptx::mbar_wait(bar(P_FULL + j), u & 1, abort_flag, kErrDecode | 5)) return false;
                ptx::tc_fence_after();
                for (int half = 0; half < 2; ++half)            // Y = P Z_hi + P Z_lo
                    for (int k = 0; k < M / 16; ++k)
                        ptx::mma_ts(tm + j * cb + y_off, tm + j * cb + k * 8,
                                    ptx::smem_desc(zaddr + (half * M + k * 16) * G::RB, G::SBO, G::SBO, G::SWZ), idescY,
                                    half > 0 || k > 0);
                ptx::mma_commit(bar(Y_FULL + j));
                return true;
            };
            for (int i = 0; ok && i < ntiles; ++i) {
                ok = issue_scores(i);
                if (nbuf == 2) {
                    if (ok && i > 0) ok = issue_values(i - 1);
                } else if (ok) {
                    ok = issue_values(i);
                }
            }
            if (ok && nbuf == 2 && ntiles > 0) issue_values(ntiles - 1);
        }
    } else if (warp >= 4) {
        const int g = (warp - 4) >> 2;                          // softmax group 0 or 1
        if (g < nbuf) {
            const int row = ((warp & 3) << 5) + lane;           // TMEM lane = token within the tile
            const uint32_t lane_addr = (uint32_t)((warp & 3) << 5) << 16;
            const uint32_t base = tm + lane_addr + g * cb;
            for (int i = g; i < ntiles; i += nbuf) {
                const int u = i / nbuf;
                if (!warp_wait(bar(S_FULL + g), u & 1, abort_flag, kErrDecode | 6)) break;
                ptx::tc_fence_after();
                uint32_t r[32];
                float mx = -INFINITY;
                for (int c = 0; c < M / 16; ++c) {              // pass 1: row maximum
                    ptx::tmem_ld16(base + c * 16, r);
                    ptx::tmem_wait_ld();
#pragma unroll
                    for (int k = 0; k < 16; ++k) mx = fmaxf(mx, __uint_as_float(r[k]));
                }
                const float neg = -mx * a.sl2;
                float sum = 0.f;
                for (int c = 0; c < M / 16; ++c) {              // pass 2: exponentials, bf16 pairs over the scores
                    ptx::tmem_ld16(base + c * 16, r);
                    ptx::tmem_wait_ld();
                    uint32_t pk[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const float p0 = ptx::ex2(fmaf(__uint_as_float(r[2 * k]), a.sl2, neg));
                        const float p1 = ptx::ex2(fmaf(__uint_as_float(r[2 * k + 1]), a.sl2, neg));
                        sum += p0 + p1;
                        pk[k] = ptx::pack_bf16(p0, p1);
                    }
                    ptx::tmem_st8(base + c * 8, pk);
                }
                ptx::tmem_wait_st();
                ptx::tc_fence_before();
                ptx::mbar_arrive(bar(P_FULL + g));
                if (!warp_wait(bar(Y_FULL + g), u & 1, abort_flag, kErrDecode | 7)) break;
                ptx::tc_fence_after();
                uint32_t y[D];
#pragma unroll
                for (int c = 0; c < D / 16; ++c) ptx::tmem_ld16(base + y_off + c * 16, y + c * 16);
                ptx::tmem_wait_ld();
                ptx::tc_fence_before();
                ptx::mbar_arrive(bar(BUF_EMPTY + g));
                const int n = (t_begin + i) * kTile + row;
                if (n < a.N) {
                    const float inv = 1.f / sum;
                    uint4 *dst = reinterpret_cast<uint4 *>(a.Y + (((size_t)b * a.N + n) * a.H + h) * D);
#pragma unroll
                    for (int c = 0; c < D / 8; ++c) {
                        uint4 v;
                        v.x = ptx::pack_bf16(__uint_as_float(y[c * 8 + 0]) * inv, __uint_as_float(y[c * 8 + 1]) * inv);
                        v.y = ptx::pack_bf16(__uint_as_float(y[c * 8 + 2]) * inv, __uint_as_float(y[c * 8 + 3]) * inv);
                        v.z = ptx::pack_bf16(__uint_as_float(y[c * 8 + 4]) * inv, __uint_as_float(y[c * 8 + 5]) * inv);
                        v.w = ptx::pack_bf16(__uint_as_float(y[c * 8 + 6]) * inv, __uint_as_float(y[c * 8 + 7]) * inv);
                        dst[c] = v;
                    }
                    if (a.lse_dec != nullptr)
                        a.lse_dec[((size_t)b * a.N + n) * a.H + h] = (mx * a.sl2 + log2f(sum)) * 0.6931471805599453f;
                }
            }
        }
    }
    // teardown: everyone arrives here (waits are bounded), then the allocating warp frees tensor memory
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tm, ncols);
    }
    if (threadIdx.x == 0 && *abort_flag != 0 && a.status != nullptr) atomicCAS(a.status, 0u, *abort_flag);
}

// ------------------------------------------------------------------------------------------------ encode

struct EncodeTcArgs {
    const uint8_t *key_mask;  // [B,N] or null
    float *part_m, *part_l, *part_acc;
    uint32_t *status;
    int B, H, N, M;
    float scale, sl2;
    int tiles;        // ceil(N / 128)
    int splits;       // CTAs along N per (b, h, latent-block pair)
    int pairs;        // ceil(ceil(M/128) / 2)
    int partials_per_split;  // 2 when M <= 128 (two slots alternate tiles), else 1
};

template <int D>
struct EncodeSmem {
    using G = TileGeom<D>;
    static constexpr size_t kv_off = 0;                         // [stage][K tile | V tile]
    __host__ __device__ static size_t q_off() { return (size_t)kEncStages * 2 * G::TILE_BYTES; }
    __host__ __device__ static size_t bar_off() { return q_off() + (size_t)2 * kTile * G::RB; }
    __host__ __device__ static size_t total() {
        size_t t = bar_off() + 512 + 1024;
        return t < kTcMinSmem ? kTcMinSmem : t;
    }
};

// Encode, split over N.  grid = (splits, H * pairs, B).  A CTA owns up to two blocks of 128 latents of head h
// ("slots", one softmax group and one TMEM score buffer + accumulator each) and a contiguous range of token
// tiles.  With M <= 128 the two slots share the one latent block and take alternate tiles.
template <int D>
__global__ void __launch_bounds__(kTcThreads, 1)
encode_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                 const __grid_constant__ CUtensorMap tmQ, EncodeTcArgs a) {
    using G = TileGeom<D>;
    using SM = EncodeSmem<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *sKV = smem + SM::kv_off;
    uint8_t *sQ = smem + SM::q_off();
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + SM::bar_off());
    enum { KV_FULL = 0, KV_EMPTY = KV_FULL + kEncStages, S_FULL = KV_EMPTY + kEncStages, P_FULL = S_FULL + 2,
           ACC_DONE = P_FULL + 2, Q_FULL, NBARS };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + NBARS);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int M = a.M;
    const int split = blockIdx.x, h = blockIdx.y / a.pairs, pair = blockIdx.y % a.pairs, b = blockIdx.z;
    const int t_begin = (int)((long)a.tiles * split / a.splits);
    const int t_end = (int)((long)a.tiles * (split + 1) / a.splits);
    const int nt = t_end - t_begin;
    const int MB = (M + kTile - 1) / kTile;
    // job q -> (tile, slot); see the kernel comment
    const bool alternate = (MB == 1);
    const int lb0 = pair * 2;                                   // latent block of slot 0
    const int nslots = alternate ? 2 : ((lb0 + 1 < MB) ? 2 : 1);
    const int nq = alternate ? nt : nt * nslots;
    const int rows_here = min(M - lb0 * kTile, 2 * kTile);      // latent rows of Q_h this CTA needs
    constexpr int SLOT_COLS = 256;                              // per slot: scores/P at [0,128), accumulator at [128,128+D)
    constexpr uint32_t NCOLS = 512;

    auto bar = [&](int i) { return ptx::smem_u32(bars + i); };

    if (threadIdx.x == 0) {
        for (int i = 0; i < NBARS; ++i) ptx::mbar_init(bar(i), (i >= P_FULL && i < P_FULL + 2) ? 128u : 1u);
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmK);
        ptx::prefetch_tensormap(&tmV);
        ptx::prefetch_tensormap(&tmQ);
    }
    if (warp == 1) ptx::tmem_alloc(ptx::smem_u32(tmem_slot), NCOLS);
    // latent rows beyond M are zero so their (discarded) lanes stay finite
    for (int i = threadIdx.x; i < (2 * kTile - rows_here) * (G::RB / 16); i += kTcThreads)
        reinterpret_cast<uint4 *>(sQ + (size_t)rows_here * G::RB)[i] = make_uint4(0, 0, 0, 0);
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tm = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            ptx::mbar_arrive_expect_tx(bar(Q_FULL), (uint32_t)(rows_here * G::RB));
            for (int r = 0; r < rows_here; r += 16)
                ptx::tma_load_2d(ptx::smem_u32(sQ + (size_t)r * G::RB), &tmQ, bar(Q_FULL), 0, h * M + lb0 * kTile + r);
            for (int i = 0; i < nt; ++i) {
                const int s = i % kEncStages;
                if (!ptx::mbar_wait(bar(KV_EMPTY + s), ((i / kEncStages) & 1) ^ 1, abort_flag, kErrEncode | 1)) break;
                ptx::mbar_arrive_expect_tx(bar(KV_FULL + s), 2 * G::TILE_BYTES);
                uint8_t *dst = sKV + (size_t)s * 2 * G::TILE_BYTES;
                ptx::tma_load_3d(ptx::smem_u32(dst), &tmK, bar(KV_FULL + s), h * D, (t_begin + i) * kTile, b);
                ptx::tma_load_3d(ptx::smem_u32(dst + G::TILE_BYTES), &tmV, bar(KV_FULL + s), h * D, (t_begin + i) * kTile, b);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idescS = ptx::instr_desc_bf16(128, kTile, 0, 0);
            const uint32_t idescV = ptx::instr_desc_bf16(128, D, 0, 1);
            const uint32_t qaddr = ptx::smem_u32(sQ);
            bool ok = ptx::mbar_wait(bar(Q_FULL), 0, abort_flag, kErrEncode | 2);
            auto tile_of = [&](int q) { return alternate ? q : q / nslots; };
            auto slot_of = [&](int q) { return alternate ? (q & 1) : q % nslots; };
            auto issue_scores = [&](int q) -> bool {
                const int t = tile_of(q), j = slot_of(q), s = t % kEncStages;
                if (!ptx::mbar_wait(bar(KV_FULL + s), (t / kEncStages) & 1, abort_flag, kErrEncode | 3)) return false;
                ptx::tc_fence_after();
                const uint32_t kaddr = ptx::smem_u32(sKV + (size_t)s * 2 * G::TILE_BYTES);
                const uint32_t qa = qaddr + (alternate ? 0 : j * kTile * G::RB);
                for (int k = 0; k < D / 16; ++k)
                    ptx::mma_ss(tm + j * SLOT_COLS, ptx::smem_desc(qa + k * 32, 16, G::SBO, G::SWZ),
                                ptx::smem_desc(kaddr + k * 32, 16, G::SBO, G::SWZ), idescS, k > 0);
                ptx::mma_commit(bar(S_FULL + j));
                return true;
            };
            auto issue_values = [&](int q) -> bool {
                const int t = tile_of(q), j = slot_of(q), s = t % kEncStages;
                const int u = alternate ? (q >> 1) : t;        // how many jobs this slot has done before
                if (!ptx::mbar_wait(bar(P_FULL + j), u & 1, abort_flag, kErrEncode | 4)) return false;
                ptx::tc_fence_after();
                const uint32_t vaddr = ptx::smem_u32(sKV + (size_t)s * 2 * G::TILE_BYTES + G::TILE_BYTES);
                for (int k = 0; k < kTile / 16; ++k)
                    ptx::mma_ts(tm + j * SLOT_COLS + kTile, tm + j * SLOT_COLS + k * 8,
                                ptx::smem_desc(vaddr + k * 16 * G::RB, G::SBO, G::SBO, G::SWZ), idescV, (u > 0 || k > 0));
                if (alternate || j == nslots - 1) ptx::mma_commit(bar(KV_EMPTY + s));  // last job of this tile
                return true;
            };
            const int stride = nslots;
            for (int q = 0; ok && q < stride && q < nq; ++q) ok = issue_scores(q);
            for (int q = 0; ok && q < nq; ++q) {
                ok = issue_values(q);
                if (ok && q + stride < nq) ok = issue_scores(q + stride);
            }
            if (ok) ptx::mma_commit(bar(ACC_DONE));
        }
    } else if (warp >= 4) {
        const int g = (warp - 4) >> 2;                          // softmax group = slot
        const int row = ((warp & 3) << 5) + lane;               // TMEM lane = latent within the block
        const uint32_t lane_addr = (uint32_t)((warp & 3) << 5) << 16;
        const uint32_t sbase = tm + lane_addr + g * SLOT_COLS, abase = sbase + kTile;
        float m_run = -INFINITY, l_run = 0.f;
        int done = 0;
        bool ok = true;
        if (g < nslots) {
            for (int q = g; q < nq; q += nslots, ++done) {
                const int t = t_begin + (alternate ? q : q / nslots);
                // validity bits of the tile's 128 tokens (tail beyond N, padding mask), one word per 32 tokens
                uint32_t wv[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int n = t * kTile + c * 32 + lane;
                    const bool valid = n < a.N && (a.key_mask == nullptr || a.key_mask[(size_t)b * a.N + n] != 0);
                    wv[c] = __ballot_sync(0xffffffffu, valid);
                }
                const uint32_t w0 = wv[0], w1 = wv[1], w2 = wv[2], w3 = wv[3];
                const bool all_valid = (w0 & w1 & w2 & w3) == 0xffffffffu;
                if (!warp_wait(bar(S_FULL + g), done & 1, abort_flag, kErrEncode | 5)) { ok = false; break; }
                ptx::tc_fence_after();
                uint32_t r[32];
                float tmax = -INFINITY;
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {                   // pass 1: tile maximum over valid tokens
                    ptx::tmem_ld32(sbase + c * 32, r);
                    ptx::tmem_wait_ld();
                    const uint32_t w = c == 0 ? w0 : c == 1 ? w1 : c == 2 ? w2 : w3;
                    if (all_valid) {
#pragma unroll
                        for (int k = 0; k < 32; ++k) tmax = fmaxf(tmax, __uint_as_float(r[k]));
                    } else {
#pragma unroll
                        for (int k = 0; k < 32; ++k)
                            if ((w >> k) & 1) tmax = fmaxf(tmax, __uint_as_float(r[k]));
                    }
                }
                const float m_new = fmaxf(m_run, tmax);
                const bool grow = done > 0 && m_new > m_run;
                if (__any_sync(0xffffffffu, grow)) {            // rescale the accumulator row (warp-uniform branch)
                    const float f = grow ? ptx::ex2((m_run - m_new) * a.sl2) : 1.f;
                    l_run *= f;
#pragma unroll
                    for (int c = 0; c < D / 16; ++c) {
                        ptx::tmem_ld16(abase + c * 16, r);
                        ptx::tmem_wait_ld();
#pragma unroll
                        for (int k = 0; k < 16; ++k) r[k] = __float_as_uint(__uint_as_float(r[k]) * f);
                        ptx::tmem_st16(abase + c * 16, r);
                    }
                }
                m_run = m_new;
                const bool dead = (m_run == -INFINITY);         // no valid token yet: all weights are zero
                const float neg = dead ? 0.f : -m_run * a.sl2;
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {                   // pass 2: weights, bf16 pairs over the scores
                    ptx::tmem_ld32(sbase + c * 32, r);
                    ptx::tmem_wait_ld();
                    const uint32_t w = c == 0 ? w0 : c == 1 ? w1 : c == 2 ? w2 : w3;
                    uint32_t pk[16];
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        float p0 = ptx::ex2(fmaf(__uint_as_float(r[2 * k]), a.sl2, neg));
                        float p1 = ptx::ex2(fmaf(__uint_as_float(r[2 * k + 1]), a.sl2, neg));
                        if (!all_valid) {
                            if (dead || !((w >> (2 * k)) & 1)) p0 = 0.f;
                            if (dead || !((w >> (2 * k + 1)) & 1)) p1 = 0.f;
                        }
                        l_run += p0 + p1;
                        pk[k] = ptx::pack_bf16(p0, p1);
                    }
                    ptx::tmem_st16(sbase + c * 16, pk);
                }
                ptx::tmem_wait_st();
                ptx::tc_fence_before();
                ptx::mbar_arrive(bar(P_FULL + g));
            }
        }
        // write this slot's partial (running max in natural-log units, sum, un-normalised rows)
        if (ok) ok = warp_wait(bar(ACC_DONE), 0, abort_flag, kErrEncode | 6);
        ptx::tc_fence_after();
        const int lb = alternate ? 0 : lb0 + g;
        const int m = lb * kTile + row;
        const bool writes = ok && (alternate || g < nslots);
        uint32_t acc[D];
        if (done > 0) {
#pragma unroll
            for (int c = 0; c < D / 16; ++c) ptx::tmem_ld16(abase + c * 16, acc + c * 16);
            ptx::tmem_wait_ld();
        } else {
#pragma unroll
            for (int k = 0; k < D; ++k) acc[k] = 0u;
        }
        if (writes && m < M) {
            const long rows = (long)a.B * a.H * M;
            const size_t prow = (size_t)(alternate ? split * 2 + g : split) * rows + ((size_t)b * a.H + h) * M + m;
            a.part_m[prow] = (m_run == -INFINITY) ? -INFINITY : m_run * a.scale;
            a.part_l[prow] = l_run;
            float4 *dst = reinterpret_cast<float4 *>(a.part_acc + prow * D);
#pragma unroll
            for (int c = 0; c < D / 4; ++c)
                dst[c] = make_float4(__uint_as_float(acc[4 * c]), __uint_as_float(acc[4 * c + 1]),
                                     __uint_as_float(acc[4 * c + 2]), __uint_as_float(acc[4 * c + 3]));
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tm, NCOLS);
    }
    if (threadIdx.x == 0 && *abort_flag != 0 && a.status != nullptr) atomicCAS(a.status, 0u, *abort_flag);
}

}  // namespace flare
