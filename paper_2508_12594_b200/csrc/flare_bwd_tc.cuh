// Tensor-core kernels of the backward for bfloat16 inputs on sm_100a (pass B: the gradient of the latent queries).
//
// dQ_m = scale * sum_n dS[m,n] k_n with
//   dS[m,n] = W_dec[n,m] (dY_n . Z_m - dd[n]) + W_enc[m,n] (dZ_m . V_n - de[m]),
//   W_dec[n,m] = exp(S[m,n] - lse_dec[n]),  W_enc[m,n] = valid(n) exp(S[m,n] - lse_enc[m]),  S = scale * q_m . k_n.
// The kernel has the shape of the encode kernel (latents on the 128 TMEM lanes, tokens on columns, the CTA's
// token range split over N, one pipeline per softmax group with its own issuing warp): per unit of 32 tokens
// three MMAs put S, A = Z dY^T and C = dZ V^T side by side in tensor memory, the group's threads turn them into
// bf16 dS over the scores, and a fourth MMA adds dS K_unit to the group's partial dQ.  Z and dZ enter as two bf16
// halves each (hi + lo): the products dY.Z_m and dZ_m.V_n are differenced against dd and de.
#pragma once

#include "flare_tc.cuh"

namespace flare {

constexpr int kBqStages = 2;     // (K, V, dY) tile triples in flight

struct BwdDqTcArgs {
    const float *Z, *dZ;       // [B,H,M,D]
    const float *lse_enc, *de; // [B,H,M]
    const float *lse_dec, *dd; // [B,N,H]
    const uint8_t *key_mask;   // [B,N] or null
    float *part;               // [P][B*H*M][D] partial dQ rows (un-scaled)
    uint32_t *status;
    int B, H, N, M;
    float sl2;                 // scale * log2(e)
    int tiles, splits, pairs, partials_per_split;
};

template <int D>
struct BwdDqSmem {
    using G = TileGeom<D>;
    static constexpr size_t tile_off = 0;                        // [stage][K | V | dY]
    __host__ __device__ static size_t q_off() { return (size_t)kBqStages * 3 * G::TILE_BYTES; }
    // Q, Z_hi, Z_lo, dZ_hi, dZ_lo: 256 latent rows each
    __host__ __device__ static size_t lat_off(int which) { return q_off() + (size_t)which * 2 * kTile * G::RB; }
    __host__ __device__ static size_t bar_off() { return lat_off(5); }
    static constexpr size_t kColBytes = 4 * kSoftmaxGroups * 3 * 32 * sizeof(float);   // per softmax warp: 3 x 32 column constants
    __host__ __device__ static size_t col_off() { return bar_off() + 512; }
    __host__ __device__ static size_t total() {
        size_t t = col_off() + kColBytes + 1024;
        return t < kTcMinSmem ? kTcMinSmem : t;
    }
};

// grid = (splits, H * pairs, B), as the encode kernel.
template <int D>
__global__ void __launch_bounds__(kTcThreads, 1)
bwd_dq_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                 const __grid_constant__ CUtensorMap tmG, const __grid_constant__ CUtensorMap tmQ, BwdDqTcArgs a) {
    using G = TileGeom<D>;
    using SM = BwdDqSmem<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *sT = smem + SM::tile_off;
    uint8_t *sQ = smem + SM::lat_off(0);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + SM::bar_off());
    constexpr int NG = kSoftmaxGroups;
    enum { T_FULL = 0, T_EMPTY = T_FULL + kBqStages, S_FULL = T_EMPTY + kBqStages, P_FULL = S_FULL + NG,
           ACC_DONE = P_FULL + NG, Q_FULL = ACC_DONE + NG, NBARS };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + NBARS);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int M = a.M;
    const int split = blockIdx.x, h = blockIdx.y / a.pairs, pair = blockIdx.y % a.pairs, b = blockIdx.z;
    const int t_begin = (int)((long)a.tiles * split / a.splits);
    const int t_end = (int)((long)a.tiles * (split + 1) / a.splits);
    const int nt = t_end - t_begin;
    const int MB = (M + kTile - 1) / kTile;
    const bool alternate = (MB == 1);                           // one latent block: the two slots take alternate tiles
    const int lb0 = pair * 2;
    const int nslots = alternate ? 2 : ((lb0 + 1 < MB) ? 2 : 1);
    const int nq = alternate ? nt : nt * nslots;
    const int rows_here = min(M - lb0 * kTile, 2 * kTile);
    constexpr int SLOT_COLS = 256, HALF = kTile / 2, UNIT = 32;
    constexpr uint32_t NCOLS = 512;
    // per group (128 columns): S at 0, A at 32, C at 64, partial dQ at 96
    auto bar = [&](int i) { return ptx::smem_u32(bars + i); };

    if (threadIdx.x == 0) {
        const uint32_t users = alternate ? 2u : 2u * (uint32_t)nslots;
        for (int i = 0; i < NBARS; ++i)
            ptx::mbar_init(bar(i), (i >= P_FULL && i < P_FULL + NG) ? 128u
                                   : (i >= T_EMPTY && i < T_EMPTY + kBqStages) ? users : 1u);
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmK);
        ptx::prefetch_tensormap(&tmV);
        ptx::prefetch_tensormap(&tmG);
        ptx::prefetch_tensormap(&tmQ);
    }
    if (warp == kFirstIssuerWarp) ptx::tmem_alloc(ptx::smem_u32(tmem_slot), NCOLS);
    // zero the latent rows beyond M (all five operands), then Z and dZ as bf16 hi/lo rows in the swizzled layout
    for (int i = threadIdx.x; i < 5 * 2 * kTile * (G::RB / 16); i += kTcThreads) {
        const int which = i / (2 * kTile * (G::RB / 16)), rem = i % (2 * kTile * (G::RB / 16));
        if (rem / (G::RB / 16) >= rows_here) reinterpret_cast<uint4 *>(smem + SM::lat_off(which))[rem] = make_uint4(0, 0, 0, 0);
    }
    for (int i = threadIdx.x; i < 2 * rows_here * (D / 8); i += kTcThreads) {
        const int which = i / (rows_here * (D / 8)), rem = i % (rows_here * (D / 8)), m = rem / (D / 8), ch = rem % (D / 8);
        const float *src = (which == 0 ? a.Z : a.dZ) + (((size_t)b * a.H + h) * M + lb0 * kTile + m) * D + ch * 8;
        const float4 lo4 = *reinterpret_cast<const float4 *>(src), hi4 = *reinterpret_cast<const float4 *>(src + 4);
        const float z[8] = {lo4.x, lo4.y, lo4.z, lo4.w, hi4.x, hi4.y, hi4.z, hi4.w};
        uint32_t vh[4], vl[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            vh[k] = ptx::pack_bf16(z[2 * k], z[2 * k + 1]);
            vl[k] = ptx::pack_bf16(z[2 * k] - __uint_as_float(vh[k] << 16), z[2 * k + 1] - __uint_as_float(vh[k] & 0xffff0000u));
        }
        const size_t off = (size_t)m * G::RB + ((ch ^ G::swz(m)) << 4);
        *reinterpret_cast<uint4 *>(smem + SM::lat_off(1 + 2 * which) + off) = make_uint4(vh[0], vh[1], vh[2], vh[3]);
        *reinterpret_cast<uint4 *>(smem + SM::lat_off(2 + 2 * which) + off) = make_uint4(vl[0], vl[1], vl[2], vl[3]);
    }
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
                const int s = i % kBqStages;
                if (!ptx::mbar_wait(bar(T_EMPTY + s), ((i / kBqStages) & 1) ^ 1, abort_flag, kErrBwdDq | 1)) break;
                ptx::mbar_arrive_expect_tx(bar(T_FULL + s), 3 * G::TILE_BYTES);
                uint8_t *dst = sT + (size_t)s * 3 * G::TILE_BYTES;
                ptx::tma_load_3d(ptx::smem_u32(dst), &tmK, bar(T_FULL + s), h * D, (t_begin + i) * kTile, b);
                ptx::tma_load_3d(ptx::smem_u32(dst + G::TILE_BYTES), &tmV, bar(T_FULL + s), h * D, (t_begin + i) * kTile, b);
                ptx::tma_load_3d(ptx::smem_u32(dst + 2 * G::TILE_BYTES), &tmG, bar(T_FULL + s), h * D, (t_begin + i) * kTile, b);
            }
        }
    } else if (warp < kFirstSoftmaxWarp) {
        const int g = warp - kFirstIssuerWarp;
        const int j = g >> 1, c = g & 1;
        if (lane == 0 && j < nslots) {
            const uint32_t idescS = ptx::instr_desc_bf16(128, UNIT, 0, 0);
            const uint32_t idescQ = ptx::instr_desc_bf16(128, D, 0, 1);
            const uint64_t blk = (uint64_t)(alternate ? 0 : j * kTile * G::RB / 16);     // the slot's latent block
            uint64_t ldesc[5];
#pragma unroll
            for (int i = 0; i < 5; ++i) ldesc[i] = ptx::smem_desc(ptx::smem_u32(smem + SM::lat_off(i)), 16, G::SBO, G::SWZ) + blk;
            const uint32_t gcol = tm + j * SLOT_COLS + c * 2 * HALF;
            const uint32_t dcol = gcol + 3 * UNIT;
            bool ok = ptx::mbar_wait(bar(Q_FULL), 0, abort_flag, kErrBwdDq | 2);
            const int jobs = (nq - j + nslots - 1) / nslots;
            const int units = 2 * jobs;
            int t = alternate ? j : 0;
            const int t_step = alternate ? 2 : 1;
            for (int n = 0; ok && n < units; ++n) {
                const int s = t % kBqStages, w = n & 1;
                if (w == 0) {
                    if (!ptx::mbar_wait(bar(T_FULL + s), (t / kBqStages) & 1, abort_flag, kErrBwdDq | 3)) break;
                    ptx::tc_fence_after();
                }
                const uint32_t tbase = ptx::smem_u32(sT + (size_t)s * 3 * G::TILE_BYTES);
                const uint64_t rowoff = (uint64_t)((c * HALF + w * UNIT) * G::RB / 16);   // the unit's 32 token rows
                const uint64_t kdesc = ptx::smem_desc(tbase, 16, G::SBO, G::SWZ) + rowoff;
                const uint64_t vdesc = ptx::smem_desc(tbase + G::TILE_BYTES, 16, G::SBO, G::SWZ) + rowoff;
                const uint64_t gdesc = ptx::smem_desc(tbase + 2 * G::TILE_BYTES, 16, G::SBO, G::SWZ) + rowoff;
                // S = Q K^T | A = (Z_hi + Z_lo) dY^T | C = (dZ_hi + dZ_lo) V^T, each 128 latents x 32 tokens
#pragma unroll
                for (int k = 0; k < D / 16; ++k) ptx::mma_ss(gcol, ldesc[0] + 2 * k, kdesc + 2 * k, idescS, k > 0);
#pragma unroll
                for (int k = 0; k < D / 16; ++k) ptx::mma_ss(gcol + UNIT, ldesc[1] + 2 * k, gdesc + 2 * k, idescS, k > 0);
#pragma unroll
                for (int k = 0; k < D / 16; ++k) ptx::mma_ss(gcol + UNIT, ldesc[2] + 2 * k, gdesc + 2 * k, idescS, 1u);
#pragma unroll
                for (int k = 0; k < D / 16; ++k) ptx::mma_ss(gcol + 2 * UNIT, ldesc[3] + 2 * k, vdesc + 2 * k, idescS, k > 0);
#pragma unroll
                for (int k = 0; k < D / 16; ++k) ptx::mma_ss(gcol + 2 * UNIT, ldesc[4] + 2 * k, vdesc + 2 * k, idescS, 1u);
                ptx::mma_commit(bar(S_FULL + g));
                if (!ptx::mbar_wait(bar(P_FULL + g), n & 1, abort_flag, kErrBwdDq | 4)) break;
                ptx::tc_fence_after();
                // dQ_part += dS_unit K_unit: the K tile as the MN-major B operand, 16 token rows further on per k-step
                const uint64_t kmn = ptx::smem_desc(tbase, G::SBO, G::SBO, G::SWZ) + rowoff;
#pragma unroll
                for (int k = 0; k < UNIT / 16; ++k)
                    ptx::mma_ts(dcol, gcol + k * 8, kmn + (uint64_t)(k * G::RB), idescQ, (n > 0 || k > 0) ? 1u : 0u);
#pragma unroll
                for (int k = 0; k < UNIT / 16; ++k) ptx::mma_ts(dcol, gcol + UNIT + k * 8, kmn + (uint64_t)(k * G::RB), idescQ, 1u);
                if (w == 1) {
                    ptx::mma_commit(bar(T_EMPTY + s));
                    t += t_step;
                }
            }
            if (ok) ptx::mma_commit(bar(ACC_DONE + g));
        }
    } else {
        const int g = (warp - kFirstSoftmaxWarp) >> 2;
        const int j = g >> 1, c = g & 1;
        const int row = ((warp & 3) << 5) + lane;
        const uint32_t lane_addr = (uint32_t)((warp & 3) << 5) << 16;
        const uint32_t gcol = tm + lane_addr + j * SLOT_COLS + c * 2 * HALF;
        const uint32_t abase = gcol + 3 * UNIT;
        const float2 sl2p = make_float2(a.sl2, a.sl2);
        const int lb = alternate ? 0 : lb0 + j;
        const int m = lb * kTile + row;
        // this thread's latent: -lse_enc in log2 units (-inf for a latent that saw no valid token or lies beyond M), -de
        float negle = -INFINITY, negde = 0.f;
        if (j < nslots && m < M) {
            const size_t r = ((size_t)b * a.H + h) * M + m;
            const float le = a.lse_enc[r];
            negle = (le == -INFINITY) ? -INFINITY : -le * 1.4426950408889634f;
            negde = -a.de[r];
        }
        const float2 neglep = make_float2(negle, negle), negdep = make_float2(negde, negde);
        float *cst = reinterpret_cast<float *>(smem + SM::col_off()) + (warp - kFirstSoftmaxWarp) * 96;   // this warp's column constants
        int done = 0;
        bool ok = true;
        auto unit = [&](auto masked, int t, int w) -> bool {
            constexpr bool kMasked = decltype(masked)::value;
            const int n = t * kTile + c * HALF + w * UNIT + lane;          // this lane fetches the constants of token n
            uint32_t wv = 0xffffffffu;
            __syncwarp();                                                   // the previous unit's reads are done
            if (n < a.N) {
                const size_t i = ((size_t)b * a.N + n) * a.H + h;
                cst[lane] = -a.lse_dec[i] * 1.4426950408889634f;
                cst[32 + lane] = -a.dd[i];
            } else {
                cst[lane] = -INFINITY;
                cst[32 + lane] = 0.f;
            }
            if (kMasked) wv = __ballot_sync(0xffffffffu, n < a.N && (a.key_mask == nullptr || a.key_mask[(size_t)b * a.N + n] != 0));
            __syncwarp();
            if (!warp_wait(bar(S_FULL + g), done & 1, abort_flag, kErrBwdDq | 5)) return false;
            ptx::tc_fence_after();
            // 8 tokens at a time: their dS goes back as two bf16 halves, hi over score columns the thread has
            // already read (4 packed columns per 8 tokens), lo likewise over the columns of A
#pragma unroll
            for (int qd = 0; qd < 4; ++qd) {
                uint32_t s[8], av[8], cv[8], pk[4], pl[4];
                ptx::tmem_ld8(gcol + qd * 8, s);
                ptx::tmem_ld8(gcol + UNIT + qd * 8, av);
                ptx::tmem_ld8(gcol + 2 * UNIT + qd * 8, cv);
                ptx::tmem_wait_ld();
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int col = qd * 8 + 2 * k;
                    const float2 sp = make_float2(__uint_as_float(s[2 * k]), __uint_as_float(s[2 * k + 1]));
                    const float2 nld = *reinterpret_cast<const float2 *>(cst + col);
                    const float2 ndd = *reinterpret_cast<const float2 *>(cst + 32 + col);
                    const float2 xd = __ffma2_rn(sp, sl2p, nld), xe = __ffma2_rn(sp, sl2p, neglep);
                    const float2 pd = make_float2(ptx::ex2(xd.x), ptx::ex2(xd.y));
                    float2 pe = make_float2(ptx::ex2(xe.x), ptx::ex2(xe.y));
                    if (kMasked) {
                        if (!((wv >> col) & 1)) pe.x = 0.f;
                        if (!((wv >> (col + 1)) & 1)) pe.y = 0.f;
                    }
                    const float2 u = __fadd2_rn(make_float2(__uint_as_float(av[2 * k]), __uint_as_float(av[2 * k + 1])), ndd);
                    const float2 v = __fadd2_rn(make_float2(__uint_as_float(cv[2 * k]), __uint_as_float(cv[2 * k + 1])), negdep);
                    const float2 ds = __ffma2_rn(pd, u, __fmul2_rn(pe, v));
                    const uint32_t hi = ptx::pack_bf16(ds.x, ds.y);
                    pk[k] = hi;
                    pl[k] = ptx::pack_bf16(ds.x - __uint_as_float(hi << 16), ds.y - __uint_as_float(hi & 0xffff0000u));
                }
                ptx::tmem_st4(gcol + qd * 4, pk);
                ptx::tmem_st4(gcol + UNIT + qd * 4, pl);
            }
            ptx::tmem_wait_st();
            ptx::tc_fence_before();
            ptx::mbar_arrive(bar(P_FULL + g));
            ++done;
            return true;
        };
        if (j < nslots) {
            for (int q = j; ok && q < nq; q += nslots) {
                const int t = t_begin + (alternate ? q : q / nslots);
                const bool plain = a.key_mask == nullptr && (t + 1) * kTile <= a.N;
#pragma unroll 1
                for (int w = 0; ok && w < 2; ++w) ok = plain ? unit(std::false_type{}, t, w) : unit(std::true_type{}, t, w);
            }
        }
        if (ok && j < nslots) ok = warp_wait(bar(ACC_DONE + g), 0, abort_flag, kErrBwdDq | 6);
        ptx::tc_fence_after();
        uint32_t acc[D];
        if (done > 0) {
#pragma unroll
            for (int dc = 0; dc < D / 16; ++dc) ptx::tmem_ld16(abase + dc * 16, acc + dc * 16);
            ptx::tmem_wait_ld();
        } else {
#pragma unroll
            for (int k = 0; k < D; ++k) acc[k] = 0u;
        }
        if (ok && j < nslots && m < M) {
            const long rows = (long)a.B * a.H * M;
            const int part = split * a.partials_per_split + (alternate ? 2 * j + c : c);
            float4 *dst = reinterpret_cast<float4 *>(a.part + ((size_t)part * rows + ((size_t)b * a.H + h) * M + m) * D);
#pragma unroll
            for (int dc = 0; dc < D / 4; ++dc)
                dst[dc] = make_float4(__uint_as_float(acc[4 * dc]), __uint_as_float(acc[4 * dc + 1]),
                                      __uint_as_float(acc[4 * dc + 2]), __uint_as_float(acc[4 * dc + 3]));
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == kFirstIssuerWarp) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tm, NCOLS);
    }
    if (threadIdx.x == 0 && *abort_flag != 0 && a.status != nullptr) atomicCAS(a.status, 0u, *abort_flag);
}

}  // namespace flare
