// Tensor-core kernels of the backward for bfloat16 inputs on sm_100a (pass B: the gradient of the latent queries).
//
// dQ_m = scale * sum_n dS[m,n] k_n with
//   dS[m,n] = W_dec[n,m] (dY_n . Z_m - dd[n]) + W_enc[m,n] (dZ_m . V_n - de[m]),
//   W_dec[n,m] = exp(S[m,n] - lse_dec[n]),  W_enc[m,n] = valid(n) exp(S[m,n] - lse_enc[m]),  S = scale * q_m . k_n.
// The kernel has the shape of the encode kernel (latents on the 128 TMEM lanes, tokens on columns, the CTA's
// token range split over N, one pipeline per softmax group with its own issuing warp): per unit of 16 tokens
// three MMAs put S, A = Z dY^T and C = dZ V^T side by side in tensor memory, the group's threads turn them into
// dS (two bf16 halves) over columns they have read, and two more MMAs add dS K_unit to the group's partial dQ.
// Units alternate between two such buffers, so the tiles of the next unit and the dQ MMAs of the previous one
// run while the group works on the current one (2 x 48 + D <= 128 columns per group).  Z and dZ enter as two bf16
// halves each (hi + lo): the products dY.Z_m and dZ_m.V_n are differenced against dd and de.
#pragma once

#include "flare_tc.cuh"

namespace flare {

constexpr int kBqStages = 3;     // (K, V, dY) tile triples in flight where all four groups of a CTA work on the same tile
constexpr int kBqMaxStages = 8;  // ... and at most where the two slots take alternate tiles (see kEncMaxStages)

struct BwdDqTcArgs {
    const __nv_bfloat16 *Q;    // [H,M,D] (read directly in the half-width form)
    const float *Z, *dZ;       // [B,H,M,D]
    const float *lse_enc, *de; // [B,H,M]
    const float *lse_dec;      // [B,N,H]
    const float *dd;           // [B,H,N] (workspace)
    const uint8_t *key_mask;   // [B,N] or null
    float *part;               // [P][B*H*M][D] partial dQ rows (un-scaled)
    uint32_t *status;
    int B, H, N, M;
    float sl2;                 // scale * log2(e)
    int tiles, splits, pairs, partials_per_split;
};

template <int D, bool kAlt>
struct BwdDqSmem {
    using G = TileGeom<D>;
    static constexpr size_t kColBytes = 4 * kSoftmaxGroups * 2 * 64 * sizeof(float);   // per softmax warp: 2 x 64 column constants
    static constexpr size_t total_for(int n) {
        return (size_t)n * 3 * G::TILE_BYTES + (size_t)5 * 2 * kTile * G::RB + 512 + kColBytes + 1024;
    }
    static constexpr int stages_for() {
        int n = kAlt ? kBqMaxStages : kBqStages;
        while (n > kBqStages && total_for(n) > 227 * 1024) --n;
        return n;
    }
    static constexpr int kStages = stages_for();                 // (K, V, dY) tile triples in flight
    static constexpr size_t tile_off = 0;                        // [stage][K | V | dY]
    __host__ __device__ static size_t q_off() { return (size_t)kStages * 3 * G::TILE_BYTES; }
    // Q, Z_hi, Z_lo, dZ_hi, dZ_lo: 256 latent rows each
    __host__ __device__ static size_t lat_off(int which) { return q_off() + (size_t)which * 2 * kTile * G::RB; }
    __host__ __device__ static size_t bar_off() { return lat_off(5); }
    __host__ __device__ static size_t col_off() { return bar_off() + 512; }
    __host__ __device__ static size_t total() {
        size_t t = col_off() + kColBytes + 1024;
        return t < kTcMinSmem ? kTcMinSmem : t;
    }
};

// grid = (splits, H * pairs, B), as the encode kernel.  DRT = 8 or 4 (with D = 16): the narrow form of the forward
// kernels (the head is DRT wide in memory; token tiles carry the neighbouring heads' features beside the head's
// own, every latent operand zeros there, and the other columns of the partial dQ are dropped).
// kPadded: the launch has padded tokens (a key mask, or N not a multiple of the tile); without it the unit body that
// tests validity is not compiled in.  kAlt: one latent block (the host picks this form for M <= 128), the two slots take
// alternate tiles and the tile ring is as deep as fits.
template <int D, int DRT = 0, bool kPadded = true, bool kAlt = false>
__global__ void __launch_bounds__(kTcThreads, 1)
bwd_dq_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                 const __grid_constant__ CUtensorMap tmG, const __grid_constant__ CUtensorMap tmQ, BwdDqTcArgs a) {
    using G = TileGeom<D>;
    using SM = BwdDqSmem<D, kAlt>;
    constexpr int nstages = SM::kStages;                        // depth of the tile ring
    constexpr bool kHalf = DRT != 0;
    constexpr int DR = kHalf ? DRT : D;                         // head width in memory
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *sT = smem + SM::tile_off;
    uint8_t *sQ = smem + SM::lat_off(0);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + SM::bar_off());
    constexpr int NG = kSoftmaxGroups;
    // per group: S_FULL and P_FULL for each of its two unit buffers
    enum { T_FULL = 0, T_EMPTY = T_FULL + nstages, S_FULL = T_EMPTY + nstages, P_FULL = S_FULL + 2 * NG,
           ACC_DONE = P_FULL + 2 * NG, Q_FULL = ACC_DONE + NG, NBARS };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + NBARS);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int M = a.M;
    const int split = blockIdx.x, h = blockIdx.y / a.pairs, pair = blockIdx.y % a.pairs, b = blockIdx.z;
    const int t_begin = (int)((long)a.tiles * split / a.splits);
    const int t_end = (int)((long)a.tiles * (split + 1) / a.splits);
    const int nt = t_end - t_begin;
    const int MB = (M + kTile - 1) / kTile;
    const bool alternate = kAlt || MB == 1;                           // one latent block: the two slots take alternate tiles
    const int lb0 = pair * 2;
    const int nslots = alternate ? 2 : ((lb0 + 1 < MB) ? 2 : 1);
    const int nq = alternate ? nt : nt * nslots;
    const int rows_here = min(M - lb0 * kTile, 2 * kTile);
    constexpr int SLOT_COLS = 256, HALF = kTile / 2, UNIT = 16, UPH = HALF / UNIT;   // units per half tile
    constexpr uint32_t NCOLS = 512;
    // per group (128 columns): two unit buffers of 48 columns (S, A, C: 16 each), partial dQ at 96
    auto bar = [&](int i) { return ptx::smem_u32(bars + i); };

    if (threadIdx.x == 0) {
        const uint32_t users = alternate ? 2u : 2u * (uint32_t)nslots;
        for (int i = 0; i < NBARS; ++i)
            ptx::mbar_init(bar(i), (i >= P_FULL && i < P_FULL + 2 * NG) ? 128u
                                   : (i >= T_EMPTY && i < T_EMPTY + nstages) ? users : 1u);
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmK);
        ptx::prefetch_tensormap(&tmV);
        ptx::prefetch_tensormap(&tmG);
        ptx::prefetch_tensormap(&tmQ);
    }
    if (warp == kFirstIssuerWarp) ptx::tmem_alloc(ptx::smem_u32(tmem_slot), NCOLS);
    // zero the latent rows beyond M (all five operands; in the half-width form all rows, whose upper halves stay
    // zero), then Z and dZ as bf16 hi/lo rows in the swizzled layout
    for (int i = threadIdx.x; i < 5 * 2 * kTile * (G::RB / 16); i += kTcThreads) {
        const int which = i / (2 * kTile * (G::RB / 16)), rem = i % (2 * kTile * (G::RB / 16));
        if (kHalf || rem / (G::RB / 16) >= rows_here) reinterpret_cast<uint4 *>(smem + SM::lat_off(which))[rem] = make_uint4(0, 0, 0, 0);
    }
    const int off = kHalf ? narrow_offset(h, DR) : 0;           // the head's first column within a token tile row
    if (kHalf) {
        __syncthreads();
        if constexpr (DR == 4) {
            const size_t r0 = ((size_t)b * a.H + h) * M + lb0 * kTile;
            stage_rows4<D>(sQ, a.Q + ((size_t)h * M + lb0 * kTile) * DR, rows_here, off);
            stage_rows4_hilo<D>(smem + SM::lat_off(1), smem + SM::lat_off(2), a.Z + r0 * DR, rows_here, off);
            stage_rows4_hilo<D>(smem + SM::lat_off(3), smem + SM::lat_off(4), a.dZ + r0 * DR, rows_here, off);
        } else {
            for (int i = threadIdx.x; i < rows_here * (DR / 8); i += kTcThreads) {
                const int m = i / (DR / 8), ch = i % (DR / 8);
                *reinterpret_cast<uint4 *>(sQ + (size_t)m * G::RB + ((ch ^ G::swz(m)) << 4)) =
                    *reinterpret_cast<const uint4 *>(a.Q + ((size_t)h * M + lb0 * kTile + m) * DR + ch * 8);
            }
        }
    }
    constexpr int ZC = DR >= 8 ? DR / 8 : 1;                    // 8-float chunks per row (none for DR = 4: staged above)
    for (int i = threadIdx.x; i < (DR >= 8 ? 2 * rows_here * ZC : 0); i += kTcThreads) {
        const int which = i / (rows_here * ZC), rem = i % (rows_here * ZC), m = rem / ZC, ch = rem % ZC;
        const float *src = (which == 0 ? a.Z : a.dZ) + (((size_t)b * a.H + h) * M + lb0 * kTile + m) * DR + ch * 8;
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
            if (kHalf) {
                ptx::mbar_arrive(bar(Q_FULL));                  // Q was written by the threads before the block barrier
            } else {
                ptx::mbar_arrive_expect_tx(bar(Q_FULL), (uint32_t)(rows_here * G::RB));
                for (int r = 0; r < rows_here; r += 16)
                    ptx::tma_load_2d(ptx::smem_u32(sQ + (size_t)r * G::RB), &tmQ, bar(Q_FULL), 0, h * M + lb0 * kTile + r);
            }
            for (int i = 0; i < nt; ++i) {
                const int s = i % nstages;
                if (!ptx::mbar_wait(bar(T_EMPTY + s), ((i / nstages) & 1) ^ 1, abort_flag, kErrBwdDq | 1)) break;
                ptx::mbar_arrive_expect_tx(bar(T_FULL + s), 3 * G::TILE_BYTES);
                uint8_t *dst = sT + (size_t)s * 3 * G::TILE_BYTES;
                ptx::tma_load_3d(ptx::smem_u32(dst), &tmK, bar(T_FULL + s), h * DR - off, (t_begin + i) * kTile, b);
                ptx::tma_load_3d(ptx::smem_u32(dst + G::TILE_BYTES), &tmV, bar(T_FULL + s), h * DR - off, (t_begin + i) * kTile, b);
                ptx::tma_load_3d(ptx::smem_u32(dst + 2 * G::TILE_BYTES), &tmG, bar(T_FULL + s), h * DR - off, (t_begin + i) * kTile, b);
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
            const uint32_t dcol = gcol + 96;
            bool ok = ptx::mbar_wait(bar(Q_FULL), 0, abort_flag, kErrBwdDq | 2);
            const int jobs = (nq - j + nslots - 1) / nslots;
            const int units = UPH * jobs;
            // Order of issue, as in the encode kernel: the three tiles of units 0 and 1, then for every unit n its dQ
            // MMAs as soon as its dS is handed over, then the tiles of unit n+2 into the buffer that dS has just left.
            int t_s = alternate ? j : 0, t_v = t_s;                         // tiles of the next tile-unit / dQ-unit
            const int t_step = alternate ? 2 : 1;
            auto issue_tiles = [&](int n) -> bool {
                const int s = t_s % nstages, w = n % UPH;
                if (w == 0 && !ptx::mbar_wait(bar(T_FULL + s), (t_s / nstages) & 1, abort_flag, kErrBwdDq | 3)) return false;
                ptx::tc_fence_after();
                const uint32_t tbase = ptx::smem_u32(sT + (size_t)s * 3 * G::TILE_BYTES);
                const uint64_t rowoff = (uint64_t)((c * HALF + w * UNIT) * G::RB / 16);   // the unit's 16 token rows
                const uint64_t kdesc = ptx::smem_desc(tbase, 16, G::SBO, G::SWZ) + rowoff;
                const uint64_t vdesc = ptx::smem_desc(tbase + G::TILE_BYTES, 16, G::SBO, G::SWZ) + rowoff;
                const uint64_t gdesc = ptx::smem_desc(tbase + 2 * G::TILE_BYTES, 16, G::SBO, G::SWZ) + rowoff;
                const uint32_t bcol = gcol + (n & 1) * 3 * UNIT;
                // S = Q K^T | A = (Z_hi + Z_lo) dY^T | C = (dZ_hi + dZ_lo) V^T, each 128 latents x 16 tokens
#pragma unroll
                for (int k = 0; k < D / 16; ++k) ptx::mma_ss(bcol, ldesc[0] + 2 * k, kdesc + 2 * k, idescS, k > 0);
#pragma unroll
                for (int k = 0; k < D / 16; ++k) ptx::mma_ss(bcol + UNIT, ldesc[1] + 2 * k, gdesc + 2 * k, idescS, k > 0);
#pragma unroll
                for (int k = 0; k < D / 16; ++k) ptx::mma_ss(bcol + UNIT, ldesc[2] + 2 * k, gdesc + 2 * k, idescS, 1u);
#pragma unroll
                for (int k = 0; k < D / 16; ++k) ptx::mma_ss(bcol + 2 * UNIT, ldesc[3] + 2 * k, vdesc + 2 * k, idescS, k > 0);
#pragma unroll
                for (int k = 0; k < D / 16; ++k) ptx::mma_ss(bcol + 2 * UNIT, ldesc[4] + 2 * k, vdesc + 2 * k, idescS, 1u);
                ptx::mma_commit(bar(S_FULL + 2 * g + (n & 1)));
                if (w == UPH - 1) t_s += t_step;
                return true;
            };
            for (int n = 0; ok && n < 2 && n < units; ++n) ok = issue_tiles(n);
            for (int n = 0; ok && n < units; ++n) {
                const int s = t_v % nstages, w = n % UPH;
                if (!ptx::mbar_wait(bar(P_FULL + 2 * g + (n & 1)), (n >> 1) & 1, abort_flag, kErrBwdDq | 4)) { ok = false; break; }
                ptx::tc_fence_after();
                // dQ_part += dS_unit K_unit (hi, then lo half of dS): the unit's 16 token rows of the K tile as the
                // MN-major B operand
                const uint64_t kmn = ptx::smem_desc(ptx::smem_u32(sT + (size_t)s * 3 * G::TILE_BYTES), G::SBO, G::SBO, G::SWZ) +
                                     (uint64_t)((c * HALF + w * UNIT) * G::RB / 16);
                const uint32_t bcol = gcol + (n & 1) * 3 * UNIT;
                ptx::mma_ts(dcol, bcol, kmn, idescQ, n > 0 ? 1u : 0u);
                ptx::mma_ts(dcol, bcol + UNIT, kmn, idescQ, 1u);
                if (w == UPH - 1) {
                    ptx::mma_commit(bar(T_EMPTY + s));
                    t_v += t_step;
                }
                if (n + 2 < units) ok = issue_tiles(n + 2);
            }
            if (ok) ptx::mma_commit(bar(ACC_DONE + g));
        }
    } else {
        const int g = (warp - kFirstSoftmaxWarp) >> 2;
        const int j = g >> 1, c = g & 1;
        const int row = ((warp & 3) << 5) + lane;
        const uint32_t lane_addr = (uint32_t)((warp & 3) << 5) << 16;
        const uint32_t gcol = tm + lane_addr + j * SLOT_COLS + c * 2 * HALF;
        const uint32_t abase = gcol + 96;
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
        // this warp's column constants for the 64 tokens of its half tile: -lse_dec (log2 units), then -dd
        float *cst = reinterpret_cast<float *>(smem + SM::col_off()) + (warp - kFirstSoftmaxWarp) * 128;
        int done = 0;
        bool ok = true;
        // One unit: 16 token columns on buffer (done & 1).  wv: validity bits of the 16 tokens (kMasked only).
        auto unit = [&](auto masked, int w, uint32_t wv) -> bool {
            constexpr bool kMasked = decltype(masked)::value;
            const int buf = done & 1;
            const uint32_t bcol = gcol + buf * 3 * UNIT;
            if (!warp_wait(bar(S_FULL + 2 * g + buf), (done >> 1) & 1, abort_flag, kErrBwdDq | 5)) return false;
            ptx::tc_fence_after();
            // 8 tokens at a time: their dS goes back as two bf16 halves over columns the thread has already read
            // (hi over S, lo over A: 4 packed columns per 8 tokens)
#pragma unroll
            for (int qd = 0; qd < 2; ++qd) {
                uint32_t s[8], av[8], cv[8], pk[4], pl[4];
                ptx::tmem_ld8(bcol + qd * 8, s);
                ptx::tmem_ld8(bcol + UNIT + qd * 8, av);
                ptx::tmem_ld8(bcol + 2 * UNIT + qd * 8, cv);
                ptx::tmem_wait_ld();
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int col = qd * 8 + 2 * k;
                    const float2 sp = make_float2(__uint_as_float(s[2 * k]), __uint_as_float(s[2 * k + 1]));
                    const float2 nld = *reinterpret_cast<const float2 *>(cst + w * UNIT + col);
                    const float2 ndd = *reinterpret_cast<const float2 *>(cst + HALF + w * UNIT + col);
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
                ptx::tmem_st4(bcol + qd * 4, pk);
                ptx::tmem_st4(bcol + UNIT + qd * 4, pl);
            }
            ptx::tmem_wait_st();
            ptx::tc_fence_before();
            ptx::mbar_arrive(bar(P_FULL + 2 * g + buf));
            ++done;
            return true;
        };
        if (j < nslots) {
            // the constants of a tile are fetched one tile ahead (two tokens per lane) and parked, as loaded, in
            // registers: nothing waits for the loads until the next tile begins
            float f_ld[2], f_dd[2];
            uint32_t f_ok[2];
            auto fetch = [&](int t) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int n = t * kTile + c * HALF + e * 32 + lane;
                    const bool in = n < a.N;
                    const size_t i = ((size_t)b * a.N + (in ? n : 0)) * a.H + h;
                    f_ld[e] = a.lse_dec[i];
                    f_dd[e] = a.dd[((size_t)b * a.H + h) * a.N + (in ? n : 0)];
                    f_ok[e] = a.key_mask == nullptr ? 1u : (uint32_t)a.key_mask[(size_t)b * a.N + (in ? n : 0)];
                }
            };
            if (j < nq) fetch(t_begin + (alternate ? j : j / nslots));
            for (int q = j; ok && q < nq; q += nslots) {
                const int t = t_begin + (alternate ? q : q / nslots);
                const bool plain = a.key_mask == nullptr && (t + 1) * kTile <= a.N;
                __syncwarp();                                               // the previous tile's reads are done
                bool v01[2];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const bool in = t * kTile + c * HALF + e * 32 + lane < a.N;
                    cst[e * 32 + lane] = in ? -f_ld[e] * 1.4426950408889634f : -INFINITY;
                    cst[HALF + e * 32 + lane] = in ? -f_dd[e] : 0.f;
                    v01[e] = in && f_ok[e] != 0;
                }
                const uint32_t wv0 = __ballot_sync(0xffffffffu, v01[0]), wv1 = __ballot_sync(0xffffffffu, v01[1]);
                __syncwarp();
                if (q + nslots < nq) fetch(t_begin + (alternate ? q + nslots : (q + nslots) / nslots));
#pragma unroll 1
                for (int w = 0; ok && w < UPH; ++w) {
                    const uint32_t wv = ((w < 2 ? wv0 : wv1) >> ((w & 1) * UNIT)) & 0xffffu;
                    if (kPadded && !plain) ok = unit(std::true_type{}, w, wv);
                    else ok = unit(std::false_type{}, w, wv);
                }
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
            float4 *dst = reinterpret_cast<float4 *>(a.part + ((size_t)part * rows + ((size_t)b * a.H + h) * M + m) * DR);
            if (DR == 4) {
                dst[0] = make_float4(__uint_as_float(off ? acc[4] : acc[0]), __uint_as_float(off ? acc[5] : acc[1]),
                                     __uint_as_float(off ? acc[6] : acc[2]), __uint_as_float(off ? acc[7] : acc[3]));
            } else {
#pragma unroll
                for (int dc = 0; dc < DR / 4; ++dc)
                    dst[dc] = make_float4(__uint_as_float(acc[4 * dc]), __uint_as_float(acc[4 * dc + 1]),
                                          __uint_as_float(acc[4 * dc + 2]), __uint_as_float(acc[4 * dc + 3]));
            }
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

// ------------------------------------------------------------------------------- pass B, token side (dK, dV)
// Tokens on the 128 TMEM lanes, latents on columns in units of kUnit, every softmax group a token tile of its
// own.  Two sweeps over the latents of a tile, as in the CUDA-core kernel: the first needs S^T = K Q^T and
// A^T = dY Z^T and leaves dd[n] = sum_m W_dec[n,m] A[n,m] in a register; the second adds C^T = V dZ^T, turns the
// three into dS^T and W_enc^T (two bf16 halves each) over the columns just read, and two more contractions
// accumulate dK_n = scale * sum_m dS[m,n] q_m and dV_n = sum_m W_enc[m,n] dZ_m.  dd goes to the workspace for
// the dQ kernel.  Columns of a group: S, A, C (kUnit each), dK (D), dV (D): 3 kUnit + 2 D <= 128.
template <int D>
struct BwdTokGeom {
    static constexpr int kUnit = D == 16 ? 32 : 16;
    static constexpr int kMaxStages = 8;
};

struct BwdTokTcArgs {
    const __nv_bfloat16 *Q;    // [H,M,D] (read directly in the half-width form)
    const float *Z, *dZ;       // [B,H,M,D]
    const float *lse_enc, *de; // [B,H,M]
    const float *lse_dec;      // [B,N,H]
    const uint8_t *key_mask;   // [B,N] or null
    __nv_bfloat16 *dK, *dV;    // [B,N,H,D]
    float *dd;                 // [B,H,N] (workspace): written in modes 0 and 1, read in mode 2
    uint32_t *status;
    int B, H, N, M;            // M: latents this launch works on (all of them, or a range)
    int mtot, m0;              // latents per head in memory, and the first one of this launch's range
    // More latents than one launch can keep in shared memory are worked off in ranges, by two series of launches:
    // mode 1 (first sweep only) adds the range's share of dd[n] to the workspace; mode 2 (second sweep only, dd
    // complete) adds the range's share of the rows of dK and dV to float32 sums in kvacc [2][B*N*H][D] and, in the
    // last range, writes the rows.  Mode 0 does both sweeps over all latents in one launch.
    int first, last;           // (the mode is a template parameter of the kernel)
    float *kvacc;
    float scale, sl2;
    int tiles, stages;
};

template <int D>
struct BwdTokSmem {
    using G = TileGeom<D>;
    __host__ __device__ static int padded_m(int M) { return (M + 31) & ~31; }
    // tiles: [stage][K | V | dY]; latents: Q, Z_hi, Z_lo, dZ_hi, dZ_lo with padded_m rows each; then -lse_enc, -de
    __host__ __device__ static size_t lat_off(int stages, int M, int which) {
        return (size_t)stages * 3 * G::TILE_BYTES + (size_t)which * padded_m(M) * G::RB;
    }
    __host__ __device__ static size_t cst_off(int stages, int M) { return lat_off(stages, M, 5); }
    __host__ __device__ static size_t bar_off(int stages, int M) { return cst_off(stages, M) + 2 * sizeof(float) * padded_m(M); }
    __host__ __device__ static size_t total(int stages, int M) {
        size_t t = bar_off(stages, M) + 512 + 1024;
        return t < kTcMinSmem ? kTcMinSmem : t;
    }
    // the most stages (at most kMaxStages) that fit beside the latent operands; 0 if not even one does
    __host__ static int stages(int M) {
        int s = BwdTokGeom<D>::kMaxStages;
        while (s > 0 && total(s, M) > (size_t)227 * 1024) --s;
        return s;
    }
};

// grid = (CTAs per head, H, B); a CTA takes the token tiles blockIdx.x, blockIdx.x + gridDim.x, ...
// DRT = 8 or 4 (with D = 16): the narrow form (head DRT wide in memory; only the head's columns of the rows of dK
// and dV are kept).
// kM: 0, or the number of latents of the launch as a compile-time constant.
// kPadded: as in the dQ kernel.
template <int D, int DRT = 0, int kMode = 0, int kM = 0, bool kPadded = true>
__global__ void __launch_bounds__(kTcThreads, 1)
bwd_token_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                    const __grid_constant__ CUtensorMap tmG, const __grid_constant__ CUtensorMap tmQ, BwdTokTcArgs a) {
    using G = TileGeom<D>;
    using SM = BwdTokSmem<D>;
    constexpr int UNIT = BwdTokGeom<D>::kUnit;
    constexpr int kMaxSt = BwdTokGeom<D>::kMaxStages;
    constexpr bool kHalf = DRT != 0;
    constexpr int DR = kHalf ? DRT : D;                         // head width in memory
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int M = kM ? kM : a.M, MU = SM::padded_m(M), stages = a.stages;
    uint8_t *sQ = smem + SM::lat_off(stages, M, 0);
    float *cst = reinterpret_cast<float *>(smem + SM::cst_off(stages, M));      // [MU] -lse_enc (log2 units), [MU] -de
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + SM::bar_off(stages, M));
    constexpr int NG = kSoftmaxGroups;
    enum { T_FULL = 0, T_EMPTY = T_FULL + kMaxSt, S_FULL = T_EMPTY + kMaxSt, P_FULL = S_FULL + NG,
           ACC_FULL = P_FULL + NG, ACC_FREE = ACC_FULL + NG, Q_FULL = ACC_FREE + NG, NBARS };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + NBARS);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = blockIdx.y, b = blockIdx.z;
    const int nt = (a.tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;   // tiles of this CTA
    const int ng = stages < NG ? stages : NG;                   // groups at work
    const int nu = (M + UNIT - 1) / UNIT;                       // latent units per sweep
    constexpr uint32_t NCOLS = 512;
    auto bar = [&](int i) { return ptx::smem_u32(bars + i); };

    if (threadIdx.x == 0) {
        for (int i = 0; i < NBARS; ++i)
            ptx::mbar_init(bar(i), ((i >= P_FULL && i < P_FULL + NG) || (i >= ACC_FREE && i < ACC_FREE + NG)) ? 128u : 1u);
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmK);
        ptx::prefetch_tensormap(&tmV);
        ptx::prefetch_tensormap(&tmG);
        ptx::prefetch_tensormap(&tmQ);
    }
    if (warp == kFirstIssuerWarp) ptx::tmem_alloc(ptx::smem_u32(tmem_slot), NCOLS);
    // latent rows M..MU-1 of all five operands are zero; their columns carry -lse_enc = -inf
    const int zfirst = kHalf ? 0 : M;                           // half-width form: every row, whose upper half stays zero
    for (int i = threadIdx.x; i < 5 * (MU - zfirst) * (G::RB / 16); i += kTcThreads) {
        const int which = i / ((MU - zfirst) * (G::RB / 16)), rem = i % ((MU - zfirst) * (G::RB / 16));
        reinterpret_cast<uint4 *>(smem + SM::lat_off(stages, M, which) + (size_t)zfirst * G::RB)[rem] = make_uint4(0, 0, 0, 0);
    }
    const int off = kHalf ? narrow_offset(h, DR) : 0;           // the head's first column within a token tile row
    if (kHalf) {
        __syncthreads();
        if constexpr (DR == 4) {
            const size_t r0 = ((size_t)b * a.H + h) * a.mtot + a.m0;
            stage_rows4<D>(sQ, a.Q + ((size_t)h * a.mtot + a.m0) * DR, M, off);
            stage_rows4_hilo<D>(smem + SM::lat_off(stages, M, 1), smem + SM::lat_off(stages, M, 2), a.Z + r0 * DR, M, off);
            stage_rows4_hilo<D>(smem + SM::lat_off(stages, M, 3), smem + SM::lat_off(stages, M, 4), a.dZ + r0 * DR, M, off);
        } else {
            for (int i = threadIdx.x; i < M * (DR / 8); i += kTcThreads) {
                const int m = i / (DR / 8), ch = i % (DR / 8);
                *reinterpret_cast<uint4 *>(sQ + (size_t)m * G::RB + ((ch ^ G::swz(m)) << 4)) =
                    *reinterpret_cast<const uint4 *>(a.Q + ((size_t)h * a.mtot + a.m0 + m) * DR + ch * 8);
            }
        }
    }
    for (int m = threadIdx.x; m < MU; m += kTcThreads) {
        float nle = -INFINITY, nde = 0.f;
        if (m < M) {
            const size_t r = ((size_t)b * a.H + h) * a.mtot + a.m0 + m;
            const float le = a.lse_enc[r];
            nle = (le == -INFINITY) ? -INFINITY : -le * 1.4426950408889634f;
            nde = -a.de[r];
        }
        cst[m] = nle;
        cst[MU + m] = nde;
    }
    constexpr int ZC = DR >= 8 ? DR / 8 : 1;                    // 8-float chunks per row (none for DR = 4: staged above)
    for (int i = threadIdx.x; i < (DR >= 8 ? 2 * M * ZC : 0); i += kTcThreads) {
        const int which = i / (M * ZC), rem = i % (M * ZC), m = rem / ZC, ch = rem % ZC;
        const float *src = (which == 0 ? a.Z : a.dZ) + (((size_t)b * a.H + h) * a.mtot + a.m0 + m) * DR + ch * 8;
        const float4 lo4 = *reinterpret_cast<const float4 *>(src), hi4 = *reinterpret_cast<const float4 *>(src + 4);
        const float z[8] = {lo4.x, lo4.y, lo4.z, lo4.w, hi4.x, hi4.y, hi4.z, hi4.w};
        uint32_t vh[4], vl[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            vh[k] = ptx::pack_bf16(z[2 * k], z[2 * k + 1]);
            vl[k] = ptx::pack_bf16(z[2 * k] - __uint_as_float(vh[k] << 16), z[2 * k + 1] - __uint_as_float(vh[k] & 0xffff0000u));
        }
        const size_t off = (size_t)m * G::RB + ((ch ^ G::swz(m)) << 4);
        *reinterpret_cast<uint4 *>(smem + SM::lat_off(stages, M, 1 + 2 * which) + off) = make_uint4(vh[0], vh[1], vh[2], vh[3]);
        *reinterpret_cast<uint4 *>(smem + SM::lat_off(stages, M, 2 + 2 * which) + off) = make_uint4(vl[0], vl[1], vl[2], vl[3]);
    }
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tm = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            if (kHalf) {
                ptx::mbar_arrive(bar(Q_FULL));                  // Q was written by the threads before the block barrier
            } else {
                ptx::mbar_arrive_expect_tx(bar(Q_FULL), (uint32_t)(M * G::RB));
                for (int r = 0; r < M; r += 16)
                    ptx::tma_load_2d(ptx::smem_u32(sQ + (size_t)r * G::RB), &tmQ, bar(Q_FULL), 0, h * a.mtot + a.m0 + r);
            }
            for (int i = 0; i < nt; ++i) {
                const int s = i % stages, t = blockIdx.x + i * gridDim.x;
                if (!ptx::mbar_wait(bar(T_EMPTY + s), ((i / stages) & 1) ^ 1, abort_flag, kErrBwdTok | 1)) break;
                ptx::mbar_arrive_expect_tx(bar(T_FULL + s), 3 * G::TILE_BYTES);
                uint8_t *dst = smem + (size_t)s * 3 * G::TILE_BYTES;
                ptx::tma_load_3d(ptx::smem_u32(dst), &tmK, bar(T_FULL + s), h * DR - off, t * kTile, b);
                ptx::tma_load_3d(ptx::smem_u32(dst + G::TILE_BYTES), &tmV, bar(T_FULL + s), h * DR - off, t * kTile, b);
                ptx::tma_load_3d(ptx::smem_u32(dst + 2 * G::TILE_BYTES), &tmG, bar(T_FULL + s), h * DR - off, t * kTile, b);
            }
        }
    } else if (warp < kFirstSoftmaxWarp) {
        const int g = warp - kFirstIssuerWarp;
        if (lane == 0 && g < ng) {
            const uint32_t idescS = ptx::instr_desc_bf16(128, UNIT, 0, 0);
            const uint32_t idescO = ptx::instr_desc_bf16(128, D, 0, 1);
            const uint32_t gcol = tm + g * 128;
            const uint32_t kcol = gcol + 3 * UNIT, vcol = kcol + D;       // the dK and dV accumulators
            bool ok = ptx::mbar_wait(bar(Q_FULL), 0, abort_flag, kErrBwdTok | 2);
            uint32_t cnt = 0;
            int k_tile = 0;
            for (int i = g; ok && i < nt; i += ng, ++k_tile) {
                const int s = i % stages;
                if (!ptx::mbar_wait(bar(T_FULL + s), (i / stages) & 1, abort_flag, kErrBwdTok | 3)) break;
                ptx::tc_fence_after();
                const uint32_t tbase = ptx::smem_u32(smem + (size_t)s * 3 * G::TILE_BYTES);
                // the tile's token rows as the K-major A operand of the three score-like contractions
                const uint64_t kdesc = ptx::smem_desc(tbase, 16, G::SBO, G::SWZ);
                const uint64_t vdesc = ptx::smem_desc(tbase + G::TILE_BYTES, 16, G::SBO, G::SWZ);
                const uint64_t gdesc = ptx::smem_desc(tbase + 2 * G::TILE_BYTES, 16, G::SBO, G::SWZ);
                for (int sweep = (kMode == 2 ? 1 : 0); ok && sweep < (kMode == 1 ? 1 : 2); ++sweep) {
                    for (int u = 0; u < nu; ++u) {
                        const uint64_t uoff = (uint64_t)(u * UNIT * G::RB / 16);      // the unit's latent rows
                        uint64_t ld[5];
#pragma unroll
                        for (int w = 0; w < 5; ++w)
                            ld[w] = ptx::smem_desc(ptx::smem_u32(smem + SM::lat_off(stages, M, w)), 16, G::SBO, G::SWZ) + uoff;
#pragma unroll
                        for (int k = 0; k < D / 16; ++k) ptx::mma_ss(gcol, kdesc + 2 * k, ld[0] + 2 * k, idescS, k > 0);
#pragma unroll
                        for (int k = 0; k < D / 16; ++k) ptx::mma_ss(gcol + UNIT, gdesc + 2 * k, ld[1] + 2 * k, idescS, k > 0);
#pragma unroll
                        for (int k = 0; k < D / 16; ++k) ptx::mma_ss(gcol + UNIT, gdesc + 2 * k, ld[2] + 2 * k, idescS, 1u);
                        if (sweep == 1) {
#pragma unroll
                            for (int k = 0; k < D / 16; ++k) ptx::mma_ss(gcol + 2 * UNIT, vdesc + 2 * k, ld[3] + 2 * k, idescS, k > 0);
#pragma unroll
                            for (int k = 0; k < D / 16; ++k) ptx::mma_ss(gcol + 2 * UNIT, vdesc + 2 * k, ld[4] + 2 * k, idescS, 1u);
                        }
                        ptx::mma_commit(bar(S_FULL + g));
                        if (!ptx::mbar_wait(bar(P_FULL + g), cnt & 1, abort_flag, kErrBwdTok | 4)) { ok = false; break; }
                        ++cnt;
                        ptx::tc_fence_after();
                        if (sweep == 1) {
                            // the previous tile's accumulators must have been read before they are overwritten
                            if (u == 0 && k_tile > 0 &&
                                !ptx::mbar_wait(bar(ACC_FREE + g), (k_tile - 1) & 1, abort_flag, kErrBwdTok | 5)) { ok = false; break; }
                            ptx::tc_fence_after();
                            // Q and dZ (hi, lo) rows of the unit as MN-major B operands, 16 latent rows per k-step
                            const uint64_t qmn = ptx::smem_desc(ptx::smem_u32(smem + SM::lat_off(stages, M, 0)), G::SBO, G::SBO, G::SWZ) + uoff;
                            const uint64_t zmn = ptx::smem_desc(ptx::smem_u32(smem + SM::lat_off(stages, M, 3)), G::SBO, G::SBO, G::SWZ) + uoff;
                            const uint64_t zln = ptx::smem_desc(ptx::smem_u32(smem + SM::lat_off(stages, M, 4)), G::SBO, G::SBO, G::SWZ) + uoff;
#pragma unroll
                            for (int k = 0; k < UNIT / 16; ++k) {
                                const uint32_t acc = (u > 0 || k > 0) ? 1u : 0u;
                                ptx::mma_ts(kcol, gcol + k * 8, qmn + (uint64_t)(k * G::RB), idescO, acc);              // dS hi
                                ptx::mma_ts(kcol, gcol + UNIT + k * 8, qmn + (uint64_t)(k * G::RB), idescO, 1u);        // dS lo
                                ptx::mma_ts(vcol, gcol + 2 * UNIT + k * 16, zmn + (uint64_t)(k * G::RB), idescO, acc);       // W_enc dZ_hi
                                ptx::mma_ts(vcol, gcol + 2 * UNIT + k * 16, zln + (uint64_t)(k * G::RB), idescO, 1u);        // W_enc dZ_lo
                                ptx::mma_ts(vcol, gcol + 2 * UNIT + k * 16 + 8, zmn + (uint64_t)(k * G::RB), idescO, 1u);    // W_enc lo x dZ_hi
                            }
                        }
                    }
                }
                if (!ok) break;
                ptx::mma_commit(bar(T_EMPTY + s));
                if (kMode != 1) ptx::mma_commit(bar(ACC_FULL + g));
            }
        }
    } else {
        const int g = (warp - kFirstSoftmaxWarp) >> 2;
        const int row = ((warp & 3) << 5) + lane;               // TMEM lane = token within the tile
        const uint32_t lane_addr = (uint32_t)((warp & 3) << 5) << 16;
        const uint32_t gcol = tm + lane_addr + g * 128;
        const uint32_t kcol = gcol + 3 * UNIT, vcol = kcol + D;
        const float2 sl2p = make_float2(a.sl2, a.sl2);
        uint32_t cnt = 0;
        int k_tile = 0;
        bool ok = true;
        // The rows of a tile are written one sweep late: while the issuing warp finishes the tile's last MMAs the
        // group already works on the first sweep of its next tile, whose MMAs do not touch the accumulators.
        bool pend = false, p_inside = false;
        size_t p_tok = 0, p_ddi = 0;
        float p_dd = 0.f;
        int p_k = 0;
        auto write_rows = [&]() -> bool {
            if (!warp_wait(bar(ACC_FULL + g), p_k & 1, abort_flag, kErrBwdTok | 8)) return false;
            ptx::tc_fence_after();
            uint32_t ak[D], avv[D];
#pragma unroll
            for (int dc = 0; dc < D / 16; ++dc) {
                ptx::tmem_ld16(kcol + dc * 16, ak + dc * 16);
                ptx::tmem_ld16(vcol + dc * 16, avv + dc * 16);
            }
            ptx::tmem_wait_ld();
            ptx::tc_fence_before();
            ptx::mbar_arrive(bar(ACC_FREE + g));
            if (p_inside) {
                if (kMode == 0) a.dd[p_ddi] = p_dd;
                float fk[DR], fv[DR];
#pragma unroll
                for (int i = 0; i < DR; ++i) {                  // the head's columns of the accumulators
                    fk[i] = __uint_as_float((DR == 4 && off) ? ak[(4 + i) % D] : ak[i]);
                    fv[i] = __uint_as_float((DR == 4 && off) ? avv[(4 + i) % D] : avv[i]);
                }
                float4 *sk = reinterpret_cast<float4 *>(a.kvacc + p_tok * DR);
                float4 *sv = reinterpret_cast<float4 *>(a.kvacc + ((size_t)a.B * a.N * a.H + p_tok) * DR);
                if (kMode == 2 && !a.first) {                  // the earlier ranges' shares
#pragma unroll
                    for (int i = 0; i < DR / 4; ++i) {
                        const float4 pk4 = sk[i], pv4 = sv[i];
                        fk[4 * i] += pk4.x; fk[4 * i + 1] += pk4.y; fk[4 * i + 2] += pk4.z; fk[4 * i + 3] += pk4.w;
                        fv[4 * i] += pv4.x; fv[4 * i + 1] += pv4.y; fv[4 * i + 2] += pv4.z; fv[4 * i + 3] += pv4.w;
                    }
                }
                if (kMode == 2 && !a.last) {
#pragma unroll
                    for (int i = 0; i < DR / 4; ++i) {
                        sk[i] = make_float4(fk[4 * i], fk[4 * i + 1], fk[4 * i + 2], fk[4 * i + 3]);
                        sv[i] = make_float4(fv[4 * i], fv[4 * i + 1], fv[4 * i + 2], fv[4 * i + 3]);
                    }
                } else {
                    uint32_t *dk = reinterpret_cast<uint32_t *>(a.dK + p_tok * DR), *dv = reinterpret_cast<uint32_t *>(a.dV + p_tok * DR);
                    uint32_t wk[DR / 2], wv[DR / 2];
#pragma unroll
                    for (int i = 0; i < DR / 2; ++i) {
                        wk[i] = ptx::pack_bf16(fk[2 * i] * a.scale, fk[2 * i + 1] * a.scale);
                        wv[i] = ptx::pack_bf16(fv[2 * i], fv[2 * i + 1]);
                    }
                    if (DR == 4) {
                        *reinterpret_cast<uint2 *>(dk) = make_uint2(wk[0], wk[1]);
                        *reinterpret_cast<uint2 *>(dv) = make_uint2(wv[0], wv[1]);
                    } else {
#pragma unroll
                        for (int q = 0; q < DR / 8; ++q) {
                            reinterpret_cast<uint4 *>(dk)[q] = make_uint4(wk[4 * q], wk[4 * q + 1], wk[4 * q + 2], wk[4 * q + 3]);
                            reinterpret_cast<uint4 *>(dv)[q] = make_uint4(wv[4 * q], wv[4 * q + 1], wv[4 * q + 2], wv[4 * q + 3]);
                        }
                    }
                }
            }
            pend = false;
            return true;
        };
        // this lane's token of a tile: its decode log-sum-exp and mask byte, fetched one tile ahead
        float f_ld = 0.f, f_dd = 0.f;
        uint32_t f_mask = 1u;
        auto fetch = [&](int i) {
            const int n = (blockIdx.x + i * gridDim.x) * kTile + row;
            const size_t nn = (size_t)b * a.N + (n < a.N ? n : 0);
            f_ld = a.lse_dec[nn * a.H + h];
            f_mask = a.key_mask == nullptr ? 1u : (uint32_t)a.key_mask[nn];
            if (kMode == 2) f_dd = a.dd[((size_t)b * a.H + h) * a.N + (n < a.N ? n : 0)];
        };
        if (g < ng && g < nt) fetch(g);
        for (int i = g; ok && g < ng && i < nt; i += ng, ++k_tile) {
            const int t = blockIdx.x + i * gridDim.x, n = t * kTile + row;
            const bool inside = n < a.N;
            const bool valid = inside && f_mask != 0;
            const size_t tok = ((size_t)b * a.N + (inside ? n : 0)) * a.H + h;
            const float negld = inside ? -f_ld * 1.4426950408889634f : -INFINITY;
            const float2 negldp = make_float2(negld, negld);
            const float dd_given = inside ? f_dd : 0.f;         // mode 2: dd[n] over all latents, from the workspace
            if (i + ng < nt) fetch(i + ng);
            const bool plain = a.key_mask == nullptr && (t + 1) * kTile <= a.N;      // uniform over the group
            // sweep 1: dd[n] = sum_m W_dec[n,m] (dY_n . Z_m)
            float2 dd2 = make_float2(0.f, 0.f);
            for (int u = 0; ok && kMode != 2 && u < nu; ++u) {
                if (!warp_wait(bar(S_FULL + g), cnt & 1, abort_flag, kErrBwdTok | 6)) { ok = false; break; }
                ++cnt;
                ptx::tc_fence_after();
#pragma unroll
                for (int hb = 0; hb < UNIT / 16; ++hb) {
                    uint32_t s[16], av[16];
                    ptx::tmem_ld16(gcol + hb * 16, s);
                    ptx::tmem_ld16(gcol + UNIT + hb * 16, av);
                    ptx::tmem_wait_ld();
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const float2 x = __ffma2_rn(make_float2(__uint_as_float(s[2 * k]), __uint_as_float(s[2 * k + 1])), sl2p, negldp);
                        dd2 = __ffma2_rn(make_float2(ptx::ex2(x.x), ptx::ex2(x.y)),
                                         make_float2(__uint_as_float(av[2 * k]), __uint_as_float(av[2 * k + 1])), dd2);
                    }
                }
                ptx::tc_fence_before();
                ptx::mbar_arrive(bar(P_FULL + g));
            }
            const float dd = kMode == 2 ? dd_given : dd2.x + dd2.y;
            const float2 negddp = make_float2(-dd, -dd);
            if (kMode == 1) {                                  // this range's share of dd[n]; no second sweep
                if (inside) {
                    const size_t ddi = ((size_t)b * a.H + h) * a.N + n;
                    a.dd[ddi] = (a.first ? 0.f : a.dd[ddi]) + dd;
                }
                continue;
            }
            if (ok && pend) ok = write_rows();                  // the previous tile's rows
            // sweep 2: dS^T and W_enc^T of every unit, handed to the issuing warp
            auto unit2 = [&](auto masked, int u) {
                constexpr bool kMasked = decltype(masked)::value;
                uint32_t pwl[4];                                    // lo halves of W_enc of an even quarter, kept for one quarter
#pragma unroll
                for (int qd = 0; qd < UNIT / 8; ++qd) {
                    uint32_t s[8], av[8], cv[8], pk[4], pl[4], pw[4], pwo[4];
                    ptx::tmem_ld8(gcol + qd * 8, s);
                    ptx::tmem_ld8(gcol + UNIT + qd * 8, av);
                    ptx::tmem_ld8(gcol + 2 * UNIT + qd * 8, cv);
                    ptx::tmem_wait_ld();
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int col = u * UNIT + qd * 8 + 2 * k;                  // latent of this pair of columns
                        const float2 sp = make_float2(__uint_as_float(s[2 * k]), __uint_as_float(s[2 * k + 1]));
                        const float2 nle = *reinterpret_cast<const float2 *>(cst + col);
                        const float2 nde = *reinterpret_cast<const float2 *>(cst + MU + col);
                        const float2 xd = __ffma2_rn(sp, sl2p, negldp), xe = __ffma2_rn(sp, sl2p, nle);
                        const float2 pd = make_float2(ptx::ex2(xd.x), ptx::ex2(xd.y));
                        float2 pe = make_float2(ptx::ex2(xe.x), ptx::ex2(xe.y));
                        if (kMasked && !valid) pe = make_float2(0.f, 0.f);
                        const float2 uu = __fadd2_rn(make_float2(__uint_as_float(av[2 * k]), __uint_as_float(av[2 * k + 1])), negddp);
                        const float2 vv = __fadd2_rn(make_float2(__uint_as_float(cv[2 * k]), __uint_as_float(cv[2 * k + 1])), nde);
                        const float2 ds = __ffma2_rn(pd, uu, __fmul2_rn(pe, vv));
                        const uint32_t hi = ptx::pack_bf16(ds.x, ds.y);
                        pk[k] = hi;
                        pl[k] = ptx::pack_bf16(ds.x - __uint_as_float(hi << 16), ds.y - __uint_as_float(hi & 0xffff0000u));
                        const uint32_t wh = ptx::pack_bf16(pe.x, pe.y);
                        pw[k] = wh;
                        pwo[k] = ptx::pack_bf16(pe.x - __uint_as_float(wh << 16), pe.y - __uint_as_float(wh & 0xffff0000u));
                    }
                    // Packed results over columns this thread has already read: dS hi over S, dS lo over A.  W_enc over
                    // C, per 16 latents (two quarters): hi in the first 8 of their 16 columns, lo in the other 8 - which
                    // the odd quarter has only just read, so the even quarter's lo waits in four registers.
                    ptx::tmem_st4(gcol + qd * 4, pk);
                    ptx::tmem_st4(gcol + UNIT + qd * 4, pl);
                    ptx::tmem_st4(gcol + 2 * UNIT + (qd >> 1) * 16 + (qd & 1) * 4, pw);
                    if (qd & 1) {
                        ptx::tmem_st4(gcol + 2 * UNIT + (qd >> 1) * 16 + 8, pwl);
                        ptx::tmem_st4(gcol + 2 * UNIT + (qd >> 1) * 16 + 12, pwo);
                    } else {
#pragma unroll
                        for (int k = 0; k < 4; ++k) pwl[k] = pwo[k];
                    }
                }
            };
            for (int u = 0; ok && u < nu; ++u) {
                if (!warp_wait(bar(S_FULL + g), cnt & 1, abort_flag, kErrBwdTok | 7)) { ok = false; break; }
                ++cnt;
                ptx::tc_fence_after();
                if (kPadded && !plain) unit2(std::true_type{}, u); else unit2(std::false_type{}, u);
                ptx::tmem_wait_st();
                ptx::tc_fence_before();
                ptx::mbar_arrive(bar(P_FULL + g));
            }
            if (!ok) break;
            pend = true; p_inside = inside; p_tok = tok; p_dd = dd; p_k = k_tile;
            p_ddi = ((size_t)b * a.H + h) * a.N + (inside ? n : 0);
        }
        if (ok && pend) ok = write_rows();
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
