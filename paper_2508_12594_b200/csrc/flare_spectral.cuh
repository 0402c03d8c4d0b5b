// Linear-time spectral analysis of the induced mixing matrix (paper: spectral-analysis appendix, Algorithm 1).
//
// With A = exp(S), S = scale * Q K^T, L_M = diag(1 / row sums of A) and L_N = diag(1 / column sums of A), the mixing
// matrix W = W_dec W_enc = L_N A^T L_M A has the non-zero eigenvalues of the M x M matrix G = J J^T,
// J = L_M^{1/2} A L_N^{1/2}.  With the log-sum-exp rows the forward already produces,
//     J[m,n] = exp(S[m,n] - lse_enc[m] / 2 - lse_dec[n] / 2),        G[m,m'] = sum_n J[m,n] J[m',n],
// so G is one more reduction over the tokens in which every (latent, token) pair costs one exponential (as in
// encode) and every pair of latents one multiply-add per token: 2 N M^2 FLOP per head, O(M^2) memory.  Nothing
// of size M x N or N x N is written.  The M x M symmetric eigenproblem (O(M^3), off the hot path) is solved by a
// small Jacobi kernel.
//
//   spectral_gram_tc_kernel    bfloat16, M <= 128, D in {16, 32}: tcgen05.  A CTA takes one head and a range of
//                              tokens; the head's latents sit on the 128 TMEM lanes.  Per 32 tokens: S = Q K^T; 128
//                              threads form J as two bf16 halves (hi + lo), back over the scores (the A operand of the
//                              next MMAs) and into shared memory (their B operand); G += J J^T with the accumulator in
//                              TMEM, as hi hi^T + hi lo^T + lo hi^T (the diagonal of G is a sum of squares: with single
//                              bf16 factors nothing cancels and G is off by 4e-3 of its largest entries).
//   spectral_gram_simt_kernel  everything else (float32 inputs, other shapes): CUDA cores, a 16 x 16 tile of G per block.
//   spectral_gram_reduce_kernel sums the token splits and writes the symmetric G.
//   spectral_jacobi_kernel     eigenvalues (and eigenvectors) of G by cyclic two-sided Jacobi rotations.
#pragma once

#include "flare_common.cuh"
#include "flare_ptx.cuh"
#include "flare_tc.cuh"

namespace flare {

struct SpectralArgs {
    const __nv_bfloat16 *Q;   // [H,M,D]
    const float *lse_enc;     // [B,H,M]
    const float *lse_dec;     // [B,N,H]
    float *part;              // [splits * kSpectralGroups][B*H][128][128] float32 partial sums of G
    uint32_t *status;
    int B, H, N, M;
    float sl2;                // scale * log2(e)
    int tiles, splits;
};

// Groups of 128 threads at work in a CTA of the tensor-core Gram kernel: each takes every third token tile with its own
// score buffer, accumulator (160 of the 512 tensor-memory columns) and partial sum.
constexpr int kSpectralGroups = 3;

template <int D>
struct SpectralSmem {
    using G = TileGeom<D>;
    static constexpr int kStages = 6;
    static constexpr size_t k_off = 0;                                      // K tiles
    static constexpr size_t q_off = (size_t)kStages * G::TILE_BYTES;        // Q rows
    static constexpr size_t pb_off = q_off + (size_t)kTile * G::RB;         // J (hi, lo) as B operands: [128 latents, 32 tokens] bf16 each
    static constexpr size_t kPbBytes = (size_t)kTile * 64;
    static constexpr size_t col_off = pb_off + kSpectralGroups * 2 * kPbBytes;   // (a hi and a lo tile per group); per softmax warp 32 column addends
    static constexpr size_t bar_off = (col_off + kSpectralGroups * 4 * 32 * sizeof(float) + 1023) & ~(size_t)1023;
    static constexpr size_t total = bar_off + 512 + 1024 < kTcMinSmem ? kTcMinSmem : bar_off + 512 + 1024;
};

// grid = (splits, H, B).  Warp 0: TMA; warps 1-3: MMA issue, one per group; warps 5-16: three groups of 128 threads, the
// latent rows on their lanes.  Group g works on the tiles g, g + 3, ... of the CTA's range and leaves its own partial sum.
template <int D>
__global__ void __launch_bounds__(kTcThreads, 1)
spectral_gram_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ, SpectralArgs a) {
    using G = TileGeom<D>;
    using GP = TileGeom<32>;                                    // the J tiles in shared memory: 32 tokens = 64 bytes per latent row
    using SM = SpectralSmem<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *sK = smem + SM::k_off, *sQ = smem + SM::q_off, *sPB = smem + SM::pb_off;
    float *colneg = reinterpret_cast<float *>(smem + SM::col_off);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + SM::bar_off);
    constexpr int kStages = SM::kStages, UNIT = 32;
    constexpr int NGS = kSpectralGroups;
    enum { K_FULL = 0, K_EMPTY = K_FULL + kStages, Q_FULL = K_EMPTY + kStages, S_FULL, P_FULL = S_FULL + NGS,
           G_DONE = P_FULL + NGS, NBARS = G_DONE + NGS };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + NBARS);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    // tensor memory, per group 160 columns: G [0,128)  S [128,160)
    constexpr uint32_t G_AA = 0, S_A = 128, GROUP_COLS = 160, NCOLS = 512;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int M = a.M;
    const int t_begin = (int)((long)a.tiles * split / a.splits), t_end = (int)((long)a.tiles * (split + 1) / a.splits);
    const int nt = t_end - t_begin;
    auto bar = [&](int i) { return ptx::smem_u32(bars + i); };

    if (threadIdx.x == 0) {
        for (int i = 0; i < NBARS; ++i) ptx::mbar_init(bar(i), (i >= P_FULL && i < P_FULL + NGS) ? 4u : 1u);   // P_FULL: one arrival per warp
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmK);
        ptx::prefetch_tensormap(&tmQ);
    }
    if (warp == kFirstIssuerWarp) ptx::tmem_alloc(ptx::smem_u32(tmem_slot), NCOLS);
    for (int i = threadIdx.x; i < kTile * (G::RB / 16); i += kTcThreads)          // latent rows beyond M stay zero
        reinterpret_cast<uint4 *>(sQ)[i] = make_uint4(0, 0, 0, 0);
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tm = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            ptx::mbar_arrive_expect_tx(bar(Q_FULL), (uint32_t)(M * G::RB));
            for (int r = 0; r < M; r += 16) ptx::tma_load_2d(ptx::smem_u32(sQ + (size_t)r * G::RB), &tmQ, bar(Q_FULL), 0, h * M + r);
            for (int i = 0; i < nt; ++i) {
                const int s = i % kStages;
                if (!ptx::mbar_wait(bar(K_EMPTY + s), ((i / kStages) & 1) ^ 1, abort_flag, kErrSpectral | 1)) break;
                ptx::mbar_arrive_expect_tx(bar(K_FULL + s), G::TILE_BYTES);
                ptx::tma_load_3d(ptx::smem_u32(sK + (size_t)s * G::TILE_BYTES), &tmK, bar(K_FULL + s), h * D, (t_begin + i) * kTile, b);
            }
        }
    } else if (warp >= kFirstIssuerWarp && warp < kFirstIssuerWarp + NGS) {
        const int g = warp - kFirstIssuerWarp;
        const int mytiles = (nt - g + NGS - 1) / NGS;
        const uint32_t gtm = tm + g * GROUP_COLS;
        if (lane == 0) {
            const uint32_t idescS = ptx::instr_desc_bf16(128, UNIT, 0, 0), idescG = ptx::instr_desc_bf16(128, 128, 0, 0);
            const uint64_t qdesc = ptx::smem_desc(ptx::smem_u32(sQ), 16, G::SBO, G::SWZ);
            const uint64_t pbdesc = ptx::smem_desc(ptx::smem_u32(sPB + (size_t)g * 2 * SM::kPbBytes), 16, GP::SBO, GP::SWZ);
            bool ok = ptx::mbar_wait(bar(Q_FULL), 0, abort_flag, kErrSpectral | 2);
            const int units = 4 * mytiles;
            auto issue_scores = [&](int u) -> bool {              // unit u: the group's tile u / 4, tokens 32 (u % 4) ... of it
                const int i = g + NGS * (u >> 2), s = i % kStages;
                if ((u & 3) == 0 && !ptx::mbar_wait(bar(K_FULL + s), (i / kStages) & 1, abort_flag, kErrSpectral | 3)) return false;
                ptx::tc_fence_after();
                const uint64_t kdesc = ptx::smem_desc(ptx::smem_u32(sK + (size_t)s * G::TILE_BYTES), 16, G::SBO, G::SWZ) +
                                       (uint64_t)(((u & 3) * UNIT * G::RB) >> 4);
#pragma unroll
                for (int k = 0; k < D / 16; ++k) ptx::mma_ss(gtm + S_A, qdesc + 2 * k, kdesc + 2 * k, idescS, k > 0);
                ptx::mma_commit(bar(S_FULL + g));
                if ((u & 3) == 3) ptx::mma_commit(bar(K_EMPTY + s));
                return true;
            };
            if (ok && units > 0) ok = issue_scores(0);
            for (int u = 0; ok && u < units; ++u) {
                if (!ptx::mbar_wait(bar(P_FULL + g), u & 1, abort_flag, kErrSpectral | 4)) break;
                ptx::tc_fence_after();
                // G += J J^T over the unit's 32 tokens (two k-steps of 16): A = J in tensor memory (hi in the first 16 columns
                // of the score buffer, lo in the other 16), B = J in shared memory (hi tile, then lo tile)
                constexpr uint64_t LO = (uint64_t)(SM::kPbBytes >> 4);
#pragma unroll
                for (int k = 0; k < 2; ++k) {
#pragma unroll
                    for (int t = 0; t < 3; ++t) {               // hi hi^T, hi lo^T, lo hi^T
                        const uint32_t acol = (t == 2 ? 16u : 0u) + 8 * k;
                        const uint64_t bsel = (t == 1 ? LO : 0) + 2 * k;
                        const uint32_t acc = (u > 0 || k > 0 || t > 0) ? 1u : 0u;
                        ptx::mma_ts(gtm + G_AA, gtm + S_A + acol, pbdesc + bsel, idescG, acc);
                    }
                }
                // the next unit's scores overwrite J in tensor memory after those MMAs (a thread's MMAs run in order); the
                // commit behind them also tells the threads that J in shared memory has been read
                if (u + 1 < units) ok = issue_scores(u + 1);
                else ptx::mma_commit(bar(G_DONE + g));
            }
        }
    } else if (warp >= kFirstSoftmaxWarp && warp < kFirstSoftmaxWarp + 4 * NGS) {
        const int g = (warp - kFirstSoftmaxWarp) >> 2;
        const int mytiles = (nt - g + NGS - 1) / NGS;
        const int row = ((warp & 3) << 5) + lane;               // TMEM lane = latent
        const int m = row;
        const uint32_t lane_addr = (uint32_t)((warp & 3) << 5) << 16;
        const uint32_t scol = tm + lane_addr + g * GROUP_COLS + S_A;
        float *cn = colneg + (warp - kFirstSoftmaxWarp) * 32;
        const float rowneg = m < M ? -0.5f * 1.4426950408889634f * a.lse_enc[((size_t)b * a.H + h) * M + m] : -INFINITY;
        const float2 sl2p = make_float2(a.sl2, a.sl2);
        uint8_t *pb = sPB + (size_t)g * 2 * SM::kPbBytes + (size_t)row * GP::RB;   // this latent's row of the group's hi tile; lo: kPbBytes on
        bool ok = true;
        const int units = 4 * mytiles;
        for (int u = 0; ok && u < units; ++u) {
            const int n = (t_begin + g + NGS * (u >> 2)) * kTile + (u & 3) * UNIT + lane;   // this lane fetches the shift of token n
            __syncwarp();
            cn[lane] = n < a.N ? -0.5f * 1.4426950408889634f * a.lse_dec[((size_t)b * a.N + n) * a.H + h] : -INFINITY;
            __syncwarp();
            if (!(ok = warp_wait(bar(S_FULL + g), u & 1, abort_flag, kErrSpectral | 5))) break;
            ptx::tc_fence_after();
            uint32_t r[32], hi[16], lo[16];
            ptx::tmem_ld32(scol, r);
            ptx::tmem_wait_ld();
#pragma unroll
            for (int k = 0; k < 8; ++k) {                       // J = 2^(s sl2 + rowneg + colneg[n]); -inf rows and columns give 0
                const float4 ng = *reinterpret_cast<const float4 *>(cn + 4 * k);
                const float2 x0 = __ffma2_rn(make_float2(__uint_as_float(r[4 * k]), __uint_as_float(r[4 * k + 1])), sl2p,
                                             make_float2(ng.x + rowneg, ng.y + rowneg));
                const float2 x1 = __ffma2_rn(make_float2(__uint_as_float(r[4 * k + 2]), __uint_as_float(r[4 * k + 3])), sl2p,
                                             make_float2(ng.z + rowneg, ng.w + rowneg));
                const float p0 = ptx::ex2(x0.x), p1 = ptx::ex2(x0.y), p2 = ptx::ex2(x1.x), p3 = ptx::ex2(x1.y);
                const uint32_t h0 = ptx::pack_bf16(p0, p1), h1 = ptx::pack_bf16(p2, p3);
                hi[2 * k] = h0;
                hi[2 * k + 1] = h1;
                lo[2 * k] = ptx::pack_bf16(p0 - __uint_as_float(h0 << 16), p1 - __uint_as_float(h0 & 0xffff0000u));
                lo[2 * k + 1] = ptx::pack_bf16(p2 - __uint_as_float(h1 << 16), p3 - __uint_as_float(h1 & 0xffff0000u));
            }
            ptx::tmem_st16(scol, hi);                           // A operand: back over the scores, hi then lo
            ptx::tmem_st16(scol + 16, lo);
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {                    // B operand: this latent's 64-byte rows, 16-byte chunks swizzled
                *reinterpret_cast<uint4 *>(pb + ((ch ^ GP::swz(row)) << 4)) = make_uint4(hi[4 * ch], hi[4 * ch + 1], hi[4 * ch + 2], hi[4 * ch + 3]);
                *reinterpret_cast<uint4 *>(pb + SM::kPbBytes + ((ch ^ GP::swz(row)) << 4)) =
                    make_uint4(lo[4 * ch], lo[4 * ch + 1], lo[4 * ch + 2], lo[4 * ch + 3]);
            }
            ptx::fence_proxy_async_smem();
            ptx::tmem_wait_st();
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar(P_FULL + g));
        }
        // the partial sum of G: this thread's lane holds row m
        if (ok && units > 0) ok = warp_wait(bar(G_DONE + g), 0, abort_flag, kErrSpectral | 6);
        ptx::tc_fence_after();
        if (ok) {
            float *dst = a.part + ((((size_t)split * NGS + g) * a.B + b) * a.H + h) * (size_t)kTile * kTile + (size_t)row * kTile;
#pragma unroll 1
            for (int c0 = 0; c0 < kTile; c0 += 32) {
                uint32_t v[32];
                if (units > 0) {
                    ptx::tmem_ld32(tm + lane_addr + g * GROUP_COLS + G_AA + c0, v);
                    ptx::tmem_wait_ld();
                } else {
#pragma unroll
                    for (int k = 0; k < 32; ++k) v[k] = 0u;
                }
#pragma unroll
                for (int k = 0; k < 32; k += 4)
                    *reinterpret_cast<float4 *>(dst + c0 + k) = make_float4(__uint_as_float(v[k]), __uint_as_float(v[k + 1]),
                                                                            __uint_as_float(v[k + 2]), __uint_as_float(v[k + 3]));
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

// Sum of the token splits into G [B,H,M,M].  One thread per element.
__global__ void __launch_bounds__(256)
spectral_gram_reduce_kernel(const float *__restrict__ part, float *__restrict__ Gout, int splits, long heads, int M) {
    const long idx = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= heads * M * M) return;
    const long bh = idx / ((long)M * M);
    const int i = (int)((idx / M) % M), j = (int)(idx % M);
    float s = 0.f;
    for (int p = 0; p < splits; ++p) s += part[((size_t)p * heads + bh) * (size_t)kTile * kTile + (size_t)i * kTile + j];
    Gout[idx] = s;
}

// G on the CUDA cores, for everything the tensor-core kernel does not take: one block per 16 x 16 tile of G of
// one (b, h); the tokens are walked in chunks of 64 whose J rows for the tile's 16 + 16 latents sit in shared memory.
template <typename T, int D>
__global__ void __launch_bounds__(256)
spectral_gram_simt_kernel(const T *__restrict__ Q, const T *__restrict__ K, const float *__restrict__ lse_enc,
                          const float *__restrict__ lse_dec, float *__restrict__ Gout, int B, int H, int N, int M, float scale) {
    constexpr int TN = 64;
    __shared__ float sQ[32][D];
    __shared__ float sK[TN][D];
    __shared__ float sJ[32][TN + 1];
    __shared__ float sLe[32];
    const int tiles_m = (M + 15) / 16;
    const int ti = blockIdx.x / tiles_m, tj = blockIdx.x % tiles_m, h = blockIdx.y, b = blockIdx.z;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    for (int i = threadIdx.x; i < 32 * D; i += 256) {
        const int rr = i / D, d = i % D, m = (rr < 16 ? ti * 16 + rr : tj * 16 + rr - 16);
        sQ[rr][d] = m < M ? to_f32(Q[((size_t)h * M + m) * D + d]) * scale : 0.f;
        if (d == 0) sLe[rr] = m < M ? lse_enc[((size_t)b * H + h) * M + m] : INFINITY;
    }
    float acc = 0.f;
    for (int n0 = 0; n0 < N; n0 += TN) {
        __syncthreads();
        for (int i = threadIdx.x; i < TN * D; i += 256) {
            const int jn = i / D, d = i % D, n = n0 + jn;
            sK[jn][d] = n < N ? to_f32(K[(((size_t)b * N + n) * H + h) * D + d]) : 0.f;
        }
        __syncthreads();
        for (int i = threadIdx.x; i < 32 * TN; i += 256) {
            const int rr = i / TN, jn = i % TN, n = n0 + jn;
            float q[D];
#pragma unroll
            for (int d = 0; d < D; ++d) q[d] = sQ[rr][d];
            const float s = score_dot<T, D>(q, sK[jn]);
            sJ[rr][jn] = n < N ? expf(s - 0.5f * sLe[rr] - 0.5f * lse_dec[((size_t)b * N + n) * H + h]) : 0.f;
        }
        __syncthreads();
#pragma unroll 8
        for (int jn = 0; jn < TN; ++jn) acc = fmaf(sJ[ty][jn], sJ[16 + tx][jn], acc);
    }
    const int mi = ti * 16 + ty, mj = tj * 16 + tx;
    if (mi < M && mj < M) Gout[(((size_t)b * H + h) * M + mi) * M + mj] = acc;
}

// Eigenvalues (descending) and, if U != null, eigenvectors (columns of U) of the symmetric matrices G [heads, M, M],
// by cyclic two-sided Jacobi rotations on disjoint index pairs (round-robin ordering: M - 1 steps of M / 2 rotations
// per sweep).  One block per matrix; G is overwritten.  Off the hot path: O(M^3) per sweep, about ten sweeps.
__global__ void __launch_bounds__(1024)
spectral_jacobi_kernel(float *__restrict__ Gall, float *__restrict__ evals, float *__restrict__ Uall, int M, int sweeps) {
    extern __shared__ float sh[];
    float *cs = sh;                         // [M/2 pairs] cosines, then sines
    int *pp = reinterpret_cast<int *>(sh + 2 * ((M + 1) / 2));   // [pairs] p, then q; then [M] ranks
    float *G = Gall + (size_t)blockIdx.x * M * M;
    float *U = Uall ? Uall + (size_t)blockIdx.x * M * M : nullptr;
    const int Me = (M + 1) & ~1, pairs = Me / 2, t = threadIdx.x, T = blockDim.x;
    if (U)
        for (int i = t; i < M * M; i += T) U[i] = (i / M == i % M) ? 1.f : 0.f;
    __syncthreads();
    // A sweep that met no off-diagonal element above 2^-22 of the largest diagonal one (float32 rotations change nothing
    // below that) was the last: six to eight sweeps in practice instead of the twelve allowed.
    __shared__ unsigned off_max, diag_max;                      // bit patterns of non-negative floats order like the floats
    for (int sweep = 0; sweep < sweeps; ++sweep) {
        if (t == 0) { off_max = 0u; diag_max = 0u; }
        __syncthreads();
        for (int i = t; i < M; i += T) atomicMax(&diag_max, __float_as_uint(fabsf(G[(size_t)i * M + i])));
        for (int step = 0; step < Me - 1; ++step) {
            // round-robin pairing of 0 .. Me-1 (index Me-1 fixed); an index >= M is a bye
            for (int k = t; k < pairs; k += T) {
                int p = k == 0 ? Me - 1 : (step + k) % (Me - 1);
                int q = (step + Me - 1 - k) % (Me - 1);
                if (p > q) { const int tmp = p; p = q; q = tmp; }
                float c = 1.f, s = 0.f;
                if (q < M) {
                    const float gpq = G[(size_t)p * M + q];
                    atomicMax(&off_max, __float_as_uint(fabsf(gpq)));
                    if (fabsf(gpq) > 1e-30f) {
                        const float tau = (G[(size_t)q * M + q] - G[(size_t)p * M + p]) / (2.f * gpq);
                        const float tt = (tau >= 0.f ? 1.f : -1.f) / (fabsf(tau) + sqrtf(1.f + tau * tau));
                        c = rsqrtf(1.f + tt * tt);
                        s = tt * c;
                    }
                }
                cs[k] = c; cs[pairs + k] = s; pp[k] = p; pp[pairs + k] = q;
            }
            __syncthreads();
            // columns: G <- G R (and U <- U R), every row independently.  Neighbouring threads take the pairs of one row:
            // a step's pairs cover every column once, so the row's sectors are all used while they are in the cache
            // (pair-major order touched one element per sector and was 3 times slower at M = 512).
            for (int i = t; i < pairs * M; i += T) {
                const int row = i / pairs, k = i % pairs, p = pp[k], q = pp[pairs + k];
                if (q >= M) continue;
                const float c = cs[k], s = cs[pairs + k];
                const float gp = G[(size_t)row * M + p], gq = G[(size_t)row * M + q];
                G[(size_t)row * M + p] = c * gp - s * gq;
                G[(size_t)row * M + q] = s * gp + c * gq;
                if (U) {
                    const float up = U[(size_t)row * M + p], uq = U[(size_t)row * M + q];
                    U[(size_t)row * M + p] = c * up - s * uq;
                    U[(size_t)row * M + q] = s * up + c * uq;
                }
            }
            __syncthreads();
            // rows: G <- R^T G, every column independently
            for (int i = t; i < pairs * M; i += T) {
                const int k = i / M, col = i % M, p = pp[k], q = pp[pairs + k];
                if (q >= M) continue;
                const float c = cs[k], s = cs[pairs + k];
                const float gp = G[(size_t)p * M + col], gq = G[(size_t)q * M + col];
                G[(size_t)p * M + col] = c * gp - s * gq;
                G[(size_t)q * M + col] = s * gp + c * gq;
            }
            __syncthreads();
        }
        if (__uint_as_float(off_max) <= 2.4e-7f * __uint_as_float(diag_max)) break;   // (uniform: shared values, read after a barrier)
    }
    // eigenvalues = diagonal, sorted descending (rank by counting; ties by index); the columns of U move alike,
    // through G's storage (its content is no longer needed)
    int *rank = pp + 2 * pairs;
    float *ev = evals + (size_t)blockIdx.x * M;
    for (int i = t; i < M; i += T) {
        const float v = G[(size_t)i * M + i];
        int r = 0;
        for (int j = 0; j < M; ++j) {
            const float w = G[(size_t)j * M + j];
            r += (w > v) || (w == v && j < i);
        }
        rank[i] = r;
        ev[r] = v;
    }
    __syncthreads();
    if (U) {
        for (int i = t; i < M * M; i += T) G[(size_t)(i / M) * M + rank[i % M]] = U[i];
        __syncthreads();
        for (int i = t; i < M * M; i += T) U[i] = G[i];
    }
}

}  // namespace flare
