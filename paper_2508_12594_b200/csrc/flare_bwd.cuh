// Backward of the FLARE mixer on the CUDA cores (float32 arithmetic, any supported dtype and shape), and the
// small reduction kernels every backward uses.  bfloat16 inputs take the tensor-core kernels instead (the dZ
// form of the encode kernel for pass A; the dQ and token kernels of the tensor-core backward for pass B when
// D <= 32); the formulas are the same.
//
// The paper times a backward pass without writing it out; these kernels apply the chain rule to its encode and
// decode equations (Section 3.2).  With S[m,n] = scale * q_m . k_n,
//   W_dec[n,m] = exp(S[m,n] - lse_dec[n]),   W_enc[m,n] = valid(n) ? exp(S[m,n] - lse_enc[m]) : 0,
// both softmax matrices are recomputed from the saved log-sum-exp rows, one score at a time:
//   pass A   dZ[m]  = sum_n W_dec[n,m] dY_n                      (reduction over tokens; split over N)
//   pass B   dd[n]  = dY_n . Y_n = sum_m W_dec[n,m] (dY_n . Z_m),   de[m] = dZ_m . Z_m
//            dS[m,n] = W_dec[n,m] (dY_n . Z_m - dd[n]) + W_enc[m,n] (dZ_m . V_n - de[m])
//            dV_n   = sum_m W_enc[m,n] dZ_m        dK_n = scale * sum_m dS[m,n] q_m       (one thread per token)
//            dQ_m   = scale * sum_b sum_n dS[m,n] k_n                                     (split over N, then summed)
// dd[n] is formed from the float32 dot products dY_n . Z_m rather than from the stored Y: Y has been rounded to
// the output type, and where the rows Z_m that a token mixes are nearly equal that rounding would dominate dS.
// Reductions add their partial results in a fixed order, so the gradients are bitwise reproducible.
#pragma once

#include "flare_common.cuh"
#include "flare_simt.cuh"

namespace flare {

constexpr int kBwdThreads = 256;
constexpr int kBwdTileN = 32;   // tokens staged in shared memory per step of the latent-parallel kernels
constexpr int kBwdLatents = 32; // latents staged in shared memory per step of the token-parallel kernel

// Pass A.  grid = (splits, H, B); block = LM latents x G token groups (as in the encode kernel).  Partial
// number split*G + g of latent row (b,h,m) goes to part[(split*G + g) * rows + row][D].
template <typename T, int D>
__global__ void __launch_bounds__(kBwdThreads)
bwd_dz_simt_kernel(const T *__restrict__ Q, const T *__restrict__ K, const T *__restrict__ dY,
                   const float *__restrict__ lse_dec, float *__restrict__ part, int B, int H, int N, int M, int LM,
                   int chunk, float scale) {
    __shared__ float sK[kBwdTileN][D];
    __shared__ float sG[kBwdTileN][D];
    __shared__ float sL[kBwdTileN];
    const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int G = kBwdThreads / LM;
    const int lm = threadIdx.x % LM, g = threadIdx.x / LM;
    const int n0 = split * chunk, n1 = min(N, n0 + chunk);
    const long rows = (long)B * H * M;
    for (int mbase = 0; mbase < M; mbase += LM) {
        const int m = mbase + lm;
        const bool live = m < M;
        float q[D], acc[D];
#pragma unroll
        for (int d = 0; d < D; ++d) {
            q[d] = live ? to_f32(Q[((size_t)h * M + m) * D + d]) * scale : 0.f;
            acc[d] = 0.f;
        }
        for (int t0 = n0; t0 < n1; t0 += kBwdTileN) {
            __syncthreads();
            for (int i = threadIdx.x; i < kBwdTileN * D; i += kBwdThreads) {
                const int j = i / D, d = i % D, n = t0 + j;
                const bool in = n < n1;
                const size_t off = (((size_t)b * N + (in ? n : 0)) * H + h) * D + d;
                sK[j][d] = in ? to_f32(K[off]) : 0.f;
                sG[j][d] = in ? to_f32(dY[off]) : 0.f;
                if (d == 0) sL[j] = in ? lse_dec[((size_t)b * N + n) * H + h] : INFINITY;  // weight 0 past the end
            }
            __syncthreads();
            if (live) {
                for (int j = g; j < kBwdTileN; j += G) {
                    const float w = expf(score_dot<T, D>(q, sK[j]) - sL[j]);
#pragma unroll
                    for (int d = 0; d < D; ++d) acc[d] = fmaf(w, sG[j][d], acc[d]);
                }
            }
        }
        if (live) {
            const size_t row = ((size_t)b * H + h) * M + m;
            float *dst = part + ((size_t)(split * G + g) * rows + row) * D;
#pragma unroll
            for (int d = 0; d < D; ++d) dst[d] = acc[d];
        }
    }
}

// dZ[row][d] = sum_p part[p][row][d], partials added in index order.  One thread per (row, d).
__global__ void __launch_bounds__(256)
bwd_dz_reduce_kernel(const float *__restrict__ part, float *__restrict__ dZ, int P, long rows, int D) {
    const long idx = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= rows * D) return;
    float s = 0.f;
    for (int p = 0; p < P; ++p) s += part[(size_t)p * rows * D + idx];
    dZ[idx] = s;
}

// de[row] = dZ_row . Z_row.  One thread per row.
__global__ void __launch_bounds__(256)
bwd_de_kernel(const float *__restrict__ dZ, const float *__restrict__ Z, float *__restrict__ de, long rows, int D) {
    const long row = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= rows) return;
    float dot = 0.f;
    for (int d = 0; d < D; ++d) dot = fmaf(dZ[row * D + d], Z[row * D + d], dot);
    de[row] = dot;
}

// Pass B, token side: dK and dV.  One thread per token of head h; grid = (ceil(N/128), H, B).
template <typename T, int D>
__global__ void __launch_bounds__(128)
bwd_token_simt_kernel(const T *__restrict__ Q, const T *__restrict__ K, const T *__restrict__ V,
                      const uint8_t *__restrict__ key_mask, const T *__restrict__ dY, const float *__restrict__ Z,
                      const float *__restrict__ dZ, const float *__restrict__ de, const float *__restrict__ lse_enc,
                      const float *__restrict__ lse_dec, T *__restrict__ dK, T *__restrict__ dV,
                      float *__restrict__ dd_out, int B, int H, int N, int M, float scale) {
    __shared__ float sQ[kBwdLatents][D];
    __shared__ float sZ[kBwdLatents][D];
    __shared__ float sDZ[kBwdLatents][D];
    __shared__ float sLe[kBwdLatents], sDe[kBwdLatents];
    const int h = blockIdx.y, b = blockIdx.z;
    const int n = blockIdx.x * 128 + threadIdx.x;
    const bool live = n < N;
    const size_t tok = (((size_t)b * N + (live ? n : 0)) * H + h) * D;
    float k[D], v[D], dy[D], dk[D], dv[D];
#pragma unroll
    for (int d = 0; d < D; ++d) {
        k[d] = live ? to_f32(K[tok + d]) : 0.f;
        v[d] = live ? to_f32(V[tok + d]) : 0.f;
        dy[d] = live ? to_f32(dY[tok + d]) : 0.f;
        dk[d] = 0.f;
        dv[d] = 0.f;
    }
    const bool valid = live && (key_mask == nullptr || key_mask[(size_t)b * N + n] != 0);
    const float ld = live ? lse_dec[((size_t)b * N + n) * H + h] : 0.f;
    // first sweep over the latents: dd = sum_m W_dec[n,m] (dY_n . Z_m)
    float dd = 0.f;
    for (int m0 = 0; m0 < M; m0 += kBwdLatents) {
        const int mc = min(kBwdLatents, M - m0);
        __syncthreads();
        for (int i = threadIdx.x; i < mc * D; i += 128) {
            const int j = i / D, d = i % D;
            sQ[j][d] = to_f32(Q[((size_t)h * M + m0 + j) * D + d]);
            sZ[j][d] = Z[(((size_t)b * H + h) * M + m0 + j) * D + d];
        }
        __syncthreads();
        for (int j = 0; j < mc; ++j) {
            const float wdec = expf(scale * score_dot<T, D>(k, sQ[j]) - ld);
            float a = 0.f;
#pragma unroll
            for (int d = 0; d < D; ++d) a = fmaf(dy[d], sZ[j][d], a);
            dd = fmaf(wdec, a, dd);
        }
    }
    if (live) dd_out[((size_t)b * H + h) * N + n] = dd;
    for (int m0 = 0; m0 < M; m0 += kBwdLatents) {
        const int mc = min(kBwdLatents, M - m0);
        __syncthreads();
        for (int i = threadIdx.x; i < mc * D; i += 128) {
            const int j = i / D, d = i % D;
            const size_t row = ((size_t)b * H + h) * M + m0 + j;
            sQ[j][d] = to_f32(Q[((size_t)h * M + m0 + j) * D + d]);
            sZ[j][d] = Z[row * D + d];
            sDZ[j][d] = dZ[row * D + d];
            if (d == 0) {
                sLe[j] = lse_enc[row];
                sDe[j] = de[row];
            }
        }
        __syncthreads();
        for (int j = 0; j < mc; ++j) {
            const float s = scale * score_dot<T, D>(k, sQ[j]);
            const float wdec = expf(s - ld);
            const float wenc = (valid && sLe[j] != -INFINITY) ? expf(s - sLe[j]) : 0.f;
            float a = 0.f, c = 0.f;
#pragma unroll
            for (int d = 0; d < D; ++d) {
                a = fmaf(dy[d], sZ[j][d], a);
                c = fmaf(sDZ[j][d], v[d], c);
            }
            const float ds = (wdec * (a - dd) + wenc * (c - sDe[j])) * scale;
#pragma unroll
            for (int d = 0; d < D; ++d) {
                dv[d] = fmaf(wenc, sDZ[j][d], dv[d]);
                dk[d] = fmaf(ds, sQ[j][d], dk[d]);
            }
        }
    }
    if (live) {
#pragma unroll
        for (int d = 0; d < D; ++d) {
            from_f32(dK[tok + d], dk[d]);
            from_f32(dV[tok + d], dv[d]);
        }
    }
}

// Pass B, latent side: partial dQ rows.  Same grid and thread map as pass A; q, z and dz of the block's latents
// sit in shared memory (rows padded by one float so that lanes reading different rows hit different banks).
template <typename T, int D>
__global__ void __launch_bounds__(kBwdThreads)
bwd_dq_simt_kernel(const T *__restrict__ Q, const T *__restrict__ K, const T *__restrict__ V,
                   const uint8_t *__restrict__ key_mask, const T *__restrict__ dY, const float *__restrict__ Z,
                   const float *__restrict__ dZ, const float *__restrict__ de, const float *__restrict__ dd,
                   const float *__restrict__ lse_enc, const float *__restrict__ lse_dec, float *__restrict__ part,
                   int B, int H, int N, int M, int LM, int chunk, float scale) {
    extern __shared__ float dyn[];
    float(*sQ)[D + 1] = reinterpret_cast<float(*)[D + 1]>(dyn);
    float(*sZ)[D + 1] = sQ + LM;
    float(*sDZ)[D + 1] = sZ + LM;
    __shared__ float sK[kBwdTileN][D];
    __shared__ float sV[kBwdTileN][D];
    __shared__ float sG[kBwdTileN][D];
    __shared__ float sLd[kBwdTileN], sDd[kBwdTileN];
    __shared__ uint8_t sValid[kBwdTileN];
    const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int G = kBwdThreads / LM;
    const int lm = threadIdx.x % LM, g = threadIdx.x / LM;
    const int n0 = split * chunk, n1 = min(N, n0 + chunk);
    const long rows = (long)B * H * M;
    for (int mbase = 0; mbase < M; mbase += LM) {
        const int m = mbase + lm;
        const bool live = m < M;
        const size_t row = ((size_t)b * H + h) * M + (live ? m : 0);
        __syncthreads();
        for (int i = threadIdx.x; i < LM * D; i += kBwdThreads) {
            const int j = i / D, d = i % D;
            const bool in = mbase + j < M;
            const size_t r = ((size_t)b * H + h) * M + (in ? mbase + j : 0);
            sQ[j][d] = in ? to_f32(Q[((size_t)h * M + mbase + j) * D + d]) : 0.f;
            sZ[j][d] = in ? Z[r * D + d] : 0.f;
            sDZ[j][d] = in ? dZ[r * D + d] : 0.f;
        }
        const float le = live ? lse_enc[row] : -INFINITY;
        const float dem = live ? de[row] : 0.f;
        float acc[D];
#pragma unroll
        for (int d = 0; d < D; ++d) acc[d] = 0.f;
        for (int t0 = n0; t0 < n1; t0 += kBwdTileN) {
            __syncthreads();
            for (int i = threadIdx.x; i < kBwdTileN * D; i += kBwdThreads) {
                const int j = i / D, d = i % D, n = t0 + j;
                const bool in = n < n1;
                const size_t off = (((size_t)b * N + (in ? n : 0)) * H + h) * D + d;
                sK[j][d] = in ? to_f32(K[off]) : 0.f;
                sV[j][d] = in ? to_f32(V[off]) : 0.f;
                sG[j][d] = in ? to_f32(dY[off]) : 0.f;
            }
            if (threadIdx.x < kBwdTileN) {
                const int j = threadIdx.x, n = t0 + j;
                const bool in = n < n1;
                sDd[j] = in ? dd[((size_t)b * H + h) * N + n] : 0.f;
                sLd[j] = in ? lse_dec[((size_t)b * N + n) * H + h] : INFINITY;
                sValid[j] = in && (key_mask == nullptr || key_mask[(size_t)b * N + n] != 0);
            }
            __syncthreads();
            if (live) {
                for (int j = g; j < kBwdTileN; j += G) {
                    float s0 = 0.f, a = 0.f, c = 0.f;
                    if constexpr (!std::is_same<T, __nv_bfloat16>::value) {   // float32 and float16 inputs
                        double sd = 0.0;
#pragma unroll
                        for (int d = 0; d < D; ++d) sd = fma((double)sQ[lm][d], (double)sK[j][d], sd);
                        s0 = (float)sd;
                    } else {
#pragma unroll
                        for (int d = 0; d < D; ++d) s0 = fmaf(sQ[lm][d], sK[j][d], s0);
                    }
#pragma unroll
                    for (int d = 0; d < D; ++d) {
                        a = fmaf(sG[j][d], sZ[lm][d], a);
                        c = fmaf(sDZ[lm][d], sV[j][d], c);
                    }
                    const float s = s0 * scale;
                    const float wdec = expf(s - sLd[j]);
                    const float wenc = (sValid[j] && le != -INFINITY) ? expf(s - le) : 0.f;
                    const float ds = wdec * (a - sDd[j]) + wenc * (c - dem);
#pragma unroll
                    for (int d = 0; d < D; ++d) acc[d] = fmaf(ds, sK[j][d], acc[d]);
                }
            }
        }
        if (live) {
            float *dst = part + ((size_t)(split * G + g) * rows + row) * D;
#pragma unroll
            for (int d = 0; d < D; ++d) dst[d] = acc[d];
        }
    }
}

// dQ[h][m][d] = scale * sum_b sum_p part[p][(b,h,m)][d].  One block per (h, m): thread (slice, d) adds the terms
// q = b * P + p with q = slice, slice + S, ... (S = 128 / D) in index order, thread (0, d) the S slice sums in index
// order: a fixed order, and the B * P loads of a row are spread over the block.
constexpr int kDqReduceThreads = 128;
__global__ void __launch_bounds__(kDqReduceThreads)
bwd_dq_reduce_kernel(const float *__restrict__ part, float *__restrict__ dQ, int P, int B, int H, int M, int D,
                     float scale) {
    __shared__ float s_a[kDqReduceThreads];
    const long hm = blockIdx.x;                                  // h * M + m
    const int t = threadIdx.x, S = kDqReduceThreads / D, d = t % D, slice = t / D;
    const long per_batch = (long)H * M, rows = (long)B * per_batch;
    float s = 0.f;
    for (int q = slice; q < B * P; q += S) {
        const int b = q / P, p = q % P;
        s += part[((size_t)p * rows + (size_t)b * per_batch + hm) * D + d];
    }
    s_a[t] = s;
    __syncthreads();
    if (slice == 0) {
        for (int k = 1; k < S; ++k) s += s_a[k * D + d];
        dQ[hm * D + d] = s * scale;
    }
}

}  // namespace flare
