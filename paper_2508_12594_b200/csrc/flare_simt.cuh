// FP32 (CUDA-core) kernels of the FLARE mixer: the float32 data path.
//
// float32 inputs must meet a 1e-5 relative tolerance, which the tensor cores' reduced-mantissa float32 mode
// cannot; these kernels use plain FMA, expf and float32 accumulation.  They follow the per-latent and per-token
// sums of the paper's design-principles appendix directly, with the usual running-maximum (online) softmax.
#pragma once

#include <type_traits>

#include "flare_common.cuh"

namespace flare {

// Score q.k of one (latent, token) pair.  For float32 and float16 inputs the products are summed in double so that
// the score, which is exponentiated, carries no float32 summation error; bfloat16 inputs sum in float.
template <typename T, int D>
__device__ __forceinline__ float score_dot(const float (&a)[D], const float *b) {
    if constexpr (!std::is_same<T, __nv_bfloat16>::value) {   // float32 and float16 inputs
        double s = 0.0;
#pragma unroll
        for (int d = 0; d < D; ++d) s = fma((double)a[d], (double)b[d], s);
        return (float)s;
    } else {
        float s = 0.f;
#pragma unroll
        for (int d = 0; d < D; ++d) s = fmaf(a[d], b[d], s);
        return s;
    }
}

constexpr int kSimtThreads = 256;
constexpr int kSimtTileN = 32;  // tokens staged in shared memory per step

// Encode, split over N.  grid = (splits, H, B).  The block's 256 threads are LM latents x G token groups
// (G = 256 / LM); thread (lm, g) folds the tokens j of its split with j % G == g into a running
// (max, sum, row) triple for latent lm and writes it as partial number split*G + g.
template <typename T, int D>
__global__ void __launch_bounds__(kSimtThreads)
encode_simt_kernel(const T *__restrict__ Q, const T *__restrict__ K, const T *__restrict__ V,
                   const uint8_t *__restrict__ key_mask, float *__restrict__ part_m, float *__restrict__ part_l,
                   float *__restrict__ part_acc, int B, int H, int N, int M, int LM, int chunk, float scale) {
    __shared__ float sK[kSimtTileN][D];
    __shared__ float sV[kSimtTileN][D];
    __shared__ uint8_t sValid[kSimtTileN];
    const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int G = kSimtThreads / LM;
    const int lm = threadIdx.x % LM, g = threadIdx.x / LM;
    const int n0 = split * chunk;
    const int n1 = min(N, n0 + chunk);
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
        float mx = -INFINITY, l = 0.f;
        for (int t0 = n0; t0 < n1; t0 += kSimtTileN) {
            __syncthreads();
            for (int i = threadIdx.x; i < kSimtTileN * D; i += kSimtThreads) {
                int j = i / D, d = i % D, n = t0 + j;
                bool in = n < n1;
                size_t off = (((size_t)b * N + (in ? n : 0)) * H + h) * D + d;
                sK[j][d] = in ? to_f32(K[off]) : 0.f;
                sV[j][d] = in ? to_f32(V[off]) : 0.f;
                if (d == 0) sValid[j] = in && (key_mask == nullptr || key_mask[(size_t)b * N + n] != 0);
            }
            __syncthreads();
            if (live) {
                for (int j = g; j < kSimtTileN; j += G) {
                    if (!sValid[j]) continue;
                    const float s = score_dot<T, D>(q, sK[j]);
                    if (s > mx) {
                        float r = expf(mx - s);  // 0 on the first token (mx = -inf)
                        l *= r;
#pragma unroll
                        for (int d = 0; d < D; ++d) acc[d] *= r;
                        mx = s;
                    }
                    float p = expf(s - mx);
                    l += p;
#pragma unroll
                    for (int d = 0; d < D; ++d) acc[d] = fmaf(p, sV[j][d], acc[d]);
                }
            }
        }
        if (live) {
            const int part = split * G + g;
            const size_t row = ((size_t)b * H + h) * M + m;
            part_m[(size_t)part * rows + row] = mx;
            part_l[(size_t)part * rows + row] = l;
#pragma unroll
            for (int d = 0; d < D; ++d) part_acc[((size_t)part * rows + row) * D + d] = acc[d];
        }
    }
}

// Log-sum-exp merge of the P partial results of every latent row (b, h, m):
//   m* = max_p m_p;  l = sum_p l_p exp(m_p - m*);  Z = sum_p acc_p exp(m_p - m*) / l;  lse = m* + log l.
// One block per row: thread (slice, d) adds the partials p = slice, slice + S, ... (S = 128 / D slices) in index
// order, thread (0, d) then adds the S slice sums in index order: a fixed order, so the result is reproducible,
// and the P loads of a row are spread over the block instead of queued in one thread (with P in the hundreds
// for small problems the serial form took longer than the encode kernel itself).
constexpr int kMergeThreads = 128;
__global__ void __launch_bounds__(kMergeThreads)
merge_kernel(const float *__restrict__ part_m, const float *__restrict__ part_l, const float *__restrict__ part_acc,
             float *__restrict__ Z, float *__restrict__ lse_enc, int P, long rows, int D) {
    __shared__ float s_a[kMergeThreads], s_b[kMergeThreads];
    const long row = blockIdx.x;
    const int t = threadIdx.x, S = kMergeThreads / D, d = t % D, slice = t / D;
    float mx = -INFINITY;
    for (int p = t; p < P; p += kMergeThreads) mx = fmaxf(mx, part_m[(size_t)p * rows + row]);
    s_a[t] = mx;
    __syncthreads();
    for (int w = kMergeThreads / 2; w > 0; w >>= 1) {
        if (t < w) s_a[t] = fmaxf(s_a[t], s_a[t + w]);
        __syncthreads();
    }
    const float mstar = s_a[0];
    __syncthreads();
    if (mstar == -INFINITY) {  // no valid token anywhere
        if (t < D) Z[row * D + t] = 0.f;
        if (lse_enc != nullptr && t == 0) lse_enc[row] = -INFINITY;
        return;
    }
    float l = 0.f, z = 0.f;
    for (int p = slice; p < P; p += S) {
        const float w = expf(part_m[(size_t)p * rows + row] - mstar);
        l = fmaf(part_l[(size_t)p * rows + row], w, l);
        z = fmaf(part_acc[((size_t)p * rows + row) * D + d], w, z);
    }
    s_a[t] = l;
    s_b[t] = z;
    __syncthreads();
    if (slice == 0) {
        for (int k = 1; k < S; ++k) {
            l += s_a[k * D + d];
            z += s_b[k * D + d];
        }
        Z[row * D + d] = z / l;
        if (lse_enc != nullptr && d == 0) lse_enc[row] = mstar + logf(l);
    }
}

// The same merge with one thread per (row, d), partials added in index order: for few partials and many rows.
__global__ void __launch_bounds__(256)
merge_serial_kernel(const float *__restrict__ part_m, const float *__restrict__ part_l, const float *__restrict__ part_acc,
                    float *__restrict__ Z, float *__restrict__ lse_enc, int P, long rows, int D) {
    const long idx = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= rows * D) return;
    const long row = idx / D;
    const int d = (int)(idx % D);
    float mstar = -INFINITY;
    for (int p = 0; p < P; ++p) mstar = fmaxf(mstar, part_m[(size_t)p * rows + row]);
    if (mstar == -INFINITY) {  // no valid token anywhere
        Z[idx] = 0.f;
        if (lse_enc != nullptr && d == 0) lse_enc[row] = -INFINITY;
        return;
    }
    float l = 0.f, z = 0.f;
    for (int p = 0; p < P; ++p) {
        float w = expf(part_m[(size_t)p * rows + row] - mstar);
        l = fmaf(part_l[(size_t)p * rows + row], w, l);
        z = fmaf(part_acc[((size_t)p * rows + row) * D + d], w, z);
    }
    Z[idx] = z / l;
    if (lse_enc != nullptr && d == 0) lse_enc[row] = mstar + logf(l);
}

constexpr int kDecodeSimtThreads = 128;
constexpr int kDecodeSimtLatents = 64;  // latents staged in shared memory per step

// Decode: one thread per token of head h; grid = (ceil(N/128), H, B).
template <typename T, int D>
__global__ void __launch_bounds__(kDecodeSimtThreads)
decode_simt_kernel(const T *__restrict__ Q, const T *__restrict__ K, const float *__restrict__ Z, T *__restrict__ Y,
                   float *__restrict__ lse_dec, int B, int H, int N, int M, float scale) {
    __shared__ float sQ[kDecodeSimtLatents][D];
    __shared__ float sZ[kDecodeSimtLatents][D];
    const int h = blockIdx.y, b = blockIdx.z;
    const int n = blockIdx.x * kDecodeSimtThreads + threadIdx.x;
    const bool live = n < N;
    const size_t tok = (((size_t)b * N + (live ? n : 0)) * H + h) * D;
    float k[D], acc[D];
#pragma unroll
    for (int d = 0; d < D; ++d) {
        k[d] = live ? to_f32(K[tok + d]) * scale : 0.f;
        acc[d] = 0.f;
    }
    float mx = -INFINITY, l = 0.f;
    for (int m0 = 0; m0 < M; m0 += kDecodeSimtLatents) {
        const int mc = min(kDecodeSimtLatents, M - m0);
        __syncthreads();
        for (int i = threadIdx.x; i < mc * D; i += kDecodeSimtThreads) {
            int j = i / D, d = i % D;
            sQ[j][d] = to_f32(Q[((size_t)h * M + m0 + j) * D + d]);
            sZ[j][d] = Z[(((size_t)b * H + h) * M + m0 + j) * D + d];
        }
        __syncthreads();
        for (int j = 0; j < mc; ++j) {
            const float s = score_dot<T, D>(k, sQ[j]);
            if (s > mx) {
                float r = expf(mx - s);
                l *= r;
#pragma unroll
                for (int d = 0; d < D; ++d) acc[d] *= r;
                mx = s;
            }
            float p = expf(s - mx);
            l += p;
#pragma unroll
            for (int d = 0; d < D; ++d) acc[d] = fmaf(p, sZ[j][d], acc[d]);
        }
    }
    if (live) {
        const float inv = 1.f / l;
#pragma unroll
        for (int d = 0; d < D; ++d) from_f32(Y[tok + d], acc[d] * inv);
        if (lse_dec != nullptr) lse_dec[((size_t)b * N + n) * H + h] = mx + logf(l);
    }
}

}  // namespace flare
