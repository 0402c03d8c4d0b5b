// Shared device/host helpers of libflare (CUDA path only; the CPU oracle shares none of this).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace flare {

// Workspace header: 256 bytes at the start of every workspace.
//   word 0: error flag (0 = fine; otherwise a code naming the wait that gave up)
//   word 1: detail (which barrier / iteration)
constexpr size_t kHeaderBytes = 256;

// Section sizes are rounded up to this, so every section starts 256-byte aligned.
constexpr size_t kAlign = 256;
__host__ __device__ inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }

// Where the pieces of an encode/forward workspace live.  P = number of partial results per latent row.
struct WorkspaceLayout {
    size_t part_m;    // float [P][B*H*M]      running maxima (natural-log units of the scaled score)
    size_t part_l;    // float [P][B*H*M]      sums of exp(score - max)
    size_t part_acc;  // float [P][B*H*M][D]   un-normalised latent rows
    size_t z;         // float [B*H*M][D]      latent sequence when the caller passes Z = NULL
    size_t total;
};

inline WorkspaceLayout make_layout(int P, long rows, int D, bool with_z) {
    WorkspaceLayout w;
    size_t off = kHeaderBytes;
    w.part_m = off;   off += align_up(sizeof(float) * (size_t)P * rows);
    w.part_l = off;   off += align_up(sizeof(float) * (size_t)P * rows);
    w.part_acc = off; off += align_up(sizeof(float) * (size_t)P * rows * D);
    w.z = off;
    if (with_z) off += align_up(sizeof(float) * (size_t)rows * D);
    w.total = off;
    return w;
}

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_f32(float &dst, float x) { dst = x; }
__device__ __forceinline__ void from_f32(__nv_bfloat16 &dst, float x) { dst = __float2bfloat16_rn(x); }
__device__ __forceinline__ float to_f32(__half x) { return __half2float(x); }
__device__ __forceinline__ void from_f32(__half &dst, float x) { dst = __float2half_rn(x); }

}  // namespace flare
