// Instruction-level measurements that the design of the kernels rests on, as kernels of the library so that they
// can be repeated on any B200 (flare_microbench): how many exponentials per clock an SM delivers with the
// special-function unit alone and with half of them on the FMA pipe, in the loop the softmax warps actually run
// (scores from tensor memory, packed weights back to it), and what an MMA hand-over costs the issuing thread.
#pragma once

#include "flare_tc.cuh"

namespace flare {

// 16 warps (the softmax warps of the forward kernels) turn 32 score columns into 16 columns of packed weights, `iters` times.
// kBody 0: running-maximum form (max, fma, ex2, sum, pack); 1: no maximum, special-function unit only; 2: no maximum,
// seven pairs of columns in sixteen (kPolyPairs) by the polynomial on the FMA pipe.  out[block] = cycles of the block's loop.
template <int kBody>
__global__ void __launch_bounds__(kTcThreads, 1) micro_softmax_kernel(int iters, float sl2, unsigned long long *out) {
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5;
    if (warp == kFirstIssuerWarp) ptx::tmem_alloc(ptx::smem_u32(&tmem_slot), 512);
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tm = tmem_slot;
    long long t0 = clock64(), t1 = t0;
    if (warp >= kFirstSoftmaxWarp) {
        const int g = (warp - kFirstSoftmaxWarp) >> 2;
        const uint32_t base = tm + ((uint32_t)((warp & 3) << 5) << 16) + g * 128;
        uint32_t z[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) z[k] = 0x3f800000u + 4096u * k + threadIdx.x;      // scores between 1 and 2
        for (int c = 0; c < 128; c += 16) ptx::tmem_st16(base + c, z);
        ptx::tmem_wait_st();
        float2 sum2 = make_float2(0.f, 0.f);
        float mx = -1e30f;
        const float2 sl2p = make_float2(sl2, sl2);
        t0 = clock64();
        for (int it = 0; it < iters; ++it) {
            const uint32_t sbase = base + (it & 1) * 32;
            uint32_t r[32], pk[16];
            ptx::tmem_ld32(sbase, r);
            ptx::tmem_wait_ld();
            if (kBody == 0) {
                mx = max_of<32>(r, mx);
                exp_chunk<32, false>(r, pk, sl2p, make_float2(-mx * sl2, -mx * sl2), sum2);
            } else {
                exp_chunk_fast<32, kBody == 2, false, 0>(r, pk, sl2p, sum2);
            }
            ptx::tmem_st16(sbase + 64, pk);
            ptx::tmem_wait_st();
        }
        t1 = clock64();
        if (sum2.x + sum2.y + mx == 123.456f) out[blockIdx.x] = 1;                      // keeps the sums alive
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (threadIdx.x == kFirstSoftmaxWarp * 32) out[blockIdx.x] = (unsigned long long)(t1 - t0);
    if (warp == kFirstIssuerWarp) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tm, 512);
    }
}

// One thread issues what a unit of the forward kernels costs it: two value MMAs (A in tensor memory, N = 48), one score
// MMA (N = 32), one commit; then polls the barrier.  out[0] = cycles it was held by the four instructions,
// out[1] = cycles from the commit to the barrier's flip (averages over `iters` rounds).  Operands are zeros.
__global__ void __launch_bounds__(64, 1) micro_mma_kernel(int iters, unsigned long long *out) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ uint64_t bar_mem;
    __shared__ uint32_t tmem_slot, flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_u32(&bar_mem), 1);
        flag = 0;
        ptx::fence_mbar_init();
    }
    for (int i = threadIdx.x; i < 24576 / 16; i += blockDim.x) reinterpret_cast<uint4 *>(smem)[i] = make_uint4(0, 0, 0, 0);
    if (warp == 0) ptx::tmem_alloc(ptx::smem_u32(&tmem_slot), 128);
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tm = tmem_slot;
    if (warp == 1 && lane == 0) {
        using G = TileGeom<16>;
        const uint64_t adesc = ptx::smem_desc(ptx::smem_u32(smem), 16, G::SBO, G::SWZ);                 // [128, 16] K-major
        const uint64_t bdesc = ptx::smem_desc(ptx::smem_u32(smem + 4096), 16, G::SBO, G::SWZ);          // [32, 16] K-major
        const uint64_t zdesc = ptx::smem_desc(ptx::smem_u32(smem + 8192), 4096, G::SBO, G::SWZ);        // three [32, 16] blocks, MN-major
        const uint32_t idS = ptx::instr_desc_bf16(128, 32, 0, 0), idY = ptx::instr_desc_bf16(128, 48, 0, 1);
        const uint32_t b = ptx::smem_u32(&bar_mem);
        long long issue = 0, flip = 0;
        bool ok = true;
        for (int it = 0; ok && it < iters; ++it) {
            const long long t0 = clock64();
            ptx::mma_ts(tm + 64, tm, zdesc, idY, 1);            // columns: scores / weights [0, 32), accumulator [64, 112)
            ptx::mma_ts(tm + 64, tm + 8, zdesc + 2, idY, 1);
            ptx::mma_ss(tm, adesc, bdesc, idS, 0);
            ptx::mma_commit(b);
            const long long t1 = clock64();
            ok = ptx::mbar_spin(b, it & 1, &flag, kErrSelftest | 2);
            issue += t1 - t0;
            flip += clock64() - t1;
        }
        out[0] = ok ? (unsigned long long)(issue / iters) : 0ull;
        out[1] = ok ? (unsigned long long)(flip / iters) : 0ull;
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tm, 128);
    }
}

}  // namespace flare
