// Tensor-core (tcgen05 + TMEM + TMA) kernels of the FLARE mixer for bfloat16 inputs on sm_100a.
//
// Both stages are two small dense contractions around a row softmax (paper Section 3.2):
//   encode  S = Q_h K_tile^T   (latents on the 128 TMEM lanes, tokens on columns)   acc += P V_tile
//   decode  S = K_tile Q_h^T   (tokens on the 128 TMEM lanes, latents on columns)   Y    = P Z_h
// Scores land in tensor memory; one thread owns one lane (one latent in encode, one token in decode), so row
// maxima and sums need no shuffles.  The bf16 weights P are written back over the scores in tensor memory and
// feed the second contraction as its A operand.
//
// Two resources limit both kernels, and neither is the one a roofline of FLOPs and bytes names.  Every
// (latent, token) pair needs one exponential on the special-function unit (16 per clock per SM), and every
// tcgen05.mma of this shape (M = 128, K = 16) holds the tensor pipe for about 107 cycles whatever its N
// (measured), so the value contraction costs one such slot per 16 latents (decode) or tokens (encode): about
// as long as the exponentials of the same block.  That cost is a latency of the issuing thread, not an occupancy
// of the pipe: four threads issuing side by side get about three times the instructions through (measured).
// The CTA is therefore four pipelines side by side: warp 0 issues TMA loads; sixteen softmax warps (four per
// scheduler) form four groups of four warps, and each group has an issuing warp of its own (warps 1-4; warp 1
// also owns the TMEM allocation).  A group owns one TMEM score buffer, or a range of columns of a shared one,
// with its own score MMA, running maximum, sum and accumulator columns; its weights go to its value
// contraction a few columns at a time as they are written.  While one group waits for its MMAs the other
// three keep the schedulers and the special-function unit fed.
#pragma once

#include <type_traits>

#include "flare_common.cuh"
#include "flare_ptx.cuh"

namespace flare {

constexpr int kSoftmaxGroups = 4;                            // groups of 4 warps (128 threads = 128 TMEM lanes)
constexpr int kFirstIssuerWarp = 1;                          // warps 1..4: one MMA-issuing warp per group
constexpr int kFirstSoftmaxWarp = kFirstIssuerWarp + kSoftmaxGroups;
constexpr int kTcThreads = (kFirstSoftmaxWarp + 4 * kSoftmaxGroups) * 32;  // 672
// The fast form of encode adds three guard warps behind the softmax warps (they check the norms of the key rows while a
// tile waits in its stage; 24 warps still get 80 registers each: six per scheduler either way).
constexpr int kGuardWarps = 3;
constexpr int kFirstGuardWarp = kTcThreads / 32;
constexpr int kTcThreadsGuarded = kTcThreads + 32 * kGuardWarps;          // 768
constexpr int kTile = 128;       // tokens per tile (decode: TMEM lanes; encode: score columns)
constexpr int kDecStages = 4;    // K tiles in flight (decode); 8 and 12 were measured 10 % slower at 32 and 128 latents
constexpr int kEncStages = 3;    // K+V tile pairs in flight (encode), where all four groups of a CTA work on the same tile
// Where the CTA's two slots take alternate tiles (one latent block: M <= 128) four tiles are in use at any time (per
// slot the one whose weights are being formed and the next, whose scores are issued ahead) and a tile lasts half as
// long, so the ring is as deep as shared memory allows: with three stages every load's latency was exposed (measured).
constexpr int kEncMaxStages = 8;
constexpr size_t kTcMinSmem = 120 * 1024;  // request at least this much so that one CTA owns an SM (and its TMEM)

// Error codes left in the workspace header by a wait that gave up.
enum : uint32_t { kErrDecode = 0x100, kErrEncode = 0x200, kErrBwdDq = 0x300, kErrBwdTok = 0x400, kErrSelftest = 0x500,
                  kErrSpectral = 0x600 };

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

// Narrow heads (half- and quarter-width forms of the kernels): the head is DR < D wide in memory and the kernels
// multiply D = 16 wide rows.  A token tile is the 16 feature columns from the 16-byte boundary at or below the
// head's first column (a TMA box must start on one), so the head's features sit `off` elements into the row
// (0, or 4 for every other head of width 4) next to its neighbours' (zeros past the last head).  The rows of the
// latent operands (Q, Z, dZ) are staged by the CTA's threads into zeroed rows at the same offset, so the
// neighbours' columns meet zeros in every product; accumulator columns outside [off, off + DR) are never read.
__device__ __forceinline__ int narrow_offset(int h, int DR) { return (h * DR) & 7; }

// rows of a [rows, 4] bf16 matrix -> columns [off, off + 4) of zeroed, swizzled D-wide rows
template <int D>
__device__ __forceinline__ void stage_rows4(uint8_t *dst, const __nv_bfloat16 *src, int rows, int off) {
    using G = TileGeom<D>;
    for (int m = threadIdx.x; m < rows; m += blockDim.x)
        *reinterpret_cast<uint2 *>(dst + (size_t)m * G::RB + (G::swz(m) << 4) + off * 2) =
            *reinterpret_cast<const uint2 *>(src + (size_t)m * 4);
}
// rows of a [rows, 4] float matrix -> two bf16 halves (hi = round(z), lo = round(z - hi)) at columns [off, off + 4)
template <int D>
__device__ __forceinline__ void stage_rows4_hilo(uint8_t *dst_hi, uint8_t *dst_lo, const float *src, int rows, int off) {
    using G = TileGeom<D>;
    for (int m = threadIdx.x; m < rows; m += blockDim.x) {
        const float4 z = *reinterpret_cast<const float4 *>(src + (size_t)m * 4);
        const uint32_t h0 = ptx::pack_bf16(z.x, z.y), h1 = ptx::pack_bf16(z.z, z.w);
        const uint32_t l0 = ptx::pack_bf16(z.x - __uint_as_float(h0 << 16), z.y - __uint_as_float(h0 & 0xffff0000u));
        const uint32_t l1 = ptx::pack_bf16(z.z - __uint_as_float(h1 << 16), z.w - __uint_as_float(h1 & 0xffff0000u));
        const size_t o = (size_t)m * G::RB + (G::swz(m) << 4) + off * 2;
        *reinterpret_cast<uint2 *>(dst_hi + o) = make_uint2(h0, h1);
        *reinterpret_cast<uint2 *>(dst_lo + o) = make_uint2(l0, l1);
    }
}

// ------------------------------------------------------------------------------------- softmax arithmetic
// p = 2^(s * sl2 + neg[k]) with one addend per column (read from shared memory, four at a time): the form the
// backward needs, where every column (token) carries its own log-sum-exp.  The weights leave as two bf16 halves,
// hi = round(p) and lo = round(p - hi): dZ feeds differences (dZ.V - dZ.Z) downstream, and with one half its
// rounding alone moved dK, dV and dQ by 2e-2 to 4e-2 of their RMS (measured).
template <int NV>
__device__ __forceinline__ void exp_chunk_cols(const uint32_t *r, uint32_t *hi, uint32_t *lo, float2 sl2p, const float *neg) {
#pragma unroll
    for (int k = 0; k < NV / 4; ++k) {
        const float4 ng = *reinterpret_cast<const float4 *>(neg + 4 * k);
        const float2 x0 = __ffma2_rn(make_float2(__uint_as_float(r[4 * k]), __uint_as_float(r[4 * k + 1])), sl2p,
                                     make_float2(ng.x, ng.y));
        const float2 x1 = __ffma2_rn(make_float2(__uint_as_float(r[4 * k + 2]), __uint_as_float(r[4 * k + 3])), sl2p,
                                     make_float2(ng.z, ng.w));
        const float p0 = ptx::ex2(x0.x), p1 = ptx::ex2(x0.y), p2 = ptx::ex2(x1.x), p3 = ptx::ex2(x1.y);
        const uint32_t h0 = ptx::pack_bf16(p0, p1), h1 = ptx::pack_bf16(p2, p3);
        hi[2 * k] = h0;
        hi[2 * k + 1] = h1;
        lo[2 * k] = ptx::pack_bf16(p0 - __uint_as_float(h0 << 16), p1 - __uint_as_float(h0 & 0xffff0000u));
        lo[2 * k + 1] = ptx::pack_bf16(p2 - __uint_as_float(h1 << 16), p3 - __uint_as_float(h1 & 0xffff0000u));
    }
}

// Row maximum over NV (16 or 32) float32 scores held as raw bits.
template <int NV>
__device__ __forceinline__ float max_of(const uint32_t *r, float m) {
#pragma unroll
    for (int k = 0; k < NV; k += 2) m = ptx::max3(m, __uint_as_float(r[k]), __uint_as_float(r[k + 1]));
    return m;
}

// p = 2^(s * sl2 + neg) for NV scores; bf16 pairs to pk, float32 sums into sum2 (two interleaved partial sums).
// With kMasked, scores whose bit in `valid` is clear (or all of them if `dead`) get weight exactly 0.
template <int NV, bool kMasked>
__device__ __forceinline__ void exp_chunk(const uint32_t *r, uint32_t *pk, float2 sl2p, float2 negp, float2 &sum2,
                                          uint32_t valid = 0xffffffffu, bool dead = false) {
#pragma unroll
    for (int k = 0; k < NV / 2; ++k) {
        const float2 x = __ffma2_rn(make_float2(__uint_as_float(r[2 * k]), __uint_as_float(r[2 * k + 1])), sl2p, negp);
        float2 p = make_float2(ptx::ex2(x.x), ptx::ex2(x.y));
        if (kMasked) {
            if (dead || !((valid >> (2 * k)) & 1)) p.x = 0.f;
            if (dead || !((valid >> (2 * k + 1)) & 1)) p.y = 0.f;
        }
        sum2 = __fadd2_rn(sum2, p);
        pk[k] = ptx::pack_bf16(p.x, p.y);
    }
}

// exp_chunk with the weights leaving as two bf16 halves (hi = round(p), lo = round(p - hi)), for an encode whose Z
// is saved for the backward: the gradients magnify the error of Z several times, and with single bf16 weights
// (Z off by 3e-3 to 4e-3 of its RMS) that alone put dK and dQ at 2e-2 to 3e-2 of theirs where N is only a few
// times M (measured; with the exact Z the same backward is at 5e-4).
template <int NV, bool kMasked>
__device__ __forceinline__ void exp_chunk_hilo(const uint32_t *r, uint32_t *hi, uint32_t *lo, float2 sl2p, float2 negp,
                                               float2 &sum2, uint32_t valid = 0xffffffffu, bool dead = false) {
#pragma unroll
    for (int k = 0; k < NV / 2; ++k) {
        const float2 x = __ffma2_rn(make_float2(__uint_as_float(r[2 * k]), __uint_as_float(r[2 * k + 1])), sl2p, negp);
        float2 p = make_float2(ptx::ex2(x.x), ptx::ex2(x.y));
        if (kMasked) {
            if (dead || !((valid >> (2 * k)) & 1)) p.x = 0.f;
            if (dead || !((valid >> (2 * k + 1)) & 1)) p.y = 0.f;
        }
        sum2 = __fadd2_rn(sum2, p);
        const uint32_t h = ptx::pack_bf16(p.x, p.y);
        hi[k] = h;
        lo[k] = ptx::pack_bf16(p.x - __uint_as_float(h << 16), p.y - __uint_as_float(h & 0xffff0000u));
    }
}

// ---------------------------------------------------------------------------- softmax without a running maximum
// The "fast" forms of the kernels evaluate p = 2^(s * sl2) as it stands: no maximum is searched, subtracted or
// tracked, no accumulator is ever rescaled, and the column ranges of a decode tile need no common reference.
// float32 and bfloat16 hold 2^x for |x| < 126; with 30 binades kept free for the sums of up to 2^20 such terms times
// values of ordinary size, that is safe while every |s * sl2| <= kFastMaxLog2.  The kernels check the sufficient
// condition |q| |k| sl2 <= kFastMaxLog2 (Cauchy-Schwarz) on the rows they hold in shared memory and raise a flag if
// it fails; the host then runs the exact form (running maximum) of the same kernel, which exits at once while the
// flag is clear.
constexpr float kFastMaxLog2 = 96.f;

// Two ways to 2^x share the work.  The special-function unit (ex2.approx) delivers 16 results per clock per SM and
// is the busiest unit of these kernels; the other half of the column pairs goes through the FMA pipe: with
// magic = 1.5 * 2^23, t = fma(s, sl2, magic) is magic + round(x) exactly, f = fma(s, sl2, magic - t) is
// x - round(x) in [-1/2, 1/2] with one rounding, a degree-3 polynomial gives 2^f within 7.5e-5 (the weights are
// rounded to bfloat16, 2e-3, right after), and adding round(x) to the exponent field is one shift-and-add on the
// bits of t.  Valid for |x| < 126, which the fast forms guarantee; scores of padded tokens (kMaskedScore) must not
// come this way.  Measured on B200 (16 warps, scores from and weights to tensor memory): 15 results per clock per SM
// with the special-function unit alone, 22 with seven pairs in sixteen on the FMA pipe (see kPolyPairs; 24 with degree 2).
constexpr int kPolyDegree = 3;
// Which of every sixteen pairs of columns take the polynomial (bit k: pair k).  Measured, softmax loop alone /
// million-point forward: 4 of 16: 19.0 exponentials per clock per SM / 1.195 ms; 5: 20.4 / 1.184; 6: 21.4 / 1.173;
// 7: 22.3-22.5 / 1.128-1.155 (this pattern the better of two); 8 (every second pair): 21.4 / 1.161; 9: 20.6 / 1.269;
// 10: 19.7 / 1.277.
constexpr unsigned kPolyPairs = 0xAAA8;
__device__ __forceinline__ float2 exp2_fma_pipe(float2 s, float2 sl2p) {
    constexpr float kMagic = 12582912.f;                        // 1.5 * 2^23
    const float2 magic = make_float2(kMagic, kMagic);
    const float2 t = __ffma2_rn(s, sl2p, magic);
    const float2 w = __ffma2_rn(t, make_float2(-1.f, -1.f), magic);   // -round(x), exact
    const float2 f = __ffma2_rn(s, sl2p, w);
    float2 p;
    if (kPolyDegree == 3) {                                     // minimax on [-1/2, 1/2], relative error 7.5e-5
        constexpr float c0 = 0.99992800f, c1 = 0.69326019f, c2 = 0.24261151f, c3 = 0.055175912f;
        p = __ffma2_rn(make_float2(c3, c3), f, make_float2(c2, c2));
        p = __ffma2_rn(p, f, make_float2(c1, c1));
        p = __ffma2_rn(p, f, make_float2(c0, c0));
    } else {                                                    // degree 2: relative error 1.7e-3
        constexpr float c0 = 1.0004400f, c1 = 0.70345056f, c2 = 0.23845598f;
        p = __ffma2_rn(make_float2(c2, c2), f, make_float2(c1, c1));
        p = __ffma2_rn(p, f, make_float2(c0, c0));
    }
    p.x = __uint_as_float(__float_as_uint(p.x) + (__float_as_uint(t.x) << 23));
    p.y = __uint_as_float(__float_as_uint(p.y) + (__float_as_uint(t.y) << 23));
    return p;
}

// p = 2^(s * sl2) for NV scores, bf16 pairs to pk.  kPoly: the pairs of kPolyPairs on the FMA pipe.
// The row sum must be that of the ROUNDED weights: without a maximum the largest weight of a row is not 1.0 but
// some 2^x with a full mantissa, and a sum of the unrounded values would normalise it away from the rounded one
// that multiplies the values (measured: Y off by 1.5e-2 of its RMS where one weight dominates a row, against 4e-3).
// kSum = 0: no sum here (a ones column of the value operand lets the tensor core add the rounded weights);
// kSum = 1: the rounded weights are widened again and added into sum2;
// kSum = 2: as 0, and the unrounded weights are added into sum2 (for a log-sum-exp output, which must not carry the
//           rounding of the weights: the backward rebuilds every weight from it).
template <int NV, bool kPoly, bool kMasked, int kSum>
__device__ __forceinline__ void exp_chunk_fast(const uint32_t *r, uint32_t *pk, float2 sl2p, float2 &sum2,
                                               uint32_t valid = 0xffffffffu) {
#pragma unroll
    for (int k = 0; k < NV / 2; ++k) {
        const float2 s = make_float2(__uint_as_float(r[2 * k]), __uint_as_float(r[2 * k + 1]));
        float2 p;
        if (kPoly && ((kPolyPairs >> (k & 15)) & 1)) {
            p = exp2_fma_pipe(s, sl2p);
        } else {
            const float2 x = __fmul2_rn(s, sl2p);
            p = make_float2(ptx::ex2(x.x), ptx::ex2(x.y));
        }
        if (kMasked) {
            if (!((valid >> (2 * k)) & 1)) p.x = 0.f;
            if (!((valid >> (2 * k + 1)) & 1)) p.y = 0.f;
        }
        pk[k] = ptx::pack_bf16(p.x, p.y);
        if (kSum == 1) sum2 = __fadd2_rn(sum2, make_float2(__uint_as_float(pk[k] << 16), __uint_as_float(pk[k] & 0xffff0000u)));
        if (kSum == 2) sum2 = __fadd2_rn(sum2, p);
    }
}

// Largest squared norm among the rows [lane, lane + 32, ...) < rows of a [rows, RB / 2] bf16 tile in shared memory
// (the 16-byte chunks of a row are permuted by the swizzle, which a sum over the whole row does not see), as an upper
// bound: the squares are summed two at a time in bf16 (one packed fma per pair of elements: the warp that runs this
// shares its schedulers with the softmax warps, so instructions are what it costs), at most 16 roundings of 2^-9 per sum (3 %),
// and the result is raised by 1/16 to stay above the exact value.
// kHalves = 2 (head-pair form: a row holds two heads side by side): the larger of the two halves' sums, since a score
// only ever meets one head's features.
template <int RB, int kHalves = 1>
__device__ __forceinline__ float tile_max_norm2(const uint8_t *tile, int rows, int lane) {
    using G = TileGeom<RB / 2>;
    float best = 0.f;
    for (int r = lane; r < rows; r += 32) {
        float n2;
        if (kHalves == 1) {
            uint32_t acc0 = 0u, acc1 = 0u;                         // two bf16x2 sums
#pragma unroll
            for (int c = 0; c < RB / 16; ++c) {
                const uint4 v = *reinterpret_cast<const uint4 *>(tile + (size_t)r * RB + c * 16);
                asm("fma.rn.bf16x2 %0, %1, %1, %0;" : "+r"(acc0) : "r"(v.x));
                asm("fma.rn.bf16x2 %0, %1, %1, %0;" : "+r"(acc1) : "r"(v.y));
                asm("fma.rn.bf16x2 %0, %1, %1, %0;" : "+r"(acc0) : "r"(v.z));
                asm("fma.rn.bf16x2 %0, %1, %1, %0;" : "+r"(acc1) : "r"(v.w));
            }
            n2 = (__uint_as_float(acc0 << 16) + __uint_as_float(acc0 & 0xffff0000u)) +
                 (__uint_as_float(acc1 << 16) + __uint_as_float(acc1 & 0xffff0000u));
        } else {
            uint32_t acc[2] = {0u, 0u};                            // one bf16x2 sum per half of the row
            const int sw = G::swz(r);
#pragma unroll
            for (int l = 0; l < RB / 16; ++l) {                    // logical chunk l sits at chunk l ^ swz(r)
                const uint4 v = *reinterpret_cast<const uint4 *>(tile + (size_t)r * RB + ((l ^ sw) << 4));
                uint32_t &a = acc[l >= RB / 32 ? 1 : 0];
                asm("fma.rn.bf16x2 %0, %1, %1, %0;" : "+r"(a) : "r"(v.x));
                asm("fma.rn.bf16x2 %0, %1, %1, %0;" : "+r"(a) : "r"(v.y));
                asm("fma.rn.bf16x2 %0, %1, %1, %0;" : "+r"(a) : "r"(v.z));
                asm("fma.rn.bf16x2 %0, %1, %1, %0;" : "+r"(a) : "r"(v.w));
            }
            n2 = fmaxf(__uint_as_float(acc[0] << 16) + __uint_as_float(acc[0] & 0xffff0000u),
                       __uint_as_float(acc[1] << 16) + __uint_as_float(acc[1] & 0xffff0000u));
        }
        n2 *= 1.0625f;
        if (!(n2 <= 3.0e38f)) n2 = INFINITY;                    // a row with a NaN or an infinity fails every check
        best = fmaxf(best, n2);
    }
    return best;
}
__device__ __forceinline__ float warp_max_nan(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// ------------------------------------------------------------------------------------------------ decode
// How the four softmax groups share tensor memory in decode.  `cs` groups split the M score columns of one
// buffer into ranges of `part_w` columns (the last may be shorter); `nbuf` buffers of `cb` columns hold
// different token tiles.  The Y accumulator of a column range sits in columns of that range that its packed
// bf16 weights leave free (`alias`), else after the scores.  Every range is a pipeline of its own: its scores
// come from their own MMA, its weights go to the value contraction a few columns at a time as they are written
// (so that the tensor pipe works on one part of the row while the exponentials of the next are evaluated), and
// the ranges of a tile meet again only when its rows of Y are written.
//
// Z enters the value contraction as two bf16 halves (hi = round(z), lo = round(z - hi), about 16 mantissa
// bits: with plain bf16 rows the rounding of Z alone reaches the error bound where max|Z| is several times
// RMS(Y)).  With a narrow head the halves sit side by side as one B operand of width 2D, so that the split
// costs no extra MMA ([P Z_hi | P Z_lo], added when Y is written).
struct DecodePlan {
    int cs, nbuf, part_w, alias, cb, ncols;
};

// Columns of one Y accumulator.
__host__ __device__ constexpr int decode_y_cols(int D) { return D <= 32 ? 2 * D : D; }

// Column choreography of one range of `len` score columns with aliasing.  The softmax walks the scores from the
// top column down in chunks of 32; a chunk's columns are free once read.  With a Y accumulator of `yc` columns,
// the first yc/16 chunks free 2*yc columns, which take those chunks' packed weights (16 columns each, top
// down) and, below them, Y; every later chunk's weights go to the bottom half of the chunk's own columns.
__host__ __device__ constexpr int decode_y_alias_col(int len, int yc) { return len - 2 * yc; }
// First column (within the range) of the packed weights of the chunk whose scores start at column `lo`.
__host__ __device__ constexpr int decode_p_col(int len, int yc, int lo, bool alias) {
    const int k = (len - 1 - lo) / 32;                         // chunk index counted from the top
    return (alias && k < yc / 16) ? len - 16 * (k + 1) : lo;
}
// Score columns per hand-over of weights to the value contraction: at most four per range and tile, and the
// first covers the 2*yc columns that make room for Y.
__host__ __device__ constexpr int decode_handover_cols(int len, int yc) {
    int u = ((len + 3) / 4 + 31) & ~31;
    if (u < 2 * yc) u = 2 * yc;
    return u < 32 ? 32 : u;
}

__host__ __device__ constexpr int decode_part_len(const DecodePlan &p, int M, int c) {
    const int start = c * p.part_w;
    const int len = M - start < p.part_w ? M - start : p.part_w;
    return len > 0 ? len : 0;
}

__host__ __device__ constexpr DecodePlan make_decode_plan(int M, int D) {
    const int yc = decode_y_cols(D);
    DecodePlan best{};
    int best_groups = 0;
    for (int cs = 1; cs <= 4; cs *= 2) {
        DecodePlan p{};
        p.cs = cs;
        p.part_w = ((M / 16 + cs - 1) / cs) * 16;
        if ((cs - 1) * p.part_w >= M) continue;                 // an empty column range
        p.alias = 1;
        for (int c = 0; c < cs; ++c)
            if (decode_part_len(p, M, c) < 2 * yc) p.alias = 0;
        p.cb = ((p.alias ? M : M + cs * yc) + 31) & ~31;
        if (p.cb > 512) continue;
        p.nbuf = 512 / p.cb < kSoftmaxGroups / cs ? 512 / p.cb : kSoftmaxGroups / cs;
        p.ncols = 32;
        while (p.ncols < p.nbuf * p.cb) p.ncols *= 2;
        if (p.nbuf * cs > best_groups) {
            best_groups = p.nbuf * cs;
            best = p;
        }
    }
    return best;
}

struct DecodeTcArgs {
    const __nv_bfloat16 *Q;  // [H,M,D] (read directly in the half-width form)
    const float *Z;      // [B,H,M,D]
    __nv_bfloat16 *Y;    // [B,N,H,D]
    float *lse_dec;      // [B,N,H] or null
    uint32_t *status;    // workspace header or null
    const uint32_t *run_if;   // exact forms: null, or a word that must be non-zero for the kernel to do anything
    uint32_t *redo;           // fast forms: set to 1 if a score may lie outside the range they are valid for
    int B, H, N, M;      // M: latents this launch works on (all of them, or a range of at most 512)
    int mtot, m0;        // latents per head in Q and Z, and the first one of this launch's range
    float *Ypart;        // kPart form of the kernel: [B,N,H,D] float32, rows normalised over the range go here instead
                         // of Y, with their log-sum-exp in lse_dec, for decode_combine_kernel
    float sl2;           // scale * log2(e)
    int tiles;           // ceil(N / 128)
    DecodePlan plan;
};

// Shared-memory carve-up of the decode kernel.
template <int D>
struct DecodeSmem {
    using G = TileGeom<D>;
    static constexpr size_t k_off = 0;
    static constexpr size_t kBarBytes = 512;
    static constexpr size_t kTail = kBarBytes + 2 * kSoftmaxGroups * kTile * sizeof(float);  // barriers + row statistics
    // K tiles in flight: as many of kDecStages as fit beside Q_h and the two halves of Z_bh.  (A K tile is free
    // again as soon as its score MMAs have run, so even one stage leaves a whole tile's softmax to hide the load.)
    __host__ __device__ static int stages(int M) {
        int s = kDecStages;
        while (s > 1 && (size_t)s * G::TILE_BYTES + (size_t)3 * M * G::RB + kTail + 2048 > 227 * 1024) --s;
        return s;
    }
    __host__ __device__ static size_t q_off(int M) { return (size_t)stages(M) * G::TILE_BYTES; }
    __host__ __device__ static size_t z_off(int M) { return q_off(M) + (size_t)M * G::RB; }  // [hi | lo], M rows each
    __host__ __device__ static size_t bar_off(int M) { return align_up(z_off(M) + (size_t)2 * M * G::RB, 1024); }
    __host__ __device__ static size_t stat_off(int M) { return bar_off(M) + kBarBytes; }
    __host__ __device__ static size_t total(int M) {
        size_t t = bar_off(M) + kTail + 1024;  // plus slack to align the base to 1024
        return t < kTcMinSmem ? kTcMinSmem : t;
    }
};

// Decode.  grid = (ctas_per_head, H, B); each CTA walks a contiguous range of 128-token tiles of one (b, h)
// with Q_h and Z_bh resident in shared memory.
//
// Narrow form (DRT = 8 or 4 with D = 16): the head is DRT wide in memory (see narrow_offset).  This is how head
// widths below the smallest MMA K-step (16) run on the tensor cores.
//
// kM: 0, or the number of latents of the launch as a compile-time constant (the plan, the column choreography and
// the chunk loops then fold to constants; the common sizes have such forms).
template <int D, int DRT = 0, bool kPart = false, int kM = 0>
__global__ void __launch_bounds__(kTcThreads, 1)
decode_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ, DecodeTcArgs a) {
    if (a.run_if != nullptr && *a.run_if == 0) return;          // behind the streaming form, as a fallback that was not needed
    constexpr bool kHalf = DRT != 0;
    constexpr int DR = kHalf ? DRT : D;                         // head width in memory
    using G = TileGeom<D>;
    using SM = DecodeSmem<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int M = kM ? kM : a.M;
    uint8_t *sK = smem + SM::k_off;
    uint8_t *sQ = smem + SM::q_off(M);
    uint8_t *sZ = smem + SM::z_off(M);
    const int nstages = SM::stages(M);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + SM::bar_off(M));
    float *stat_m = reinterpret_cast<float *>(smem + SM::stat_off(M));   // [group][128] row maxima (log2 units)
    float *stat_l = stat_m + kSoftmaxGroups * kTile;                      // [group][128] row sums
    constexpr int NG = kSoftmaxGroups;
    // S_FULL, Y_FULL: one per group (column range of a buffer); P_CHUNK: four hand-overs per group; BUF_EMPTY: per buffer
    enum { K_FULL = 0, K_EMPTY = K_FULL + kDecStages, S_FULL = K_EMPTY + kDecStages, P_CHUNK = S_FULL + NG,
           Y_FULL = P_CHUNK + 4 * NG, BUF_EMPTY = Y_FULL + NG, Q_FULL = BUF_EMPTY + NG, NBARS };
    static_assert(NBARS * 8 + 8 <= SM::kBarBytes, "barrier area too small");
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + NBARS);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = blockIdx.y, b = blockIdx.z;
    const int off = kHalf ? narrow_offset(h, DR) : 0;           // the head's first column within a token tile row
    const int t_begin = (int)((long)a.tiles * blockIdx.x / gridDim.x);
    const int t_end = (int)((long)a.tiles * (blockIdx.x + 1) / gridDim.x);
    const int ntiles = t_end - t_begin;

    constexpr DecodePlan kPlan = make_decode_plan(kM ? kM : 16, D);
    const DecodePlan pl = kM ? kPlan : a.plan;
    const int cs = pl.cs, nbuf = pl.nbuf, cb = pl.cb;
    constexpr int YC = decode_y_cols(D);
    constexpr bool kWide = YC == 2 * D;                         // one MMA over [Z_hi | Z_lo] (N = 2D) per 16 latents
    // column of the Y accumulator of range c, relative to its buffer
    auto y_col = [&](int c) {
        if (!pl.alias) return M + c * YC;
        return c * pl.part_w + decode_y_alias_col(decode_part_len(pl, M, c), YC);
    };

    auto bar = [&](int i) { return ptx::smem_u32(bars + i); };

    if (threadIdx.x == 0) {
        for (int i = 0; i < NBARS; ++i) {
            const bool counted = (i >= P_CHUNK && i < P_CHUNK + 4 * NG) || (i >= BUF_EMPTY && i < BUF_EMPTY + NG);
            const bool per_range = i >= K_EMPTY && i < K_EMPTY + kDecStages;   // every range's issuer releases the K tile
            ptx::mbar_init(bar(i), counted ? 128u : per_range ? (uint32_t)cs : 1u);
        }
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmK);
        ptx::prefetch_tensormap(&tmQ);
    }
    if (warp == kFirstIssuerWarp) ptx::tmem_alloc(ptx::smem_u32(tmem_slot), (uint32_t)pl.ncols);
    // Z_bh -> two bf16 halves (hi = round(z), lo = round(z - hi)); rows of RB bytes in the swizzled layout the
    // MMA's B operand expects (latent-major rows), the lo half M rows after the hi half.
    {
        const float *Zg = a.Z + (((size_t)b * a.H + h) * a.mtot + a.m0) * DR;
        if (kHalf) {   // upper halves of the rows of Q, Z_hi and Z_lo are zero
            for (int i = threadIdx.x; i < M * (D / 8); i += kTcThreads) {
                reinterpret_cast<uint4 *>(sQ)[i] = make_uint4(0, 0, 0, 0);
                reinterpret_cast<uint4 *>(sZ)[i] = make_uint4(0, 0, 0, 0);
                reinterpret_cast<uint4 *>(sZ + (size_t)M * G::RB)[i] = make_uint4(0, 0, 0, 0);
            }
            __syncthreads();
            if constexpr (DR == 4) {
                stage_rows4<D>(sQ, a.Q + ((size_t)h * a.mtot + a.m0) * DR, M, off);
                stage_rows4_hilo<D>(sZ, sZ + (size_t)M * G::RB, Zg, M, off);
            } else {
                for (int i = threadIdx.x; i < M * (DR / 8); i += kTcThreads) {
                    const int m = i / (DR / 8), c = i % (DR / 8);
                    *reinterpret_cast<uint4 *>(sQ + (size_t)m * G::RB + ((c ^ G::swz(m)) << 4)) =
                        *reinterpret_cast<const uint4 *>(a.Q + ((size_t)h * a.mtot + a.m0 + m) * DR + c * 8);
                }
            }
        }
        constexpr int ZC = DR >= 8 ? DR / 8 : 1;                // 8-float chunks per row of Z (none for DR = 4: staged above)
        for (int i = threadIdx.x; i < (DR >= 8 ? M * ZC : 0); i += kTcThreads) {
            const int m = i / ZC, c = i % ZC;
            const float4 lo = *reinterpret_cast<const float4 *>(Zg + (size_t)m * DR + c * 8);
            const float4 hi = *reinterpret_cast<const float4 *>(Zg + (size_t)m * DR + c * 8 + 4);
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
            if (kHalf) {
                ptx::mbar_arrive(bar(Q_FULL));                  // Q was written by the threads before the block barrier
            } else {
                // Q_h: M/16 boxes of 16 rows
                ptx::mbar_arrive_expect_tx(bar(Q_FULL), (uint32_t)(M * G::RB));
                for (int r = 0; r < M; r += 16)
                    ptx::tma_load_2d(ptx::smem_u32(sQ + (size_t)r * G::RB), &tmQ, bar(Q_FULL), 0, h * a.mtot + a.m0 + r);
            }
        }
        if (lane == 0) {
            for (int i = 0; i < ntiles; ++i) {
                const int s = i % nstages;
                if (!ptx::mbar_wait(bar(K_EMPTY + s), ((i / nstages) & 1) ^ 1, abort_flag, kErrDecode | 1)) break;
                ptx::mbar_arrive_expect_tx(bar(K_FULL + s), G::TILE_BYTES);
                ptx::tma_load_3d(ptx::smem_u32(sK + (size_t)s * G::TILE_BYTES), &tmK, bar(K_FULL + s), h * DR - off,
                                 (t_begin + i) * kTile, b);
            }
        }
    } else if (warp < kFirstSoftmaxWarp) {
        const int g = warp - kFirstIssuerWarp;                  // the group this warp issues MMAs for
        if (lane == 0 && g < nbuf * cs) {
            // One issuing thread per group: the scores of the group's next tile as soon as its K tile has landed and
            // its buffer is drained, then the value contraction of each hand-over of weights as it arrives.
            const int j = g / cs, c = g % cs;
            const int len = decode_part_len(pl, M, c), hcols = decode_handover_cols(len, YC);
            const uint32_t idescY = ptx::instr_desc_bf16(128, YC, 0, 1);
            // Q rows of this range (K-major B operand of the score MMA); descriptor address fields are in 16-byte units
            const uint64_t qdesc = ptx::smem_desc(ptx::smem_u32(sQ), 16, G::SBO, G::SWZ) + (uint64_t)((c * pl.part_w * G::RB) >> 4);
            // Z rows of this range as the MN-major B operand: 8-row groups SBO apart; in the wide form the lo half is
            // the second block along N, M rows further on
            const uint64_t zdesc = ptx::smem_desc(ptx::smem_u32(sZ), kWide ? (uint32_t)(M * G::RB) : (uint32_t)G::SBO,
                                                  G::SBO, G::SWZ) + (uint64_t)((c * pl.part_w * G::RB) >> 4);
            const uint32_t sbuf = tm + j * cb + c * pl.part_w;  // the range's scores / packed weights
            const uint32_t dcol = tm + j * cb + y_col(c);
            bool ok = ptx::mbar_wait(bar(Q_FULL), 0, abort_flag, kErrDecode | 2);
            for (int i = j, u = 0; ok && i < ntiles; i += nbuf, ++u) {
                const int s = i % nstages;
                if (!ptx::mbar_wait(bar(K_FULL + s), (i / nstages) & 1, abort_flag, kErrDecode | 3)) break;
                if (!ptx::mbar_wait(bar(BUF_EMPTY + j), (u & 1) ^ 1, abort_flag, kErrDecode | 4)) break;
                ptx::tc_fence_after();
                const uint64_t kdesc = ptx::smem_desc(ptx::smem_u32(sK + (size_t)s * G::TILE_BYTES), 16, G::SBO, G::SWZ);
                for (int n0 = 0; n0 < len; n0 += 256) {         // S[:, range] = K_tile Q_range^T, N <= 256 per MMA
                    const int nn = len - n0 < 256 ? len - n0 : 256;
                    const uint32_t idescS = ptx::instr_desc_bf16(128, nn, 0, 0);
                    const uint64_t qd = qdesc + (uint64_t)((n0 * G::RB) >> 4);
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) ptx::mma_ss(sbuf + n0, kdesc + 2 * k, qd + 2 * k, idescS, k > 0);
                }
                ptx::mma_commit(bar(S_FULL + g));
                ptx::mma_commit(bar(K_EMPTY + s));              // one arrival per range: the K tile is free after the last
                for (int top = len, ho = 0; ok && top > 0; ++ho) {   // hand-overs go from the top column down
                    if (!ptx::mbar_wait(bar(P_CHUNK + 4 * g + ho), u & 1, abort_flag, kErrDecode | 5)) { ok = false; break; }
                    ptx::tc_fence_after();
                    const int bottom = top - hcols > 0 ? top - hcols : 0;
                    while (top > bottom) {                      // chunks of 32 score columns (a last one of 16)
                        const int w = top - bottom >= 32 ? 32 : 16, lo = top - w;
                        const uint32_t acol = sbuf + decode_p_col(len, YC, lo, pl.alias != 0);
                        for (int sub = 0; sub < w / 16; ++sub) {    // 16 latents: 8 packed columns, 16 rows of Z
                            const uint64_t bd = zdesc + (uint64_t)(((lo + 16 * sub) * G::RB) >> 4);
                            ptx::mma_ts(dcol, acol + sub * 8, bd, idescY, (top == len && sub == 0) ? 0u : 1u);
                            if (!kWide) ptx::mma_ts(dcol, acol + sub * 8, bd + (uint64_t)((M * G::RB) >> 4), idescY, 1u);
                        }
                        top = lo;
                    }
                }
                if (ok) ptx::mma_commit(bar(Y_FULL + g));
            }
        }
    } else if (warp - kFirstSoftmaxWarp < 4 * nbuf * cs) {
        const int g = (warp - kFirstSoftmaxWarp) >> 2;          // softmax group
        const int j = g / cs, c = g % cs;                       // its buffer and column range
        const int row = ((warp & 3) << 5) + lane;               // TMEM lane = token within the tile
        const uint32_t lane_addr = (uint32_t)((warp & 3) << 5) << 16;
        const uint32_t buf = tm + lane_addr + j * cb;
        const int len = decode_part_len(pl, M, c);
        const int hcols = decode_handover_cols(len, YC);
        const bool alias = pl.alias != 0;
        const uint32_t sbase = buf + c * pl.part_w;             // own scores, and own packed weights over them
        const float2 sl2p = make_float2(a.sl2, a.sl2);
        float *my_m = stat_m + g * kTile + row, *my_l = stat_l + g * kTile + row;
        for (int i = j, u = 0; i < ntiles; i += nbuf, ++u) {
            if (!warp_wait(bar(S_FULL + g), u & 1, abort_flag, kErrDecode | 6)) break;
            ptx::tc_fence_after();
            uint32_t r[32];
            float mx = -INFINITY;
            int col = 0;
            for (; col + 32 <= len; col += 32) {                // pass 1: row maximum over the range
                ptx::tmem_ld32(sbase + col, r);
                ptx::tmem_wait_ld();
                mx = max_of<32>(r, mx);
            }
            if (col < len) {
                ptx::tmem_ld16(sbase + col, r);
                ptx::tmem_wait_ld();
                mx = max_of<16>(r, mx);
            }
            const float neg = -mx * a.sl2;
            const float2 negp = make_float2(neg, neg);
            float2 sum2 = make_float2(0.f, 0.f);
            uint32_t pk[16];
            // pass 2, from the top column down: exponentials, bf16 pairs into columns already read (see
            // decode_p_col); every `hcols` score columns are handed to the value contraction
            for (int hi = len, ho = 0; hi > 0; ++ho) {
                const int bottom = hi - hcols > 0 ? hi - hcols : 0;
                for (int top = hi; top > bottom;) {
                    if (top - bottom >= 32) {
                        const int lo = top - 32;
                        ptx::tmem_ld32(sbase + lo, r);
                        ptx::tmem_wait_ld();
                        exp_chunk<32, false>(r, pk, sl2p, negp, sum2);
                        ptx::tmem_st16(sbase + decode_p_col(len, YC, lo, alias), pk);
                        top = lo;
                    } else {
                        const int lo = top - 16;
                        ptx::tmem_ld16(sbase + lo, r);
                        ptx::tmem_wait_ld();
                        exp_chunk<16, false>(r, pk, sl2p, negp, sum2);
                        ptx::tmem_st8(sbase + decode_p_col(len, YC, lo, alias), pk);
                        top = lo;
                    }
                }
                if (bottom == 0 && cs > 1) {                    // statistics travel with the last hand-over
                    *my_m = mx * a.sl2;
                    *my_l = sum2.x + sum2.y;
                }
                ptx::tmem_wait_st();
                ptx::tc_fence_before();
                ptx::mbar_arrive(bar(P_CHUNK + 4 * g + ho));
                hi = bottom;
            }
            const float sum = sum2.x + sum2.y;
            if (u % cs != c) continue;                          // the ranges take turns writing the tile's rows
            // every range's statistics are in shared memory once its threads have arrived on its last hand-over,
            // and its Y accumulator is complete once its Y_FULL has fired
            bool all = true;
            for (int cc = 0; cc < cs && all; ++cc) {
                const int gg = j * cs + cc, lcc = decode_part_len(pl, M, cc);
                const int last = (lcc + decode_handover_cols(lcc, YC) - 1) / decode_handover_cols(lcc, YC) - 1;
                all = warp_wait(bar(P_CHUNK + 4 * gg + last), u & 1, abort_flag, kErrDecode | 8) &&
                      warp_wait(bar(Y_FULL + gg), u & 1, abort_flag, kErrDecode | 7);
            }
            if (!all) break;
            ptx::tc_fence_after();
            // merge the ranges: weights 2^(m_c - m), total sum l
            float mtot = mx * a.sl2, ltot = sum, wgt[4] = {1.f, 1.f, 1.f, 1.f};
            if (cs > 1) {
                float mc[4], lc[4];
                mtot = -INFINITY;
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    mc[cc] = cc < cs ? stat_m[(j * cs + cc) * kTile + row] : -INFINITY;
                    lc[cc] = cc < cs ? stat_l[(j * cs + cc) * kTile + row] : 0.f;
                    mtot = fmaxf(mtot, mc[cc]);
                }
                ltot = 0.f;
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    wgt[cc] = ptx::ex2(mc[cc] - mtot);
                    ltot = fmaf(wgt[cc], lc[cc], ltot);
                }
            }
            const float inv = 1.f / ltot;
            const int n = (t_begin + i) * kTile + row;
            uint4 *dst = reinterpret_cast<uint4 *>(a.Y + (((size_t)b * a.N + (n < a.N ? n : 0)) * a.H + h) * DR);
#pragma unroll
            for (int dc = 0; dc < D / 16; ++dc) {
                float y[16];
                uint32_t t[16];
#pragma unroll
                for (int k = 0; k < 16; ++k) y[k] = 0.f;
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    if (cc < cs) {
#pragma unroll
                        for (int half = 0; half < (kWide ? 2 : 1); ++half) {   // wide form: hi and lo products
                            ptx::tmem_ld16(buf + y_col(cc) + half * D + dc * 16, t);
                            ptx::tmem_wait_ld();
#pragma unroll
                            for (int k = 0; k < 16; ++k) y[k] = fmaf(__uint_as_float(t[k]), wgt[cc], y[k]);
                        }
                    }
                }
                if (kPart) {                                    // a range of the latents: float32 rows for the combine kernel
                    if (n < a.N) {
                        float4 *pd = reinterpret_cast<float4 *>(a.Ypart + (((size_t)b * a.N + n) * a.H + h) * DR + dc * 16);
                        if (DR == 4) {
                            pd[0] = make_float4((off ? y[4] : y[0]) * inv, (off ? y[5] : y[1]) * inv,
                                                (off ? y[6] : y[2]) * inv, (off ? y[7] : y[3]) * inv);
                        } else {
#pragma unroll
                            for (int k = 0; k < (DR < 16 ? DR : 16) / 4; ++k)
                                pd[k] = make_float4(y[4 * k] * inv, y[4 * k + 1] * inv, y[4 * k + 2] * inv, y[4 * k + 3] * inv);
                        }
                    }
                } else if (DR == 4) {
                    if (n < a.N)
                        *reinterpret_cast<uint2 *>(dst) =
                            make_uint2(ptx::pack_bf16((off ? y[4] : y[0]) * inv, (off ? y[5] : y[1]) * inv),
                                       ptx::pack_bf16((off ? y[6] : y[2]) * inv, (off ? y[7] : y[3]) * inv));
                } else if (n < a.N) {
                    dst[2 * dc] = make_uint4(ptx::pack_bf16(y[0] * inv, y[1] * inv), ptx::pack_bf16(y[2] * inv, y[3] * inv),
                                             ptx::pack_bf16(y[4] * inv, y[5] * inv), ptx::pack_bf16(y[6] * inv, y[7] * inv));
                    if (DR > 8 + 16 * dc)
                        dst[2 * dc + 1] =
                            make_uint4(ptx::pack_bf16(y[8] * inv, y[9] * inv), ptx::pack_bf16(y[10] * inv, y[11] * inv),
                                       ptx::pack_bf16(y[12] * inv, y[13] * inv), ptx::pack_bf16(y[14] * inv, y[15] * inv));
                }
            }
            ptx::tc_fence_before();
            ptx::mbar_arrive(bar(BUF_EMPTY + j));
            if (n < a.N && a.lse_dec != nullptr)
                a.lse_dec[((size_t)b * a.N + n) * a.H + h] = (mtot + log2f(ltot)) * 0.6931471805599453f;
        }
    }
    // teardown: everyone arrives here (waits are bounded), then the allocating warp frees tensor memory
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == kFirstIssuerWarp) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tm, (uint32_t)pl.ncols);
    }
    if (threadIdx.x == 0 && *abort_flag != 0 && a.status != nullptr) atomicCAS(a.status, 0u, *abort_flag);
}

// ------------------------------------------------------------------------------------- decode, streaming form
// Decode without a row maximum (see kFastMaxLog2) needs no whole row of scores before the first exponential, so
// it can run as a stream like encode: a group owns a whole token tile (tokens on the 128 lanes; the four groups of
// a CTA work on four different tiles) and walks the latents in units of 32 columns on two alternating score
// buffers:  S_unit = K_tile Q_unit^T,  P = 2^(S sl2) as packed bf16 back over the scores,
// Y += P [Z_hi | Z_lo | 1]_unit.  Units follow one another across tile boundaries without a pause: the rows of a
// finished tile are normalised and stored after the first unit of the next one.  The accumulator column after
// [P Z_hi | P Z_lo] is the row's sum of rounded weights (see exp_chunk_fast).  D = 32: Z_lo enters as a second,
// accumulating MMA into the columns of Z_hi, which keeps the accumulator at 48 columns.
//
// What shapes the pipeline (measured on B200): the thread that issues a tcgen05.mma or a tcgen05.commit is held
// about 130 cycles per instruction, a barrier flips 170 cycles after its commit was issued, and a waiting warp
// notices 100 to 200 cycles later.  A group's issuing thread is therefore its bottleneck as soon as it has more
// than a handful of such instructions per unit (with separate commits and waits for scores and weights: 1300
// cycles per unit, measured with the arithmetic taken out).  Its loop is: wait for the weights of unit n; the
// two value MMAs of unit n; the score MMA of unit n + 2 into the buffer those weights have just been read from
// (the tensor core runs a thread's MMAs in order); ONE commit, which tells the threads both that the scores of
// unit n + 2 are there and that everything before them is done.
template <int D>
struct DecodeStreamSmem {
    using G = TileGeom<D>;
    static constexpr size_t kBarBytes = 1024;
    __host__ __device__ static int stages(int M) {
        int s = 8;
        while (s > 4 && (size_t)s * G::TILE_BYTES + (size_t)4 * M * G::RB + kBarBytes + 2048 > 227 * 1024) --s;
        return s;
    }
    __host__ __device__ static size_t q_off(int M) { return (size_t)stages(M) * G::TILE_BYTES; }
    __host__ __device__ static size_t z_off(int M) { return q_off(M) + (size_t)M * G::RB; }      // [hi | lo | ones], M rows each
    __host__ __device__ static size_t bar_off(int M) { return align_up(z_off(M) + (size_t)3 * M * G::RB, 1024); }
    __host__ __device__ static size_t total(int M) {
        size_t t = bar_off(M) + kBarBytes + 1024;
        return t < kTcMinSmem ? kTcMinSmem : t;
    }
    __host__ __device__ static bool fits(int M) { return bar_off(M) + kBarBytes + 1024 <= 227 * 1024; }
};

// kM: 0, or the number of latents of the launch as a compile-time constant (a multiple of 64): the unit loops are
// then unrolled and every descriptor offset, buffer index and barrier parity within a tile is a constant, which
// matters most for the issuing thread (its scalar instructions wait for issue slots among the softmax warps).
// kLse: the log-sum-exp rows are wanted (lse_dec; always with kPart): the threads then also add up the unrounded weights.
template <int D, int DRT = 0, bool kPart = false, int kM = 0, bool kLse = false>
__global__ void __launch_bounds__(kTcThreadsGuarded, 1)
decode_stream_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ, DecodeTcArgs a) {
    static_assert(D == 16 || D == 32, "head widths 16 (and narrower, as part of 16) and 32");
    constexpr bool kHalf = DRT != 0;
    constexpr int DR = kHalf ? DRT : D;                         // head width in memory
    using G = TileGeom<D>;
    using SM = DecodeStreamSmem<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    static_assert(kM % 64 == 0, "compile-time latent counts are multiples of 64");
    const int M = kM ? kM : a.M;
    const int nstages = SM::stages(M);
    uint8_t *sK = smem;
    uint8_t *sQ = smem + SM::q_off(M);
    uint8_t *sZ = smem + SM::z_off(M);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + SM::bar_off(M));
    constexpr int NG = kSoftmaxGroups, kMaxStages = 8, UNIT = 32;
    // S_FULL[2] per group: the scores of a unit are in its buffer (and all earlier MMAs of the group are done);
    // P_FULL[2]: the unit's weights are over them (one arrival per warp); Y_FULL / Y_FREE: a tile's rows are complete / read
    enum { K_FULL = 0, K_EMPTY = K_FULL + kMaxStages, Q_FULL = K_EMPTY + kMaxStages, S_FULL = Q_FULL + 1,
           P_FULL = S_FULL + 2 * NG, Y_FULL = P_FULL + 2 * NG, Y_FREE = Y_FULL + NG, NBARS = Y_FREE + NG };
    static_assert(NBARS * 8 + 16 <= SM::kBarBytes, "barrier area too small");
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + NBARS);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    constexpr int Y_COL = 2 * UNIT, GROUP_COLS = 128;          // a group's columns: two score buffers, then 48 of Y
    constexpr int YN = 48;                                      // N of the value MMA that carries the ones block
    constexpr int SUM_COL = 32;                                 // accumulator column of the row sum

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tid = threadIdx.x < kTcThreads ? (int)threadIdx.x : (1 << 30);   // the guard warps stage nothing
    const int h = blockIdx.y, b = blockIdx.z;
    const int off = kHalf ? narrow_offset(h, DR) : 0;
    const int t_begin = (int)((long)a.tiles * blockIdx.x / gridDim.x);
    const int t_end = (int)((long)a.tiles * (blockIdx.x + 1) / gridDim.x);
    const int ntiles = t_end - t_begin;
    const int units = (M + UNIT - 1) / UNIT;                    // per tile; the last may have 16 columns
    auto bar = [&](int i) { return ptx::smem_u32(bars + i); };

    if (threadIdx.x == 0) {
        for (int i = 0; i < NBARS; ++i) {
            const bool by_warps = (i >= P_FULL && i < P_FULL + 2 * NG) || (i >= Y_FREE && i < Y_FREE + NG);
            const bool guarded = i >= K_EMPTY && i < K_EMPTY + kMaxStages;     // released by its group and its guard warp
            ptx::mbar_init(bar(i), by_warps ? 4u : guarded ? 2u : 1u);
        }
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmK);
        ptx::prefetch_tensormap(&tmQ);
    }
    if (warp == kFirstIssuerWarp) ptx::tmem_alloc(ptx::smem_u32(tmem_slot), 512);
    {   // Z_bh -> [hi | lo | ones] blocks of M latent-major rows in the swizzled layout of an MN-major B operand
        const float *Zg = a.Z + (((size_t)b * a.H + h) * a.mtot + a.m0) * DR;
        if (kHalf) {
            for (int i = tid; i < M * (D / 8); i += kTcThreads) {
                reinterpret_cast<uint4 *>(sQ)[i] = make_uint4(0, 0, 0, 0);
                reinterpret_cast<uint4 *>(sZ)[i] = make_uint4(0, 0, 0, 0);
                reinterpret_cast<uint4 *>(sZ + (size_t)M * G::RB)[i] = make_uint4(0, 0, 0, 0);
            }
            __syncthreads();
            if constexpr (DR == 4) {
                stage_rows4<D>(sQ, a.Q + ((size_t)h * a.mtot + a.m0) * DR, M, off);
                stage_rows4_hilo<D>(sZ, sZ + (size_t)M * G::RB, Zg, M, off);
            } else {
                for (int i = tid; i < M * (DR / 8); i += kTcThreads) {
                    const int m = i / (DR / 8), c = i % (DR / 8);
                    *reinterpret_cast<uint4 *>(sQ + (size_t)m * G::RB + ((c ^ G::swz(m)) << 4)) =
                        *reinterpret_cast<const uint4 *>(a.Q + ((size_t)h * a.mtot + a.m0 + m) * DR + c * 8);
                }
            }
        }
        constexpr int ZC = DR >= 8 ? DR / 8 : 1;
        for (int i = tid; i < (DR >= 8 ? M * ZC : 0); i += kTcThreads) {
            const int m = i / ZC, c = i % ZC;
            const float4 lo = *reinterpret_cast<const float4 *>(Zg + (size_t)m * DR + c * 8);
            const float4 hi = *reinterpret_cast<const float4 *>(Zg + (size_t)m * DR + c * 8 + 4);
            const float z[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
            uint32_t vh[4], vl[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                vh[k] = ptx::pack_bf16(z[2 * k], z[2 * k + 1]);
                vl[k] = ptx::pack_bf16(z[2 * k] - __uint_as_float(vh[k] << 16), z[2 * k + 1] - __uint_as_float(vh[k] & 0xffff0000u));
            }
            uint8_t *dst = sZ + (size_t)m * G::RB + ((c ^ G::swz(m)) << 4);
            *reinterpret_cast<uint4 *>(dst) = make_uint4(vh[0], vh[1], vh[2], vh[3]);
            *reinterpret_cast<uint4 *>(dst + (size_t)M * G::RB) = make_uint4(vl[0], vl[1], vl[2], vl[3]);
        }
        uint8_t *ones = sZ + (size_t)2 * M * G::RB;             // a one in column 0 of every latent row
        for (int i = tid; i < M * (G::RB / 16); i += kTcThreads) {
            const int m = i / (G::RB / 16), c = i % (G::RB / 16);
            *reinterpret_cast<uint4 *>(ones + (size_t)m * G::RB + ((c ^ G::swz(m)) << 4)) = make_uint4(c == 0 ? 0x00003F80u : 0u, 0, 0, 0);
        }
        ptx::fence_proxy_async_smem();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tm = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            if (kHalf) {
                ptx::mbar_arrive(bar(Q_FULL));
            } else {
                ptx::mbar_arrive_expect_tx(bar(Q_FULL), (uint32_t)(M * G::RB));
                for (int r = 0; r < M; r += 16)
                    ptx::tma_load_2d(ptx::smem_u32(sQ + (size_t)r * G::RB), &tmQ, bar(Q_FULL), 0, h * a.mtot + a.m0 + r);
            }
        }
        for (int i = 0; i < ntiles; ++i) {
            const int s = i % nstages;
            if (!warp_wait(bar(K_EMPTY + s), ((i / nstages) & 1) ^ 1, abort_flag, kErrDecode | 1)) break;
            if (lane == 0) {
                ptx::mbar_arrive_expect_tx(bar(K_FULL + s), G::TILE_BYTES);
                ptx::tma_load_3d(ptx::smem_u32(sK + (size_t)s * G::TILE_BYTES), &tmK, bar(K_FULL + s), h * DR - off,
                                 (t_begin + i) * kTile, b);
            }
        }
    } else if (warp >= kFirstGuardWarp) {
        // Guard warps, one tile in three each: |q| |k| sl2 <= kFastMaxLog2 for every latent row of the launch and every
        // key row of the tile, checked while the tile sits in its stage (whole rows: in the narrow forms they hold the
        // neighbouring heads' features too, which only makes the check stricter).
        bool tame = warp_wait(bar(Q_FULL), 0, abort_flag, kErrDecode | 9);
        const float q2 = warp_max_nan(tile_max_norm2<G::RB>(sQ, M, lane));
        const float lim = kFastMaxLog2 / a.sl2;
        const float k2_limit = lim * lim / fmaxf(q2, 1e-30f);
        if (!(q2 <= 3.0e38f)) tame = false;
        for (int j = warp - kFirstGuardWarp; j < ntiles; j += kGuardWarps) {
            const int sj = j % nstages;
            if (!warp_wait(bar(K_FULL + sj), (j / nstages) & 1, abort_flag, kErrDecode | 10)) break;
            const float k2 = warp_max_nan(tile_max_norm2<G::RB>(sK + (size_t)sj * G::TILE_BYTES, kTile, lane));
            if (!(k2 <= k2_limit)) tame = false;
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar(K_EMPTY + sj));
        }
        if (!tame && lane == 0 && a.redo != nullptr) *a.redo = 1u;
    } else if (warp < kFirstSoftmaxWarp) {
        const int g = warp - kFirstIssuerWarp;
        const int mytiles = (ntiles - g + NG - 1) / NG;          // tiles g, g + 4, ... of the CTA's range
        if (lane == 0 && mytiles > 0) {
            const uint32_t gcol = tm + g * GROUP_COLS;
            const uint32_t idescY = ptx::instr_desc_bf16(128, YN, 0, 1);
            const uint32_t idescLo = ptx::instr_desc_bf16(128, D, 0, 1);       // D = 32: the accumulating Z_lo product
            const uint64_t qdesc = ptx::smem_desc(ptx::smem_u32(sQ), 16, G::SBO, G::SWZ);
            // value operand: Z_hi rows of the unit; next block along N: Z_lo (D = 16, then the ones block) or the ones
            // block (D = 32), LBO bytes further on
            const uint64_t zdesc = ptx::smem_desc(ptx::smem_u32(sZ), (uint32_t)((D == 16 ? 1 : 2) * M * G::RB), G::SBO, G::SWZ);
            const uint64_t zlo = ptx::smem_desc(ptx::smem_u32(sZ + (size_t)M * G::RB), (uint32_t)G::SBO, G::SBO, G::SWZ);
            const int total = mytiles * units;
            bool ok = ptx::mbar_wait(bar(Q_FULL), 0, abort_flag, kErrDecode | 2);
            const uint32_t kstep = (uint32_t)(G::TILE_BYTES >> 4);
            const uint64_t kdesc0 = ptx::smem_desc(ptx::smem_u32(sK), 16, G::SBO, G::SWZ);
            if constexpr (kM != 0) {
                // Unrolled over the tile's units: unit c of every tile uses buffer c & 1 (the number of units is even),
                // so within a tile every buffer, descriptor offset and barrier parity is a constant.
                constexpr int U = kM / UNIT;
                constexpr uint32_t idescS = ptx::instr_desc_bf16(128, UNIT, 0, 0);
                const uint32_t sfull = bar(S_FULL + 2 * g), pfull = bar(P_FULL + 2 * g);
                int stage = g % nstages, wrap = 0;               // K stage of the tile whose scores are issued next, and its phase
                uint64_t kdesc = 0;
                auto scores = [&](int c) {                        // S of unit c (a constant after unrolling) of the tile at kdesc, and the commit
#pragma unroll
                    for (int k = 0; k < D / 16; ++k)
                        ptx::mma_ss(gcol + (c & 1) * UNIT, kdesc + 2 * k, qdesc + (uint64_t)((c * UNIT * G::RB) >> 4) + 2 * k, idescS, k > 0);
                    ptx::mma_commit(sfull + 8 * (c & 1));
                };
                auto open_tile = [&]() -> bool {                  // wait for the K tile of the S stream's next tile
                    if (!ptx::mbar_wait(bar(K_FULL + stage), (uint32_t)wrap, abort_flag, kErrDecode | 3)) return false;
                    ptx::tc_fence_after();
                    kdesc = kdesc0 + (uint64_t)(kstep * (uint32_t)stage);
                    return true;
                };
                auto close_tile = [&]() {                         // its last scores are issued: the stage is free, on to the next tile
                    ptx::mma_commit(bar(K_EMPTY + stage));
                    stage += NG;
                    if (stage >= nstages) { stage -= nstages; wrap ^= 1; }
                };
                ok = ok && open_tile();
                if (ok) {
                    scores(0);
                    scores(1);
                    if (U == 2) close_tile();
                }
                for (int tu = 0; ok && tu < mytiles; ++tu) {
                    const uint32_t par = (uint32_t)((tu * (U / 2)) & 1);    // parity of the tile's first two units on their buffers
                    const bool more = tu + 1 < mytiles;
#pragma unroll
                    for (int c = 0; c < U; ++c) {
                        if (!ptx::mbar_spin(pfull + 8 * (c & 1), par ^ (uint32_t)((c >> 1) & 1), abort_flag, kErrDecode | 5)) { ok = false; break; }
                        if (c == 0 && tu > 0 && !ptx::mbar_spin(bar(Y_FREE + g), (uint32_t)((tu - 1) & 1), abort_flag, kErrDecode | 11)) { ok = false; break; }
                        ptx::tc_fence_after();
                        const uint32_t pcol = gcol + (c & 1) * UNIT;
                        const uint64_t zr = zdesc + (uint64_t)((c * UNIT * G::RB) >> 4), zl = zlo + (uint64_t)((c * UNIT * G::RB) >> 4);
                        ptx::mma_ts(gcol + Y_COL, pcol, zr, idescY, c == 0 ? 0u : 1u);
                        if (D == 32) ptx::mma_ts(gcol + Y_COL, pcol, zl, idescLo, 1u);
                        ptx::mma_ts(gcol + Y_COL, pcol + 8, zr + (uint64_t)(G::RB), idescY, 1u);
                        if (D == 32) ptx::mma_ts(gcol + Y_COL, pcol + 8, zl + (uint64_t)(G::RB), idescLo, 1u);
                        if (c == U - 1) ptx::mma_commit(bar(Y_FULL + g));
                        // the scores of the unit two further on go into the buffer just read; the commit behind them covers
                        // the value MMAs above as well
                        if (c + 2 < U) {
                            scores(c + 2);
                            if (c + 2 == U - 1) close_tile();
                        } else if (more) {
                            if (c + 2 == U && !open_tile()) { ok = false; break; }
                            scores(c + 2 - U);
                            if (c + 2 - U == U - 1) close_tile();
                        }
                    }
                }
            } else {
                // This thread's own instructions are on the critical path of the group (they run one at a time, each
                // waiting for its issue slot among the softmax warps), so both streams of work below keep their
                // position in running counters instead of dividing: the score units (two ahead of the value units) ...
                int s_c = 0, s_stage = g % nstages, s_wrap = (g / nstages) & 1, s_n = 0;   // chunk, K stage and its phase, unit
                const int last_nn = M - (units - 1) * UNIT;
                const uint32_t idescS_full = ptx::instr_desc_bf16(128, UNIT, 0, 0), idescS_last = ptx::instr_desc_bf16(128, last_nn, 0, 0);
                auto issue_scores = [&]() -> bool {                   // (the caller commits)
                    if (s_c == 0) {
                        if (!ptx::mbar_wait(bar(K_FULL + s_stage), (uint32_t)s_wrap, abort_flag, kErrDecode | 3)) return false;
                        ptx::tc_fence_after();
                    }
                    const uint64_t kdesc = kdesc0 + (uint64_t)(kstep * (uint32_t)s_stage);
                    const uint64_t qd = qdesc + (uint64_t)((uint32_t)(s_c * UNIT * G::RB) >> 4);
                    const uint32_t idescS = s_c == units - 1 ? idescS_last : idescS_full;
                    const uint32_t w = (uint32_t)(s_n & 1);
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) ptx::mma_ss(gcol + w * UNIT, kdesc + 2 * k, qd + 2 * k, idescS, k > 0);
                    ptx::mma_commit(bar(S_FULL + 2 * g) + 8 * w);
                    ++s_n;
                    if (++s_c == units) {                           // the tile's last scores: its stage is free, on to the next tile
                        ptx::mma_commit(bar(K_EMPTY + s_stage));
                        s_c = 0;
                        s_stage += NG;
                        if (s_stage >= nstages) { s_stage -= nstages; s_wrap ^= 1; }
                    }
                    return true;
                };
                for (int n = 0; ok && n < 2 && n < total; ++n) ok = issue_scores();
                // ... and the value units
                int c = 0, tu = 0;
                for (int n = 0; ok && n < total; ++n) {
                    const uint32_t w = (uint32_t)(n & 1);           // the unit's buffer: its weights lie over its scores
                    if (!ptx::mbar_spin(bar(P_FULL + 2 * g) + 8 * w, (uint32_t)((n >> 1) & 1), abort_flag, kErrDecode | 5)) break;
                    // a tile's first value MMA overwrites the accumulator: the previous tile's rows must have been read
                    if (c == 0 && tu > 0 && !ptx::mbar_spin(bar(Y_FREE + g), (uint32_t)((tu - 1) & 1), abort_flag, kErrDecode | 11)) break;
                    ptx::tc_fence_after();
                    const int subs = (c == units - 1 ? last_nn : UNIT) / 16;
                    const uint64_t rowoff = (uint64_t)((uint32_t)(c * UNIT * G::RB) >> 4);
                    const uint32_t pcol = gcol + w * UNIT;
                    ptx::mma_ts(gcol + Y_COL, pcol, zdesc + rowoff, idescY, c == 0 ? 0u : 1u);
                    if (D == 32) ptx::mma_ts(gcol + Y_COL, pcol, zlo + rowoff, idescLo, 1u);
                    if (subs == 2) {                                // the unit's second 16 latents: 8 packed columns, 16 rows of Z on
                        ptx::mma_ts(gcol + Y_COL, pcol + 8, zdesc + rowoff + (uint64_t)(G::RB), idescY, 1u);
                        if (D == 32) ptx::mma_ts(gcol + Y_COL, pcol + 8, zlo + rowoff + (uint64_t)(G::RB), idescLo, 1u);
                    }
                    if (++c == units) {
                        ptx::mma_commit(bar(Y_FULL + g));
                        c = 0;
                        ++tu;
                    }
                    if (n + 2 < total && !(ok = issue_scores())) break;   // into the buffer just read; its commit covers the value MMAs too
                }
            }
        }
    } else {
        const int g = (warp - kFirstSoftmaxWarp) >> 2;
        const int mytiles = (ntiles - g + NG - 1) / NG;
        const int row = ((warp & 3) << 5) + lane;               // TMEM lane = token within the tile
        const uint32_t gcol = tm + ((uint32_t)((warp & 3) << 5) << 16) + g * GROUP_COLS;
        const float2 sl2p = make_float2(a.sl2, a.sl2);
        float2 sum2 = make_float2(0.f, 0.f);                    // kLse: the tile's row sum of unrounded weights so far
        float l_exact = 0.f;                                    // ... and that of the tile whose rows are still to be written
        constexpr int kSum = kLse ? 2 : 0;
        // normalise and store the rows of tile tu (this group's tu-th), whose value MMAs are all issued
        auto epilogue = [&](int tu) -> bool {
            if (!warp_wait(bar(Y_FULL + g), tu & 1, abort_flag, kErrDecode | 7)) return false;
            ptx::tc_fence_after();
            uint32_t y[48];
            ptx::tmem_ld32(gcol + Y_COL, *reinterpret_cast<uint32_t(*)[32]>(y));
            ptx::tmem_ld16(gcol + Y_COL + 32, y + 32);
            ptx::tmem_wait_ld();
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar(Y_FREE + g));    // the accumulator may be overwritten
            const float l = __uint_as_float(y[SUM_COL]);
            const float inv = 1.f / l;
            const int n = (t_begin + g + tu * NG) * kTile + row;
            if (n < a.N) {
                // the head's DR values: accumulator columns [off, off + DR) (off is 0 except for every other head of width 4)
                float v[DR];
#pragma unroll
                for (int k = 0; k < DR; ++k) {
                    if (D == 16) {
                        const float a0 = __uint_as_float(y[k]) + __uint_as_float(y[16 + k]);
                        const float a4 = DR == 4 ? __uint_as_float(y[4 + k]) + __uint_as_float(y[20 + k]) : a0;
                        v[k] = ((DR == 4 && off) ? a4 : a0) * inv;
                    } else {
                        v[k] = __uint_as_float(y[k]) * inv;
                    }
                }
                const size_t rowidx = ((size_t)b * a.N + n) * a.H + h;
                if (kPart) {
                    float4 *pd = reinterpret_cast<float4 *>(a.Ypart + rowidx * DR);
#pragma unroll
                    for (int k = 0; k < DR / 4; ++k) pd[k] = make_float4(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]);
                } else if (DR == 4) {
                    *reinterpret_cast<uint2 *>(a.Y + rowidx * DR) = make_uint2(ptx::pack_bf16(v[0], v[1]), ptx::pack_bf16(v[2], v[3]));
                } else {
                    uint4 *dst = reinterpret_cast<uint4 *>(a.Y + rowidx * DR);
#pragma unroll
                    for (int k = 0; k < DR / 8; ++k)
                        dst[k] = make_uint4(ptx::pack_bf16(v[8 * k], v[8 * k + 1]), ptx::pack_bf16(v[8 * k + 2], v[8 * k + 3]),
                                            ptx::pack_bf16(v[8 * k + 4], v[8 * k + 5]), ptx::pack_bf16(v[8 * k + 6], v[8 * k + 7]));
                }
                if (kLse) a.lse_dec[rowidx] = log2f(l_exact) * 0.6931471805599453f;
            }
            return true;
        };
        bool ok = true;
        int n = 0;                                              // unit counter of this group's stream
        const int total = mytiles * units;
        // A wait on a barrier costs a warp about 150 cycles even when the phase is long complete, and the warp has
        // nothing else to do meanwhile.  So the wait for the next unit's scores is asked early, without blocking,
        // before the exponentials of this unit, and falls back to a blocking wait only if the answer was no.
        bool s_ready = false;
        for (int tu = 0; ok && tu < mytiles; ++tu) {
            for (int c = 0; ok && c < units; ++c, ++n) {
                const int w = n & 1;
                const int nn = kM ? UNIT : (M - c * UNIT < UNIT ? M - c * UNIT : UNIT);
                if (!s_ready && !(ok = warp_wait(bar(S_FULL + 2 * g + w), (n >> 1) & 1, abort_flag, kErrDecode | 6))) break;
                ptx::tc_fence_after();
                uint32_t r[32], pk[16];
                if (nn == UNIT) ptx::tmem_ld32(gcol + w * UNIT, r);
                else ptx::tmem_ld16(gcol + w * UNIT, r);
                ptx::tmem_wait_ld();
                bool s_probe = false;
                if (nn == UNIT) {
                    exp_chunk_fast<16, true, false, kSum>(r, pk, sl2p, sum2);
                    s_probe = n + 1 < total && ptx::mbar_test(bar(S_FULL + 2 * g + (w ^ 1)), ((n + 1) >> 1) & 1);
                    exp_chunk_fast<16, true, false, kSum>(r + 16, pk + 8, sl2p, sum2);
                    ptx::tmem_st16(gcol + w * UNIT, pk);
                } else {
                    exp_chunk_fast<16, true, false, kSum>(r, pk, sl2p, sum2);
                    ptx::tmem_st8(gcol + w * UNIT, pk);
                }
                ptx::tmem_wait_st();
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(bar(P_FULL + 2 * g + w));
                s_ready = __all_sync(0xffffffffu, s_probe);
                // the previous tile's rows, while the tensor core works on this unit
                if (c == 0 && tu > 0) ok = epilogue(tu - 1);
                if (kLse && c == units - 1) {                   // the tile's sum is complete; the next tile starts its own
                    l_exact = sum2.x + sum2.y;
                    sum2 = make_float2(0.f, 0.f);
                }
            }
        }
        if (ok && mytiles > 0) epilogue(mytiles - 1);
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == kFirstIssuerWarp) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tm, 512);
    }
    if (threadIdx.x == 0 && *abort_flag != 0 && a.status != nullptr) atomicCAS(a.status, 0u, *abort_flag);
}

// Decode over more latents than one launch holds: every launch decodes a range of the latents into float32 rows
// normalised over that range (Ypart[c]) with the range's log-sum-exp (lse_part[c]); this kernel joins the C ranges,
//   lse = log sum_c exp(lse_c),   Y = sum_c exp(lse_c - lse) Ypart[c],
// the same algebra as the split-N merge of the encode stage.  One thread per (token, head) row of DR elements.
template <int DR>
__global__ void __launch_bounds__(256)
decode_combine_kernel(const float *__restrict__ Ypart, const float *__restrict__ lse_part, int C, long rows,
                      __nv_bfloat16 *__restrict__ Y, float *__restrict__ lse_dec) {
    const long row = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= rows) return;
    float lc[8], mx = -INFINITY;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        lc[c] = c < C ? lse_part[(size_t)c * rows + row] : -INFINITY;
        mx = fmaxf(mx, lc[c]);
    }
    float w[8], sum = 0.f;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        w[c] = c < C ? expf(lc[c] - mx) : 0.f;
        sum += w[c];
    }
    const float inv = 1.f / sum;
    float y[DR];
#pragma unroll
    for (int k = 0; k < DR; ++k) y[k] = 0.f;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        if (c < C) {
            const float4 *src = reinterpret_cast<const float4 *>(Ypart + ((size_t)c * rows + row) * DR);
#pragma unroll
            for (int k = 0; k < DR / 4; ++k) {
                const float4 v = src[k];
                y[4 * k] = fmaf(w[c], v.x, y[4 * k]);
                y[4 * k + 1] = fmaf(w[c], v.y, y[4 * k + 1]);
                y[4 * k + 2] = fmaf(w[c], v.z, y[4 * k + 2]);
                y[4 * k + 3] = fmaf(w[c], v.w, y[4 * k + 3]);
            }
        }
    }
    uint32_t *dst = reinterpret_cast<uint32_t *>(Y + (size_t)row * DR);
#pragma unroll
    for (int k = 0; k < DR / 2; ++k) dst[k] = ptx::pack_bf16(y[2 * k] * inv, y[2 * k + 1] * inv);
    if (lse_dec != nullptr) lse_dec[row] = mx + logf(sum);
}

// ------------------------------------------------------------------------------------------------ encode

struct EncodeTcArgs {
    const __nv_bfloat16 *Q;   // [H,M,D] (read directly in the head-pair form)
    const float *lse_dec;     // [B,N,H]: only for the backward's dZ form of the kernel
    const uint8_t *key_mask;  // [B,N] or null
    float *part_m, *part_l, *part_acc;
    uint32_t *status;
    const uint32_t *run_if;   // exact forms: null, or a word that must be non-zero for the kernel to do anything
    uint32_t *redo;           // fast forms: set to 1 if a score may lie outside the range they are valid for
    int B, H, N, M;
    float scale, sl2;
    int tiles;        // ceil(N / 128)
    int splits;       // CTAs along N per (b, h, latent-block pair)
    int pairs;        // ceil(ceil(M/128) / 2)
    int partials_per_split;  // 4 when M <= 128 (two slots alternate tiles, two column halves each), else 2
};

// DG: columns of a K/V tile row as the kernel sees it (D, or 2D in the head-pair form).  kAlt: the CTA's two slots
// take alternate tiles (one latent block); the ring is then as deep as fits, at most kEncMaxStages.
template <int DG, bool kAlt>
struct EncodeSmem {
    using G = TileGeom<DG>;
    static constexpr size_t kColBytes = 4 * kSoftmaxGroups * 2 * 32 * sizeof(float);   // per softmax warp: 2 x 32 column addends
    // score bias of padded tokens: per stage a [128 tokens, 16] bf16 tile, then one [128 latents, 16] tile of ones
    static constexpr size_t kBiasTile = kTile * 32;
    // the tile of ones of the fast form exists only where its accumulator has room for the sum's column (DG + 16 <= 64)
    static constexpr size_t kOnesBytes = DG + 16 <= 64 ? (size_t)kTile * G::RB : 0;
    static constexpr size_t total_for(int n) {
        size_t t = (size_t)n * 2 * G::TILE_BYTES + (size_t)2 * kTile * G::RB + 512 + kColBytes;
        t = (t + 1023) & ~(size_t)1023;
        t = (t + (size_t)(n + 1) * kBiasTile + 1023) & ~(size_t)1023;
        return t + kOnesBytes + 1024;
    }
    static constexpr int stages_for() {
        int n = kAlt ? kEncMaxStages : kEncStages;
        while (n > kEncStages && total_for(n) > 227 * 1024) --n;
        return n;
    }
    static constexpr int kStages = stages_for();                // K+V tile pairs in flight
    static constexpr size_t kv_off = 0;                         // [stage][K tile | V tile]
    __host__ __device__ static size_t q_off() { return (size_t)kStages * 2 * G::TILE_BYTES; }
    __host__ __device__ static size_t bar_off() { return q_off() + (size_t)2 * kTile * G::RB; }
    __host__ __device__ static size_t col_off() { return bar_off() + 512; }
    __host__ __device__ static size_t bias_off() { return (col_off() + kColBytes + 1023) & ~(size_t)1023; }
    // fast form: a [128 tokens, DG] tile with a one in column 0 of every row, the value operand's second block along N
    __host__ __device__ static size_t ones_off() { return (bias_off() + (kStages + 1) * kBiasTile + 1023) & ~(size_t)1023; }
    __host__ __device__ static size_t total() {
        size_t t = ones_off() + kOnesBytes + 1024;
        return t < kTcMinSmem ? kTcMinSmem : t;
    }
};

// Padding in encode.  A token that takes no part in the softmax (masked, or beyond N in the last tile) gets the
// score kMaskedScore instead of a test per element: one more MMA k-step adds ones[latent] x bias[token] to the
// tile's scores, with bias = kMaskedScore or 0 (exactly representable, so the scores of valid tokens do not
// change).  Such a score never wins a maximum against a valid one and its weight 2^(score - max) is exactly 0.
// A row that has seen no valid token yet has a running maximum at or below kDeadBelow and is treated as empty.
constexpr float kMaskedScore = -1.0e30f;
constexpr float kDeadBelow = -1.0e29f;

// Encode, split over N.  grid = (splits, H * pairs, B).  A CTA owns up to two blocks of 128 latents of head h
// ("slots", one TMEM score buffer each) and a contiguous range of token tiles.  With M <= 128 the two slots
// share the one latent block and take alternate tiles.  Each slot is served by two softmax groups that split
// the tile's 128 token columns in halves; a half is a pipeline of its own, with its own issuing warp, running
// maximum, sum and accumulator, i.e. its own partial result for the merge kernel.  A half is worked off in
// units of 32 tokens on two alternating score buffers: while the group evaluates the exponentials of one
// unit, the score MMA of the next and the value MMAs of the previous one run, so that the group never waits
// for the tensor pipe in steady state.
//
// Head-pair form (kPair; M <= 64, H even, D <= 32): with at most 64 latents half of the 128 lanes would idle, so
// a CTA takes two adjacent heads at once.  Lanes 0-63 hold the latents of head 2p, lanes 64-127 those of head
// 2p+1; the A operand is the block-diagonal [Q_2p 0; 0 Q_2p+1] over the 2D feature columns the two heads occupy
// side by side in a token row, so one MMA with K = 2D gives every lane its own head's scores, and the value MMA
// with N = 2D gives lanes 0-63 their rows in accumulator columns [0, D) and lanes 64-127 theirs in [D, 2D).
//
// dZ form (kDz; pass A of the backward): the same kernel with dY in place of V and the decode weights in place of
// the encode weights, dZ_m = sum_n exp(S[m,n] - lse_dec[n]) dY_n.  Every column (token) carries its own shift
// and the weights are already normalised, so there is no running maximum, no rescaling and no sum; tokens
// beyond N get the shift -inf.  Every group leaves one partial sum of dZ per split (part_acc).
//
// Narrow form (DRT = 8 or 4 with D = 16; not with kPair): the head is DRT wide in memory, as in the decode kernel:
// K and V tile rows carry the neighbouring heads' features beside the head's own, Q rows zeros there; accumulator
// columns outside the head's (weights times the neighbours' values) are dropped.
//
// kHiLo: the weights go to the value contraction as two bf16 halves (see exp_chunk_hilo), as in the dZ form.
//
// kMaskBody: padded tokens are handled by a second form of the unit body that tests every element (the form for
// calls with a key mask, where every tile has padding); without it they are handled in the scores (kMaskedScore),
// which costs a bias tile and one more MMA per unit of the tiles that have padding, and nothing elsewhere.
//
// kFast: no running maximum (see kFastMaxLog2): weights 2^(s * sl2) as they stand, half of them by the polynomial
// on the FMA pipe (not with kHiLo, whose point is accuracy), no rescaling, partial maximum 0.  Three more warps
// (the guard warps) check the norms of the key rows of every tile against those of the CTA's latent rows; in the
// producer warp that check sat between two loads and cost 10 % at D = 32 (measured).
template <int D, bool kPair, bool kDz = false, int DRT = 0, bool kHiLo = false, bool kMaskBody = false, bool kFast = false, bool kAlt = kPair>
__global__ void __launch_bounds__(kFast ? kTcThreadsGuarded : kTcThreads, 1)
encode_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                 const __grid_constant__ CUtensorMap tmQ, EncodeTcArgs a) {
    static_assert(!(kFast && kDz), "the dZ form has no maximum to drop");
    if (!kFast && a.run_if != nullptr && *a.run_if == 0) return;      // the exact form as a fallback that was not needed
    constexpr bool kHalf = DRT != 0;
    static_assert(!(kPair && kHalf), "head pairing and the narrow form exclude each other");
    constexpr int DG = kPair ? 2 * D : D;
    constexpr int DR = kHalf ? DRT : D;                         // head width in memory
    using G = TileGeom<DG>;
    using SM = EncodeSmem<DG, kAlt>;
    static_assert(kAlt || !kPair, "head pairs share one latent block");
    constexpr int nstages = SM::kStages;                        // depth of the K/V ring
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *sKV = smem + SM::kv_off;
    uint8_t *sQ = smem + SM::q_off();
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + SM::bar_off());
    constexpr int NG = kSoftmaxGroups;
    // per group: S_FULL and P_FULL for each of its two score buffers, PV_DONE (one phase per unit), ACC_DONE
    enum { KV_FULL = 0, KV_EMPTY = KV_FULL + nstages, S_FULL = KV_EMPTY + nstages, P_FULL = S_FULL + 2 * NG,
           PV_DONE = P_FULL + 2 * NG, ACC_DONE = PV_DONE + NG, Q_FULL = ACC_DONE + NG, NBARS };
    static_assert(NBARS * 8 + 8 <= 512, "barrier area too small");
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + NBARS);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tid = threadIdx.x < kTcThreads ? (int)threadIdx.x : (1 << 30);   // the guard warps stage nothing
    const int M = a.M;
    // h: the head, or in the head-pair form the first head of the pair
    const int split = blockIdx.x, h = (kPair ? 2 : 1) * (blockIdx.y / a.pairs), pair = blockIdx.y % a.pairs, b = blockIdx.z;
    const int t_begin = (int)((long)a.tiles * split / a.splits);
    const int t_end = (int)((long)a.tiles * (split + 1) / a.splits);
    const int nt = t_end - t_begin;
    const int MB = (M + kTile - 1) / kTile;
    // job q -> (tile, slot); see the kernel comment
    // (the host picks the kAlt form for MB == 1; kept a run-time value in the other form, where it is always false: as
    // a compile-time constant the same kernel measured 3 % slower, 0.613 against 0.592 ms on the million-point shape)
    const bool alternate = kAlt || MB == 1;
    const int lb0 = pair * 2;                                   // latent block of slot 0
    const int nslots = alternate ? 2 : ((lb0 + 1 < MB) ? 2 : 1);
    const int nq = alternate ? nt : nt * nslots;
    const int rows_q = min(M - lb0 * kTile, 2 * kTile);                  // latent rows of this CTA
    const int off = kHalf ? narrow_offset(h, DR) : 0;                    // the head's first column within a tile row
    const int rows_here = (kPair || kHalf) ? 0 : rows_q;                 // ... fetched by TMA
    constexpr int SLOT_COLS = 256;   // per slot and half (128 columns): two score buffers of UNIT columns, accumulator at 64
    constexpr int HALF = kTile / 2;
    constexpr int UNIT = 32;         // tokens per unit of work of a group
    constexpr uint32_t NCOLS = 512;
    // Fast form with single weights: the value operand gets a second block along N whose column 0 is all ones, so
    // accumulator column DG is the sum of the rounded weights (see exp_chunk_fast); where the accumulator has no
    // room for it (DG = 64) the threads add the rounded weights themselves.
    constexpr bool kOnes = kFast && !kHiLo && DG + 16 <= 2 * UNIT;
    constexpr int kSumMode = kOnes ? 0 : 1;
    uint8_t *sOnes = smem + SM::ones_off();
    constexpr int ACC_COL = 2 * UNIT;                           // a group's columns: two score buffers, then the accumulator

    auto bar = [&](int i) { return ptx::smem_u32(bars + i); };

    if (threadIdx.x == 0) {
        // a K/V tile is released by the issuers of all the groups that use it
        const uint32_t users = alternate ? 2u : 2u * (uint32_t)nslots;
        for (int i = 0; i < NBARS; ++i)
            ptx::mbar_init(bar(i), (i >= P_FULL && i < P_FULL + 2 * NG) ? (kFast ? 4u : 128u)   // fast form: one arrival per warp
                                   : (i >= KV_EMPTY && i < KV_EMPTY + nstages) ? users + (kFast ? 1u : 0u)   // and its guard warp
                                   : (i >= KV_FULL && i < KV_FULL + nstages) ? 2u : 1u);   // the TMA loads, the bias tile
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmK);
        ptx::prefetch_tensormap(&tmV);
        ptx::prefetch_tensormap(&tmQ);
    }
    if (warp == kFirstIssuerWarp) ptx::tmem_alloc(ptx::smem_u32(tmem_slot), NCOLS);
    // latent rows beyond M are zero so their (discarded) lanes stay finite
    for (int i = tid; i < (2 * kTile - rows_here) * (G::RB / 16); i += kTcThreads)
        reinterpret_cast<uint4 *>(sQ + (size_t)rows_here * G::RB)[i] = make_uint4(0, 0, 0, 0);
    uint8_t *sBias = smem + SM::bias_off();                     // [stage] bias tiles, then the tile of ones
    if (!kDz) {
        using GB = TileGeom<16>;
        uint8_t *ones = sBias + (size_t)nstages * SM::kBiasTile;
        for (int r = tid; r < kTile; r += kTcThreads) {   // row r = [1, 0, ..., 0]: the first 16-byte chunk, swizzled
            reinterpret_cast<uint4 *>(ones + (size_t)r * GB::RB)[GB::swz(r)] = make_uint4(0x00003F80u, 0, 0, 0);
            reinterpret_cast<uint4 *>(ones + (size_t)r * GB::RB)[GB::swz(r) ^ 1] = make_uint4(0, 0, 0, 0);
        }
    }
    if (kOnes) {
        for (int i = tid; i < kTile * (G::RB / 16); i += kTcThreads) {
            const int r = i / (G::RB / 16), ch = i % (G::RB / 16);
            *reinterpret_cast<uint4 *>(sOnes + (size_t)r * G::RB + ((ch ^ G::swz(r)) << 4)) =
                make_uint4(ch == 0 ? 0x00003F80u : 0u, 0, 0, 0);
        }
    }
    if (kPair) {
        // block-diagonal A operand: row r < 64 = [Q[h][r] | 0], row 64 + r = [0 | Q[h+1][r]], 16-byte chunks swizzled
        __syncthreads();
        for (int i = tid; i < 2 * M * (D / 8); i += kTcThreads) {
            const int which = i / (M * (D / 8)), rem = i % (M * (D / 8)), m = rem / (D / 8), ch = rem % (D / 8);
            const uint4 v = *reinterpret_cast<const uint4 *>(a.Q + ((size_t)(h + which) * M + m) * D + ch * 8);
            const int r = which * 64 + m, chunk = which * (D / 8) + ch;
            *reinterpret_cast<uint4 *>(sQ + (size_t)r * G::RB + ((chunk ^ G::swz(r)) << 4)) = v;
        }
    }
    if (kHalf) {
        // rows [Q[h][m] | 0]: the lower DR/8 chunks of every row, the rest stays zero
        __syncthreads();
        if constexpr (DR == 4) {
            stage_rows4<DG>(sQ, a.Q + ((size_t)h * M + lb0 * kTile) * DR, rows_q, off);
        } else {
            for (int i = tid; i < rows_q * (DR / 8); i += kTcThreads) {
                const int m = i / (DR / 8), ch = i % (DR / 8);
                *reinterpret_cast<uint4 *>(sQ + (size_t)m * G::RB + ((ch ^ G::swz(m)) << 4)) =
                    *reinterpret_cast<const uint4 *>(a.Q + ((size_t)h * M + lb0 * kTile + m) * DR + ch * 8);
            }
        }
    }
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tm = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            if (kPair || kHalf) {
                ptx::mbar_arrive(bar(Q_FULL));                  // Q was written by the threads before the block barrier
            } else {
                ptx::mbar_arrive_expect_tx(bar(Q_FULL), (uint32_t)(rows_here * G::RB));
                for (int r = 0; r < rows_here; r += 16)
                    ptx::tma_load_2d(ptx::smem_u32(sQ + (size_t)r * G::RB), &tmQ, bar(Q_FULL), 0, h * M + lb0 * kTile + r);
            }
        }
        // The whole warp walks the tiles: lane 0 waits for the stage and issues the loads; for a tile with padding
        // (masked tokens, or tokens beyond N) every lane first writes four rows of the stage's bias tile.
        for (int i = 0; i < nt; ++i) {
            const int s = i % nstages, t = t_begin + i;
            if (!warp_wait(bar(KV_EMPTY + s), ((i / nstages) & 1) ^ 1, abort_flag, kErrEncode | 1)) break;
            const bool plain = kDz || kMaskBody || (a.key_mask == nullptr && (t + 1) * kTile <= a.N);
            if (!plain) {
                using GB = TileGeom<16>;
                uint8_t *bt = sBias + (size_t)s * SM::kBiasTile;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int r = lane * 4 + k, n = t * kTile + r;
                    const bool valid = n < a.N && (a.key_mask == nullptr || a.key_mask[(size_t)b * a.N + n] != 0);
                    const uint32_t first = valid ? 0u : (uint32_t)__bfloat16_as_ushort(__float2bfloat16(kMaskedScore));
                    reinterpret_cast<uint4 *>(bt + (size_t)r * GB::RB)[GB::swz(r)] = make_uint4(first, 0, 0, 0);
                    reinterpret_cast<uint4 *>(bt + (size_t)r * GB::RB)[GB::swz(r) ^ 1] = make_uint4(0, 0, 0, 0);
                }
                ptx::fence_proxy_async_smem();
                __syncwarp();
            }
            if (lane == 0) {
                ptx::mbar_arrive(bar(KV_FULL + s));             // the bias tile (or none needed)
                ptx::mbar_arrive_expect_tx(bar(KV_FULL + s), 2 * G::TILE_BYTES);
                uint8_t *dst = sKV + (size_t)s * 2 * G::TILE_BYTES;
                ptx::tma_load_3d(ptx::smem_u32(dst), &tmK, bar(KV_FULL + s), h * DR - off, t * kTile, b);
                ptx::tma_load_3d(ptx::smem_u32(dst + G::TILE_BYTES), &tmV, bar(KV_FULL + s), h * DR - off, t * kTile, b);
            }
        }
    } else if (kFast && warp >= kFirstGuardWarp) {
        // Guard warps (fast form), one tile in three each: the largest |k|^2 a tile may hold so that |q| |k| sl2 <=
        // kFastMaxLog2 for the CTA's latent rows, checked while the tile sits in its stage; the stage is released by
        // its users and its guard.  (Whole rows of both operands: in the head-pair and narrow forms they hold the
        // neighbouring heads' features too, which only makes the check stricter.)
        bool tame = warp_wait(bar(Q_FULL), 0, abort_flag, kErrEncode | 8);
        const float q2 = warp_max_nan(tile_max_norm2<G::RB>(sQ, 2 * kTile, lane));
        const float lim = kFastMaxLog2 / a.sl2;
        const float k2_limit = lim * lim / fmaxf(q2, 1e-30f);
        if (!(q2 <= 3.0e38f)) tame = false;                     // NaN or infinity in Q
        for (int j = warp - kFirstGuardWarp; j < nt; j += kGuardWarps) {
            const int sj = j % nstages;
            if (!warp_wait(bar(KV_FULL + sj), (j / nstages) & 1, abort_flag, kErrEncode | 9)) break;
            const float k2 = warp_max_nan(tile_max_norm2<G::RB, kPair ? 2 : 1>(sKV + (size_t)sj * 2 * G::TILE_BYTES, kTile, lane));
            if (!(k2 <= k2_limit)) tame = false;
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar(KV_EMPTY + sj));
        }
        if (!tame && lane == 0) *a.redo = 1u;
    } else if (warp < kFirstSoftmaxWarp) {
        const int g = warp - kFirstIssuerWarp;                  // the group this warp issues MMAs for
        const int j = g >> 1, c = g & 1;                        // its slot and column half
        if (lane == 0 && j < nslots) {
            const uint32_t idescS = ptx::instr_desc_bf16(128, UNIT, 0, 0);
            const uint32_t idescV = ptx::instr_desc_bf16(128, kOnes ? DG + 16 : DG, 0, 1);
            // Q rows of the slot's latent block (K-major A operand); descriptor address fields are in 16-byte units
            const uint64_t qdesc = ptx::smem_desc(ptx::smem_u32(sQ), 16, G::SBO, G::SWZ) +
                                   (uint64_t)(alternate ? 0 : j * kTile * G::RB / 16);
            const uint32_t gcol = tm + j * SLOT_COLS + c * 2 * HALF;        // the group's 128 columns
            const uint32_t dcol = gcol + ACC_COL;                           // its accumulator
            bool ok = ptx::mbar_wait(bar(Q_FULL), 0, abort_flag, kErrEncode | 2);
            const int jobs = (nq - j + nslots - 1) / nslots;                // tiles this group works on
            const int units = 2 * jobs;
            // Order of issue: S(0), S(1), then for every unit n: its value MMAs as soon as its weights are handed
            // over, then the scores of unit n+2 into the buffer those weights have just left.  Every wait blocks
            // in hardware, so the issuing warp takes no issue slots from the softmax warps while it waits.
            int t_s = alternate ? j : 0, t_v = t_s;                         // tiles (relative to t_begin) of the next S / PV unit
            const int t_step = alternate ? 2 : 1;
            if constexpr (kFast) {
                // The fast form's loop, with as few instructions of this thread per unit as it takes (they are on the
                // critical path of the group: each waits for an issue slot among the softmax warps, and a tcgen05.mma or
                // commit holds the thread for 50 to 130 cycles): descriptors are a base plus a stage and a unit offset;
                // one wait per tile for the loads and one per unit for the weights; ONE commit per unit, behind the score
                // MMA of the unit two further on, which tells the threads both that those scores are there and that the
                // value MMAs before them (which read the buffer the scores went into) are done.
                const uint32_t stage_step = (uint32_t)((2 * G::TILE_BYTES) >> 4), unit_step = (uint32_t)((UNIT * G::RB) >> 4);
                const uint64_t kd0 = ptx::smem_desc(ptx::smem_u32(sKV), 16, G::SBO, G::SWZ) + (uint64_t)((c * HALF * G::RB) >> 4);
                const uint32_t v0 = ptx::smem_u32(sKV + G::TILE_BYTES);
                const uint64_t vd0 = ptx::smem_desc(v0, kOnes ? ptx::smem_u32(sOnes) - v0 : (uint32_t)G::SBO, G::SBO, G::SWZ) +
                                     (uint64_t)((c * HALF * G::RB) >> 4);
                // a stage further on, the V tile starts stage_step later and (kOnes) the ones tile is that much nearer (LBO: bits 16-29)
                const uint64_t vstep = (uint64_t)stage_step - (kOnes ? ((uint64_t)stage_step << 16) : 0ull);
                const uint32_t sfull = bar(S_FULL + 2 * g), pfull = bar(P_FULL + 2 * g);
                // without kMaskBody only a last partial tile has padding; its scores get the bias MMA (see kMaskedScore)
                const int bias_tile = (!kMaskBody && a.N % kTile != 0) ? a.tiles - 1 - t_begin : -1;
                int ss = t_s % nstages, sp = (t_s / nstages) & 1, sv = ss;
                auto scores = [&](int w) {                        // the scores of unit w of the S stream's tile, and the commit
                    const uint64_t kd = kd0 + (uint64_t)(stage_step * (uint32_t)ss + unit_step * (uint32_t)w);
#pragma unroll
                    for (int k = 0; k < DG / 16; ++k) ptx::mma_ss(gcol + w * UNIT, qdesc + 2 * k, kd + 2 * k, idescS, k > 0);
                    if (!kMaskBody && t_s == bias_tile) {
                        using GB = TileGeom<16>;
                        const uint64_t odesc = ptx::smem_desc(ptx::smem_u32(sBias + (size_t)nstages * SM::kBiasTile), 16, GB::SBO, GB::SWZ);
                        const uint64_t bdesc = ptx::smem_desc(ptx::smem_u32(sBias + (size_t)ss * SM::kBiasTile), 16, GB::SBO, GB::SWZ) +
                                               (uint64_t)((c * HALF + w * UNIT) * GB::RB / 16);
                        ptx::mma_ss(gcol + w * UNIT, odesc, bdesc, idescS, 1u);
                    }
                    ptx::mma_commit(sfull + 8 * w);
                };
                auto open_tile = [&]() -> bool {
                    if (!ptx::mbar_wait(bar(KV_FULL + ss), (uint32_t)sp, abort_flag, kErrEncode | 3)) return false;
                    ptx::tc_fence_after();
                    return true;
                };
                auto next_s = [&]() {
                    t_s += t_step;
                    ss += t_step;
                    if (ss >= nstages) { ss -= nstages; sp ^= 1; }
                };
                if (ok && jobs > 0 && (ok = open_tile())) {
                    scores(0);
                    scores(1);
                    next_s();
                }
                for (int job = 0; ok && job < jobs; ++job) {
#pragma unroll
                    for (int w = 0; w < 2; ++w) {
                        if (!ptx::mbar_spin(pfull + 8 * w, (uint32_t)(job & 1), abort_flag, kErrEncode | 4)) { ok = false; break; }
                        ptx::tc_fence_after();
                        const uint64_t vd = vd0 + vstep * (uint64_t)sv + (uint64_t)(unit_step * (uint32_t)w);
#pragma unroll
                        for (int k = 0; k < UNIT / 16; ++k) {
                            ptx::mma_ts(dcol, gcol + w * UNIT + k * 8, vd + (uint64_t)(k * G::RB), idescV, (job > 0 || w > 0 || k > 0) ? 1u : 0u);
                            if (kHiLo) ptx::mma_ts(dcol, gcol + w * UNIT + 16 + k * 8, vd + (uint64_t)(k * G::RB), idescV, 1u);
                        }
                        if (w == 1) {                             // the tile's last unit: one arrival per group
                            ptx::mma_commit(bar(KV_EMPTY + sv));
                            sv += t_step;
                            if (sv >= nstages) sv -= nstages;
                        }
                        if (job + 1 < jobs) {                     // the same unit of the group's next tile, into the buffer just read
                            if (w == 0 && !open_tile()) { ok = false; break; }
                            scores(w);
                            if (w == 1) next_s();
                        }
                    }
                }
                if (ok) ptx::mma_commit(bar(ACC_DONE + g));
            } else {
                int s_stage = t_s % nstages, s_phase = (t_s / nstages) & 1;   // stage and phase of the S stream's tile
                auto issue_scores = [&](int n) -> bool {
                    const int s = s_stage, w = n & 1;                        // w: which 32 tokens of the half; also the buffer
                    if (!ptx::mbar_wait(bar(KV_FULL + s), s_phase, abort_flag, kErrEncode | 3)) return false;
                    ptx::tc_fence_after();
                    // S_unit = Q_block K_unit^T: the unit's 32 token rows of the K tile are the B operand
                    const uint64_t kdesc = ptx::smem_desc(ptx::smem_u32(sKV + (size_t)s * 2 * G::TILE_BYTES), 16, G::SBO, G::SWZ) +
                                           (uint64_t)((c * HALF + w * UNIT) * G::RB / 16);
#pragma unroll
                    for (int k = 0; k < DG / 16; ++k) ptx::mma_ss(gcol + w * UNIT, qdesc + 2 * k, kdesc + 2 * k, idescS, k > 0);
                    const int tile = t_begin + t_s;
                    if (!kDz && !kMaskBody && !(a.key_mask == nullptr && (tile + 1) * kTile <= a.N)) {
                        // scores += ones x bias: padded tokens drop to kMaskedScore (see there)
                        using GB = TileGeom<16>;
                        const uint64_t odesc = ptx::smem_desc(ptx::smem_u32(sBias + (size_t)nstages * SM::kBiasTile), 16, GB::SBO, GB::SWZ);
                        const uint64_t bdesc = ptx::smem_desc(ptx::smem_u32(sBias + (size_t)s * SM::kBiasTile), 16, GB::SBO, GB::SWZ) +
                                               (uint64_t)((c * HALF + w * UNIT) * GB::RB / 16);
                        ptx::mma_ss(gcol + w * UNIT, odesc, bdesc, idescS, 1u);
                    }
                    ptx::mma_commit(bar(S_FULL + 2 * g + w));
                    if (w == 1) {
                        t_s += t_step;
                        s_stage += t_step;
                        if (s_stage >= nstages) { s_stage -= nstages; s_phase ^= 1; }
                    }
                    return true;
                };
                for (int n = 0; ok && n < 2 && n < units; ++n) ok = issue_scores(n);
                int v_stage = t_v % nstages;
                for (int n = 0; ok && n < units; ++n) {
                    const int w = n & 1, s = v_stage;
                    if (!ptx::mbar_wait(bar(P_FULL + 2 * g + w), (n >> 1) & 1, abort_flag, kErrEncode | 4)) break;
                    ptx::tc_fence_after();
                    // acc += P_unit V_unit: V tile as the MN-major B operand, 16 token rows further on per k-step
                    const uint64_t vdesc = ptx::smem_desc(ptx::smem_u32(sKV + (size_t)s * 2 * G::TILE_BYTES + G::TILE_BYTES),
                                                          G::SBO, G::SBO, G::SWZ) + (uint64_t)((c * HALF + w * UNIT) * G::RB / 16);
#pragma unroll
                    for (int k = 0; k < UNIT / 16; ++k) {
                        ptx::mma_ts(dcol, gcol + w * UNIT + k * 8, vdesc + (uint64_t)(k * G::RB), idescV, (n > 0 || k > 0) ? 1u : 0u);
                        if (kDz || kHiLo)    // the lo halves of the weights sit 16 columns further on
                            ptx::mma_ts(dcol, gcol + w * UNIT + 16 + k * 8, vdesc + (uint64_t)(k * G::RB), idescV, 1u);
                    }
                    ptx::mma_commit(bar(PV_DONE + g));
                    if (w == 1) {                                           // the tile's last unit: one arrival per group
                        ptx::mma_commit(bar(KV_EMPTY + s));
                        t_v += t_step;
                        v_stage += t_step;
                        if (v_stage >= nstages) v_stage -= nstages;
                    }
                    if (n + 2 < units) ok = issue_scores(n + 2);
                }
                if (ok) ptx::mma_commit(bar(ACC_DONE + g));
            }
        }
    } else {
        const int g = (warp - kFirstSoftmaxWarp) >> 2;          // softmax group
        const int j = g >> 1, c = g & 1;                        // its slot and column half
        const int row = ((warp & 3) << 5) + lane;               // TMEM lane = latent within the block
        const uint32_t lane_addr = (uint32_t)((warp & 3) << 5) << 16;
        const uint32_t gcol = tm + lane_addr + j * SLOT_COLS + c * 2 * HALF;   // the group's 128 columns
        const uint32_t abase = gcol + ACC_COL;                                // its accumulator
        const float2 sl2p = make_float2(a.sl2, a.sl2);
        float m_run = -INFINITY;
        float2 l2 = make_float2(0.f, 0.f);
        int done = 0;                                           // units finished
        bool ok = true;
        float *colneg = reinterpret_cast<float *>(smem + SM::col_off()) + (warp - kFirstSoftmaxWarp) * 64;   // this warp's addends
        // dZ form of a unit: weights exp(S - lse_dec[token]), no maximum, no sum.
        auto unit_dz = [&](int t, int w) -> bool {
            const uint32_t sbase = gcol + w * UNIT;
            const int n = t * kTile + c * HALF + w * UNIT + lane;          // this lane fetches the shift of token n
            const int hh = h + (kPair ? (row >> 6) : 0);                   // the head of this lane's latent
            __syncwarp();                                                   // the previous unit's reads are done
            colneg[lane] = n < a.N ? -a.lse_dec[((size_t)b * a.N + n) * a.H + hh] * 1.4426950408889634f : -INFINITY;
            __syncwarp();
            if (!warp_wait(bar(S_FULL + 2 * g + w), (done >> 1) & 1, abort_flag, kErrEncode | 5)) return false;
            ptx::tc_fence_after();
            uint32_t r[32], pk[16], pl[16];
            ptx::tmem_ld32(sbase, r);
            ptx::tmem_wait_ld();
            exp_chunk_cols<32>(r, pk, pl, sl2p, colneg);
            ptx::tmem_st16(sbase, pk);                          // hi halves over the first 16 score columns,
            ptx::tmem_st16(sbase + 16, pl);                     // lo halves over the other 16
            ptx::tmem_wait_st();
            ptx::tc_fence_before();
            ptx::mbar_arrive(bar(P_FULL + 2 * g + w));
            ++done;
            return true;
        };
        // One unit of work: 32 token columns of this group's half, on score buffer w.  kMasked: some of the tile's
        // tokens may be padding or lie beyond N (their weights are exactly 0); the plain form has no such tests.
        auto unit = [&](auto masked, int t, int w) -> bool {
            constexpr bool kMasked = decltype(masked)::value;
            uint32_t wv = 0xffffffffu;
            if (kMasked) {
                const int n = t * kTile + c * HALF + w * UNIT + lane;
                wv = __ballot_sync(0xffffffffu, n < a.N && (a.key_mask == nullptr || a.key_mask[(size_t)b * a.N + n] != 0));
            }
            const uint32_t sbase = gcol + w * UNIT;             // the unit's scores, and its packed weights over them
            if (!warp_wait(bar(S_FULL + 2 * g + w), (done >> 1) & 1, abort_flag, kErrEncode | 5)) return false;
            ptx::tc_fence_after();
            uint32_t r[32];
            ptx::tmem_ld32(sbase, r);                           // the scores stay in registers for both passes
            ptx::tmem_wait_ld();
            float tmax = -INFINITY;
            if (!kMasked) {
                tmax = max_of<32>(r, tmax);
            } else {
#pragma unroll
                for (int k = 0; k < 32; ++k)
                    if ((wv >> k) & 1) tmax = fmaxf(tmax, __uint_as_float(r[k]));
            }
            const float m_new = fmaxf(m_run, tmax);
            const bool grow = done > 0 && m_new > m_run;
            if (__any_sync(0xffffffffu, grow)) {                // rescale the accumulator row (warp-uniform branch)
                // the value MMAs of every earlier unit must have landed in the accumulator first
                if (!warp_wait(bar(PV_DONE + g), (done - 1) & 1, abort_flag, kErrEncode | 7)) return false;
                ptx::tc_fence_after();
                const float f = grow ? ptx::ex2((m_run - m_new) * a.sl2) : 1.f;
                l2.x *= f;
                l2.y *= f;
                uint32_t ar[16];
#pragma unroll
                for (int dc = 0; dc < DG / 16; ++dc) {
                    ptx::tmem_ld16(abase + dc * 16, ar);
                    ptx::tmem_wait_ld();
#pragma unroll
                    for (int k = 0; k < 16; ++k) ar[k] = __float_as_uint(__uint_as_float(ar[k]) * f);
                    ptx::tmem_st16(abase + dc * 16, ar);
                }
            }
            m_run = m_new;
            const bool dead = m_run < kDeadBelow;               // no valid token yet: all weights are zero
            const float neg = dead ? 0.f : -m_run * a.sl2;
            const float2 negp = make_float2(neg, neg);
            uint32_t pk[16];
            if (kHiLo) {
                uint32_t pl[16];
                exp_chunk_hilo<32, kMasked>(r, pk, pl, sl2p, negp, l2, wv, dead);
                ptx::tmem_st16(sbase, pk);                      // hi halves over the first 16 score columns,
                ptx::tmem_st16(sbase + 16, pl);                 // lo halves over the other 16
            } else {
                exp_chunk<32, kMasked>(r, pk, sl2p, negp, l2, wv, dead);
                ptx::tmem_st16(sbase, pk);
            }
            ptx::tmem_wait_st();                                // weights (and a rescaled accumulator) are in place
            ptx::tc_fence_before();
            ptx::mbar_arrive(bar(P_FULL + 2 * g + w));
            ++done;
            return true;
        };
        // Fast form of a unit: weights 2^(s * sl2), no maximum, nothing to rescale.  kMasked as above; kPoly: half of
        // the exponentials on the FMA pipe (never where padding sits in the scores as kMaskedScore).
        auto unit_fast = [&](auto masked, auto poly, int t, int w) -> bool {
            constexpr bool kMasked = decltype(masked)::value;
            constexpr bool kPoly = decltype(poly)::value && !kHiLo;
            uint32_t wv = 0xffffffffu;
            if (kMasked) {
                const int n = t * kTile + c * HALF + w * UNIT + lane;
                wv = __ballot_sync(0xffffffffu, n < a.N && (a.key_mask == nullptr || a.key_mask[(size_t)b * a.N + n] != 0));
            }
            const uint32_t sbase = gcol + w * UNIT;
            if (!warp_wait(bar(S_FULL + 2 * g + w), (done >> 1) & 1, abort_flag, kErrEncode | 5)) return false;
            ptx::tc_fence_after();
            uint32_t r[32], pk[16];
            ptx::tmem_ld32(sbase, r);
            ptx::tmem_wait_ld();
            if (kHiLo) {
                uint32_t pl[16];
                exp_chunk_hilo<32, kMasked>(r, pk, pl, sl2p, make_float2(0.f, 0.f), l2, wv, false);
                ptx::tmem_st16(sbase, pk);
                ptx::tmem_st16(sbase + 16, pl);
            } else {
                exp_chunk_fast<32, kPoly, kMasked, kSumMode>(r, pk, sl2p, l2, wv);
                ptx::tmem_st16(sbase, pk);
            }
            ptx::tmem_wait_st();
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar(P_FULL + 2 * g + w));
            ++done;
            return true;
        };
        if (j < nslots) {
            for (int q = j; ok && q < nq; q += nslots) {
                const int t = t_begin + (alternate ? q : q / nslots);
                const bool full = a.key_mask == nullptr && (t + 1) * kTile <= a.N;    // no padding in this tile (warp-uniform)
                const bool plain = !kMaskBody || full;
#pragma unroll 1
                for (int w = 0; ok && w < 2; ++w) {             // the half's two units, on alternating buffers
                    if (kDz) ok = unit_dz(t, w);
                    else if (kFast && kMaskBody) ok = plain ? unit_fast(std::false_type{}, std::true_type{}, t, w)
                                                            : unit_fast(std::true_type{}, std::true_type{}, t, w);
                    else if (kFast) ok = full ? unit_fast(std::false_type{}, std::true_type{}, t, w)
                                              : unit_fast(std::false_type{}, std::false_type{}, t, w);
                    else if (kMaskBody && !plain) ok = unit(std::true_type{}, t, w);
                    else ok = unit(std::false_type{}, t, w);    // (without kMaskBody padding is in the scores already)
                }
            }
        }
        // write this group's partial (running max in natural-log units, sum, un-normalised rows)
        if (ok && j < nslots) ok = warp_wait(bar(ACC_DONE + g), 0, abort_flag, kErrEncode | 6);
        ptx::tc_fence_after();
        const int lb = alternate ? 0 : lb0 + j;
        // head-pair form: lanes 64-127 belong to the second head, whose rows are accumulator columns [D, 2D)
        const int second = kPair ? (row >> 6) : 0;
        const int m = kPair ? (row & 63) : lb * kTile + row;
        const bool writes = ok && j < nslots;
        uint32_t acc[D];
        if (done > 0) {
#pragma unroll
            for (int dc = 0; dc < D / 16; ++dc) ptx::tmem_ld16(abase + second * D + dc * 16, acc + dc * 16);
            if (kOnes) {                                        // column DG: the sum of the weights
                uint32_t t8[8];
                ptx::tmem_ld8(abase + DG, t8);
                ptx::tmem_wait_ld();
                l2 = make_float2(__uint_as_float(t8[0]), 0.f);
            }
            ptx::tmem_wait_ld();
        } else {
#pragma unroll
            for (int k = 0; k < D; ++k) acc[k] = 0u;
        }
        if (kFast) m_run = (l2.x + l2.y > 0.f) ? 0.f : -INFINITY;   // weights relative to 2^0; a row with no valid token
        if (writes && m < M) {
            const long rows = (long)a.B * a.H * M;
            const int part = split * a.partials_per_split + (alternate ? 2 * j + c : c);
            const size_t prow = (size_t)part * rows + ((size_t)b * a.H + h + second) * M + m;
            if (!kDz) {
                a.part_m[prow] = (m_run < kDeadBelow) ? -INFINITY : m_run * a.scale;
                a.part_l[prow] = l2.x + l2.y;
            }
            float4 *dst = reinterpret_cast<float4 *>(a.part_acc + prow * DR);
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

// The bounded wait of the kernels above, on its own: one thread waits for at most `budget_ns` on a barrier phase
// that nothing ever completes, then takes the same way out as a kernel whose wait gave up (code into the block's
// abort flag, from there into the workspace header).  Lets a caller see FLARE_ERR_TIMEOUT without a hung kernel.
__global__ void selftest_wait_kernel(uint32_t *status, unsigned long long budget_ns) {
    __shared__ uint64_t bar_mem;
    __shared__ uint32_t flag;
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_u32(&bar_mem), 1);
        flag = 0;
        ptx::fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) ptx::mbar_wait_for(ptx::smem_u32(&bar_mem), 0, &flag, kErrSelftest | 1, budget_ns);
    __syncthreads();
    if (threadIdx.x == 0 && flag != 0 && status != nullptr) atomicCAS(status, 0u, flag);
}

}  // namespace flare
