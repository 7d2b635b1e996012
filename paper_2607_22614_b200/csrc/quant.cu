// fp32 -> fp8 e4m3 with one fp32 scale per 128 x 128 block of the rollout tensor (sm_100a).
//
// One CTA per block: 256 threads hold the block's 16 384 values in registers (eight 256-bit loads in
// flight per thread, three CTAs per SM, each row of the block one contiguous 512 B request), reduce |x| to the block
// maximum with shuffles and one shared-memory step, then
// divide by the block's scale, convert two values per cvt.rn.satfinite.e4m3x2.f32 and store
// each row as one contiguous 128 B request.  The bound is HBM: 4 B read + 1 B written per element (+ 4 B
// per 16 384 elements for the scale).
//
// The definition is code = e4m3(fl32(x / scale)).  A correctly rounded fp32 division costs about twenty
// instructions, which would make the kernel issue-bound, so the quotient is taken as t = x * fl32(1 / scale)
// wherever that provably gives the same code: t and the true quotient differ by at most 2 ulp, so they can
// round to different e4m3 codes only if t lies within a few ulp of a midpoint between two codes (its 20 dropped
// mantissa bits within 4 of 0x80000) or below 2^-6, where the e4m3 grid is no longer 3 mantissa bits wide.
// A thread's eight values of a row take the exact division together when any of them is in doubt (about one
// group in 10^3 for weight-like data).  Whole, aligned blocks (nearly all of them) run a predicate-free body.
// Parking part of the block in shared memory (cp.async) to raise the CTAs per SM was measured and is slower:
// the block stays in registers, 256 threads x 64 values, three CTAs per SM.
#include <cuda_runtime.h>

#include "dr_internal.h"

namespace dr {
namespace {

#ifndef DR_Q_THREADS
#define DR_Q_THREADS 256
#endif
#ifndef DR_Q_MIN_BLOCKS
#define DR_Q_MIN_BLOCKS 3
#endif
constexpr int kQThreads = DR_Q_THREADS;
constexpr int kRowsPerPass = kQThreads / 16;   // 16 threads cover one 128-column block row
constexpr int kPasses = 128 / kRowsPerPass;    // block rows per thread
static_assert(kQThreads >= 128 && 128 % kRowsPerPass == 0, "thread count must tile the block");

__device__ __forceinline__ void ld256f(const void* p, float (&v)[8])
{
    asm volatile("ld.global.nc.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
                 : "l"(p));
}
__device__ __forceinline__ void ld128f(const void* p, float* v)
{
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3])
                 : "l"(p));
}
__device__ __forceinline__ float ld32f(const void* p)
{
    float v;
    asm volatile("ld.global.nc.L1::no_allocate.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}
// two fp32 -> two e4m3 bytes: round to nearest even, saturate to +-448; a NaN of either sign comes out
// as 0x7F (checked against the oracle on sources made of every bit pattern)
__device__ __forceinline__ uint32_t cvt_e4m3x2(float lo, float hi)
{
    uint16_t d;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(d) : "f"(hi), "f"(lo));
    return d;
}
// Eight values of one block row -> eight e4m3 codes of x / scale, packed into two words.
// The codes are first taken from the products with the reciprocal.  Product and true quotient differ by at most
// 2 ulp, so they can round to different codes only (A) next to a midpoint between two codes: the 20 mantissa bits
// e4m3 drops lie within 4 of 0x80000, tested with one multiply-add per value (shifting the 20 bits to the top and
// subtracting (0x80000 - 4) << 12 leaves a value <= 8 << 12) and a min tree; or (B) below 2^-6, where the e4m3
// grid is no longer 3 mantissa bits wide: tested on the packed codes, four at a time (a code of magnitude
// <= small_code = 8 means the product rounded to 2^-6 or less).  In either case all eight are redone with the
// correctly rounded division.  small_code = 0x7F sends every group there (blocks whose reciprocal is not normal).
__device__ __forceinline__ uint2 pack8(const float* t)
{
    const uint32_t h0 = cvt_e4m3x2(t[0], t[1]), h1 = cvt_e4m3x2(t[2], t[3]);
    const uint32_t h2 = cvt_e4m3x2(t[4], t[5]), h3 = cvt_e4m3x2(t[6], t[7]);
    return make_uint2(h0 | (h1 << 16), h2 | (h3 << 16));
}
__device__ __forceinline__ uint2 quantise8(const float* x, float scale, float recip, uint32_t small_code)
{
    float t[8];
    uint32_t d[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        t[k] = __fmul_rn(x[k], recip);
        d[k] = __float_as_uint(t[k]) * 4096u - 0x7FFFC000u;
    }
#pragma unroll
    for (int w = 4; w >= 1; w /= 2)  // min tree (three-input minima were measured and are slower)
#pragma unroll
        for (int k = 0; k < w; ++k) d[k] = min(d[k], d[k + w]);
    const uint32_t dmin = d[0];
    uint2 q = pack8(t);
    // per byte: magnitude + (0x7F - small_code) reaches bit 7 exactly when the magnitude exceeds small_code
    const uint32_t bias = (0x7Fu - small_code) * 0x01010101u;
    const uint32_t big = ((q.x & 0x7F7F7F7Fu) + bias) & ((q.y & 0x7F7F7F7Fu) + bias) & 0x80808080u;
    if (dmin <= 0x8000u || big != 0x80808080u) {
#pragma unroll
        for (int k = 0; k < 8; ++k) t[k] = __fdiv_rn(x[k], scale);
        q = pack8(t);
    }
    return q;
}

// One 128 x 128 block.  FAST: the block is whole (128 rows, 128 columns inside the tensor), its rows allow
// 256-bit loads and the buffers' bases are 32-byte aligned, so no access needs a predicate.
template <bool FAST>
__device__ __forceinline__ void quant_block(const QTensor& T, uint32_t bi, uint32_t bj, uint32_t nrows,
                                            const uint64_t* row_src, float* warp_max, float* s_scale,
                                            const char* __restrict__ flat, char* __restrict__ arena, int allow256)
{
    const uint32_t r0 = bi * 128, c0 = bj * 128;
    const uint32_t cu = threadIdx.x & 15;   // 8-column unit inside the block row
    const uint32_t rb = threadIdx.x >> 4;   // row inside a pass
    const uint32_t col = c0 + cu * 8;
    float v[kPasses][8];
    float amax = 0.0f;
#pragma unroll
    for (int p = 0; p < kPasses; ++p) {
        const uint32_t row = p * kRowsPerPass + rb;
        if (FAST) {
            ld256f(flat + (row_src[row] + col) * 4, v[p]);
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) v[p][k] = 0.0f;
            if (row < nrows && col < T.cols) {
                const char* src = flat + (row_src[row] + col) * 4;
                // T.aligned speaks of offsets from the flat base; the base itself is only promised to be 16-byte
                // aligned, so the 256-bit form also needs a 32-byte aligned base (allow256)
                if (T.aligned && allow256) {
                    ld256f(src, v[p]);
                } else if (T.aligned) {
                    ld128f(src, &v[p][0]);
                    ld128f(src + 16, &v[p][4]);
                } else {
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        if (col + k < T.cols) v[p][k] = ld32f(src + 4 * k);
                }
            }
        }
    }
#pragma unroll
    for (int p = 0; p < kPasses; ++p)
#pragma unroll
        for (int k = 0; k < 8; ++k) amax = fmaxf(amax, fabsf(v[p][k]));  // fmaxf drops NaN operands
#pragma unroll
    for (int o = 16; o; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, o));
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = amax;
    __syncthreads();
    if (threadIdx.x == 0) {
        float m = warp_max[0];
#pragma unroll
        for (int w = 1; w < kQThreads / 32; ++w) m = fmaxf(m, warp_max[w]);
        // amax / 448, held inside the normal fp32 range: 2^-126 for blocks whose amax / 448 underflows (the
        // all-zero block among them), FLT_MAX for a block holding an infinity
        float scale = fminf(fmaxf(__fdiv_rn(m, 448.0f), 1.17549435e-38f), 3.40282347e+38f);
        *s_scale = scale;
        *(float*)(arena + T.scale_off + ((uint64_t)bi * T.nbc + bj) * 4) = scale;
    }
    __syncthreads();
    const float scale = *s_scale;
    const float recip = __frcp_rn(scale);
    // the product form needs a normal reciprocal (scale <= 2^126: always, except for the infinity block);
    // otherwise every group takes the exact division
    const uint32_t small_code = recip >= 1.17549435e-38f ? 8u : 0x7Fu;

#pragma unroll
    for (int p = 0; p < kPasses; ++p) {
        const uint32_t row = p * kRowsPerPass + rb;
        if (!FAST && (row >= nrows || col >= T.cols)) continue;
        const uint2 q = quantise8(v[p], scale, recip, small_code);
        char* dst = arena + T.payload_off + (uint64_t)(r0 + row) * T.cols + col;
        if (FAST || T.aligned) {
            asm volatile("st.global.L1::no_allocate.v2.b32 [%0], {%1,%2};" ::"l"(dst), "r"(q.x), "r"(q.y) : "memory");
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if (col + k < T.cols) dst[k] = (char)(((k < 4 ? q.x : q.y) >> (8 * (k & 3))) & 0xFF);
        }
    }
}

// The general form is a call, not inlined: compiled into the kernel body it costs the whole-block path registers
// (156 instead of 32 bytes of spills at the 80 registers that three CTAs per SM allow).
__device__ __noinline__ void quant_block_ragged(const QTensor& T, uint32_t bi, uint32_t bj, uint32_t nrows,
                                                const uint64_t* row_src, float* warp_max, float* s_scale,
                                                const char* __restrict__ flat, char* __restrict__ arena, int allow256)
{
    quant_block<false>(T, bi, bj, nrows, row_src, warp_max, s_scale, flat, arena, allow256);
}

__global__ void __launch_bounds__(kQThreads, DR_Q_MIN_BLOCKS)
    quant_kernel(const QTensor* __restrict__ tensors, uint32_t n_tensors, const QPart* __restrict__ parts,
                 const uint32_t* __restrict__ hints, uint32_t hint_shift, const char* __restrict__ flat,
                 char* __restrict__ arena, int allow256, uint64_t block_begin)
{
    __shared__ uint64_t row_src[128];  // flat element offset of (row, first column of the tensor)
    __shared__ float warp_max[kQThreads / 32];
    __shared__ float s_scale;

    const uint64_t b = block_begin + blockIdx.x;
    // block -> tensor: hint plus a short walk (all threads, same addresses: broadcast loads)
    uint32_t ti = hints[b >> hint_shift];
    while (ti + 1 < n_tensors && tensors[ti + 1].block0 <= b) ++ti;
    const QTensor T = tensors[ti];
    const uint32_t lb = (uint32_t)(b - T.block0);
    const uint32_t bi = lb / T.nbc, bj = lb - bi * T.nbc;
    const uint32_t r0 = bi * 128;
    const uint32_t nrows = min(128u, T.rows - r0);

    // each of the first 128 threads finds the source row of one block row (binary search over the parts)
    if (threadIdx.x < 128) {
        uint64_t off = 0;
        const uint32_t r = r0 + threadIdx.x;
        if (threadIdx.x < nrows) {
            uint32_t lo = T.part0, hi = T.part0 + T.n_parts;  // last part with dst_row0 <= r
            while (hi - lo > 1) {
                uint32_t mid = lo + (hi - lo) / 2;
                if (parts[mid].dst_row0 <= r) lo = mid; else hi = mid;
            }
            const QPart P = parts[lo];
            off = P.src_off + (uint64_t)(r - P.dst_row0) * P.src_stride;
        }
        row_src[threadIdx.x] = off;
    }
    __syncthreads();
    if (nrows == 128 && bj * 128 + 128 <= T.cols && T.aligned && allow256)
        quant_block<true>(T, bi, bj, nrows, row_src, warp_max, &s_scale, flat, arena, allow256);
    else
        quant_block_ragged(T, bi, bj, nrows, row_src, warp_max, &s_scale, flat, arena, allow256);
}

// ---- the inverse: e4m3 codes times the block's scale, back to the flat fp32 positions ----------------------
// Same decomposition (one CTA per 128 x 128 block, 16 threads per block row, eight values per thread and row),
// no reduction: 1 B read + 4 B written per element.  value(code) is exact in fp16 (cvt.rn.f16x2.e4m3x2), the
// product with the scale is one fp32 multiplication, and any NaN (a NaN code, a NaN scale, 0 * Inf) becomes the
// quiet NaN 0x7FC00000.
__device__ __forceinline__ void e4m3x2_to_f32(uint32_t two, float& lo, float& hi)
{
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)two));
    asm("cvt.f32.f16 %0, %1;" : "=f"(lo) : "h"((uint16_t)(h2 & 0xFFFF)));
    asm("cvt.f32.f16 %0, %1;" : "=f"(hi) : "h"((uint16_t)(h2 >> 16)));
}
__global__ void __launch_bounds__(kQThreads)
    dequant_kernel(const QTensor* __restrict__ tensors, uint32_t n_tensors, const QPart* __restrict__ parts,
                   const uint32_t* __restrict__ hints, uint32_t hint_shift, const char* __restrict__ arena,
                   char* __restrict__ flat, int allow256)
{
    __shared__ uint64_t row_src[128];
    const uint64_t b = blockIdx.x;
    uint32_t ti = hints[b >> hint_shift];
    while (ti + 1 < n_tensors && tensors[ti + 1].block0 <= b) ++ti;
    const QTensor T = tensors[ti];
    const uint32_t lb = (uint32_t)(b - T.block0);
    const uint32_t bi = lb / T.nbc, bj = lb - bi * T.nbc;
    const uint32_t r0 = bi * 128, c0 = bj * 128;
    const uint32_t nrows = min(128u, T.rows - r0);
    if (threadIdx.x < 128) {
        uint64_t off = 0;
        const uint32_t r = r0 + threadIdx.x;
        if (threadIdx.x < nrows) {
            uint32_t lo = T.part0, hi = T.part0 + T.n_parts;
            while (hi - lo > 1) {
                uint32_t mid = lo + (hi - lo) / 2;
                if (parts[mid].dst_row0 <= r) lo = mid; else hi = mid;
            }
            const QPart P = parts[lo];
            off = P.src_off + (uint64_t)(r - P.dst_row0) * P.src_stride;
        }
        row_src[threadIdx.x] = off;
    }
    const float scale = *(const float*)(arena + T.scale_off + ((uint64_t)bi * T.nbc + bj) * 4);
    const bool finite_scale = (__float_as_uint(scale) & 0x7F800000u) != 0x7F800000u;
    __syncthreads();

    const uint32_t cu = threadIdx.x & 15, rb = threadIdx.x >> 4;
    const uint32_t col = c0 + cu * 8;
    uint32_t q[kPasses][2];
#pragma unroll
    for (int p = 0; p < kPasses; ++p) {
        const uint32_t row = p * kRowsPerPass + rb;
        q[p][0] = q[p][1] = 0;
        if (row < nrows && col < T.cols) {
            const char* src = arena + T.payload_off + (uint64_t)(r0 + row) * T.cols + col;
            if (T.aligned) {
                asm volatile("ld.global.nc.L1::no_allocate.v2.b32 {%0,%1}, [%2];" : "=r"(q[p][0]), "=r"(q[p][1]) : "l"(src));
            } else {
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    if (col + k < T.cols) q[p][k >> 2] |= (uint32_t)(uint8_t)src[k] << (8 * (k & 3));
            }
        }
    }
#pragma unroll
    for (int p = 0; p < kPasses; ++p) {
        const uint32_t row = p * kRowsPerPass + rb;
        if (row >= nrows || col >= T.cols) continue;
        uint32_t y[8];
        // A product can only be NaN if a code is a NaN code (magnitude 0x7F: + 1 reaches bit 7) or the scale is not
        // finite; without either, the eight products need no NaN check.
        const uint32_t nan_code = (((q[p][0] & 0x7F7F7F7Fu) + 0x01010101u) | ((q[p][1] & 0x7F7F7F7Fu) + 0x01010101u)) & 0x80808080u;
        const bool check = nan_code != 0 || !finite_scale;
#pragma unroll
        for (int k = 0; k < 8; k += 2) {
            float lo, hi;
            e4m3x2_to_f32((q[p][k >> 2] >> (8 * (k & 3))) & 0xFFFF, lo, hi);
            lo = __fmul_rn(lo, scale);
            hi = __fmul_rn(hi, scale);
            y[k] = __float_as_uint(lo);
            y[k + 1] = __float_as_uint(hi);
        }
        if (check) {
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if ((y[k] & 0x7FFFFFFFu) > 0x7F800000u) y[k] = 0x7FC00000u;
        }
        char* dst = flat + (row_src[row] + col) * 4;
        if (T.aligned && allow256) {
            asm volatile("st.global.L1::no_allocate.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(dst), "r"(y[0]), "r"(y[1]),
                         "r"(y[2]), "r"(y[3]), "r"(y[4]), "r"(y[5]), "r"(y[6]), "r"(y[7])
                         : "memory");
        } else if (T.aligned) {
            asm volatile("st.global.L1::no_allocate.v4.b32 [%0], {%1,%2,%3,%4};" ::"l"(dst), "r"(y[0]), "r"(y[1]), "r"(y[2]),
                         "r"(y[3])
                         : "memory");
            asm volatile("st.global.L1::no_allocate.v4.b32 [%0], {%1,%2,%3,%4};" ::"l"(dst + 16), "r"(y[4]), "r"(y[5]),
                         "r"(y[6]), "r"(y[7])
                         : "memory");
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if (col + k < T.cols) *(uint32_t*)(dst + 4 * k) = y[k];
        }
    }
}

}  // namespace

int launch_quant(const dr_plan* p, const void* flat, void* arena, void* stream, uint64_t block_lo, uint64_t block_hi)
{
    if (block_hi > p->info.quant_blocks) block_hi = p->info.quant_blocks;
    if (block_lo >= block_hi) return DR_OK;
    const uint64_t blocks = block_hi - block_lo;
    if (blocks > 0x7FFFFFFFull) {
        set_error("too many quantisation blocks");
        return DR_ERR_UNSUPPORTED;
    }
    quant_kernel<<<(unsigned)blocks, kQThreads, 0, (cudaStream_t)stream>>>(
        p->d_qtensors, (uint32_t)p->qtensors.size(), p->d_qparts, p->d_qhints, p->qhint_shift, (const char*)flat,
        (char*)arena, (((uintptr_t)flat | (uintptr_t)arena) & 31) == 0, block_lo);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        set_error("quant kernel launch: %s", cudaGetErrorString(e));
        return DR_ERR_CUDA;
    }
    return DR_OK;
}

int launch_dequant(const dr_plan* p, const void* arena, void* flat, void* stream)
{
    const uint64_t blocks = p->info.quant_blocks;
    if (blocks == 0) return DR_OK;
    if (blocks > 0x7FFFFFFFull) {
        set_error("too many quantisation blocks");
        return DR_ERR_UNSUPPORTED;
    }
    dequant_kernel<<<(unsigned)blocks, kQThreads, 0, (cudaStream_t)stream>>>(
        p->d_qtensors, (uint32_t)p->qtensors.size(), p->d_qparts, p->d_qhints, p->qhint_shift, (const char*)arena,
        (char*)flat, (((uintptr_t)flat | (uintptr_t)arena) & 31) == 0);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        set_error("dequant kernel launch: %s", cudaGetErrorString(e));
        return DR_ERR_CUDA;
    }
    return DR_OK;
}

}  // namespace dr
