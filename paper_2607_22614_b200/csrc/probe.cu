// Trivial contiguous streaming kernels in the repack kernel's launch shape (512 threads, one CTA per 48 KB
// of 32-byte units, 256-bit accesses past L1): what this GPU sustains for a given read : write mix.  The bench
// runs them beside the repack so that its bandwidth can be compared with a ceiling measured in the same run.
#include <cuda_runtime.h>

#include "dr_internal.h"

namespace dr {
namespace {

constexpr int kT = 512, kU = 3;  // threads per CTA, 32-byte units per thread

struct W8 {
    uint32_t w[8];
};
struct W4 {
    uint32_t w[4];
};
__device__ __forceinline__ W8 ld256(const void* p)
{
    W8 v;
    asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]), "=r"(v.w[4]), "=r"(v.w[5]), "=r"(v.w[6]),
                   "=r"(v.w[7])
                 : "l"(p));
    return v;
}
__device__ __forceinline__ W4 ld128(const void* p)
{
    W4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3])
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void st256(void* p, const W8& v)
{
    asm volatile("st.global.L1::no_allocate.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(v.w[0]), "r"(v.w[1]),
                 "r"(v.w[2]), "r"(v.w[3]), "r"(v.w[4]), "r"(v.w[5]), "r"(v.w[6]), "r"(v.w[7])
                 : "memory");
}
__device__ __forceinline__ void st128(void* p, const W4& v)
{
    asm volatile("st.global.L1::no_allocate.v4.b32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.w[0]), "r"(v.w[1]), "r"(v.w[2]),
                 "r"(v.w[3])
                 : "memory");
}

// One unit = the thread's access on the wider side: 32 bytes read (read, copy, narrow) or 32 bytes written
// (write, widen).
template <int MODE>
__global__ void __launch_bounds__(kT) probe_kernel(const char* __restrict__ a, char* __restrict__ b, uint32_t* sink)
{
    const uint64_t u0 = (uint64_t)blockIdx.x * kT * kU + threadIdx.x;
    if (MODE == DR_PROBE_READ) {
        W8 v[kU];
        uint32_t acc = 0;
#pragma unroll
        for (int j = 0; j < kU; ++j) v[j] = ld256(a + (u0 + j * kT) * 32);
#pragma unroll
        for (int j = 0; j < kU; ++j)
#pragma unroll
            for (int i = 0; i < 8; ++i) acc ^= v[j].w[i];
        if (acc == 0x9E3779B9u && sink) *sink = acc;  // keeps the loads alive; practically never taken
    } else if (MODE == DR_PROBE_WRITE) {
        W8 v;
#pragma unroll
        for (int i = 0; i < 8; ++i) v.w[i] = threadIdx.x + i;
#pragma unroll
        for (int j = 0; j < kU; ++j) st256(b + (u0 + j * kT) * 32, v);
    } else if (MODE == DR_PROBE_COPY) {
        W8 v[kU];
#pragma unroll
        for (int j = 0; j < kU; ++j) v[j] = ld256(a + (u0 + j * kT) * 32);
#pragma unroll
        for (int j = 0; j < kU; ++j) st256(b + (u0 + j * kT) * 32, v[j]);
    } else if (MODE == DR_PROBE_NARROW) {
        W8 v[kU];
#pragma unroll
        for (int j = 0; j < kU; ++j) v[j] = ld256(a + (u0 + j * kT) * 32);
#pragma unroll
        for (int j = 0; j < kU; ++j) {
            W4 o;
#pragma unroll
            for (int i = 0; i < 4; ++i)
                asm("cvt.rn.bf16x2.f32 %0, %1, %2;"
                    : "=r"(o.w[i])
                    : "f"(__uint_as_float(v[j].w[2 * i + 1])), "f"(__uint_as_float(v[j].w[2 * i])));
            st128(b + (u0 + j * kT) * 16, o);
        }
    } else if (MODE == DR_PROBE_NARROW4) {  // 32 bytes in, 8 bytes out per unit (the fp8 forward's mix)
        W8 v[kU];
#pragma unroll
        for (int j = 0; j < kU; ++j) v[j] = ld256(a + (u0 + j * kT) * 32);
#pragma unroll
        for (int j = 0; j < kU; ++j) {
            const uint32_t lo = (v[j].w[0] & 0xFF) | ((v[j].w[1] & 0xFF) << 8) | ((v[j].w[2] & 0xFF) << 16) | (v[j].w[3] << 24);
            const uint32_t hi = (v[j].w[4] & 0xFF) | ((v[j].w[5] & 0xFF) << 8) | ((v[j].w[6] & 0xFF) << 16) | (v[j].w[7] << 24);
            asm volatile("st.global.L1::no_allocate.v2.b32 [%0], {%1,%2};" ::"l"(b + (u0 + j * kT) * 8), "r"(lo), "r"(hi) : "memory");
        }
    } else if (MODE == DR_PROBE_WIDEN4) {  // 8 bytes in, 32 bytes out per unit (the fp8 inverse's mix)
        uint32_t lo[kU], hi[kU];
#pragma unroll
        for (int j = 0; j < kU; ++j)
            asm volatile("ld.global.nc.L1::no_allocate.v2.b32 {%0,%1}, [%2];" : "=r"(lo[j]), "=r"(hi[j]) : "l"(a + (u0 + j * kT) * 8));
#pragma unroll
        for (int j = 0; j < kU; ++j) {
            W8 o;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                o.w[i] = (lo[j] >> (8 * i)) << 23;
                o.w[4 + i] = (hi[j] >> (8 * i)) << 23;
            }
            st256(b + (u0 + j * kT) * 32, o);
        }
    } else {  // DR_PROBE_WIDEN
        W4 v[kU];
#pragma unroll
        for (int j = 0; j < kU; ++j) v[j] = ld128(a + (u0 + j * kT) * 16);
#pragma unroll
        for (int j = 0; j < kU; ++j) {
            W8 o;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                o.w[2 * i] = v[j].w[i] << 16;
                o.w[2 * i + 1] = v[j].w[i] & 0xFFFF0000u;
            }
            st256(b + (u0 + j * kT) * 32, o);
        }
    }
}

}  // namespace
}  // namespace dr

extern "C" int dr_probe_stream(uint32_t mode, const void* a_dev, void* b_dev, uint64_t n_bytes, void* cuda_stream)
{
    using namespace dr;
    const uint64_t tile = (uint64_t)kT * kU * 32;  // bytes of the wider side per CTA
    if (mode > DR_PROBE_WIDEN4 || n_bytes == 0 || n_bytes % tile || (mode != DR_PROBE_WRITE && !a_dev) ||
        (mode != DR_PROBE_READ && !b_dev)) {
        set_error("dr_probe_stream: bad mode, NULL buffer, or byte count not a multiple of %llu", (unsigned long long)tile);
        return DR_ERR_INVALID;
    }
    if (((uintptr_t)a_dev | (uintptr_t)b_dev) & 31) {
        set_error("dr_probe_stream: buffers must be 32-byte aligned");
        return DR_ERR_ALIGN;
    }
    const uint64_t ctas = n_bytes / tile;
    if (ctas > 0x7FFFFFFFull) {
        set_error("dr_probe_stream: too many bytes for one launch");
        return DR_ERR_UNSUPPORTED;
    }
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const char* a = (const char*)a_dev;
    char* b = (char*)b_dev;
    const unsigned g = (unsigned)ctas;
    switch (mode) {
    case DR_PROBE_READ: probe_kernel<DR_PROBE_READ><<<g, kT, 0, s>>>(a, b, nullptr); break;
    case DR_PROBE_WRITE: probe_kernel<DR_PROBE_WRITE><<<g, kT, 0, s>>>(a, b, nullptr); break;
    case DR_PROBE_COPY: probe_kernel<DR_PROBE_COPY><<<g, kT, 0, s>>>(a, b, nullptr); break;
    case DR_PROBE_NARROW: probe_kernel<DR_PROBE_NARROW><<<g, kT, 0, s>>>(a, b, nullptr); break;
    case DR_PROBE_NARROW4: probe_kernel<DR_PROBE_NARROW4><<<g, kT, 0, s>>>(a, b, nullptr); break;
    case DR_PROBE_WIDEN4: probe_kernel<DR_PROBE_WIDEN4><<<g, kT, 0, s>>>(a, b, nullptr); break;
    default: probe_kernel<DR_PROBE_WIDEN><<<g, kT, 0, s>>>(a, b, nullptr); break;
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        set_error("probe kernel launch: %s", cudaGetErrorString(e));
        return DR_ERR_CUDA;
    }
    return DR_OK;
}
