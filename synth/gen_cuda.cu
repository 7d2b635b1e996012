/*
 * Seeded synthetic state generator (device side).
 *
 * Same counter-based function as the host generator: a pure function of
 * (seed, buffer_id, index) made of 64-bit integer mixing and one fp32
 * multiply.  It exists so that tens of GB of state can be created, and
 * later re-derived for a byte-exact comparison, without a host copy.  Input
 * generation and comparison only: no layout map, no cast, no staging logic.
 */
#include <cuda_runtime.h>
#include <cstdint>

namespace {

constexpr uint64_t kG = 0x9E3779B97F4A7C15ull;

__device__ __forceinline__ uint64_t mix(uint64_t x)
{
    x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27; x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    return x;
}

__device__ __forceinline__ uint32_t lanes16(uint64_t w)
{
    return (uint32_t)(w & 0xFFFF) + (uint32_t)((w >> 16) & 0xFFFF) +
           (uint32_t)((w >> 32) & 0xFFFF) + (uint32_t)(w >> 48);
}

__device__ __forceinline__ uint32_t gen_bits(uint64_t seed, uint32_t buffer_id, uint64_t index)
{
    uint64_t z = seed ^ ((uint64_t)buffer_id * 0xD1B54A32D192ED03ull);
    uint64_t a = mix(z + (index + 1) * kG);
    uint64_t b = mix(a + kG);
    uint64_t c = mix(b + kG);
    int32_t s = (int32_t)(lanes16(a) + lanes16(b)) - 262140;
    uint32_t kb = buffer_id == 1 ? 0x32A0879Eu : buffer_id == 2 ? 0x2DA461EAu : 0x34C8A986u;
    uint32_t u = __float_as_uint(__fmul_rn(__int2float_rn(s), __uint_as_float(kb)));
    if (buffer_id == 0 && c % 100 == 0) u = (u & 0xFFFF0000u) | 0x8000u;
    if (buffer_id == 2) u &= 0x7FFFFFFFu;
    return u;
}

__global__ void fill_f32_kernel(uint32_t* out, uint64_t seed, uint32_t buffer_id, uint64_t start, uint64_t n)
{
    uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
        out[i] = gen_bits(seed, buffer_id, start + i);
}

__global__ void fill_bf16_kernel(uint16_t* out, uint64_t seed, uint32_t buffer_id, uint64_t start, uint64_t n)
{
    uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
        out[i] = (uint16_t)(gen_bits(seed, buffer_id, start + i) >> 16);
}

__global__ void mismatch_f32_kernel(const uint32_t* buf, uint64_t seed, uint32_t buffer_id, uint64_t start,
                                    uint64_t n, unsigned long long* count)
{
    uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    unsigned long long bad = 0;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
        bad += buf[i] != gen_bits(seed, buffer_id, start + i);
    for (int o = 16; o; o >>= 1) bad += __shfl_xor_sync(0xFFFFFFFFu, bad, o);
    if ((threadIdx.x & 31) == 0 && bad) atomicAdd(count, bad);
}

int grid_for(uint64_t n)
{
    uint64_t b = (n + 255) / 256;
    return (int)(b < 1 ? 1 : b > 148 * 16 ? 148 * 16 : b);
}

}  // namespace

extern "C" {

/* Fill device fp32 buffer `dev[0..n)` with elements start..start+n of `buffer_id`. Asynchronous on `stream`. */
int synth_cuda_fill_f32(void* dev, uint64_t seed, uint32_t buffer_id, uint64_t start, uint64_t n, void* stream)
{
    if (n == 0) return 0;
    fill_f32_kernel<<<grid_for(n), 256, 0, (cudaStream_t)stream>>>((uint32_t*)dev, seed, buffer_id, start, n);
    return (int)cudaGetLastError();
}

int synth_cuda_fill_bf16(void* dev, uint64_t seed, uint32_t buffer_id, uint64_t start, uint64_t n, void* stream)
{
    if (n == 0) return 0;
    fill_bf16_kernel<<<grid_for(n), 256, 0, (cudaStream_t)stream>>>((uint16_t*)dev, seed, buffer_id, start, n);
    return (int)cudaGetLastError();
}

/* Adds to *dev_count (a device uint64 the caller zeroed) the number of elements of dev[0..n) whose bits differ
 * from the generator's elements start..start+n. Asynchronous on `stream`. */
int synth_cuda_mismatch_f32(const void* dev, uint64_t seed, uint32_t buffer_id, uint64_t start, uint64_t n,
                            void* dev_count, void* stream)
{
    if (n == 0) return 0;
    mismatch_f32_kernel<<<grid_for(n), 256, 0, (cudaStream_t)stream>>>((const uint32_t*)dev, seed, buffer_id, start, n,
                                                                       (unsigned long long*)dev_count);
    return (int)cudaGetLastError();
}

}  // extern "C"
