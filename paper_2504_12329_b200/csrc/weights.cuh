// Seeded random-init weights, generated on the device.
//
// Element idx of a tensor with stream key K is built from outputs 3*idx+1 .. 3*idx+3 of the
// SplitMix64 stream with initial state K (Steele, Lea, Flood 2014): their twelve 16-bit fields are
// summed (an Irwin-Hall(12) variate, standard deviation ~65536), centred, scaled to unit variance
// and multiplied by 0.02, then rounded to bf16 (nearest even).  Only integer operations, one exact
// power-of-two scaling and one IEEE multiply are involved, so any conforming implementation
// produces the same bits.
#pragma once
#include "st_common.cuh"

namespace st {

constexpr uint64_t kGamma = 0x9e3779b97f4a7c15ULL;

__host__ __device__ __forceinline__ uint64_t splitmix_out(uint64_t z)
{
    z = (z ^ (z >> 30)) * 0xbf58476d1ce4e5b9ULL;
    z = (z ^ (z >> 27)) * 0x94d049bb133111ebULL;
    return z ^ (z >> 31);
}

// Key of the stream of tensor `tid` of model `tag` under `seed`.
__host__ __device__ inline uint64_t tensor_stream_key(uint64_t seed, uint32_t tag, uint32_t tid)
{
    uint64_t k = splitmix_out(seed + kGamma);
    k = splitmix_out(k + kGamma + tag);
    return splitmix_out(k + kGamma + tid);
}

__device__ __forceinline__ uint32_t sum16x4(uint64_t r)
{
    return (uint32_t)(r & 0xffffu) + (uint32_t)((r >> 16) & 0xffffu) + (uint32_t)((r >> 32) & 0xffffu) +
           (uint32_t)(r >> 48);
}

__device__ __forceinline__ float seeded_weight(uint64_t key, uint64_t idx)
{
    const uint64_t c = key + (3 * idx + 1) * kGamma;
    const uint32_t s = sum16x4(splitmix_out(c)) + sum16x4(splitmix_out(c + kGamma)) +
                       sum16x4(splitmix_out(c + 2 * kGamma));
    const float z = (float)((int32_t)s - 6 * 65535) * 1.52587890625e-05f;  // exact: * 2^-16
    return __fmul_rn(0.02f, z);
}

// out[(r * row_mul + row_add) * cols + c] = element (r0 + r) * cols + c of the stream, as bf16 bits.
// row_mul/row_add let several logical tensors interleave their rows in one physical matrix.
__global__ void fill_bf16_kernel(uint16_t *out, uint64_t key, uint64_t r0, uint64_t rows, uint64_t cols,
                                 uint32_t row_mul, uint32_t row_add)
{
    const uint64_t n = rows * cols;
    for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t r = i / cols, c = i - r * cols;
        out[(r * row_mul + row_add) * cols + c] = f32_to_bf16_bits(seeded_weight(key, (r0 + r) * cols + c));
    }
}

// Same values widened to fp32 (biases are kept in fp32 on the device; the values are bf16-exact).
__global__ void fill_f32_kernel(float *out, uint64_t key, uint64_t n)
{
    for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x)
        out[i] = __uint_as_float((uint32_t)f32_to_bf16_bits(seeded_weight(key, i)) << 16);
}

__global__ void fill_const_f32_kernel(float *out, float v, uint64_t n)
{
    for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x)
        out[i] = v;
}

}  // namespace st
