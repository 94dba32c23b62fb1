// Shared device-side definitions of the Speculative Thinking decode library (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace st {

// Which rows a model pass works on.  Written by the host (explicit prefill/decode calls) or by the
// router kernel (generation), read by every kernel of the pass.
struct StepDesc {
    int32_t pos0;     // position of the first ingested token (= cached length before the pass)
    int32_t m;        // number of tokens ingested by the pass
    int32_t tok_off;  // tokens of the pass are tok[tok_off .. tok_off + m)
    int32_t emit;     // 1: the pass ends with LM head + sampling; 0: ingest only
};

// Device status bits (sticky).
enum : int32_t {
    DEV_BAD_TOKEN = 1,     // token id outside the vocabulary
    DEV_BAD_PAGE = 2,      // block table entry outside the pool
    DEV_WAIT_EXPIRED = 4,  // a bounded wait ran out
    DEV_LOG_FULL = 8       // an emission / handoff log overflowed
};

__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

__device__ __forceinline__ uint4 ldg_nc_v4(const void *p)
{
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ uint16_t f32_to_bf16_bits(float f)
{
    uint32_t u = __float_as_uint(f);
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

// The KV cache holds IEEE half precision (11 significand bits): with bf16 (8 bits) the rounding of K and V
// alone costs more than the logit tolerance once it has accumulated over 64 layers.
__device__ __forceinline__ uint16_t kv_bits(float f) { return __half_as_ushort(__float2half_rn(f)); }
__device__ __forceinline__ float kv_lo(uint32_t v) { return __half2float(__ushort_as_half((unsigned short)(v & 0xffffu))); }
__device__ __forceinline__ float kv_hi(uint32_t v) { return __half2float(__ushort_as_half((unsigned short)(v >> 16))); }

// Programmatic dependent launch.  pdl_launch: the next kernel of the stream, if it was launched with programmatic
// stream serialization, may become resident once every CTA of this grid has got here (or exited).  pdl_wait: block
// until the grids before this one have completed and their writes are visible; a thread calls it before its first
// access to memory they produce.  Both do nothing in a launch without the attribute.
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// v + the K-split partial sums ws[s * split_stride .. +3], s < k_splits <= 8, added in split order.  All loads are
// issued before the first addition, so a row costs one trip to L2 instead of one per split.
__device__ __forceinline__ float4 add_splits4(float4 v, const float *ws, size_t split_stride, int k_splits)
{
    float4 w[8];
#pragma unroll
    for (int s = 0; s < 8; ++s)
        if (s < k_splits) w[s] = __ldcg(reinterpret_cast<const float4 *>(ws + (size_t)s * split_stride));
#pragma unroll
    for (int s = 0; s < 8; ++s)
        if (s < k_splits) { v.x += w[s].x; v.y += w[s].y; v.z += w[s].z; v.w += w[s].w; }
    return v;
}

// a = hi + lo with hi = bf16(a), lo = bf16(a - hi): 16 significand bits in two bf16 values.
__device__ __forceinline__ void split_bf16(float a, uint16_t &hi, uint16_t &lo)
{
    hi = f32_to_bf16_bits(a);
    lo = f32_to_bf16_bits(a - __uint_as_float((uint32_t)hi << 16));
}

}  // namespace st
