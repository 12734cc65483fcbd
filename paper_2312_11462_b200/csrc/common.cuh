// Shared device/host helpers of the review-step library (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include "../../include/csd.h"

namespace csd {

// ---- host side --------------------------------------------------------------------------------
// Device status word: one int in mapped pinned host memory, written by kernels through its
// device alias and read by the host after a stream synchronise.  Null until first use.
int* status_word_device();          // device-visible alias (allocates the mapping on first call)
csd_status note_cuda(cudaError_t e); // records the error text, returns CSD_ERR_CUDA (or CSD_OK)
void count_launch(int n = 1);        // launch counter read by csd_cascade_generate
long long launches_so_far();

#define CSD_CUDA(expr)                                        \
    do {                                                      \
        cudaError_t e__ = (expr);                             \
        if (e__ != cudaSuccess) return csd::note_cuda(e__);   \
    } while (0)

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Launch configuration with programmatic stream serialization: the kernel may start while its
// predecessor in the stream is still running and must execute griddepcontrol.wait before it
// touches anything the predecessor writes.
struct PdlLaunch {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    PdlLaunch(dim3 grid, dim3 block, size_t smem, cudaStream_t st) {
        cfg = cudaLaunchConfig_t{};
        cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
    }
};

// ---- device side ------------------------------------------------------------------------------
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void set_status(int* status, int code) {
    if (status) atomicCAS(status, 0, code);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// two bf16 packed in a 32-bit word -> two fp32 (bf16 is the top half of an fp32)
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ float bf16_bits_to_float(uint16_t h) { return __uint_as_float(((uint32_t)h) << 16); }
__device__ __forceinline__ uint16_t float_to_bf16_bits(float f) {
    return __bfloat16_as_ushort(__float2bfloat16_rn(f));
}

// x = b1 + b2 + b3 with bf16 terms (8 + 8 + 8 mantissa bits: exact for an fp32 value); the
// tensor-core GEMM takes its fp32 rows in this form
__device__ __forceinline__ void split3(float x, uint16_t& b1, uint16_t& b2, uint16_t& b3) {
    b1 = float_to_bf16_bits(x);
    const float r1 = x - bf16_bits_to_float(b1);
    b2 = float_to_bf16_bits(r1);
    b3 = float_to_bf16_bits(r1 - bf16_bits_to_float(b2));
}

// 128-bit streaming load that does not allocate in L1 (weights are read exactly once)
__device__ __forceinline__ uint4 ldg_stream(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

}  // namespace csd
