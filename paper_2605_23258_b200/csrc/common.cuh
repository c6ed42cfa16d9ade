// Device-side helpers shared by the kernels of libvector.
#ifndef VECTOR_COMMON_CUH_
#define VECTOR_COMMON_CUH_

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace vec {

void count_launch();      // host: one more kernel launched by the library

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

__device__ __forceinline__ void store_out(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_out(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// Monotone map from fp32 to uint32: a < b  <=>  ordered_key(a) < ordered_key(b)
// (-0 sorts just below +0; NaNs are not expected).
__device__ __forceinline__ uint32_t ordered_key(float f) {
    uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
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


// Rotary angle of channel pair c at position pos: pos * theta^(-2c/d).  The product is formed and
// reduced to [-pi, pi] in fp64 (positions reach 1e5 rad, where fp32 would be off by 1e-2), the sine
// and cosine of the remainder are taken in fp32.
__device__ __forceinline__ void rope_cos_sin(double pos, double inv_freq, float& cs, float& sn) {
    const double ang = pos * inv_freq;
    const double n = rint(ang * 0.15915494309189535);
    const double r = fma(-n, 6.283185307179586, ang);
    sincosf((float)r, &sn, &cs);
}
// The same for the tuned kernels, from the pair's 64-bit phase (turns per position as a fraction
// of 2^64, f = its low and high words): the top 32 bits of pos * phase modulo 2^64 are the angle
// in turns modulo one, exact to 2^-32 of a turn for any 32-bit position; read as a signed number
// they lie in [-1/2, 1/2), so the angle handed to sine and cosine lies in [-pi, pi).
__device__ __forceinline__ void rope_phase_cos_sin(uint32_t pos, uint2 f, float& cs, float& sn) {
    const uint32_t turns = pos * f.y + __umulhi(pos, f.x);
    const float ang = (float)(int)turns * 1.4629180792671596e-9f;      // 2 pi / 2^32
    __sincosf(ang, &sn, &cs);
}
// A shorter form for where issue slots are what costs (decode): the phase rounded to 32 bits.  The
// 32-bit product pos * phase32 is the angle in turns modulo one, taken as a signed number in
// [-1/2, 1/2); the phase's rounding leaves pos * 2^-33 of a turn (1e-4 rad at position 131072,
// 8e-4 rad at 2^20), well under the fp16 spacing of the turned key.
__device__ __forceinline__ void rope_phase32_cos_sin(uint32_t pos, uint32_t phase32, float& cs, float& sn) {
    const float ang = (float)(int)(pos * phase32) * 1.4629180792671596e-9f;      // 2 pi / 2^32
    __sincosf(ang, &sn, &cs);
}
// Inverse frequencies theta^(-2c/d), c < d/2, into shared memory (fp64); callers synchronise.
__device__ __forceinline__ void rope_fill_inv_freq(double* inv_freq, int d, float theta) {
    for (int c = threadIdx.x; c < d / 2; c += blockDim.x) inv_freq[c] = pow((double)theta, -2.0 * (double)c / (double)d);
}

// Kernel launch that may carry the programmatic-dependent attribute: with `dependent` the kernel may
// be scheduled while the kernel before it in the stream drains (once every block of that one has
// executed griddepcontrol.launch_dependents, or exited); it must execute griddepcontrol.wait before
// it touches that kernel's output.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_maybe_dependent(bool dependent, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                          cudaStream_t st, Args... args) {
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = dependent ? 1 : 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    count_launch();
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace vec
#endif
