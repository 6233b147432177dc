// Shared declarations of the xsv CUDA library: cache layout in HBM, the
// per-layer view handed to kernels, small device helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#define XSV_D 64   // channels per head (head_dim)
#define XSV_G 64   // quantisation group size (tokens for K, channels for V)
#ifndef XSV_MAX_BATCH
#define XSV_MAX_BATCH 8   // streams per batched launch (also in the public header)
#endif

// Bits of the sticky device status word.
#define XSV_DEV_TIMEOUT 1
#define XSV_DEV_RANGE 2
// Beside XSV_DEV_TIMEOUT: which wait of the attention kernel ran out (diagnostic only).
#define XSV_DEV_SITE_STAGE 0x100     // a producer waiting for a free kv stage
#define XSV_DEV_SITE_S 0x200         // a softmax warp waiting for S
#define XSV_DEV_SITE_PV 0x400        // a softmax warp waiting for the completion of P V
#define XSV_DEV_SITE_Q 0x800         // the MMA warp waiting for a unit's query tiles
#define XSV_DEV_SITE_K 0x1000        // the MMA warp waiting for a kv stage to be filled
#define XSV_DEV_SITE_P 0x4000        // the MMA warp waiting for a sub-tile's probabilities
#define XSV_DEV_SITE_SELFTEST 0x2000

// One layer's cache as the kernels see it.  All arrays live in one slab.
//   kcodes/vcodes [H][cap][rowb] : packed codes of one (head, token) row, code c
//                                  at bit offset c*bits of the row (little endian);
//                                  rowb = 64*bits/8 bytes.  bits == 16: the raw
//                                  16-bit elements.
//   kscale/kzero  [H][capg][64]  : Eq. 10 parameters per channel per 64-token group: the scale and the
//                                  offset (the group's minimum, in value units).
//   vscale/vzero  [H][cap]       : the same per token (64 channels).
//   origin        [cap]          : frame_index * F + token_index of each slot.
struct LayerView {
    uint8_t* kcodes;
    float* kscale;
    float* kzero;
    uint8_t* vcodes;
    float* vscale;
    float* vzero;
    long long* origin;
    long long cap;
    int capg;
    int rowb;
    int bits;
};

template <typename T> __device__ __forceinline__ float xsv_to_float(T v);
template <> __device__ __forceinline__ float xsv_to_float<__half>(__half v) { return __half2float(v); }
template <> __device__ __forceinline__ float xsv_to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T xsv_from_float(float v);
template <> __device__ __forceinline__ __half xsv_from_float<__half>(float v) { return __float2half_rn(v); }
template <> __device__ __forceinline__ __nv_bfloat16 xsv_from_float<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// Pack two floats into one 32-bit register of two 16-bit values (lo = a).
template <typename T> __device__ __forceinline__ uint32_t xsv_pack2(float a, float b);
template <> __device__ __forceinline__ uint32_t xsv_pack2<__half>(float a, float b) {
    __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}
template <> __device__ __forceinline__ uint32_t xsv_pack2<__nv_bfloat16>(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}

// Exact int -> float for |v| < 2^22 without the conversion unit: 1.5 * 2^23 + v
// is exact in float32 and so is the subtraction that follows.
__device__ __forceinline__ float xsv_small_int_to_float(int v) {
    return __fadd_rn(__int_as_float(0x4B400000 + v), -12582912.f);
}

// Eq. 12 in the minimum-offset form: x~ = code * s + z, a float32 multiply then a float32 add (two roundings,
// never a fused multiply-add: the re-quantisation of kept keys starts from these values and must see the same
// bits everywhere).
__device__ __forceinline__ float xsv_dequant(int code, float z, float s) {
    return __fadd_rn(__fmul_rn(xsv_small_int_to_float(code), s), z);
}

// Eq. 10 in float32, one rounding per operation: s = (mx - mn) / n, offset z = mn; degenerate groups
// (s below the smallest normal, which includes mx == mn) take s = 1.
__device__ __forceinline__ void xsv_quant_params(float mn, float mx, int n, float& s, float& z) {
    s = __fdiv_rn(__fsub_rn(mx, mn), __int2float_rn(n));
    if (!(s >= 1.17549435e-38f)) s = 1.f;
    z = mn;
}

// Eq. 9: clamp(round((x - z) / s), 0, n), round = nearest-even, with (x - z) one float32 subtraction and the
// quotient the IEEE float32 one.  inv_s = 1 / s (correctly rounded).  y * inv_s lies within 2^-22 |y / s| of
// the true quotient, as does the rounded quotient itself; unless y * inv_s comes within 2^-20 |y / s| of a
// rounding boundary (a half-integer) both therefore round to the same integer, and the division is skipped.
// Near a boundary the exact division decides.
__device__ __forceinline__ int xsv_quant_code(float x, float s, float inv_s, float z, int n) {
    const float d = __fsub_rn(x, z);
    const float y = __fmul_rn(d, inv_s);
    int q;
    if (fabsf(y) < 2097152.f) {
        // round to nearest even by adding and subtracting 1.5 * 2^23 (exact for |y| < 2^21); the integer is
        // in the low mantissa bits of the sum
        const float t = __fadd_rn(y, 12582912.f);
        const float r = __fadd_rn(t, -12582912.f);
        q = __float_as_int(t) - 0x4B400000;
        if (fabsf(fabsf(y - r) - 0.5f) < fabsf(y) * 9.5367431640625e-7f) q = __float2int_rn(rintf(__fdiv_rn(d, s)));
    } else {
        q = __float2int_rn(rintf(__fdiv_rn(d, s)));   // saturating
    }
    return q < 0 ? 0 : (q > n ? n : q);
}

// Programmatic dependent launch.  A kernel launched with xsv_launch_dep may be scheduled while the kernel before
// it in the stream is still running (once all of that kernel's blocks have called xsv_dep_release or exited); it must
// call xsv_dep_sync() before it touches anything the earlier kernel reads or writes: the call returns when that kernel
// has completed and its writes are visible.  Every kernel of the step calls xsv_dep_release() first, so that its own
// successor is scheduled early too; what is saved is the launch latency between dependent kernels.  Without the
// launch attribute both calls do nothing.
__device__ __forceinline__ void xsv_dep_release() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void xsv_dep_sync() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

bool xsv_dep_launch_enabled();   // false when the environment variable XSV_NO_DEP_LAUNCH is set (host side)

template <typename... KArgs, typename... Args>
inline cudaError_t xsv_launch_dep(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                  Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = xsv_dep_launch_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Launch counter (host side), bumped by every kernel launch of the library.
void xsv_count_launch(int n = 1);
