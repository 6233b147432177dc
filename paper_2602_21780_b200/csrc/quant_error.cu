// Quantisation error of the two granularities of Eq. 11 (the quantity of
// Table 1): quantise a [heads][tokens][64] tensor per channel over groups of 64
// tokens, or per token over its 64 channels (Eq. 9-10), dequantise (Eq. 12) and
// average the squared error.  One block per (64-token group, head); the sums
// are accumulated in float64 in a fixed order (deterministic).
#include <vector>

#include "../../include/xsv.h"
#include "xsv_kernels.h"

namespace {

template <typename T>
__global__ void __launch_bounds__(256) quant_error_kernel(const T* __restrict__ x, int n_tokens, int bits, int per_channel,
                                                          double* __restrict__ partial, int* __restrict__ status) {
    __shared__ float tile[XSV_G][XSV_D + 1];
    __shared__ float ps[64], pz[64];
    __shared__ double red[8];
    const int g = blockIdx.x, h = blockIdx.y, tid = threadIdx.x;
    const int t0 = g * XSV_G, cnt = min(XSV_G, n_tokens - t0), nmax = (1 << bits) - 1;
    for (int i = tid; i < cnt * XSV_D; i += 256) {
        const int r = i >> 6, c = i & 63;
        tile[r][c] = xsv_to_float<T>(x[((size_t)h * n_tokens + t0 + r) * XSV_D + c]);
    }
    __syncthreads();
    if (tid < 64) {
        // per channel: thread = channel, over the group's tokens; per token: thread = token, over its channels
        const int len = per_channel ? cnt : XSV_D;
        if (per_channel || tid < cnt) {
            float mn = INFINITY, mx = -INFINITY;
            for (int k = 0; k < len; ++k) {
                const float v = per_channel ? tile[k][tid] : tile[tid][k];
                mn = fminf(mn, v);
                mx = fmaxf(mx, v);
            }
            float s, z;
            xsv_quant_params(mn, mx, nmax, s, z);
            ps[tid] = s;
            pz[tid] = z;
        }
    }
    __syncthreads();
    double acc = 0.0;
    for (int i = tid; i < cnt * XSV_D; i += 256) {
        const int r = i >> 6, c = i & 63, k = per_channel ? c : r;
        const float v = tile[r][c], s = ps[k];
        const int code = xsv_quant_code(v, s, __frcp_rn(s), pz[k], nmax);
        const double e = (double)v - (double)xsv_dequant(code, pz[k], s);
        acc += e * e;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    if ((tid & 31) == 0) red[tid >> 5] = acc;
    __syncthreads();
    if (tid == 0) {
        double s = 0.0;
        for (int k = 0; k < 8; ++k) s += red[k];
        partial[(size_t)h * gridDim.x + g] = s;
    }
}

__global__ void __launch_bounds__(256) quant_error_sum_kernel(const double* __restrict__ partial, int n, double count,
                                                              double* __restrict__ out) {
    __shared__ double red[256];
    double s = 0.0;
    for (int i = threadIdx.x; i < n; i += 256) s += partial[i];
    red[threadIdx.x] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int k = 0; k < 256; ++k) t += red[k];
        *out = t / count;
    }
}

}  // namespace

extern "C" xsv_status xsv_quantization_mse(const void* x, int heads, long long n_tokens, xsv_dtype dtype, int bits,
                                           int per_channel, double* mse_host, void* stream) {
    if (!x || !mse_host || heads <= 0 || n_tokens <= 0 || n_tokens > (1LL << 30)) return XSV_ERR_ARG;
    if (dtype != XSV_F16 && dtype != XSV_BF16) return XSV_ERR_ARG;
    if (bits != 2 && bits != 4 && bits != 8) return XSV_ERR_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const int groups = (int)((n_tokens + XSV_G - 1) / XSV_G);
    const size_t n_part = (size_t)groups * heads;
    double* scratch = nullptr;
    if (cudaMallocAsync((void**)&scratch, (n_part + 2) * sizeof(double), st) != cudaSuccess) {
        cudaGetLastError();
        return XSV_ERR_OOM;
    }
    int* status = reinterpret_cast<int*>(scratch + n_part + 1);
    cudaMemsetAsync(status, 0, sizeof(int), st);
    dim3 grid(groups, heads);
    if (dtype == XSV_F16)
        quant_error_kernel<__half><<<grid, 256, 0, st>>>((const __half*)x, (int)n_tokens, bits, per_channel ? 1 : 0, scratch, status);
    else
        quant_error_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)x, (int)n_tokens, bits, per_channel ? 1 : 0, scratch, status);
    quant_error_sum_kernel<<<1, 256, 0, st>>>(scratch, (int)n_part, (double)heads * (double)n_tokens * XSV_D, scratch + n_part);
    xsv_count_launch(2);
    double result = 0.0;
    int dev_status = 0;
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaMemcpyAsync(&result, scratch + n_part, sizeof(double), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(&dev_status, status, sizeof(int), cudaMemcpyDeviceToHost, st);
    cudaFreeAsync(scratch, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return XSV_ERR_CUDA;
    *mse_host = result;
    (void)dev_status;
    return XSV_OK;
}
