// Importance scores without any allocation: the scratch of the pooled-query
// reduction lives in a fixed device array that is part of the library image.
#include <mutex>

#include "../../include/xsv.h"
#include "xsv_kernels.h"

#define XSV_STATIC_MAX_HEADS 64

// Partial sums of the pooling-weighted queries, [heads][XSV_QCHUNKS][64] floats.
// 128 KB, held by every GPU that loads the library until the process exits.
static __device__ __align__(256) float g_static_qpart[XSV_STATIC_MAX_HEADS * XSV_QCHUNKS * 64];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_mu;
float* g_qpart_addr[kMaxDevices];   // device address of g_static_qpart, per device, once resolved

// In host code `g_static_qpart` is only a handle for the runtime, not a device
// address; the address a kernel can use comes from cudaGetSymbolAddress, asked
// once per device while that device is current.
xsv_status static_scratch(float** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return XSV_ERR_CUDA;
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_qpart_addr[dev]) {
        float* p = nullptr;
        if (cudaGetSymbolAddress((void**)&p, g_static_qpart) != cudaSuccess || !p) {
            cudaGetLastError();
            return XSV_ERR_CUDA;
        }
        g_qpart_addr[dev] = p;
    }
    *out = g_qpart_addr[dev];
    return XSV_OK;
}
}  // namespace

extern "C" xsv_status xsv_importance_scores_static(const void* Q, const void* keys, int heads, int n_tokens,
                                                   long long n_keys, xsv_dtype dtype, int n_special, int pool_group,
                                                   float* scores, void* stream) {
    if (!Q || !keys || !scores || heads <= 0 || n_tokens <= 0 || n_keys <= 0 || n_keys > (1LL << 30)) return XSV_ERR_ARG;
    if (heads > XSV_STATIC_MAX_HEADS) return XSV_ERR_LIMIT;
    if (dtype != XSV_F16 && dtype != XSV_BF16) return XSV_ERR_ARG;
    if (n_special < 0 || n_special > n_tokens || pool_group <= 0) return XSV_ERR_ARG;
    if (((uintptr_t)Q | (uintptr_t)keys) & 15) return XSV_ERR_SHAPE;
    float* qpart = nullptr;
    xsv_status s = static_scratch(&qpart);
    if (s != XSV_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    LayerView lv{};
    lv.kcodes = (uint8_t*)const_cast<void*>(keys);
    lv.cap = n_keys;
    lv.rowb = XSV_D * 2;
    lv.bits = 16;
    const int n_pooled = n_special + (n_tokens - n_special + pool_group - 1) / pool_group;
    const float qnorm = 1.0f / ((float)heads * (float)n_pooled);
    // The first kernel overwrites every partial sum the second one reads
    // (heads * XSV_QCHUNKS rows), so nothing left by an earlier call is used and
    // nothing needs clearing.
    cudaError_t e = xsv_launch_qtilde(Q, (int)dtype, heads, n_tokens, n_special, pool_group, qpart, st);
    if (e == cudaSuccess) e = xsv_launch_score_raw(lv, (int)dtype, heads, 0, (int)n_keys, qpart, qnorm, scores, st);
    return e == cudaSuccess ? XSV_OK : XSV_ERR_CUDA;
}
