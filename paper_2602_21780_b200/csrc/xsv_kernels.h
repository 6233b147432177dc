// Host-side launchers of the xsv kernels (one per phase of the step).
#pragma once
#include "xsv_common.cuh"
#include "xsv_device.h"

// dtype: 0 = fp16, 1 = bf16 (xsv_dtype).

// Multiprocessors of the current device (queried once per device).
int xsv_sm_count();

// Eq. 3-4 folded by linearity: per-(head, chunk) partial sums of the pooling-weighted
// queries; qpart [H * XSV_QCHUNKS][64].
#define XSV_QCHUNKS 8
cudaError_t xsv_launch_qtilde(const void* Q, int dtype, int H, int F, int n_special, int g,
                              float* qpart, cudaStream_t st);

// Eq. 5-7: scores[j] for the middle segment positions [T_first, T_c).
cudaError_t xsv_launch_score(const LayerView& lv, int H, int T_first, int T_c, const float* qpart,
                             float qnorm /* 1 / (H * N_pooled) */, float* scores, cudaStream_t st);

// bits == 16: same scores from the raw 16-bit keys.
cudaError_t xsv_launch_score_raw(const LayerView& lv, int dtype, int H, int T_first, int T_c,
                                 const float* qpart, float qnorm, float* scores, cudaStream_t st);

// Eq. 8: top-k of scores[0..n) (score descending, position ascending).  Writes
// srcmap[0..k) = T_first + selected positions (ascending) and
// dscal[0] = number of frozen key groups = min(first evicted position, T_c) / 64.
cudaError_t xsv_launch_select(const float* scores, int n, int k, int T_first, int T_c, int* srcmap,
                              int* dscal, cudaStream_t st);

// Eq. 9-11 for the new cache order, one launch (bits < 16).
// Keys: the key groups are rebuilt.  New position p < n_old_new comes from cache position
//   (p < T_first ? p : srcmap[p - T_first]) (srcmap == nullptr: identity); p >= n_old_new is token
//   p - n_old_new of the frame.  Groups below the frozen count (fz_dev ? *fz_dev : fz_host) are copied
//   verbatim (skipped when src and dst are the same buffer).
// Values: kept rows move verbatim (codes, scale, zero-point, origin) to new positions [0, n_old_new) when
//   dst != src; the frame's rows are quantised per token into [n_old_new, n_old_new + F), with their origins
//   origin0 + token index.
//   with_values == false leaves the values to xsv_launch_values.
cudaError_t xsv_launch_compress(const LayerView& src, const LayerView& dst, const void* Kf, const void* Vf,
                                int dtype, int H, int F, int n_old_new, int T_new, int T_first,
                                const int* srcmap, const int* fz_dev, int fz_host, long long origin0,
                                bool with_values, int* status, cudaStream_t st);

// The value part of the above as launches of its own (two small kernels), for a stream other than the keys'.
cudaError_t xsv_launch_values(const LayerView& src, const LayerView& dst, const void* Vf, int dtype, int H, int F,
                              int n_old_new, int T_first, const int* srcmap, long long origin0, int* status,
                              cudaStream_t st);

// bits == 16: gather / append raw 16-bit rows of K and V (no quantisation).
cudaError_t xsv_launch_raw_update(const LayerView& src, const LayerView& dst, const void* Kf,
                                  const void* Vf, int H, int F, int n_old_new, int T_first,
                                  const int* srcmap, long long origin0, cudaStream_t st);

// Eq. 2 + Eq. 12: out = softmax(Q [K~;K]^T / 8) [V~;V]; warp-level mma.sync kernel.
cudaError_t xsv_launch_attn_mma(const LayerView& lv, int T_c, const void* Q, const void* K, const void* V,
                                void* out, int dtype, int H, int F, cudaStream_t st);

// Same contract; tcgen05 + TMEM kernel, to be followed by xsv_launch_attn_tc5_merge
// with the same arguments: a small kernel that merges the parts of query tiles
// shared by several CTAs.  `workspace` holds those parts:
// xsv_attn_tc5_workspace_bytes() bytes of device memory; nullptr returns
// cudaErrorNotSupported.  A bounded wait that runs out sets XSV_DEV_TIMEOUT in
// *status.  spare_sms multiprocessors are left without a CTA (for a kernel that
// runs beside this one on another stream).
size_t xsv_attn_tc5_workspace_bytes();
cudaError_t xsv_launch_attn_tc5(const LayerView& lv, int T_c, const void* Q, const void* K, const void* V,
                                void* out, int dtype, int H, int F, float* workspace, int* status,
                                int spare_sms, cudaStream_t st);
cudaError_t xsv_launch_attn_tc5_merge(const LayerView& lv, int T_c, const void* Q, const void* K, const void* V,
                                      void* out, int dtype, int H, int F, float* workspace, int* status,
                                      int spare_sms, cudaStream_t st);

// The attention of several independent streams (each with its own cache view, inputs, output and status word) and
// the merge that follows, as one launch each; all streams share dtype, bit width and head count.  `workspace` as above.
cudaError_t xsv_launch_attn_tc5_batch(int n, const LayerView* lvs, const int* T_cs, const void* const* Qs,
                                      const void* const* Ks, const void* const* Vs, void* const* outs, int dtype, int H,
                                      const int* Fs, float* workspace, int* const* statuses, cudaStream_t st);
// Streams per attention launch that xsv_launch_attn_tc5_batch would choose for these cache and frame lengths on a
// device with `sms` multiprocessors (host arithmetic only); -1 for bad arguments.
int xsv_attn_batch_group_size(int n, const int* T_cs, const int* Fs, int H, int sms);

// One small kernel whose only wait can never be satisfied: it must come back after the
// attention kernel's wait limit with XSV_DEV_TIMEOUT set in *status (device int).
cudaError_t xsv_launch_wait_selftest(int* status, cudaStream_t st);
