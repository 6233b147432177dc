// Bandwidth-bound kernels of the step: pooled-query reduction and importance
// scores (Eq. 3-7), top-k selection (Eq. 8), quantise-and-pack of the new
// cache order (Eq. 9-11).
#include <cstdlib>

#include "xsv_kernels.h"

namespace {

// ---------------------------------------------------------------------------
// Eq. 3-4 (+ the row mean of Eq. 7) by linearity:
//   q~[c] = 1/(H*N_pooled) * sum_h sum_i w_i Q[h,i,c],
//   w_i = 1 for special tokens, 1/|group| for a patch token in a pooling group.
// This kernel writes the fixed-order partial sums per (head, token chunk).
// ---------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) qtilde_partial_kernel(const T* __restrict__ Q, int F, int n_special,
                                                             int g, float* __restrict__ qpart) {
    xsv_dep_release();
    xsv_dep_sync();
    const int h = blockIdx.y, chunk = blockIdx.x;
    const int per = (F + XSV_QCHUNKS - 1) / XSV_QCHUNKS;
    const int i0 = chunk * per, i1 = min(F, i0 + per);
    const int c8 = threadIdx.x & 7, r = threadIdx.x >> 3;      // 8 channels (one 16-byte load), 32 rows in flight
    const int n_patch = F - n_special;
    float a[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) a[e] = 0.f;
    // six rows per thread at a time, all loads issued before the first use
    for (int base = i0 + r; base < i1; base += 32 * 6) {
        uint4 v[6];
        float w[6];
#pragma unroll
        for (int k = 0; k < 6; ++k) {
            const int i = base + 32 * k;
            v[k] = make_uint4(0u, 0u, 0u, 0u);
            w[k] = 0.f;
            if (i < i1) {
                v[k] = *reinterpret_cast<const uint4*>(Q + ((size_t)h * F + i) * XSV_D + 8 * c8);
                w[k] = 1.f;
                if (i >= n_special) {
                    const int gi = (i - n_special) / g;
                    w[k] = 1.f / (float)min(g, n_patch - gi * g);
                }
            }
        }
#pragma unroll
        for (int k = 0; k < 6; ++k) {
            T e8[8];
            *reinterpret_cast<uint4*>(e8) = v[k];
#pragma unroll
            for (int e = 0; e < 8; ++e) a[e] = fmaf(w[k], xsv_to_float<T>(e8[e]), a[e]);
        }
    }
    // the four row lanes of a warp, then the eight warps, in a fixed order
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        a[e] += __shfl_xor_sync(0xFFFFFFFFu, a[e], 8);
        a[e] += __shfl_xor_sync(0xFFFFFFFFu, a[e], 16);
    }
    __shared__ float red[8][64];
    if ((threadIdx.x & 31) < 8) {
#pragma unroll
        for (int e = 0; e < 8; ++e) red[threadIdx.x >> 5][8 * c8 + e] = a[e];
    }
    __syncthreads();
    if (threadIdx.x < 64) {
        float s = 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) s += red[k][threadIdx.x];
        qpart[((size_t)h * XSV_QCHUNKS + chunk) * 64 + threadIdx.x] = s;
    }
}

// q~ = sum_h sum_i w_i Q[h,i,:] from the n_part partial rows, summed in one fixed order by every block that needs
// it (the partial rows are 32 KB and stay in the L2; a kernel of its own for this sum cost more than the reads).
// 256 threads: four per channel, each sums every fourth row with its loads eight at a time; qt[64] in shared memory.
__device__ __forceinline__ void qtilde_sum(const float* __restrict__ qpart, int n_part, float qnorm, float (*red)[64], float* qt) {
    const int c = threadIdx.x & 63, part = threadIdx.x >> 6;
    float s = 0.f;
    for (int k0 = part; k0 < n_part; k0 += 4 * 8) {
        float v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = (k0 + 4 * j < n_part) ? qpart[(size_t)(k0 + 4 * j) * 64 + c] : 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) s += v[j];
    }
    red[part][c] = s;
    __syncthreads();
    if (threadIdx.x < 64) qt[c] = (((red[0][c] + red[1][c]) + red[2][c]) + red[3][c]) * qnorm;
    __syncthreads();
}

// ---------------------------------------------------------------------------
// Eq. 5-7: S[j] = (1/H) sum_h q~ . K~[h, T_first + j, :] over the middle segment.
// By linearity q~ . K~[h,p,:] = sum_c (q~_c s_c) code_c + sum_c q~_c z_c, with
// (s, z) the scale and offset of the key group of p: one block per key group, so the
// weights q~_c s_c and the bias are prepared once per head and a token costs one
// multiply-add per code.  256 threads = 64 tokens x 4 head slices; a warp reads
// 32 consecutive packed rows of one head.  A thread first issues the loads of
// its (up to four) rows, then helps with the weights, so the two round trips to
// memory overlap.  Codes are widened without the conversion unit:
// (word & mask_k) | 2^23 read as a float, minus 2^23, is code * 2^(bits k); the
// weight carries the 2^-(bits k).
// ---------------------------------------------------------------------------
constexpr int SCORE_TPB = 256;             // 64 tokens x 4 slices of the heads
constexpr int SCORE_ROWS = 4;              // rows a thread holds in registers at a time

template <int BITS>
__global__ void __launch_bounds__(SCORE_TPB) score_kernel(LayerView lv, int H, int T_first, int T_c,
                                                          const float* __restrict__ qpart, int n_part, float qnorm,
                                                          float* __restrict__ scores) {
    xsv_dep_release();
    // The kernels before this one in the stream (the partial sums of the queries, the merge of the previous step's
    // attention) do not touch the cache: the packed rows and the groups' parameters are loaded before the wait for
    // them, and only the partial sums are read after it.
    __shared__ float q_red[4][64];
    __shared__ __align__(16) float q_t[64];
    constexpr int ROWB = XSV_D * BITS / 8;
    constexpr int NV = ROWB / 16;              // 16-byte loads per row
    constexpr int SUB = (BITS == 8) ? 2 : (BITS == 4 ? 4 : 8);   // codes per 16-bit sub-word
    constexpr uint32_t NMAX = (1u << BITS) - 1u;
    extern __shared__ __align__(16) float sm[];
    float* sW = sm;                             // [H][64] weights q~_c * s_c * 2^-(bits * position of c in its sub-word)
    float* sB = sW + (size_t)H * 64;            // [H] bias sum_c q~_c z_c
    float* part = sB + ((H + 3) & ~3);          // [4][64] per-slice sums

    const int g = (T_first >> 6) + blockIdx.x;  // key group of this block
    const int tok = threadIdx.x & 63, slice = threadIdx.x >> 6, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int p = g * 64 + tok;
    const bool valid = p >= T_first && p < T_c;

    float acc = 0.f;
    for (int hb = 0; hb < H; hb += 4 * SCORE_ROWS) {
        uint4 rows[SCORE_ROWS][NV];
#pragma unroll
        for (int r = 0; r < SCORE_ROWS; ++r) {
            const int h = hb + slice + 4 * r;
            if (valid && h < H) {
                const uint4* row = reinterpret_cast<const uint4*>(lv.kcodes + ((size_t)h * lv.cap + p) * ROWB);
#pragma unroll
                for (int v = 0; v < NV; ++v) rows[r][v] = row[v];
            } else {
#pragma unroll
                for (int v = 0; v < NV; ++v) rows[r][v] = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        if (hb == 0) {
            // the group's parameters of the first two heads of this warp: loaded, like the rows, before the wait
            float sc[2][2], zz[2][2];
            auto load_params = [&](int h0) {
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    const int h = h0 + t * (SCORE_TPB / 32);
                    const size_t m = ((size_t)min(h, H - 1) * lv.capg + g) * 64;
                    sc[t][0] = lv.kscale[m + lane]; sc[t][1] = lv.kscale[m + lane + 32];
                    zz[t][0] = lv.kzero[m + lane]; zz[t][1] = lv.kzero[m + lane + 32];
                }
            };
            load_params(warp);
            xsv_dep_sync();
            qtilde_sum(qpart, n_part, qnorm, q_red, q_t);
            // weights and bias: one warp per head at a time, lane l takes channels l and l + 32 (same position in
            // their sub-words)
            const float q0 = q_t[lane], q1 = q_t[lane + 32];
            const float pos = __int_as_float((127 - BITS * ((lane & 7) % SUB)) << 23);
            for (int h0 = warp; h0 < H; h0 += 2 * (SCORE_TPB / 32)) {     // two heads per pass: eight loads in flight
                if (h0 != warp) load_params(h0);
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    const int h = h0 + t * (SCORE_TPB / 32);
                    const float w0 = q0 * sc[t][0], w1 = q1 * sc[t][1];
                    float b = q0 * zz[t][0] + q1 * zz[t][1];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) b += __shfl_xor_sync(0xFFFFFFFFu, b, o);
                    if (h < H) {
                        sW[h * 64 + lane] = w0 * pos;
                        sW[h * 64 + lane + 32] = w1 * pos;
                        if (lane == 0) sB[h] = b;
                    }
                }
            }
            __syncthreads();
        }
#pragma unroll
        for (int r = 0; r < SCORE_ROWS; ++r) {
            const int h = hb + slice + 4 * r;
            if (h < H) {
                const float4* w4 = reinterpret_cast<const float4*>(sW + h * 64);
                float a = 0.f;
#pragma unroll
                for (int v = 0; v < NV; ++v) {
                    const uint32_t ww[4] = {rows[r][v].x, rows[r][v].y, rows[r][v].z, rows[r][v].w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
#pragma unroll
                        for (int j = 0; j < 2; ++j) {           // the word's two 16-bit sub-words
                            const uint32_t sub = ww[k] >> (16 * j);
#pragma unroll
                            for (int e4 = 0; e4 < SUB / 4; ++e4) {
                                const int c = ((v * 4 + k) * 2 + j) * SUB + 4 * e4;   // channel of the first of four codes
                                const float4 wv = w4[c / 4];
                                const float wq[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const uint32_t mk = (sub & (NMAX << (BITS * (4 * e4 + e)))) | 0x4B000000u;
                                    a = fmaf(wq[e], __uint_as_float(mk) - 8388608.f, a);
                                }
                            }
                            if (SUB == 2) {
                                // 8-bit codes: two per sub-word, weights read in pairs
                                const int c = ((v * 4 + k) * 2 + j) * 2;
                                const float2 wv = reinterpret_cast<const float2*>(sW + h * 64)[c / 2];
                                a = fmaf(wv.x, __uint_as_float((sub & 0xFFu) | 0x4B000000u) - 8388608.f, a);
                                a = fmaf(wv.y, __uint_as_float((sub & 0xFF00u) | 0x4B000000u) - 8388608.f, a);
                            }
                        }
                    }
                }
                acc += a + sB[h];
            }
        }
    }
    part[slice * 64 + tok] = acc;
    __syncthreads();
    if (threadIdx.x < 64 && valid)
        scores[p - T_first] = (((part[tok] + part[64 + tok]) + part[128 + tok]) + part[192 + tok]) / (float)H;
}

// bits == 16: keys are raw 16-bit values.  64 tokens x 4 head slices per block as above; a warp reads 32 consecutive
// rows (4 KB) of one head, a thread one 128-byte row at a time with the next one already in flight.
template <typename T>
__global__ void __launch_bounds__(SCORE_TPB) score_raw_kernel(LayerView lv, int H, int T_first, int T_c,
                                                              const float* __restrict__ qpart, int n_part, float qnorm,
                                                              float* __restrict__ scores) {
    xsv_dep_release();
    xsv_dep_sync();
    __shared__ __align__(16) float qt[64];
    __shared__ float part[4][64];
    qtilde_sum(qpart, n_part, qnorm, part, qt);
    const int tok = threadIdx.x & 63, slice = threadIdx.x >> 6;
    const int j = blockIdx.x * 64 + tok;
    const int p = T_first + j;
    const bool valid = p < T_c;
    uint4 cur[8], nxt[8];
    auto load_row = [&](int h, uint4 (&r)[8]) {
        if (valid && h < H) {
            const uint4* row = reinterpret_cast<const uint4*>(lv.kcodes + ((size_t)h * lv.cap + p) * (XSV_D * 2));
#pragma unroll
            for (int v = 0; v < 8; ++v) r[v] = row[v];
        } else {
#pragma unroll
            for (int v = 0; v < 8; ++v) r[v] = make_uint4(0u, 0u, 0u, 0u);
        }
    };
    load_row(slice, cur);
    __syncthreads();
    float acc = 0.f;
    for (int h = slice; h < H; h += 4) {
        load_row(h + 4, nxt);
        float a = 0.f;
#pragma unroll
        for (int v = 0; v < 8; ++v) {
            const uint32_t u[4] = {cur[v].x, cur[v].y, cur[v].z, cur[v].w};
            const float4 q0 = reinterpret_cast<const float4*>(qt)[2 * v], q1 = reinterpret_cast<const float4*>(qt)[2 * v + 1];
            const float qq[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                T lo, hi;
                *reinterpret_cast<uint16_t*>(&lo) = (uint16_t)(u[e] & 0xFFFFu);
                *reinterpret_cast<uint16_t*>(&hi) = (uint16_t)(u[e] >> 16);
                a = fmaf(qq[2 * e], xsv_to_float<T>(lo), a);
                a = fmaf(qq[2 * e + 1], xsv_to_float<T>(hi), a);
            }
        }
        acc += a;
#pragma unroll
        for (int v = 0; v < 8; ++v) cur[v] = nxt[v];
    }
    part[slice][tok] = acc;
    __syncthreads();
    if (threadIdx.x < 64 && valid)
        scores[j] = (((part[0][tok] + part[1][tok]) + part[2][tok]) + part[3][tok]) / (float)H;
}

// ---------------------------------------------------------------------------
// Eq. 8: top-k by radix select on an order-preserving integer image of the
// float32 scores, ties broken by position, then an ordered compaction.
// One block of 1024 threads; n is at most a few tens of thousands.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t score_key(float s) {
    if (s == 0.f) s = 0.f;   // -0 and +0 compare equal: give them one key
    uint32_t u = __float_as_uint(s);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__global__ void __launch_bounds__(1024) select_kernel(const float* __restrict__ scores, int n, int k,
                                                      int T_first, int T_c, int* __restrict__ srcmap,
                                                      int* __restrict__ dscal) {
    xsv_dep_release();
    xsv_dep_sync();
    __shared__ int hist[256];
    __shared__ uint32_t s_prefix;
    __shared__ int s_remaining;
    __shared__ int w_gt[32], w_eq[32], w_off[32], w_eqb[32];
    __shared__ int s_first_evicted;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    uint32_t thr = 0xFFFFFFFFu;
    int need_eq = 0;
    if (k > 0) {
        uint32_t prefix = 0, mask = 0;
        if (tid == 0) s_remaining = k;
        for (int pass = 3; pass >= 0; --pass) {
            const int shift = pass * 8;
            if (tid < 256) hist[tid] = 0;
            __syncthreads();
            for (int j = tid; j < n; j += 1024) {
                uint32_t key = score_key(scores[j]);
                if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1);
            }
            __syncthreads();
            if (tid == 0) {
                int remaining = s_remaining, cum = 0, digit = 0;
                for (int b = 255; b >= 0; --b) {
                    if (cum + hist[b] >= remaining) { digit = b; break; }
                    cum += hist[b];
                }
                s_remaining = remaining - cum;
                s_prefix = prefix | ((uint32_t)digit << shift);
            }
            __syncthreads();
            prefix = s_prefix;
            mask |= 255u << shift;
        }
        thr = prefix;
        need_eq = s_remaining;     // how many of the keys equal to thr are taken (lowest positions)
    }
    if (tid == 0) s_first_evicted = n;
    // ordered compaction: warp w owns the contiguous range [w*seg, (w+1)*seg)
    const int seg = ((n + 31) / 32 + 31) / 32 * 32;
    const int a = min(n, warp * seg), b = min(n, a + seg);
    const int bend = a + (b - a + 31) / 32 * 32;     // whole stripes, so every lane joins the ballots
    int cgt = 0, ceq = 0;
    for (int j = a + lane; j < bend; j += 32) {
        uint32_t key = j < b ? score_key(scores[j]) : 0u;
        bool gt = j < b && key > thr, eq = j < b && key == thr && k > 0;
        cgt += __popc(__ballot_sync(0xFFFFFFFFu, gt));
        ceq += __popc(__ballot_sync(0xFFFFFFFFu, eq));
    }
    if (lane == 0) { w_gt[warp] = cgt; w_eq[warp] = ceq; }
    __syncthreads();
    if (warp == 0) {
        // exclusive scans over the 32 warps, in warp order
        int eq = w_eq[lane], gt = w_gt[lane];
        int eq_incl = eq;
        for (int o = 1; o < 32; o <<= 1) { int t = __shfl_up_sync(0xFFFFFFFFu, eq_incl, o); if (lane >= o) eq_incl += t; }
        int eq_before = eq_incl - eq;
        int take_eq = max(0, min(eq, need_eq - eq_before));
        int kept = gt + take_eq;
        int k_incl = kept;
        for (int o = 1; o < 32; o <<= 1) { int t = __shfl_up_sync(0xFFFFFFFFu, k_incl, o); if (lane >= o) k_incl += t; }
        w_off[lane] = k_incl - kept;
        w_eqb[lane] = eq_before;
    }
    __syncthreads();
    int off = w_off[warp], eqb = w_eqb[warp];
    int first_ev = n;
    const uint32_t lt = (1u << lane) - 1u;
    for (int j = a + lane; j < bend; j += 32) {
        uint32_t key = j < b ? score_key(scores[j]) : 0u;
        bool gt = j < b && key > thr, eq = j < b && key == thr && k > 0;
        uint32_t beq = __ballot_sync(0xFFFFFFFFu, eq);
        int rank = eqb + __popc(beq & lt);
        bool keep = gt || (eq && rank < need_eq);
        uint32_t bk = __ballot_sync(0xFFFFFFFFu, keep);
        if (keep) srcmap[off + __popc(bk & lt)] = T_first + j;
        if (j < b && !keep) first_ev = min(first_ev, j);
        off += __popc(bk);
        eqb += __popc(beq);
    }
    for (int o = 16; o > 0; o >>= 1) first_ev = min(first_ev, __shfl_xor_sync(0xFFFFFFFFu, first_ev, o));
    if (lane == 0 && first_ev < n) atomicMin(&s_first_evicted, first_ev);
    __syncthreads();
    if (tid == 0) dscal[0] = min(T_first + s_first_evicted, T_c) >> 6;
}

// ---------------------------------------------------------------------------
// Eq. 8 again, for n <= 1024 * KPT: thread t keeps the keys of the KPT
// consecutive positions [t KPT, (t + 1) KPT) in registers (16-byte loads), so
// the scores are read from memory once.
//
// The k-th largest key is found by bisection on its bits, from the highest bit
// in which the keys differ downwards.  A step counts the keys >= (prefix | bit)
// -- one warp reduction, one shared-memory atomic per warp, one barrier -- and
// the search stops as soon as a candidate splits off exactly k keys, which for
// scores without ties happens after about log2(n) + a few steps.  Only the keys
// inside the current interval [prefix, prefix + 2^(b+1)) are still undecided;
// once they number at most 2048 they are copied to shared memory and the
// remaining steps look at one or two keys per thread instead of KPT.
//
// Ordered compaction: block-wide exclusive scans of the per-thread counts give
// every thread the output offset of its first kept position; the kept
// positions are staged in shared memory and copied out coalesced.  Same total
// order as select_kernel (score descending, position ascending).
// ---------------------------------------------------------------------------
constexpr int SEL_ACT = 2048;             // undecided keys that fit the shared-memory stage of the bisection

// Exclusive prefix sum of v over the 1024 threads of the block; *total receives the sum.  ws: 33 ints.
__device__ __forceinline__ int sel_block_scan(int v, int* ws, int* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o); if (lane >= o) incl += t; }
    __syncthreads();               // ws may still be read from an earlier scan
    if (lane == 31) ws[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const int x = ws[lane];
        int xi = x;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xFFFFFFFFu, xi, o); if (lane >= o) xi += t; }
        ws[lane] = xi - x;
        if (lane == 31) ws[32] = xi;
    }
    __syncthreads();
    *total = ws[32];
    return ws[warp] + incl - v;
}

template <int KPT>
__global__ void __launch_bounds__(1024) select_reg_kernel(const float* __restrict__ scores, int n, int k, int T_first,
                                                          int T_c, int* __restrict__ srcmap, int* __restrict__ dscal) {
    xsv_dep_release();
    xsv_dep_sync();
    extern __shared__ __align__(16) int sel_sm[];     // [1024 * KPT]: undecided keys, later the kept positions
    __shared__ int cnt[36];
    __shared__ uint32_t s_lo, s_hi;
    __shared__ int s_nact;
    __shared__ int ws[33];
    __shared__ int s_first_evicted;
    constexpr uint32_t FULL = 0xFFFFFFFFu;
    const int tid = threadIdx.x, lane = tid & 31;
    const int j0 = tid * KPT;
    uint32_t key[KPT];                    // positions past n hold key 0
    if ((reinterpret_cast<uintptr_t>(scores) & 15) == 0) {
#pragma unroll
        for (int v = 0; v < KPT / 4; ++v) {
            const int j = j0 + 4 * v;
            if (j + 3 < n) {
                const float4 f = *reinterpret_cast<const float4*>(scores + j);
                key[4 * v] = score_key(f.x); key[4 * v + 1] = score_key(f.y);
                key[4 * v + 2] = score_key(f.z); key[4 * v + 3] = score_key(f.w);
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) key[4 * v + e] = (j + e < n) ? score_key(scores[j + e]) : 0u;
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < KPT; ++i) key[i] = (j0 + i < n) ? score_key(scores[j0 + i]) : 0u;
    }

    uint32_t thr = 0xFFFFFFFFu;
    int need_eq = 0;
    if (k >= n) {
        thr = 0u;                  // every key is kept
        need_eq = n;
    } else if (k > 0) {
        if (tid < 36) cnt[tid] = 0;
        if (tid == 0) { s_lo = 0xFFFFFFFFu; s_hi = 0u; s_nact = 0; }
        __syncthreads();
        uint32_t lo = 0xFFFFFFFFu, hi = 0u;
#pragma unroll
        for (int i = 0; i < KPT; ++i)
            if (j0 + i < n) { lo = min(lo, key[i]); hi = max(hi, key[i]); }
        lo = __reduce_min_sync(FULL, lo);
        hi = __reduce_max_sync(FULL, hi);
        if (lane == 0) { atomicMin(&s_lo, lo); atomicMax(&s_hi, hi); }
        __syncthreads();
        lo = s_lo;
        hi = s_hi;
        if (lo == hi) {            // all keys equal: the k lowest positions
            thr = lo;
            need_eq = k;
        } else {
            int b = 31 - __clz(lo ^ hi);
            uint32_t v = (b == 31) ? 0u : (lo & ~((2u << b) - 1u));     // the leading bits all keys share
            // Invariants: ge_v keys are >= v, `above` of them are >= v + 2^(b+1) (the end of the undecided interval),
            // above < k <= ge_v.
            int ge_v = n, above = 0, step = 0;
            bool exact = false;
            // stage 1: all keys, in registers
            for (; b >= 0 && ge_v - above > SEL_ACT; --b, ++step) {
                const uint32_t cand = v | (1u << b);
                int c = 0;
#pragma unroll
                for (int i = 0; i < KPT; ++i) c += (key[i] >= cand) ? 1 : 0;
                c = __reduce_add_sync(FULL, c);
                if (lane == 0 && c != 0) atomicAdd(&cnt[step], c);
                __syncthreads();
                c = cnt[step];
                if (c >= k) {
                    v = cand;
                    ge_v = c;
                    if (c == k) { exact = true; break; }
                } else {
                    above = c;
                }
            }
            if (!exact && b >= 0) {
                // stage 2: the undecided keys (v <= key < v + 2^(b+1)), one or two per thread, from shared memory
                const uint32_t width = (b == 31) ? 0xFFFFFFFFu : ((2u << b) - 1u);      // interval length - 1
                int mine = 0;
#pragma unroll
                for (int i = 0; i < KPT; ++i) mine += (j0 + i < n && key[i] - v <= width && key[i] >= v) ? 1 : 0;
                int incl = mine;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(FULL, incl, o); if (lane >= o) incl += t; }
                int base = 0;
                if (lane == 31 && incl != 0) base = atomicAdd(&s_nact, incl);
                base = __shfl_sync(FULL, base, 31) + incl - mine;
#pragma unroll
                for (int i = 0; i < KPT; ++i)
                    if (j0 + i < n && key[i] - v <= width && key[i] >= v) sel_sm[base++] = (int)key[i];
                __syncthreads();
                const int n_act = s_nact;          // == ge_v - above
                const uint32_t a0 = tid < n_act ? (uint32_t)sel_sm[tid] : 0u;
                const uint32_t a1 = tid + 1024 < n_act ? (uint32_t)sel_sm[tid + 1024] : 0u;
                const int above0 = above;          // keys beyond the staged interval
                for (; b >= 0; --b, ++step) {
                    const uint32_t cand = v | (1u << b);
                    int c = ((a0 >= cand) ? 1 : 0) + ((a1 >= cand) ? 1 : 0);
                    c = __reduce_add_sync(FULL, c);
                    if (lane == 0 && c != 0) atomicAdd(&cnt[step], c);
                    __syncthreads();
                    c = cnt[step] + above0;       // all keys >= cand
                    if (c >= k) {
                        v = cand;
                        if (c == k) { exact = true; break; }
                    } else {
                        above = c;
                    }
                }
            }
            if (exact) {           // exactly k keys are >= v
                thr = v - 1u;
                need_eq = 0;
            } else {               // v is the k-th largest key; `above` keys are larger
                thr = v;
                need_eq = k - above;
            }
        }
    }
    if (tid == 0) s_first_evicted = n;

    // ordered compaction.  Positions past n hold key 0, which is never above the threshold; they can only tie with it,
    // and ties are looked at only when some are to be kept (need_eq is the same in every thread).
    uint32_t keep = 0;                    // bit i: position j0 + i is kept
#pragma unroll
    for (int i = 0; i < KPT; ++i) keep |= (key[i] > thr) ? (1u << i) : 0u;
    int total = 0;
    if (need_eq > 0) {
        uint32_t eqm = 0;
#pragma unroll
        for (int i = 0; i < KPT; ++i) eqm |= (j0 + i < n && key[i] == thr) ? (1u << i) : 0u;
        const int eq_before = sel_block_scan(__popc(eqm), ws, &total);
        int take = max(0, min(__popc(eqm), need_eq - eq_before));
        while (take > 0) {                // the lowest positions among the ties
            const uint32_t low = eqm & (0u - eqm);
            keep |= low;
            eqm ^= low;
            --take;
        }
    }
    int off = sel_block_scan(__popc(keep), ws, &total);
#pragma unroll
    for (int i = 0; i < KPT; ++i)
        if (keep & (1u << i)) sel_sm[off++] = T_first + j0 + i;
    const uint32_t owned = (j0 >= n) ? 0u : ((n - j0 >= KPT) ? ((KPT == 32) ? 0xFFFFFFFFu : ((1u << (KPT & 31)) - 1u)) : ((1u << (n - j0)) - 1u));
    const uint32_t dropped = owned & ~keep;
    int first_ev = dropped ? j0 + __ffs(dropped) - 1 : n;
    first_ev = __reduce_min_sync(FULL, first_ev);
    if (lane == 0 && first_ev < n) atomicMin(&s_first_evicted, first_ev);
    __syncthreads();
    for (int i = tid; i < total; i += 1024) srcmap[i] = sel_sm[i];
    if (tid == 0) dscal[0] = min(T_first + s_first_evicted, T_c) >> 6;
}

// ---------------------------------------------------------------------------
// Eq. 9-11 for keys.  One warp per (new 64-token group, head), no block-level
// synchronisation; warps walk the (group, head) items with a stride of the
// whole grid.  A warp first copies the packed rows of the group's 64 members
// into its slice of shared memory (all loads in flight at once) together with
// the parameters of the old groups they come from (kept tokens stay in order,
// so a new group draws on a short run of old groups).  Lane (tq, w) owns the
// 8 channels [8w, 8w + 8) of the members tq, tq + 4, ..., tq + 60: eight lanes
// cover one packed row, and a row's 8 new codes are one store of 8 * bits bits.
// Pass 1 dequantises (Eq. 12) or widens the frame's 16-bit keys and keeps a
// running min / max per channel; two shuffles finish the reduction over the 64
// tokens.  Each lane derives the parameters of two channels (Eq. 10) and
// publishes them through shared memory.  Pass 2 re-derives the values and
// writes the codes (Eq. 9).
//
// The arithmetic is arranged for the pipes it runs on (integer and min/max
// instructions issue at half the rate of float multiply-adds):
//  * a code is not shifted down before it is widened: (word & mask_k) | 2^23,
//    read as a float, is 2^23 + code * 2^(bits k); minus 2^23 and times the
//    staged s * 2^-(bits k) that is code * s with the rounding of Eq. 12's
//    multiply, and the group's offset is added in a second operation;
//  * the clamp of Eq. 9 is a saturating multiply by 1/n, and a row's codes are
//    summed into 16-bit sub-words by multiply-adds (n * 2^(bits k) each) and
//    converted once per sub-word.
// ---------------------------------------------------------------------------
constexpr int RQ_WIN = 4;                  // old groups whose parameters are staged; tokens from further on read global memory
constexpr int RQ_THREADS = 256;

template <int BITS>
struct RqCfg {
    static constexpr int ROWB = XSV_D * BITS / 8;
    static constexpr int SUB = (BITS == 8) ? 2 : (BITS == 4 ? 4 : 8);   // codes per 16-bit sub-word
    static constexpr int NSUB = 8 / SUB;                                // sub-words per lane (8 codes)
    static constexpr int CODE_WORDS = XSV_G * ROWB / 4;
    // per warp, in 4-byte words: old scales and offsets, new scale / reciprocal / offset (+ 64 spare),
    // old positions, packed rows
    static constexpr int WORDS = 2 * RQ_WIN * 64 + 4 * 64 + 64 + CODE_WORDS;
    static constexpr int OFF_CODES = 2 * RQ_WIN * 64 + 4 * 64 + 64;
};

__device__ __forceinline__ float rq_min3(float a, float b, float c) {
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float rq_max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float rq_mul_sat(float a, float b) {
    float d;
    asm("mul.rn.sat.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}

// 16-bit sub-word j of a lane's 8 codes (the upper half of the register is ignored by the masks).
template <int BITS>
__device__ __forceinline__ uint32_t rq_sub(uint64_t ch, int j) { return (uint32_t)(ch >> (16 * j)); }

// General form of Eq. 12 for a row whose old group is outside the staged window or has parameters the fast
// form cannot take: parameters from memory, one conversion per code.
template <int BITS>
__device__ __forceinline__ void rq_fetch_slow(const float* __restrict__ ks, const float* __restrict__ kz, uint64_t ch, float (&x)[8]) {
    constexpr uint32_t NMAX = (1u << BITS) - 1u;
#pragma unroll
    for (int e = 0; e < 8; ++e) x[e] = xsv_dequant((int)((uint32_t)(ch >> (e * BITS)) & NMAX), kz[e], ks[e]);
}

template <typename T>
__device__ __forceinline__ void rq_fetch_fresh(const T* __restrict__ row, float (&x)[8]) {
    const uint4 a = *reinterpret_cast<const uint4*>(row);
    const uint32_t u[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        T lo, hi;
        *reinterpret_cast<uint16_t*>(&lo) = (uint16_t)(u[e] & 0xFFFFu);
        *reinterpret_cast<uint16_t*>(&hi) = (uint16_t)(u[e] >> 16);
        x[2 * e] = xsv_to_float<T>(lo);
        x[2 * e + 1] = xsv_to_float<T>(hi);
    }
}

// Values of kept tokens move verbatim (codes row, scale, zero-point, origin): one warp per (64 new positions, head).
template <int BITS>
__device__ __forceinline__ void rq_gather_v_item(const LayerView& src, const LayerView& dst, int H, int n_old_new,
                                                 int T_first, const int* __restrict__ srcmap, int item, int lane) {
    constexpr int ROWB = XSV_D * BITS / 8, PPR = ROWB / 16;
    const int h = item % H, p0 = (item / H) * 64;
    int spv[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const int p = p0 + lane + 32 * k;
        spv[k] = p < n_old_new ? ((srcmap != nullptr && p >= T_first) ? srcmap[p - T_first] : p) : -1;
    }
    uint4 v[2 * PPR];
#pragma unroll
    for (int j = 0; j < 2 * PPR; ++j) {
        const int idx = lane + 32 * j, row = idx / PPR, piece = idx % PPR;
        const int sp = __shfl_sync(0xFFFFFFFFu, spv[row >> 5], row & 31);
        v[j] = make_uint4(0u, 0u, 0u, 0u);
        if (sp >= 0) v[j] = *reinterpret_cast<const uint4*>(src.vcodes + ((size_t)h * src.cap + sp) * ROWB + 16 * piece);
    }
#pragma unroll
    for (int j = 0; j < 2 * PPR; ++j) {
        const int idx = lane + 32 * j, row = idx / PPR, piece = idx % PPR;
        if (p0 + row < n_old_new)
            *reinterpret_cast<uint4*>(dst.vcodes + ((size_t)h * dst.cap + p0 + row) * ROWB + 16 * piece) = v[j];
    }
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const int p = p0 + lane + 32 * k;
        if (spv[k] >= 0) {
            dst.vscale[(size_t)h * dst.cap + p] = src.vscale[(size_t)h * src.cap + spv[k]];
            dst.vzero[(size_t)h * dst.cap + p] = src.vzero[(size_t)h * src.cap + spv[k]];
            if (h == 0) dst.origin[p] = src.origin[spv[k]];
        }
    }
}

// Eq. 9-11 for the frame's values: one warp per (4 tokens, head); a row of 64 channels at a time, two channels per
// lane, shuffle reductions for min / max.
constexpr int RQ_VROWS = 4;
template <typename T, int BITS>
__device__ __forceinline__ void rq_quant_v_item(const LayerView& dst, const T* __restrict__ Vf, int H, int F,
                                                int n_old_new, long long origin0, int* __restrict__ status, int item,
                                                int lane) {
    constexpr int ROWB = XSV_D * BITS / 8;
    constexpr int NMAX = (1 << BITS) - 1;
    constexpr int LPW = 16 / BITS;            // lanes that share one 32-bit word
    const int h = item % H, f0 = (item / H) * RQ_VROWS;
#pragma unroll 4
    for (int i = 0; i < RQ_VROWS; ++i) {
        const int f = f0 + i;
        if (f >= F) break;
        const uint32_t raw = *reinterpret_cast<const uint32_t*>(Vf + ((size_t)h * F + f) * XSV_D + 2 * lane);
        T lo, hi;
        *reinterpret_cast<uint16_t*>(&lo) = (uint16_t)(raw & 0xFFFFu);
        *reinterpret_cast<uint16_t*>(&hi) = (uint16_t)(raw >> 16);
        const float x0 = xsv_to_float<T>(lo), x1 = xsv_to_float<T>(hi);
        float mn = fminf(x0, x1), mx = fmaxf(x0, x1);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            mn = fminf(mn, __shfl_xor_sync(0xFFFFFFFFu, mn, o));
            mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
        }
        float s, z;
        xsv_quant_params(mn, mx, NMAX, s, z);
        const float inv_s = __frcp_rn(s);
        const uint32_t c0 = (uint32_t)xsv_quant_code(x0, s, inv_s, z, NMAX), c1 = (uint32_t)xsv_quant_code(x1, s, inv_s, z, NMAX);
        uint32_t w = (c0 | (c1 << BITS)) << (2 * BITS * (lane % LPW));
#pragma unroll
        for (int o = 1; o < LPW; o <<= 1) w |= __shfl_xor_sync(0xFFFFFFFFu, w, o);
        const int p = n_old_new + f;
        if (lane % LPW == 0)
            *reinterpret_cast<uint32_t*>(dst.vcodes + ((size_t)h * dst.cap + p) * ROWB + 4 * (lane / LPW)) = w;
        if (lane == 0) {
            dst.vscale[(size_t)h * dst.cap + p] = s;
            dst.vzero[(size_t)h * dst.cap + p] = z;
            if (h == 0) dst.origin[p] = origin0 + f;
        }
    }
}

// The frame's value rows alone (used when the values are handled on another stream than the keys).
template <typename T, int BITS>
__global__ void __launch_bounds__(256) quant_v_kernel(LayerView dst, const T* __restrict__ Vf, int H, int F, int n_old_new,
                                                      long long origin0, int n_vq, int* __restrict__ status) {
    xsv_dep_release();
    xsv_dep_sync();
    const int item = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (item < n_vq) rq_quant_v_item<T, BITS>(dst, Vf, H, F, n_old_new, origin0, status, item, threadIdx.x & 31);
}

template <typename T, int BITS>
__global__ void __launch_bounds__(RQ_THREADS, 3) requant_k_kernel(LayerView src, LayerView dst, const T* __restrict__ Kf,
                                                               const T* __restrict__ Vf, int H, int F, int n_old_new,
                                                               int T_new, int T_first, const int* __restrict__ srcmap,
                                                               const int* __restrict__ fz_dev, int fz_host,
                                                               int g_base, int n_items, int n_vg, int n_vq,
                                                               long long origin0, int* __restrict__ status) {
    xsv_dep_release();
    xsv_dep_sync();
    using C = RqCfg<BITS>;
    constexpr int ROWB = C::ROWB, SUB = C::SUB, NSUB = C::NSUB;
    constexpr int NMAX = (1 << BITS) - 1;
    constexpr uint32_t FULL = 0xFFFFFFFFu;
    constexpr float KINV = 1.f / (float)NMAX;
    extern __shared__ __align__(16) float rq_sm[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wpb = blockDim.x >> 5;
    const int tq = lane >> 3, w = lane & 7;
    float* w_s = rq_sm + (size_t)warp * C::WORDS;
    float* w_zc = w_s + RQ_WIN * 64;
    float* n_s = w_zc + RQ_WIN * 64;
    float* n_i = n_s + 64;
    float* n_zf = n_i + 64;                                   // the new groups' offsets
    int* s_sp = reinterpret_cast<int*>(n_zf + 128);
    uint8_t* s_codes = reinterpret_cast<uint8_t*>(w_s + C::OFF_CODES);
    const int fz = fz_dev ? *fz_dev : fz_host;
    const bool same = (src.kcodes == dst.kcodes);
    // position of this lane's staging channels (lane and lane + 32: same position) inside their 16-bit sub-word
    const int pos_shift = BITS * ((lane & 7) % SUB);
    const float pos_scale = __int_as_float((127 - pos_shift) << 23);

    // Warp slot: warp * (blocks) + block, so that a partial round of items is spread over all blocks (and so over all
    // multiprocessors).  The heavy key-group items are dealt out first, round by round; the short value items then go
    // to the slots that received one key item fewer (to all slots if the key items came out even).
    const int slot = warp * gridDim.x + blockIdx.x, n_slots = gridDim.x * wpb;
    {
        const int extra = n_items % n_slots;                  // slots [0, extra) hold one more key item
        const int first = (extra == 0) ? 0 : extra;
        if (slot >= first) {
            for (int j = slot - first; j < n_vg + n_vq; j += n_slots - first) {
                if (j < n_vg) rq_gather_v_item<BITS>(src, dst, H, n_old_new, T_first, srcmap, j, lane);
                else rq_quant_v_item<T, BITS>(dst, Vf, H, F, n_old_new, origin0, status, j - n_vg, lane);
            }
        }
    }
    for (int it = slot; it < n_items; it += n_slots) {
        const int gi = g_base + it / H, h = it % H;
        const int p0 = gi * XSV_G;
        const int cnt = min(XSV_G, T_new - p0);
        const size_t prm = ((size_t)h * dst.capg + gi) * 64;

        if (gi < fz) {   // frozen: the group keeps its members, positions, codes and parameters
            if (same) continue;
            const uint32_t* s = reinterpret_cast<const uint32_t*>(src.kcodes + ((size_t)h * src.cap + p0) * ROWB);
            uint32_t* d = reinterpret_cast<uint32_t*>(dst.kcodes + ((size_t)h * dst.cap + p0) * ROWB);
#pragma unroll 4
            for (int i = lane; i < XSV_G * ROWB / 4; i += 32) d[i] = s[i];
            const size_t sprm = ((size_t)h * src.capg + gi) * 64;
            dst.kscale[prm + lane] = src.kscale[sprm + lane];
            dst.kscale[prm + lane + 32] = src.kscale[sprm + lane + 32];
            dst.kzero[prm + lane] = src.kzero[sprm + lane];
            dst.kzero[prm + lane + 32] = src.kzero[sprm + lane + 32];
            continue;
        }

        // old position of every member (-1: a token of the frame, -2: past the end)
        int spv[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const int tk = lane + 32 * k, p = p0 + tk;
            int sp = -2;
            if (tk < cnt) sp = (p >= n_old_new) ? -1 : ((srcmap != nullptr && p >= T_first) ? srcmap[p - T_first] : p);
            s_sp[tk] = sp;
            spv[k] = sp;
        }
        __syncwarp();
        const int g_lo = s_sp[0] >> 6;     // members are in ascending old position; -1 >> 6 == -1: none cached
        uint32_t slow_rows = 0;
        if (g_lo >= 0) {
            // packed rows of the cached members
            constexpr int PPR = ROWB / 16;
#pragma unroll
            for (int j = 0; j < 2 * PPR; ++j) {
                const int idx = lane + 32 * j, row = idx / PPR, piece = idx % PPR;
                const int sp = s_sp[row];
                if (sp >= 0)
                    reinterpret_cast<uint4*>(s_codes)[idx] =
                        *reinterpret_cast<const uint4*>(src.kcodes + ((size_t)h * src.cap + sp) * ROWB + 16 * piece);
            }
            // parameters of the staged old groups: lane l takes channels l and l + 32 of each row
            bool slow[RQ_WIN];
            const float* ksp = src.kscale + ((size_t)h * src.capg + g_lo) * 64 + lane;
            const float* kzp = src.kzero + ((size_t)h * src.capg + g_lo) * 64 + lane;
#pragma unroll
            for (int r = 0; r < RQ_WIN; ++r) {
                slow[r] = false;
                if (g_lo + r < src.capg) {
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        const float z = kzp[r * 64 + 32 * k];
                        const float sc = ksp[r * 64 + 32 * k];
                        const bool ok = sc >= 7.8886090522101181e-31f /* 2^-100: the scaling by 2^-(bits k) stays exact */;
                        w_s[r * 64 + 32 * k + lane] = sc * pos_scale;
                        w_zc[r * 64 + 32 * k + lane] = z;
                        slow[r] |= !ok;
                    }
                }
            }
#pragma unroll
            for (int r = 0; r < RQ_WIN; ++r) slow_rows |= __any_sync(FULL, slow[r]) ? (1u << r) : 0u;
        }
        __syncwarp();

        // members whose old group lies in the first g + 1 staged rows (they are the first nb[g] members)
        int nb[RQ_WIN];
#pragma unroll
        for (int g = 0; g < RQ_WIN; ++g) {
            const bool a = spv[0] >= 0 && (spv[0] >> 6) - g_lo <= g, b = spv[1] >= 0 && (spv[1] >> 6) - g_lo <= g;
            nb[g] = __popc(__ballot_sync(FULL, a)) + __popc(__ballot_sync(FULL, b));
        }

        const uint8_t* const cbase = s_codes + tq * ROWB + w * BITS;   // this lane's octet of member tq; member tq + 4 i is 4 i rows on
        auto chunk_of = [&](int i) -> uint64_t {
            const uint8_t* cp = cbase + i * (4 * ROWB);
            if (BITS == 2) return *reinterpret_cast<const uint16_t*>(cp);
            if (BITS == 4) return *reinterpret_cast<const uint32_t*>(cp);
            const uint2 t = *reinterpret_cast<const uint2*>(cp);
            return (uint64_t)t.x | ((uint64_t)t.y << 32);
        };
        // Walks this lane's members tq, tq + 4, ...: run by run of members that share a staged old group (the group's
        // constants are loaded once per run; two members per step where the run allows), then whatever is left -- old
        // groups outside the window or with parameters the fast form cannot take, and the frame's tokens -- one by one
        // in the general form.  one(i, x) / two(i, x0, x1) receive the values of member tq + 4 i (and tq + 4 i + 4).
        auto walk = [&](auto&& one, auto&& two) {
            int i = 0;
            if (g_lo >= 0) {
#pragma unroll 1
                for (int g = 0; g < RQ_WIN; ++g) {
                    const int i_end = min(16, max(0, (nb[g] - tq + 3) >> 2));
                    if (i >= i_end) continue;
                    if ((slow_rows >> g) & 1u) break;
                    const float4 s0 = *reinterpret_cast<const float4*>(w_s + g * 64 + 8 * w), s1 = *reinterpret_cast<const float4*>(w_s + g * 64 + 8 * w + 4);
                    const float4 c0 = *reinterpret_cast<const float4*>(w_zc + g * 64 + 8 * w), c1 = *reinterpret_cast<const float4*>(w_zc + g * 64 + 8 * w + 4);
                    const float sv[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
                    const float cv[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
                    auto deq = [&](uint64_t ch, float (&x)[8]) {
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const uint32_t m = (rq_sub<BITS>(ch, e / SUB) & ((uint32_t)NMAX << (BITS * (e % SUB)))) | 0x4B000000u;
                            x[e] = __fadd_rn(__fmul_rn(__fadd_rn(__uint_as_float(m), -8388608.f), sv[e]), cv[e]);
                        }
                    };
#pragma unroll 1
                    for (; i + 1 < i_end; i += 2) {
                        const uint64_t ch0 = chunk_of(i), ch1 = chunk_of(i + 1);
                        float x0[8], x1[8];
                        deq(ch0, x0);
                        deq(ch1, x1);
                        two(i, x0, x1);
                    }
                    if (i < i_end) {
                        float x0[8];
                        deq(chunk_of(i), x0);
                        one(i, x0);
                        ++i;
                    }
                }
            }
#pragma unroll 1
            for (; i < 16; ++i) {
                const int tk = tq + 4 * i;
                const int sp = s_sp[tk];
                if (sp == -2) break;
                float x[8];
                if (sp >= 0) {
                    const size_t m = ((size_t)h * src.capg + (sp >> 6)) * 64 + 8 * w;
                    rq_fetch_slow<BITS>(src.kscale + m, src.kzero + m, chunk_of(i), x);
                } else {
                    rq_fetch_fresh<T>(Kf + ((size_t)h * F + (p0 + tk - n_old_new)) * XSV_D + 8 * w, x);
                }
                one(i, x);
            }
        };

        float mn[8], mx[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) { mn[e] = INFINITY; mx[e] = -INFINITY; }
        walk(
            [&](int, const float (&x)[8]) {
#pragma unroll
                for (int e = 0; e < 8; ++e) { mn[e] = fminf(mn[e], x[e]); mx[e] = fmaxf(mx[e], x[e]); }
            },
            [&](int, const float (&x0)[8], const float (&x1)[8]) {
#pragma unroll
                for (int e = 0; e < 8; ++e) { mn[e] = rq_min3(mn[e], x0[e], x1[e]); mx[e] = rq_max3(mx[e], x0[e], x1[e]); }
            });
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            mn[e] = fminf(mn[e], __shfl_xor_sync(FULL, mn[e], 8));
            mx[e] = fmaxf(mx[e], __shfl_xor_sync(FULL, mx[e], 8));
            mn[e] = fminf(mn[e], __shfl_xor_sync(FULL, mn[e], 16));
            mx[e] = fmaxf(mx[e], __shfl_xor_sync(FULL, mx[e], 16));
        }
        // Eq. 10: this lane derives the parameters of channels 8w + 2tq and 8w + 2tq + 1
        float s2[2], z2[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const float a = tq == 0 ? mn[k] : tq == 1 ? mn[2 + k] : tq == 2 ? mn[4 + k] : mn[6 + k];
            const float b = tq == 0 ? mx[k] : tq == 1 ? mx[2 + k] : tq == 2 ? mx[4 + k] : mx[6 + k];
            xsv_quant_params(a, b, NMAX, s2[k], z2[k]);
            const int c = 8 * w + 2 * tq + k;
            n_s[c] = s2[k];
            n_i[c] = __frcp_rn(s2[k]);
            n_zf[c] = z2[k];
        }
        __syncwarp();
        float iv[8], fv[8], ns[8];
        {
            const float4 i0 = *reinterpret_cast<const float4*>(n_i + 8 * w), i1 = *reinterpret_cast<const float4*>(n_i + 8 * w + 4);
            const float4 f0 = *reinterpret_cast<const float4*>(n_zf + 8 * w), f1 = *reinterpret_cast<const float4*>(n_zf + 8 * w + 4);
            const float4 a0 = *reinterpret_cast<const float4*>(n_s + 8 * w), a1 = *reinterpret_cast<const float4*>(n_s + 8 * w + 4);
            iv[0] = i0.x; iv[1] = i0.y; iv[2] = i0.z; iv[3] = i0.w; iv[4] = i1.x; iv[5] = i1.y; iv[6] = i1.z; iv[7] = i1.w;
            fv[0] = f0.x; fv[1] = f0.y; fv[2] = f0.z; fv[3] = f0.w; fv[4] = f1.x; fv[5] = f1.y; fv[6] = f1.z; fv[7] = f1.w;
            ns[0] = -a0.x; ns[1] = -a0.y; ns[2] = -a0.z; ns[3] = -a0.w; ns[4] = -a1.x; ns[5] = -a1.y; ns[6] = -a1.z; ns[7] = -a1.w;
        }
        uint8_t* const obase = dst.kcodes + ((size_t)h * dst.cap + p0 + tq) * ROWB + w * BITS;
        auto put = [&](int i, const float (&x)[8]) {
            // Eq. 9 in the float domain: d = x - offset (one subtraction), then round(d / s).  Re-quantised values sit
            // on rounding boundaries of the new grid whenever the old and new scales are in a small rational ratio, so
            // the quotient must be the IEEE one every time: with 1/s correctly rounded, y0 = d (1/s) followed by two
            // remainder corrections y += (d - y s) (1/s), each one fused multiply-add pair, is the correctly rounded
            // d / s (the first correction makes y faithful, the second exact).  Then: round to nearest even by adding
            // and subtracting 1.5 * 2^23, clamp to [0, n] by a saturating multiply with 1/n, and sum
            // n * u * 2^(bits k) into the sub-word (the sum is within 2^-6 of the integer it stands for, so the
            // conversion restores it).  The quotient lies in [0, n] up to rounding, far inside the exact range.
            uint64_t out;
            {
                float acc[NSUB];
#pragma unroll
                for (int j = 0; j < NSUB; ++j) acc[j] = 0.f;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float d = __fsub_rn(x[e], fv[e]);
                    float y = __fmul_rn(d, iv[e]);
                    y = __fmaf_rn(__fmaf_rn(y, ns[e], d), iv[e], y);
                    y = __fmaf_rn(__fmaf_rn(y, ns[e], d), iv[e], y);
                    const float r = __fadd_rn(__fadd_rn(y, 12582912.f), -12582912.f);
                    const float u = rq_mul_sat(r, KINV);
                    acc[e / SUB] = __fmaf_rn(u, (float)(NMAX << (BITS * (e % SUB))), acc[e / SUB]);
                }
                out = 0;
#pragma unroll
                for (int j = 0; j < NSUB; ++j) out |= (uint64_t)__float2uint_rn(acc[j]) << (16 * j);
            }
            uint8_t* rowp = obase + i * (4 * ROWB);
            if (BITS == 2) *reinterpret_cast<uint16_t*>(rowp) = (uint16_t)out;
            else if (BITS == 4) *reinterpret_cast<uint32_t*>(rowp) = (uint32_t)out;
            else *reinterpret_cast<uint2*>(rowp) = make_uint2((uint32_t)out, (uint32_t)(out >> 32));
        };
        walk(put, [&](int i, const float (&x0)[8], const float (&x1)[8]) { put(i, x0); put(i + 1, x1); });
        // the parameters go out last: in place, the group's old parameters may still have been read from memory above
        *reinterpret_cast<float2*>(dst.kscale + prm + 8 * w + 2 * tq) = make_float2(s2[0], s2[1]);
        *reinterpret_cast<float2*>(dst.kzero + prm + 8 * w + 2 * tq) = make_float2(z2[0], z2[1]);
        __syncwarp();   // the staged rows are rewritten by the next item
    }
}

// ---------------------------------------------------------------------------
// Values of kept tokens move verbatim: codes row, scale, zero-point, origin.
// One thread per (head, new position, 16-byte piece).
// ---------------------------------------------------------------------------
template <int ROWB>
__global__ void __launch_bounds__(256) gather_v_kernel(LayerView src, LayerView dst, int H, int n_old_new,
                                                       int T_first, const int* __restrict__ srcmap) {
    xsv_dep_release();
    xsv_dep_sync();
    constexpr int PPR = ROWB / 16;
    const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
    const long long total = (long long)H * n_old_new * PPR;
    if (idx >= total) return;
    const int piece = (int)(idx % PPR);
    const long long hp = idx / PPR;
    const int p = (int)(hp % n_old_new), h = (int)(hp / n_old_new);
    const int sp = (srcmap != nullptr && p >= T_first) ? srcmap[p - T_first] : p;
    const uint4* s = reinterpret_cast<const uint4*>(src.vcodes + ((size_t)h * src.cap + sp) * ROWB) + piece;
    uint4* d = reinterpret_cast<uint4*>(dst.vcodes + ((size_t)h * dst.cap + p) * ROWB) + piece;
    *d = *s;
    if (piece == 0) {
        if (dst.bits < 16) {
            dst.vscale[(size_t)h * dst.cap + p] = src.vscale[(size_t)h * src.cap + sp];
            dst.vzero[(size_t)h * dst.cap + p] = src.vzero[(size_t)h * src.cap + sp];
        }
        if (h == 0) dst.origin[p] = src.origin[sp];
    }
}

// Same for raw 16-bit key rows (bits == 16).
__global__ void __launch_bounds__(256) gather_kraw_kernel(LayerView src, LayerView dst, int H, int n_old_new,
                                                          int T_first, const int* __restrict__ srcmap) {
    xsv_dep_release();
    xsv_dep_sync();
    constexpr int PPR = 8;
    const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
    const long long total = (long long)H * n_old_new * PPR;
    if (idx >= total) return;
    const int piece = (int)(idx % PPR);
    const long long hp = idx / PPR;
    const int p = (int)(hp % n_old_new), h = (int)(hp / n_old_new);
    const int sp = (srcmap != nullptr && p >= T_first) ? srcmap[p - T_first] : p;
    const uint4* s = reinterpret_cast<const uint4*>(src.kcodes + ((size_t)h * src.cap + sp) * 128) + piece;
    uint4* d = reinterpret_cast<uint4*>(dst.kcodes + ((size_t)h * dst.cap + p) * 128) + piece;
    *d = *s;
}

// Append the fresh frame's raw rows of K and V (bits == 16) and their origins.
__global__ void __launch_bounds__(256) append_raw_kernel(LayerView dst, const uint4* __restrict__ Kf,
                                                         const uint4* __restrict__ Vf, int H, int F,
                                                         int n_old_new, long long origin0) {
    xsv_dep_release();
    xsv_dep_sync();
    const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
    const long long total = (long long)H * F * 8;
    if (idx >= total) return;
    const int piece = (int)(idx % 8);
    const long long hf = idx / 8;
    const int f = (int)(hf % F), h = (int)(hf / F);
    const size_t d = ((size_t)h * dst.cap + n_old_new + f) * 8 + piece;
    reinterpret_cast<uint4*>(dst.kcodes)[d] = Kf[idx];
    reinterpret_cast<uint4*>(dst.vcodes)[d] = Vf[idx];
    if (h == 0 && piece == 0) dst.origin[n_old_new + f] = origin0 + f;
}

}  // namespace

// ------------------------------ launchers ----------------------------------
bool xsv_dep_launch_enabled() {
    static const bool on = (getenv("XSV_NO_DEP_LAUNCH") == nullptr);
    return on;
}

int xsv_current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return -1;
    }
    return dev;
}

int xsv_sm_count() {
    static XsvPerDeviceInt table;
    const int dev = xsv_current_device();
    int n = table.get(dev);
    if (n == 0) {
        if (dev < 0 || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        table.set(dev, n);
    }
    return n;
}

cudaError_t xsv_launch_qtilde(const void* Q, int dtype, int H, int F, int n_special, int g, float* qpart,
                              cudaStream_t st) {
    dim3 grid(XSV_QCHUNKS, H);
    if (dtype == 0) xsv_launch_dep(qtilde_partial_kernel<__half>, grid, dim3(256), 0, st, (const __half*)Q, F, n_special, g, qpart);
    else xsv_launch_dep(qtilde_partial_kernel<__nv_bfloat16>, grid, dim3(256), 0, st, (const __nv_bfloat16*)Q, F, n_special, g, qpart);
    xsv_count_launch(1);
    return cudaGetLastError();
}

cudaError_t xsv_launch_score(const LayerView& lv, int H, int T_first, int T_c, const float* qpart, float qnorm,
                             float* scores, cudaStream_t st) {
    const int n = T_c - T_first;
    if (n <= 0) return cudaSuccess;
    const int grid = ((T_c - 1) >> 6) - (T_first >> 6) + 1;      // key groups that hold a middle token
    const size_t smem = ((size_t)H * 64 + ((H + 3) & ~3) + 4 * 64) * sizeof(float);
    cudaError_t e = cudaSuccess;
#define XSV_SCORE(B)                                                                                       \
    {                                                                                                      \
        static XsvPerDeviceInt attr_set;   /* largest opt-in size configured per device */               \
        const int dev = xsv_current_device();                                                              \
        if (smem > 48 * 1024 && attr_set.get(dev) < (int)smem) {                                           \
            e = cudaFuncSetAttribute(score_kernel<B>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
            if (e != cudaSuccess) return e;                                                                \
            attr_set.set(dev, (int)smem);                                                                  \
        }                                                                                                  \
        xsv_launch_dep(score_kernel<B>, dim3(grid), dim3(SCORE_TPB), smem, st, lv, H, T_first, T_c, qpart, H * XSV_QCHUNKS, qnorm, scores); \
    }
    switch (lv.bits) {
        case 2: XSV_SCORE(2) break;
        case 4: XSV_SCORE(4) break;
        case 8: XSV_SCORE(8) break;
        default: return cudaErrorInvalidValue;
    }
#undef XSV_SCORE
    xsv_count_launch();
    return cudaGetLastError();
}

cudaError_t xsv_launch_score_raw(const LayerView& lv, int dtype, int H, int T_first, int T_c, const float* qpart,
                                 float qnorm, float* scores, cudaStream_t st) {
    const int n = T_c - T_first;
    if (n <= 0) return cudaSuccess;
    const int grid = (n + 63) / 64;
    if (dtype == 0) xsv_launch_dep(score_raw_kernel<__half>, dim3(grid), dim3(SCORE_TPB), 0, st, lv, H, T_first, T_c, qpart, H * XSV_QCHUNKS, qnorm, scores);
    else xsv_launch_dep(score_raw_kernel<__nv_bfloat16>, dim3(grid), dim3(SCORE_TPB), 0, st, lv, H, T_first, T_c, qpart, H * XSV_QCHUNKS, qnorm, scores);
    xsv_count_launch();
    return cudaGetLastError();
}

cudaError_t xsv_launch_select(const float* scores, int n, int k, int T_first, int T_c, int* srcmap, int* dscal,
                              cudaStream_t st) {
#define XSV_SEL(KPT)                                                                                             \
    {                                                                                                            \
        static XsvPerDeviceInt attr_set;                                                                         \
        const int dev = xsv_current_device();                                                                    \
        if (!attr_set.get(dev)) {                                                                                \
            cudaError_t e = cudaFuncSetAttribute(select_reg_kernel<KPT>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                                 1024 * KPT * 4);                                                \
            if (e != cudaSuccess) return e;                                                                      \
            attr_set.set(dev, 1);                                                                                \
        }                                                                                                        \
        xsv_launch_dep(select_reg_kernel<KPT>, dim3(1), dim3(1024), 1024 * KPT * 4, st, scores, n, k, T_first, T_c, srcmap, dscal); \
    }
    if (n <= 1024 * 8) XSV_SEL(8)
    else if (n <= 1024 * 16) XSV_SEL(16)
    else if (n <= 1024 * 24) XSV_SEL(24)
    else if (n <= 1024 * 32) XSV_SEL(32)
    else xsv_launch_dep(select_kernel, dim3(1), dim3(1024), 0, st, scores, n, k, T_first, T_c, srcmap, dscal);
#undef XSV_SEL
    xsv_count_launch();
    return cudaGetLastError();
}

cudaError_t xsv_launch_compress(const LayerView& src, const LayerView& dst, const void* Kf, const void* Vf, int dtype,
                                int H, int F, int n_old_new, int T_new, int T_first, const int* srcmap,
                                const int* fz_dev, int fz_host, long long origin0, bool with_values, int* status,
                                cudaStream_t st) {
    const int ngroups = (T_new + XSV_G - 1) / XSV_G;
    const bool same = src.kcodes == dst.kcodes;
    const int g0 = (fz_dev == nullptr && same) ? fz_host : 0;   // in place: skip the frozen prefix
    const int n_items = max(0, ngroups - g0) * H, wpb = RQ_THREADS / 32;
    const int n_vg = (same || !with_values) ? 0 : ((n_old_new + 63) / 64) * H;     // value rows that move
    const int n_vq = with_values ? ((F + RQ_VROWS - 1) / RQ_VROWS) * H : 0;        // value rows of the frame
    const int n_all = n_items + n_vg + n_vq;
    if (n_all <= 0) return cudaSuccess;
#define XSV_RQ(TT, B)                                                                                                \
    {                                                                                                                \
        const size_t smem = (size_t)wpb * RqCfg<B>::WORDS * 4;                                                       \
        static XsvPerDeviceInt per_sm_of;   /* resident blocks per multiprocessor: the grid is one wave of them */   \
        const int dev = xsv_current_device();                                                                        \
        int per_sm = per_sm_of.get(dev);                                                                             \
        if (per_sm == 0) {                                                                                           \
            cudaFuncSetAttribute(requant_k_kernel<TT, B>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);   \
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, requant_k_kernel<TT, B>, RQ_THREADS, smem) != \
                    cudaSuccess || per_sm <= 0)                                                                      \
                per_sm = 2;                                                                                          \
            per_sm_of.set(dev, per_sm);                                                                              \
        }                                                                                                            \
        const int grid = min((n_all + wpb - 1) / wpb, xsv_sm_count() * per_sm);                                      \
        xsv_launch_dep(requant_k_kernel<TT, B>, dim3(grid), dim3(RQ_THREADS), smem, st, src, dst, (const TT*)Kf,     \
                       (const TT*)Vf, H, F, n_old_new, T_new, T_first, srcmap, fz_dev, fz_host, g0, n_items, n_vg,   \
                       n_vq, origin0, status);                                                                       \
    }
    if (dtype == 0) {
        switch (src.bits) {
            case 2: XSV_RQ(__half, 2); break;
            case 4: XSV_RQ(__half, 4); break;
            case 8: XSV_RQ(__half, 8); break;
            default: return cudaErrorInvalidValue;
        }
    } else {
        switch (src.bits) {
            case 2: XSV_RQ(__nv_bfloat16, 2); break;
            case 4: XSV_RQ(__nv_bfloat16, 4); break;
            case 8: XSV_RQ(__nv_bfloat16, 8); break;
            default: return cudaErrorInvalidValue;
        }
    }
#undef XSV_RQ
    xsv_count_launch();
    return cudaGetLastError();
}

cudaError_t xsv_launch_values(const LayerView& src, const LayerView& dst, const void* Vf, int dtype, int H, int F,
                              int n_old_new, int T_first, const int* srcmap, long long origin0, int* status,
                              cudaStream_t st) {
    if (src.vcodes != dst.vcodes && n_old_new > 0) {
        const long long total = (long long)H * n_old_new * (src.rowb / 16);
        const int grid = (int)((total + 255) / 256);
        switch (src.rowb) {
            case 16: xsv_launch_dep(gather_v_kernel<16>, dim3(grid), dim3(256), 0, st, src, dst, H, n_old_new, T_first, srcmap); break;
            case 32: xsv_launch_dep(gather_v_kernel<32>, dim3(grid), dim3(256), 0, st, src, dst, H, n_old_new, T_first, srcmap); break;
            case 64: xsv_launch_dep(gather_v_kernel<64>, dim3(grid), dim3(256), 0, st, src, dst, H, n_old_new, T_first, srcmap); break;
            default: return cudaErrorInvalidValue;
        }
        xsv_count_launch();
    }
    const int n_vq = ((F + RQ_VROWS - 1) / RQ_VROWS) * H;
    const int grid = (n_vq + 7) / 8;
#define XSV_QV(TT, B) xsv_launch_dep(quant_v_kernel<TT, B>, dim3(grid), dim3(256), 0, st, dst, (const TT*)Vf, H, F, n_old_new, origin0, n_vq, status)
    if (dtype == 0) {
        switch (dst.bits) {
            case 2: XSV_QV(__half, 2); break;
            case 4: XSV_QV(__half, 4); break;
            case 8: XSV_QV(__half, 8); break;
            default: return cudaErrorInvalidValue;
        }
    } else {
        switch (dst.bits) {
            case 2: XSV_QV(__nv_bfloat16, 2); break;
            case 4: XSV_QV(__nv_bfloat16, 4); break;
            case 8: XSV_QV(__nv_bfloat16, 8); break;
            default: return cudaErrorInvalidValue;
        }
    }
#undef XSV_QV
    xsv_count_launch();
    return cudaGetLastError();
}

cudaError_t xsv_launch_raw_update(const LayerView& src, const LayerView& dst, const void* Kf, const void* Vf,
                                  int H, int F, int n_old_new, int T_first, const int* srcmap, long long origin0,
                                  cudaStream_t st) {
    if (src.kcodes != dst.kcodes && n_old_new > 0) {
        const long long total = (long long)H * n_old_new * 8;
        const int grid = (int)((total + 255) / 256);
        xsv_launch_dep(gather_kraw_kernel, dim3(grid), dim3(256), 0, st, src, dst, H, n_old_new, T_first, srcmap);
        xsv_launch_dep(gather_v_kernel<128>, dim3(grid), dim3(256), 0, st, src, dst, H, n_old_new, T_first, srcmap);
        xsv_count_launch(2);
    }
    const long long total = (long long)H * F * 8;
    xsv_launch_dep(append_raw_kernel, dim3((int)((total + 255) / 256)), dim3(256), 0, st, dst, (const uint4*)Kf, (const uint4*)Vf, H, F,
                                                                  n_old_new, origin0);
    xsv_count_launch();
    return cudaGetLastError();
}
