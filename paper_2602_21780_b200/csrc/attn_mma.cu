// Eq. 2 + Eq. 12: attention of one frame's queries over [dequantised cache ;
// fresh frame], warp-level mma.sync version (portable baseline; the tcgen05
// kernel in attn_tc5.cu is the fast path).
//
// One CTA = one head x 128 queries (8 warps x 16 rows).  Keys/values are taken
// 64 tokens at a time: cache tiles coincide with the key quantisation groups,
// so one (scale, zero-point) row per channel serves a whole tile.  Packed codes
// are unpacked and dequantised in registers (float32, Eq. 12), rounded to fp16
// and written to shared memory with a 16-byte XOR swizzle; QK^T and PV run on
// m16n8k16 tensor-core MMAs with float32 accumulation and a float32 online
// softmax.
//
// Operands are fp16 inside the kernel for both input types: bf16 inputs convert
// exactly (saturating beyond +-65504), and the dequantised keys keep an 11-bit
// significand -- rounding them to bf16 alone costs more than the 1e-2 output
// tolerance on peaked softmax rows.
#include "xsv_kernels.h"

namespace {

constexpr int BM = 128;   // queries per CTA
constexpr int BN = 64;    // keys per tile

__device__ __forceinline__ void mma_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// two floats -> packed fp16x2 (lo = a), saturating to the finite range
__device__ __forceinline__ uint32_t pack_h2(float a, float b) {
    uint32_t r;
    asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;\n" : "=r"(r) : "f"(b), "f"(a));
    return r;
}
// a 32-bit word of two input elements (fp16 or bf16) -> packed fp16x2
template <typename T> __device__ __forceinline__ uint32_t to_h2(uint32_t w);
template <> __device__ __forceinline__ uint32_t to_h2<__half>(uint32_t w) { return w; }
template <> __device__ __forceinline__ uint32_t to_h2<__nv_bfloat16>(uint32_t w) {
    return pack_h2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

// Byte offset of 16-byte chunk `chunk` (0..7) of row `row` in a [64][64] 16-bit tile.
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }

// Unpack + dequantise 16 consecutive codes starting at channel c0 (bit offset
// c0*BITS of the row), using per-channel (ks, kz) or per-token (s, z) scale and offset: code * s + z (Eq. 12).
template <int BITS, bool PER_CHANNEL>
__device__ __forceinline__ void dequant16(const uint8_t* rowptr, int c0, const float* ks, const float* kz, float s,
                                          float z, uint32_t (&out)[8]) {
    constexpr uint32_t M = (1u << BITS) - 1u;
    constexpr int NW = 16 * BITS / 32 > 0 ? 16 * BITS / 32 : 1;     // 32-bit words holding 16 codes
    uint32_t w[NW];
    if (BITS == 2) {
        w[0] = *reinterpret_cast<const uint32_t*>(rowptr + c0 / 4);
    } else if (BITS == 4) {
        uint2 t = *reinterpret_cast<const uint2*>(rowptr + c0 / 2);
        w[0] = t.x; w[NW - 1] = t.y;
    } else {
        uint4 t = *reinterpret_cast<const uint4*>(rowptr + c0);
        w[0] = t.x; w[1 % NW] = t.y; w[2 % NW] = t.z; w[3 % NW] = t.w;
    }
    constexpr int CPW = 32 / BITS;
#pragma unroll
    for (int e = 0; e < 16; e += 2) {
        float c_a = (float)((w[e / CPW] >> ((e % CPW) * BITS)) & M);
        float c_b = (float)((w[(e + 1) / CPW] >> (((e + 1) % CPW) * BITS)) & M);
        float a, b;
        if (PER_CHANNEL) {
            a = __fadd_rn(__fmul_rn(c_a, ks[c0 + e]), kz[c0 + e]);
            b = __fadd_rn(__fmul_rn(c_b, ks[c0 + e + 1]), kz[c0 + e + 1]);
        } else {
            a = __fadd_rn(__fmul_rn(c_a, s), z);
            b = __fadd_rn(__fmul_rn(c_b, s), z);
        }
        out[e / 2] = pack_h2(a, b);
    }
}

template <typename T, int BITS>
__global__ void __launch_bounds__(256) attn_mma_kernel(LayerView lv, int T_c, const T* __restrict__ Q,
                                                       const T* __restrict__ Kf, const T* __restrict__ Vf,
                                                       T* __restrict__ out, int F) {
    constexpr int ROWB = XSV_D * BITS / 8;
    __shared__ __align__(128) uint8_t sK[BN * 128];
    __shared__ __align__(128) uint8_t sV[BN * 128];
    __shared__ float sKs[64], sKz[64];

    const int h = blockIdx.y, q0 = blockIdx.x * BM;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gid = lane >> 2, tig = lane & 3;
    const uint32_t sK_u = (uint32_t)__cvta_generic_to_shared(sK), sV_u = (uint32_t)__cvta_generic_to_shared(sV);

    // Q fragments (A operand), 4 k-steps of 16 channels
    uint32_t qa[4][4];
    {
        const int r0 = q0 + warp * 16 + gid, r1 = r0 + 8;
        const uint32_t* g0 = reinterpret_cast<const uint32_t*>(Q + ((size_t)h * F + r0) * XSV_D);
        const uint32_t* g1 = reinterpret_cast<const uint32_t*>(Q + ((size_t)h * F + r1) * XSV_D);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            qa[ks][0] = r0 < F ? to_h2<T>(g0[ks * 8 + tig]) : 0u;
            qa[ks][1] = r1 < F ? to_h2<T>(g1[ks * 8 + tig]) : 0u;
            qa[ks][2] = r0 < F ? to_h2<T>(g0[ks * 8 + 4 + tig]) : 0u;
            qa[ks][3] = r1 < F ? to_h2<T>(g1[ks * 8 + 4 + tig]) : 0u;
        }
    }
    float o[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    const float sc = 0.125f * 1.4426950408889634f;   // 1/sqrt(64) * log2(e)

    const int n_ct = (T_c + BN - 1) / BN;             // cache tiles (== key quantisation groups)
    const int n_ft = (F + BN - 1) / BN;               // fresh tiles
    for (int t = 0; t < n_ct + n_ft; ++t) {
        const bool cached = t < n_ct;
        const int base = cached ? t * BN : (t - n_ct) * BN;
        const int cnt = min(BN, (cached ? T_c : F) - base);
        __syncthreads();   // previous tile fully consumed
        if (cached && BITS < 16) {
            if (tid < 64) sKs[tid] = lv.kscale[((size_t)h * lv.capg + t) * 64 + tid];
            else if (tid < 128) sKz[tid - 64] = lv.kzero[((size_t)h * lv.capg + t) * 64 + tid - 64];
            __syncthreads();
        }
        {
            // thread -> (row, quarter): 16 channels = two 16-byte chunks of K and of V
            const int row = tid >> 2, qtr = tid & 3;
            uint32_t kk[8] = {0, 0, 0, 0, 0, 0, 0, 0}, vv[8] = {0, 0, 0, 0, 0, 0, 0, 0};
            if (row < cnt) {
                if (cached && BITS < 16) {
                    const size_t r = (size_t)h * lv.cap + base + row;
                    dequant16<BITS < 16 ? BITS : 4, true>(lv.kcodes + r * ROWB, qtr * 16, sKs, sKz, 0.f, 0.f, kk);
                    dequant16<BITS < 16 ? BITS : 4, false>(lv.vcodes + r * ROWB, qtr * 16, nullptr, nullptr,
                                                               lv.vscale[r], lv.vzero[r], vv);
                } else {
                    const uint4 *kp, *vp;
                    if (cached) {
                        const size_t r = (size_t)h * lv.cap + base + row;
                        kp = reinterpret_cast<const uint4*>(lv.kcodes + r * 128) + qtr * 2;
                        vp = reinterpret_cast<const uint4*>(lv.vcodes + r * 128) + qtr * 2;
                    } else {
                        const size_t r = (size_t)h * F + base + row;
                        kp = reinterpret_cast<const uint4*>(Kf + r * XSV_D) + qtr * 2;
                        vp = reinterpret_cast<const uint4*>(Vf + r * XSV_D) + qtr * 2;
                    }
                    uint4 a = kp[0], b = kp[1], c = vp[0], d = vp[1];
                    kk[0] = to_h2<T>(a.x); kk[1] = to_h2<T>(a.y); kk[2] = to_h2<T>(a.z); kk[3] = to_h2<T>(a.w);
                    kk[4] = to_h2<T>(b.x); kk[5] = to_h2<T>(b.y); kk[6] = to_h2<T>(b.z); kk[7] = to_h2<T>(b.w);
                    vv[0] = to_h2<T>(c.x); vv[1] = to_h2<T>(c.y); vv[2] = to_h2<T>(c.z); vv[3] = to_h2<T>(c.w);
                    vv[4] = to_h2<T>(d.x); vv[5] = to_h2<T>(d.y); vv[6] = to_h2<T>(d.z); vv[7] = to_h2<T>(d.w);
                }
            }
            *reinterpret_cast<uint4*>(sK + tile_off(row, qtr * 2)) = make_uint4(kk[0], kk[1], kk[2], kk[3]);
            *reinterpret_cast<uint4*>(sK + tile_off(row, qtr * 2 + 1)) = make_uint4(kk[4], kk[5], kk[6], kk[7]);
            *reinterpret_cast<uint4*>(sV + tile_off(row, qtr * 2)) = make_uint4(vv[0], vv[1], vv[2], vv[3]);
            *reinterpret_cast<uint4*>(sV + tile_off(row, qtr * 2 + 1)) = make_uint4(vv[4], vv[5], vv[6], vv[7]);
        }
        __syncthreads();

        // S = Q K^T : 8 key blocks of 8
        float s[8][4];
#pragma unroll
        for (int nb = 0; nb < 8; ++nb) s[nb][0] = s[nb][1] = s[nb][2] = s[nb][3] = 0.f;
#pragma unroll
        for (int nb = 0; nb < 8; ++nb) {
#pragma unroll
            for (int kp = 0; kp < 2; ++kp) {   // two k-steps (32 channels) per ldmatrix.x4
                uint32_t b[4];
                // matrices: (ch chunk 4kp+0), (4kp+1), (4kp+2), (4kp+3) of key rows nb*8..+7
                const int r = nb * 8 + (lane & 7), chunk = kp * 4 + (lane >> 3);
                ldmatrix_x4(b, sK_u + tile_off(r, chunk));
                mma_f16(s[nb], qa[kp * 2], b[0], b[1]);
                mma_f16(s[nb], qa[kp * 2 + 1], b[2], b[3]);
            }
        }
        // mask the tail of a partial tile, scale into the log2 domain
#pragma unroll
        for (int nb = 0; nb < 8; ++nb) {
            const int c = nb * 8 + tig * 2;
            s[nb][0] = (c < cnt) ? s[nb][0] * sc : -INFINITY;
            s[nb][1] = (c + 1 < cnt) ? s[nb][1] * sc : -INFINITY;
            s[nb][2] = (c < cnt) ? s[nb][2] * sc : -INFINITY;
            s[nb][3] = (c + 1 < cnt) ? s[nb][3] * sc : -INFINITY;
        }
        float mx0 = m0, mx1 = m1;
#pragma unroll
        for (int nb = 0; nb < 8; ++nb) {
            mx0 = fmaxf(mx0, fmaxf(s[nb][0], s[nb][1]));
            mx1 = fmaxf(mx1, fmaxf(s[nb][2], s[nb][3]));
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xFFFFFFFFu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xFFFFFFFFu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xFFFFFFFFu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xFFFFFFFFu, mx1, 2));
        const float r0 = exp2f(m0 - mx0), r1 = exp2f(m1 - mx1);   // 0 on the first tile (m = -inf)
        m0 = mx0; m1 = mx1;
        float ls0 = 0.f, ls1 = 0.f;
#pragma unroll
        for (int nb = 0; nb < 8; ++nb) {
            s[nb][0] = exp2f(s[nb][0] - mx0); s[nb][1] = exp2f(s[nb][1] - mx0);
            s[nb][2] = exp2f(s[nb][2] - mx1); s[nb][3] = exp2f(s[nb][3] - mx1);
            ls0 += s[nb][0] + s[nb][1];
            ls1 += s[nb][2] + s[nb][3];
        }
        l0 = l0 * r0 + ls0;
        l1 = l1 * r1 + ls1;
#pragma unroll
        for (int i = 0; i < 8; ++i) { o[i][0] *= r0; o[i][1] *= r0; o[i][2] *= r1; o[i][3] *= r1; }

        // O += P V : 4 k-steps of 16 keys, 8 channel blocks of 8
#pragma unroll
        for (int kk2 = 0; kk2 < 4; ++kk2) {
            uint32_t pa[4];
            pa[0] = pack_h2(s[2 * kk2][0], s[2 * kk2][1]);
            pa[1] = pack_h2(s[2 * kk2][2], s[2 * kk2][3]);
            pa[2] = pack_h2(s[2 * kk2 + 1][0], s[2 * kk2 + 1][1]);
            pa[3] = pack_h2(s[2 * kk2 + 1][2], s[2 * kk2 + 1][3]);
#pragma unroll
            for (int np = 0; np < 4; ++np) {   // two channel blocks per ldmatrix.x4.trans
                uint32_t b[4];
                // matrices: (keys kk2*16+0..7, chunk 2np), (keys +8..15, chunk 2np), (keys 0..7, chunk 2np+1), (keys 8..15, chunk 2np+1)
                const int r = kk2 * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, chunk = np * 2 + (lane >> 4);
                ldmatrix_x4_trans(b, sV_u + tile_off(r, chunk));
                mma_f16(o[np * 2], pa, b[0], b[1]);
                mma_f16(o[np * 2 + 1], pa, b[2], b[3]);
            }
        }
    }
    // row sums across the 4 lanes of a quad, normalise, store
    l0 += __shfl_xor_sync(0xFFFFFFFFu, l0, 1); l0 += __shfl_xor_sync(0xFFFFFFFFu, l0, 2);
    l1 += __shfl_xor_sync(0xFFFFFFFFu, l1, 1); l1 += __shfl_xor_sync(0xFFFFFFFFu, l1, 2);
    const float i0 = 1.f / l0, i1 = 1.f / l1;
    const int r0 = q0 + warp * 16 + gid, r1 = r0 + 8;
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) {
        const int c = nb * 8 + tig * 2;
        if (r0 < F) *reinterpret_cast<uint32_t*>(out + ((size_t)h * F + r0) * XSV_D + c) = xsv_pack2<T>(o[nb][0] * i0, o[nb][1] * i0);
        if (r1 < F) *reinterpret_cast<uint32_t*>(out + ((size_t)h * F + r1) * XSV_D + c) = xsv_pack2<T>(o[nb][2] * i1, o[nb][3] * i1);
    }
}

}  // namespace

cudaError_t xsv_launch_attn_mma(const LayerView& lv, int T_c, const void* Q, const void* K, const void* V, void* out,
                                int dtype, int H, int F, cudaStream_t st) {
    dim3 grid((F + BM - 1) / BM, H);
#define XSV_AT(TT, B) attn_mma_kernel<TT, B><<<grid, 256, 0, st>>>(lv, T_c, (const TT*)Q, (const TT*)K, (const TT*)V, (TT*)out, F)
    if (dtype == 0) {
        switch (lv.bits) {
            case 2: XSV_AT(__half, 2); break;
            case 4: XSV_AT(__half, 4); break;
            case 8: XSV_AT(__half, 8); break;
            case 16: XSV_AT(__half, 16); break;
            default: return cudaErrorInvalidValue;
        }
    } else {
        switch (lv.bits) {
            case 2: XSV_AT(__nv_bfloat16, 2); break;
            case 4: XSV_AT(__nv_bfloat16, 4); break;
            case 8: XSV_AT(__nv_bfloat16, 8); break;
            case 16: XSV_AT(__nv_bfloat16, 16); break;
            default: return cudaErrorInvalidValue;
        }
    }
#undef XSV_AT
    xsv_count_launch();
    return cudaGetLastError();
}
