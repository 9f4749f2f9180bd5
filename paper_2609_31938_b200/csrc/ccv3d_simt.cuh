// Plain FP32-FMA kernels: the direct causal Conv3D (FP32 layers, and the
// BF16 reference route), the cache-update copy, and the chain glue.
//
// The direct kernel evaluates Eq. (2) as written: for an output element it
// walks (ci, dt, dh, dw), picks the source frame of tap dt from the cache or
// from x (Eq. (1) with p_l = 0: Z frame t+dt), treats out-of-image taps as
// zero and adds the bias once.  FP32 accumulation in registers; one rounding
// at the store.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ccv3d {

__device__ __forceinline__ float ld_as_float(const float* p) { return __ldg(p); }
__device__ __forceinline__ float ld_as_float(const __nv_bfloat16* p) {
    return __bfloat162float(__ldg(p));
}
__device__ __forceinline__ void st_from_float(float* p, float v) { *p = v; }
__device__ __forceinline__ void st_from_float(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

struct SimtParams {
    const void* x;
    const void* cache;  // [N,Cin,cf,H,W]; may be null: first chunk, absent frames are skipped
    int cf;             // history frames the cache holds (0..kt-1); older ones are absent (zero)
    const void* w;      // original [Cout,Cin,kt,kh,kw] order, storage dtype
    const float* bias;  // FP32, [Cout]
    void* out;
    int N, Cin, Cout, T, H, W, kt, kh, kw;   // T, H, W: input extents
    int To, Ho, Wo;                          // output extents
    int st;                                  // temporal stride: output frame t reads Z frames t*st + dt*dil_t
    int act;                                 // 1: SiLU on conv + bias before the output rounding
    int sh, sw, ph, pw, dh, dw, dil_t;       // spatial stride, padding, dilation; temporal dilation (Eq. (1)-(2))
};
// With tc = d_t (kt-1): Z = [absent x (tc-cf) ; cache ; x]; frame tau < tc of Z is cache frame tau-(tc-cf) when that is >= 0.

constexpr int SIMT_CO = 8;       // output channels per thread (1 for calls too small to fill the device otherwise)
constexpr int SIMT_THREADS = 128;

// grid.x: ceil(N*To*Ho*Wo / SIMT_THREADS), grid.y: ceil(Cout / CO).  The order of accumulation of an output element
// does not depend on CO.
template <typename TIn, typename TOut, int CO = SIMT_CO>
__global__ void __launch_bounds__(SIMT_THREADS) conv3d_direct_kernel(const SimtParams p) {
    constexpr int SIMT_CO = CO;
    const int64_t HW = (int64_t)p.H * p.W, HWo = (int64_t)p.Ho * p.Wo;
    const int64_t npix = (int64_t)p.N * p.To * HWo;
    const int64_t pix = (int64_t)blockIdx.x * SIMT_THREADS + threadIdx.x;
    if (pix >= npix) return;
    const int w0 = (int)(pix % p.Wo);
    const int h0 = (int)((pix / p.Wo) % p.Ho);
    const int t = (int)((pix / HWo) % p.To);
    const int n = (int)(pix / (HWo * p.To));
    const int co0 = blockIdx.y * SIMT_CO;
    const int tc = p.dil_t * (p.kt - 1);
    const int taps = p.kt * p.kh * p.kw;

    float acc[SIMT_CO];
#pragma unroll
    for (int j = 0; j < SIMT_CO; ++j) acc[j] = (co0 + j < p.Cout) ? p.bias[co0 + j] : 0.f;

    const TIn* x = (const TIn*)p.x;
    const TIn* cache = (const TIn*)p.cache;
    const TIn* wt = (const TIn*)p.w;
    for (int ci = 0; ci < p.Cin; ++ci) {
        for (int dt = 0; dt < p.kt; ++dt) {
            const int tau = t * p.st + dt * p.dil_t;  // frame of Z = [cache ; x], Eq. (1)
            const TIn* frame;
            if (tau < tc) {
                const int cfr = tau - (tc - p.cf);
                if (!cache || cfr < 0) continue;
                frame = cache + (((int64_t)n * p.Cin + ci) * p.cf + cfr) * HW;
            } else {
                frame = x + (((int64_t)n * p.Cin + ci) * p.T + (tau - tc)) * HW;
            }
            for (int dh = 0; dh < p.kh; ++dh) {
                const int hs = h0 * p.sh + dh * p.dh - p.ph;
                if (hs < 0 || hs >= p.H) continue;
                for (int dw = 0; dw < p.kw; ++dw) {
                    const int ws = w0 * p.sw + dw * p.dw - p.pw;
                    if (ws < 0 || ws >= p.W) continue;
                    const float v = ld_as_float(frame + (int64_t)hs * p.W + ws);
                    const int64_t wofs = ((int64_t)ci * p.kt + dt) * p.kh * p.kw + dh * p.kw + dw;
#pragma unroll
                    for (int j = 0; j < SIMT_CO; ++j) {
                        if (co0 + j < p.Cout)
                            acc[j] = fmaf(v, ld_as_float(wt + (int64_t)(co0 + j) * p.Cin * taps + wofs), acc[j]);
                    }
                }
            }
        }
    }
    TOut* out = (TOut*)p.out;
    if (p.act) {
#pragma unroll
        for (int j = 0; j < SIMT_CO; ++j) acc[j] = acc[j] / (1.f + expf(-acc[j]));
    }
#pragma unroll
    for (int j = 0; j < SIMT_CO; ++j)
        if (co0 + j < p.Cout)
            st_from_float(out + (((int64_t)n * p.Cout + co0 + j) * p.To + t) * HWo + (int64_t)h0 * p.Wo + w0, acc[j]);
}

// new_cache[n,ci,j,:,:] = Z[n,ci,T+j,:,:], Z = [cache ; x]; pure bit copy in units of `unit` bytes
// (16 when the frame size allows it, else the element size).
// grid.x covers one frame in units, grid.y strides over the N*Cin*(kt-1) planes.
template <typename U>
__global__ void cache_update_kernel(const U* __restrict__ x, const U* __restrict__ cache, U* __restrict__ new_cache,
                                    int Cin, int T, int tc, int cf, int64_t frame_units, int64_t planes) {
    for (int64_t plane = blockIdx.y; plane < planes; plane += gridDim.y) {  // plane = (n*Cin + ci)*tc + j
        const int j = (int)(plane % tc);
        const int64_t nc = plane / tc;
        const int tau = T + j;
        const U* src = nullptr;
        if (tau < tc) {
            const int cfr = tau - (tc - cf);
            if (cache && cfr >= 0) src = cache + (nc * cf + cfr) * frame_units;
        } else {
            src = x + (nc * T + (tau - tc)) * frame_units;
        }
        U* dst = new_cache + plane * frame_units;
        for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < frame_units;
             i += (int64_t)gridDim.x * blockDim.x) {
            if (src) {
                dst[i] = src[i];
            } else {
                U z;
                memset(&z, 0, sizeof(U));
                dst[i] = z;
            }
        }
    }
}

// FP32 bias from the stored bias (or zeros), padded with zeros up to n_pad.
template <typename TIn>
__global__ void bias_to_f32_kernel(const TIn* __restrict__ b, float* __restrict__ out, int n, int n_pad) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n_pad) out[i] = (b && i < n) ? ld_as_float(b + i) : 0.f;
}

// ---- image-row slabs (height-split halo exchange) ----
// Copies `rows` image rows of every plane: unit = 16-byte vectors (V = uint4) or bytes (V = unsigned char);
// chunk = units per slab of rows, pitches in units per plane, src == nullptr writes zeros.
template <typename V>
__global__ void rows_copy_kernel(V* __restrict__ dst, int64_t dst_pitch, const V* __restrict__ src, int64_t src_pitch,
                                 int64_t planes, int64_t chunk) {
    const int64_t total = planes * chunk;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t pl = i / chunk, off = i - pl * chunk;
        dst[pl * dst_pitch + off] = src ? __ldg(src + pl * src_pitch + off) : V{};
    }
}

// ---- chain glue ----
__global__ void add_bf16_kernel(const __nv_bfloat16* __restrict__ a, const __nv_bfloat16* __restrict__ b,
                                __nv_bfloat16* __restrict__ y, int64_t n) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        y[i] = __float2bfloat16_rn(__bfloat162float(a[i]) + __bfloat162float(b[i]));
}

// 8 elements (16 bytes) per thread; n8 = n / 8, all pointers 16-byte aligned
__global__ void add_bf16_vec_kernel(const uint4* __restrict__ a, const uint4* __restrict__ b, uint4* __restrict__ y,
                                    int64_t n8) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += (int64_t)gridDim.x * blockDim.x) {
        const uint4 va = __ldg(a + i), vb = __ldg(b + i);
        const uint32_t wa[4] = {va.x, va.y, va.z, va.w}, wb[4] = {vb.x, vb.y, vb.z, vb.w};
        uint32_t wy[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float lo = __uint_as_float(wa[k] << 16) + __uint_as_float(wb[k] << 16);
            const float hi = __uint_as_float(wa[k] & 0xFFFF0000u) + __uint_as_float(wb[k] & 0xFFFF0000u);
            const __nv_bfloat162 r = __floats2bfloat162_rn(lo, hi);
            wy[k] = *reinterpret_cast<const uint32_t*>(&r);
        }
        y[i] = make_uint4(wy[0], wy[1], wy[2], wy[3]);
    }
}

// y[nc, t*rt + r, 2h + a, 2w + b] = x[nc, t, h, w]
__global__ void upsample_bf16_kernel(const __nv_bfloat16* __restrict__ x, __nv_bfloat16* __restrict__ y,
                                     int64_t NC, int T, int H, int W, int rt) {
    const int64_t total = NC * T * rt * (int64_t)(2 * H) * (2 * W);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int wo = (int)(i % (2 * W));
        const int ho = (int)((i / (2 * W)) % (2 * H));
        const int to = (int)((i / ((int64_t)4 * W * H)) % (T * rt));
        const int64_t nc = i / ((int64_t)4 * W * H * T * rt);
        y[i] = x[((nc * T + to / rt) * H + ho / 2) * W + wo / 2];
    }
}

// Same, W % 4 == 0 and 16-byte aligned bases: a thread reads 4 input pixels (8 bytes), doubles them to 8 output
// pixels (16 bytes) and writes that vector to the 2 output rows of each of the rt output frames.
__global__ void upsample_bf16_vec_kernel(const uint2* __restrict__ x, uint4* __restrict__ y, int64_t NC, int T, int H,
                                         int W, int rt) {
    const int W4 = W / 4;
    const int64_t total = NC * T * (int64_t)H * W4;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int w4 = (int)(i % W4);
        const int h = (int)((i / W4) % H);
        const int t = (int)((i / ((int64_t)W4 * H)) % T);
        const int64_t nc = i / ((int64_t)W4 * H * T);
        const uint2 v = __ldg(x + i);
        uint4 o;
        o.x = __byte_perm(v.x, v.x, 0x1010);   // pixel 0 twice
        o.y = __byte_perm(v.x, v.x, 0x3232);   // pixel 1 twice
        o.z = __byte_perm(v.y, v.y, 0x1010);
        o.w = __byte_perm(v.y, v.y, 0x3232);
        const int64_t row_vecs = W4;           // 16-byte vectors per output row (2W pixels)
        for (int r = 0; r < rt; ++r) {
            uint4* dst = y + (((nc * T * rt + (int64_t)t * rt + r) * (2 * H) + 2 * h) * row_vecs + w4);
            dst[0] = o;
            dst[row_vecs] = o;
        }
    }
}

}  // namespace ccv3d
