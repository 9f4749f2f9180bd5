// Layout kernels of the tensor-core route: weight packing, the channels-last staging pass (BF16 and FP32 with
// the TF32 hi/lo split), frame-ring moves.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ccv3d {

// ------------------------------------------------------------------------------------------------
// weight packing (create time)
// ------------------------------------------------------------------------------------------------
// Wq[dt][cb][nt][sp][r][e]: for temporal tap dt, input-channel block cb, output-channel tile nt and spatial
// tap sp = dh*kw + dw, a tile of NPAD rows (output channels) x KB input channels, stored as the exact
// shared-memory image the tensor core expects for a K-major operand with 128-byte (KB = 64) or 64-byte
// (KB = 32) swizzle: the 16-byte chunk c of row r sits at chunk position c ^ (r & 7), respectively
// c ^ ((r >> 1) & 3).  A tile, or a run of consecutive spatial taps, is then one contiguous bulk copy.
// Zero outside the real channel extents.
__global__ void pack_weights_kernel(const __nv_bfloat16* __restrict__ w, __nv_bfloat16* __restrict__ wq, int Cout,
                                    int Cin, int kt, int spatial, int CB, int KB, int NT, int NPAD) {
    const int64_t total = (int64_t)kt * CB * NT * spatial * NPAD * KB;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        int64_t q = i;
        const int e = (int)(q % KB); q /= KB;
        const int r = (int)(q % NPAD); q /= NPAD;
        const int sp = (int)(q % spatial); q /= spatial;
        const int nt = (int)(q % NT); q /= NT;
        const int cb = (int)(q % CB);
        const int dt = (int)(q / CB);
        const int chunk_stored = e >> 3;
        const int chunk = chunk_stored ^ (KB == 64 ? (r & 7) : ((r >> 1) & 3));
        const int ci = cb * KB + chunk * 8 + (e & 7);
        const int co = nt * NPAD + r;
        __nv_bfloat16 v = __float2bfloat16_rn(0.f);
        if (ci < Cin && co < Cout) v = w[(((int64_t)co * Cin + ci) * kt + dt) * spatial + sp];
        wq[i] = v;
    }
}

// ------------------------------------------------------------------------------------------------
// staging: NCTHW -> channels-last blocks, fused with the cache update
// ------------------------------------------------------------------------------------------------
struct StageParams {
    const __nv_bfloat16* x;      // [N,Cin,T,H,W]
    const __nv_bfloat16* cache;  // [N,Cin,cf,H,W] or null
    int cf;                      // history frames the cache holds (0..tc); Z frame f < tc is cache frame f-(tc-cf) if >= 0
    __nv_bfloat16* zs;           // [N][F][CB][H][W][KB], F = tc + T
    __nv_bfloat16* new_cache;    // [N,Cin,tc,H,W] or null
    int N, Cin, T, H, W, tc, CB;
    int f_begin;                 // first Z frame to stage (tc when there is no cache and nothing older is needed)
    int h_begin;                 // first image row of this launch (grid.y rows are staged)
    int ring_F = 0, ring_f0 = 0; // ring_F > 0 (separate staging kernel only): zs is a frame ring of ring_F slots and
                                 // Z frame f goes to slot (ring_f0 + f) mod ring_F
    // Phase-decomposed copy for layers with a spatial stride (separate staging kernel only; ph_sh = 0: off):
    // zs is [N][F][CB][ph_sh*ph_sw][ph_Hp][ph_Wp][KB], pixel (h, w) goes to phase (h % ph_sh) * ph_sw + w % ph_sw at
    // (h / ph_sh, w / ph_sw); the launch covers ph_Hp*ph_sh rows and ph_Wp*ph_sw columns, zeros beyond the image.
    int ph_sh = 0, ph_sw = 0, ph_Hp = 0, ph_Wp = 0;
};

constexpr int STG_PX = 64;  // pixels of one image row handled per block

// grid: (ceil(W/64), rows of this launch, N*(F - f_begin)*CB); block: 32 * (KB/8) threads.
// VEC: W % 8 == 0 and all bases 16-byte aligned -> 16-byte loads along w.
template <int KB, bool VEC>
__global__ void __launch_bounds__(32 * (KB / 8)) stage_frames_kernel(const StageParams p) {
    constexpr int NTHR = 32 * (KB / 8);
    constexpr int PITCH = STG_PX / 2 + 1;  // 32-bit words per channel row (+1: bank spread)
    __shared__ uint32_t tile[KB * PITCH];

    const int F = p.tc + p.T;
    const int nf = F - p.f_begin;
    int z = blockIdx.z;
    const int cb = z % p.CB;
    z /= p.CB;
    const int f = p.f_begin + z % nf;
    const int n = z / nf;
    const int h = p.h_begin + blockIdx.y;
    const int w0 = blockIdx.x * STG_PX;
    const int64_t HW = (int64_t)p.H * p.W;

    // source frame of Z: cache frames first (oldest first), then x
    const __nv_bfloat16* src = nullptr;  // base of channel 0 of this (n, frame); channel stride cstride
    int64_t cstride = 0;
    if (f < p.tc) {
        const int cfr = f - (p.tc - p.cf);
        if (p.cache && cfr >= 0) {
            src = p.cache + ((int64_t)n * p.Cin * p.cf + cfr) * HW;
            cstride = (int64_t)p.cf * HW;
        }
    } else {
        src = p.x + ((int64_t)n * p.Cin * p.T + (f - p.tc)) * HW;
        cstride = (int64_t)p.T * HW;
    }
    // does this frame belong to the updated cache?  new_cache[j] = Z[T + j]
    const int jc = f - p.T;
    __nv_bfloat16* ncdst = nullptr;
    if (p.new_cache && jc >= 0 && jc < p.tc) ncdst = p.new_cache + ((int64_t)n * p.Cin * p.tc + jc) * HW;
    const int64_t ncstride = (int64_t)p.tc * HW;

    // ---- load phase: KB channel rows of up to 64 pixels ----
    if (h >= p.H) src = nullptr, ncdst = nullptr;           // (phase-decomposed copy: rows below the image are zeros)
    if (VEC) {
        // 8 vectors of 8 pixels per row
        for (int i = threadIdx.x; i < KB * 8; i += NTHR) {
            const int c = i >> 3, v = i & 7;
            const int ci = cb * KB + c;
            const int w = w0 + v * 8;
            uint4 val = make_uint4(0u, 0u, 0u, 0u);
            if (w < p.W && ci < p.Cin) {
                if (src) val = __ldg(reinterpret_cast<const uint4*>(src + ci * cstride + (int64_t)h * p.W + w));
                if (ncdst) *reinterpret_cast<uint4*>(ncdst + ci * ncstride + (int64_t)h * p.W + w) = val;
            }
            uint32_t* row = tile + c * PITCH + v * 4;
            row[0] = val.x; row[1] = val.y; row[2] = val.z; row[3] = val.w;
        }
    } else {
        unsigned short* t16 = reinterpret_cast<unsigned short*>(tile);
        for (int i = threadIdx.x; i < KB * STG_PX; i += NTHR) {
            const int c = i / STG_PX, px = i % STG_PX;
            const int ci = cb * KB + c;
            const int w = w0 + px;
            unsigned short val = 0;
            if (w < p.W && ci < p.Cin) {
                if (src) val = __ldg(reinterpret_cast<const unsigned short*>(src + ci * cstride + (int64_t)h * p.W + w));
                if (ncdst) *reinterpret_cast<unsigned short*>(ncdst + ci * ncstride + (int64_t)h * p.W + w) = val;
            }
            t16[c * (2 * PITCH) + px] = val;
        }
    }
    __syncthreads();

    // ---- store phase: each thread builds the 16-byte channel octet of two neighbouring pixels ----
    constexpr int OCT = KB / 8;
    const int oct = threadIdx.x % OCT;
    const int pp = threadIdx.x / OCT;  // pixel pair 0..31
    uint32_t lo[4], hi[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint32_t a = tile[(oct * 8 + 2 * k) * PITCH + pp];      // channel 2k:   pixels (2pp, 2pp+1)
        const uint32_t b = tile[(oct * 8 + 2 * k + 1) * PITCH + pp];  // channel 2k+1
        lo[k] = __byte_perm(a, b, 0x5410);                            // pixel 2pp:   (ch 2k, ch 2k+1)
        hi[k] = __byte_perm(a, b, 0x7632);                            // pixel 2pp+1
    }
    const int FS = p.ring_F > 0 ? p.ring_F : F;         // frame slots per sample
    int fs = p.ring_f0 + f;
    if (fs >= FS) fs -= FS;
    const int wa = w0 + 2 * pp;
    if (p.ph_sh > 0) {
        // phase images: pixel (h, w) -> phase (h % s_h, w % s_w), position (h / s_h, w / s_w); columns up to Wp * s_w
        const int64_t img = (int64_t)p.ph_Hp * p.ph_Wp;
        __nv_bfloat16* base = p.zs + ((((int64_t)n * FS + fs) * p.CB + cb) * (p.ph_sh * p.ph_sw) + (h % p.ph_sh) * p.ph_sw) * img * KB +
                              (int64_t)(h / p.ph_sh) * p.ph_Wp * KB;
        const int wlim = p.ph_Wp * p.ph_sw;
        if (wa < wlim)
            *reinterpret_cast<uint4*>(base + ((wa % p.ph_sw) * img + wa / p.ph_sw) * KB + oct * 8) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        if (wa + 1 < wlim)
            *reinterpret_cast<uint4*>(base + (((wa + 1) % p.ph_sw) * img + (wa + 1) / p.ph_sw) * KB + oct * 8) =
                make_uint4(hi[0], hi[1], hi[2], hi[3]);
        return;
    }
    __nv_bfloat16* dst = p.zs + ((((int64_t)n * FS + fs) * p.CB + cb) * HW + (int64_t)h * p.W) * KB;
    if (wa < p.W) *reinterpret_cast<uint4*>(dst + (int64_t)wa * KB + oct * 8) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    if (wa + 1 < p.W)
        *reinterpret_cast<uint4*>(dst + (int64_t)(wa + 1) * KB + oct * 8) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
}

// ------------------------------------------------------------------------------------------------
// FP32 layers on the tensor cores ("3xTF32"): packing and staging with the hi/lo split
// ------------------------------------------------------------------------------------------------
// The tensor core reads an FP32 operand as TF32 by ignoring its low 13 mantissa bits; what it ignores is kept
// as a second operand, lo(v) = v - hi(v) (exact in FP32; itself truncated to TF32 when used, which leaves a
// relative error of about 2^-21 per product).
__device__ __forceinline__ float tf32_lo(float v) { return v - __uint_as_float(__float_as_uint(v) & 0xFFFFE000u); }

// Wq[pass][dt][cb][nt][sp][r][e], e < 32 FP32 input channels of block cb: pass 0 holds lo(w) (multiplied with the
// activations' values), passes 1 and 2 hold w (multiplied with the activations' remainders, then with their
// values); rows of 128 bytes stored as the 128-byte-swizzled shared-memory image (16-byte chunk c of row r at
// chunk position c ^ (r & 7)).  Zero outside the real channel extents.
__global__ void pack_weights_f32_kernel(const float* __restrict__ w, float* __restrict__ wq, int Cout, int Cin, int kt,
                                        int spatial, int CB, int NT, int NPAD) {
    const int64_t total = (int64_t)3 * kt * CB * NT * spatial * NPAD * 32;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        int64_t q = i;
        const int e = (int)(q % 32); q /= 32;
        const int r = (int)(q % NPAD); q /= NPAD;
        const int sp = (int)(q % spatial); q /= spatial;
        const int nt = (int)(q % NT); q /= NT;
        const int cb = (int)(q % CB); q /= CB;
        const int dt = (int)(q % kt);
        const int pass = (int)(q / kt);
        const int chunk = (e >> 2) ^ (r & 7);
        const int ci = cb * 32 + chunk * 4 + (e & 3);
        const int co = nt * NPAD + r;
        float val = 0.f;
        if (ci < Cin && co < Cout) {
            val = w[(((int64_t)co * Cin + ci) * kt + dt) * spatial + sp];
            if (pass == 0) val = tf32_lo(val);
        }
        wq[i] = val;
    }
}

struct StageF32Params {
    const float* x;          // [N,Cin,T,H,W]
    const float* cache;      // [N,Cin,cf,H,W] or null
    int cf;
    float* zs;               // [N][F][2*CBr][H][W][32]: block 2*cb = the values, block 2*cb+1 = their TF32 remainders
    float* new_cache;        // [N,Cin,tc,H,W] or null
    int N, Cin, T, H, W, tc, CBr;
    int f_begin;
};

// grid: (ceil(W/32), H, N*(F - f_begin)*CBr); block 256.  [32 channels][32 pixels] of an image row -> 32 pixels x
// (32 values, 32 remainders), plus the bit-exact cache update from the same registers.
__global__ void __launch_bounds__(256) stage_frames_f32_kernel(const StageF32Params p) {
    __shared__ float tile[32 * 33];
    const int F = p.tc + p.T;
    const int nf = F - p.f_begin;
    int z = blockIdx.z;
    const int cb = z % p.CBr; z /= p.CBr;
    const int f = p.f_begin + z % nf;
    const int n = z / nf;
    const int h = blockIdx.y;
    const int w0 = blockIdx.x * 32;
    const int64_t HW = (int64_t)p.H * p.W;
    const float* src = nullptr;
    int64_t cstride = 0;
    if (f < p.tc) {
        const int cfr = f - (p.tc - p.cf);
        if (p.cache && cfr >= 0) {
            src = p.cache + ((int64_t)n * p.Cin * p.cf + cfr) * HW;
            cstride = (int64_t)p.cf * HW;
        }
    } else {
        src = p.x + ((int64_t)n * p.Cin * p.T + (f - p.tc)) * HW;
        cstride = (int64_t)p.T * HW;
    }
    const int jc = f - p.T;                               // new_cache[j] = Z[T + j]
    float* ncdst = (p.new_cache && jc >= 0 && jc < p.tc) ? p.new_cache + ((int64_t)n * p.Cin * p.tc + jc) * HW : nullptr;
    const int64_t ncstride = (int64_t)p.tc * HW;
    for (int i = threadIdx.x; i < 32 * 32; i += 256) {
        const int c = i >> 5, px = i & 31;
        const int ci = cb * 32 + c, w = w0 + px;
        float v = 0.f;
        if (w < p.W && ci < p.Cin) {
            if (src) v = __ldg(src + ci * cstride + (int64_t)h * p.W + w);
            if (ncdst) ncdst[ci * ncstride + (int64_t)h * p.W + w] = v;
        }
        tile[c * 33 + px] = v;
    }
    __syncthreads();
    const int px = threadIdx.x >> 3, q = threadIdx.x & 7;    // pixel, channel quad
    const int w = w0 + px;
    if (w < p.W) {
        float4 hi, lo;
        hi.x = tile[(4 * q + 0) * 33 + px]; hi.y = tile[(4 * q + 1) * 33 + px];
        hi.z = tile[(4 * q + 2) * 33 + px]; hi.w = tile[(4 * q + 3) * 33 + px];
        lo.x = tf32_lo(hi.x); lo.y = tf32_lo(hi.y); lo.z = tf32_lo(hi.z); lo.w = tf32_lo(hi.w);
        float* dst = p.zs + ((((int64_t)n * F + f) * (2 * p.CBr) + 2 * cb) * HW + (int64_t)h * p.W + w) * 32 + 4 * q;
        *reinterpret_cast<float4*>(dst) = hi;
        *reinterpret_cast<float4*>(dst + HW * 32) = lo;
    }
}

// ------------------------------------------------------------------------------------------------
// frame rings: the inverse move (ring -> NCTHW) and the nearest-neighbour upsample between rings
// ------------------------------------------------------------------------------------------------
struct RingGeom {
    __nv_bfloat16* base;         // [N][F][CB][H][W][KB]
    int N, F, CB, H, W, KB;
};

// grid: (ceil(W/64), H, N*T*CB); block 256.  [64 pixels][KB channels] of an image row -> KB channel rows of 64 pixels.
template <int KB>
__global__ void __launch_bounds__(256) ring_store_kernel(const RingGeom r, int slot0, int T, int C, __nv_bfloat16* __restrict__ y) {
    constexpr int PITCH = KB + 2;                         // BF16 elements per pixel row (+2: bank spread)
    __shared__ __align__(16) unsigned short tile[STG_PX * PITCH];
    int z = blockIdx.z;
    const int cb = z % r.CB; z /= r.CB;
    const int t = z % T;
    const int n = z / T;
    const int h = blockIdx.y;
    const int w0 = blockIdx.x * STG_PX;
    const int64_t HW = (int64_t)r.H * r.W;
    int fs = slot0 + t;
    if (fs >= r.F) fs -= r.F;
    const __nv_bfloat16* src = r.base + ((((int64_t)n * r.F + fs) * r.CB + cb) * HW + (int64_t)h * r.W + w0) * KB;
    const int npx = (r.W - w0 < STG_PX) ? r.W - w0 : STG_PX;
    constexpr int OCT = KB / 8;
    for (int i = threadIdx.x; i < npx * OCT; i += 256) {   // contiguous 16-byte chunks
        const int px = i / OCT, oct = i % OCT;
        const uint4 u = __ldg(reinterpret_cast<const uint4*>(src) + i);
        uint32_t* d = reinterpret_cast<uint32_t*>(tile + px * PITCH + oct * 8);
        d[0] = u.x; d[1] = u.y; d[2] = u.z; d[3] = u.w;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < KB * STG_PX; i += 256) {
        const int c = i / STG_PX, px = i % STG_PX;
        if (px < npx)
            reinterpret_cast<unsigned short*>(y)[(((int64_t)n * C + cb * KB + c) * T + t) * HW + (int64_t)h * r.W + w0 + px] =
                tile[px * PITCH + c];
    }
}

// One thread per 16-byte chunk of the source frames; each chunk is written to 2x2 pixels of rt output frames.
__global__ void __launch_bounds__(256) ring_upsample_kernel(const RingGeom in, int in_slot0, const RingGeom out, int out_slot0,
                                                            int T, int rt) {
    const int OCT = in.KB / 8;
    const int64_t per_frame = (int64_t)in.CB * in.H * in.W * OCT;
    const int64_t total = (int64_t)in.N * T * per_frame;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        int64_t q = i;
        const int oct = (int)(q % OCT); q /= OCT;
        const int w = (int)(q % in.W); q /= in.W;
        const int h = (int)(q % in.H); q /= in.H;
        const int cb = (int)(q % in.CB); q /= in.CB;
        const int t = (int)(q % T);
        const int n = (int)(q / T);
        int fs = in_slot0 + t;
        if (fs >= in.F) fs -= in.F;
        const uint4 u = __ldg(reinterpret_cast<const uint4*>(
            in.base + ((((int64_t)n * in.F + fs) * in.CB + cb) * in.H * in.W + (int64_t)h * in.W + w) * in.KB + oct * 8));
        for (int j = 0; j < rt; ++j) {
            int os = (out_slot0 + t * rt + j) % out.F;
            __nv_bfloat16* o = out.base + ((((int64_t)n * out.F + os) * out.CB + cb) * out.H * out.W +
                                           (int64_t)(2 * h) * out.W + 2 * w) * out.KB + oct * 8;
            *reinterpret_cast<uint4*>(o) = u;
            *reinterpret_cast<uint4*>(o + out.KB) = u;
            *reinterpret_cast<uint4*>(o + (int64_t)out.W * out.KB) = u;
            *reinterpret_cast<uint4*>(o + (int64_t)(out.W + 1) * out.KB) = u;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// cooperative staging: what the stager warps inside the convolution kernels share with the host
// ------------------------------------------------------------------------------------------------
// The same tile move as stage_frames_kernel<KB, true>, run by the 128 threads of the stager warps: a task is
// [KB channels][PX or 2 PX pixels] of one image row of one Z frame = 8 or 16 KB, fetched by TMA straight from x or the
// cache as two or four raw boxes [32 channels][64 pixels] (128-byte rows, 128-byte swizzle), transposed on the way out
// of shared memory by ldmatrix.trans and written channels-last with 16-byte stores; a frame of the updated cache goes
// back out of the same raw boxes with TMA stores.
struct StagerMaps {       // raw NCTHW views (w, h, frame, c, n), box [32 channels][1][1][64 pixels]
    CUtensorMap x, cache, nc;
};

constexpr int STAGER_MAX_SLOTS = 4;        // tasks in flight per team (a slot holds a task's raw boxes of 4 KB each)

struct StagerRec {        // one task as the issuing thread decoded it, read by the whole team
    __nv_bfloat16* dst;   // channels-last destination of pixel (h, w0)
    int w0, h, n, c0;     // first pixel, image row, sample, first channel of the block
    int fr_nc;            // frame of the updated cache this task also writes, or -1
    int present;          // 0: absent history (zeros, nothing was fetched)
};

// Raw boxes of 4 KB per task: 8 KB tasks next to wide tiles (one pixel block per CTA), 16 KB tasks - twice the pixels -
// next to narrow ones (two pixel blocks), which stage twice the input bytes per MMA cycle and whose stager teams are
// bound by their per-task instructions.
template <int NB>
struct STAGER_BOXES { static constexpr int value = NB == 2 ? 4 : 2; };

template <int KB>
struct StagerGeom {
    static constexpr int PX = (KB == 64) ? 64 : 128;      // pixels of an image row per 8 KB of a task
};

__device__ __forceinline__ void stager_bar() { asm volatile("bar.sync 2, 128;" ::: "memory"); }
// barrier of the 128 stager threads that also ANDs a flag over them (a wait that gave up in one thread ends the
// team together: nobody is left waiting at a barrier for a thread that returned)
__device__ __forceinline__ bool stager_bar_and(bool v) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.and.pred q, 2, 128, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)v)
        : "memory");
    return r != 0;
}

}  // namespace ccv3d
