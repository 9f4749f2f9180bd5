// The implicit-GEMM kernel (conv3d_tcgen05_kernel) with its parameter blocks, and the bounded-wait self-test.
#pragma once
#include <type_traits>
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ccv3d {

// ------------------------------------------------------------------------------------------------
// the implicit-GEMM kernel
// ------------------------------------------------------------------------------------------------
struct TcParams {
    int N, T, H, W, Cout;
    int F;            // frames of Z held in the staging buffer (kt-1 + T)
    int kt, kh, kw;
    int CB;           // input-channel blocks of KB
    int NT, NPAD;     // output-channel tiles and their (padded) width, NPAD % 16 == 0, <= 256
    int tiles_h, tiles_w, total_tiles;   // tile rows handled by this launch, tile columns, tiles of this launch
    int main_tiles;           // > 0: work items main_tiles .. total_tiles-1 are the launch's last tiles at HALF width (the
                              // last wave would be at most half full: twice the items, each half as long); see TileView
    int ty_begin;                        // first tile row of this launch (a launch may cover a band of the image)
    int first_frame;  // Z frames below this are absent (first chunk): their taps are skipped
    int out_f32;      // 1: out is FP32, 0: BF16
    int per_tap_a;    // 1: one A load per tap (box without halo), 0: one halo load per (dt, ci-block)
    int TPB;          // spatial taps per weight stage (1 or kw); kh*kw % TPB == 0
    int epi_tma;      // 1: epilogue stages BF16 tiles in shared memory and stores them with TMA; 0: direct stores;
                      // 2: the output is a frame ring (channels-last), staged pixel-major and stored with TMA
    int ECH;          // output channels per epilogue chunk (32 or 16) when epi_tma
    int SA, SB, ACC;  // ring depths and accumulator buffers
    uint32_t a_slot, b_slot, b_tap;  // bytes per ring slot (multiples of 1024) and per tap inside a weight slot
    uint32_t b_src_tap;       // bytes per tap in the packed weights when that differs from b_tap (split_n), else 0
    int split_n;              // 1: NT and NPAD describe half-width output-channel tiles of a layer packed at full width
    uint32_t e_slot;          // bytes of one epilogue staging buffer (two are allocated when epi_tma)
    uint32_t raw_slot;        // fused mode: bytes of one raw [32 ch][BH rows][32 px] box (two are allocated)
    int tc, cf;               // fused mode: kt-1 and the history frames the cache holds; Z frame f < tc is cache frame f-(tc-cf)
    uint32_t tmem_cols;       // power of two >= NB*NPAD*ACC
    long long wait_limit_clk; // bound of every mbarrier wait, in SM clocks
    unsigned int* band_ctr;   // cooperative staging: per 16-row band, the number of CTAs that have staged their share
    int nbands;               // cooperative staging: 16-row bands of the input image
    int band_first;           // cooperative staging: bands below this were staged before the launch (by stage_frames_kernel)
    int stg_slots;            // cooperative staging: raw slots (tasks in flight) of the stager team, 2..STAGER_MAX_SLOTS
    // general geometry (Eq. (2) with the layer's own padding and dilation, Eq. (1) with d_t); when `general` is 0
    // the kernel uses pad = (k-1)/2 and unit dilation.  H and W above are the OUTPUT extents; the input extents
    // only live in the tensor map.  Spatial stride > 1 is served by the per-tap mode with a strided tensor map.
    int general, pad_h, pad_w, dil_h, dil_w, dil_t, str_h, str_w, str_t;   // T above counts OUTPUT frames (T_o)
    // Spatial stride > 1 from a phase-decomposed staging copy (phased = 1): the staged frames are split into
    // S2 = s_h * s_w phase images (pixel (h, w) lives in phase (h % s_h) * s_w + w % s_w at (h / s_h, w / s_w)), in which
    // consecutive output pixels are consecutive pixels again, so that each phase needs one halo tile and its taps are
    // descriptor offsets into it: tap (a, c) reads phase image pixel (oh + floor((a d_h - p_h) / s_h), ow + ...).
    int phased, S2;
    int ph_bw, ph_bh;                     // halo extents beyond the tile (largest offset range of any phase)
    unsigned char ph_first[17];           // taps of phase q: entries ph_first[q] .. ph_first[q+1]-1 of the lists below
    unsigned char ph_tap[49];             // spatial tap index a*kw + c
    unsigned char ph_roff[49], ph_coff[49];   // the tap's row / column offset inside its phase's halo tile
    signed char ph_h0[16], ph_w0[16];     // halo origin of a phase relative to the tile origin (in phase-image pixels)
    int f0;                   // ring input: the slot of Z frame 0; Z frame f lives in slot (f0 + f) mod F (0 for a staged copy)
    const __nv_bfloat16* res; // optional residual ring [N][res_F][res_CB][H][W][res_KB] holding Cout channels, or null
    int res_F, res_f0, res_CB, res_KB;   // residual frame t is slot (res_f0 + t) mod res_F
    int out_F, out_f0, out_KB;           // epi_tma == 2: output frame t goes to slot (out_f0 + t) mod out_F
    int act;                             // 1: SiLU on conv + bias before the output rounding (and before the residual)
    int up_rt;                           // epi_tma == 2, > 0: the output ring is 2H x 2W; every pixel is written 2x2 times into
                                         // each of the up_rt slots (out_f0 + t*up_rt + j) mod out_F (nearest-neighbour upsample)
#ifdef CCV3D_DEV_TRACE
    unsigned long long* trace;   // dev builds: clock64 stamps of CTA 0
#endif
    const float* bias;        // [NT*NPAD]
    const uint8_t* wq;        // packed weight tiles [dt][cb][nt][sp] of b_tap bytes each
    void* out;
    unsigned int* status;     // 0 = fine; else (block << 8) | site
};

enum : uint32_t {
    SITE_A_EMPTY = 1, SITE_B_EMPTY = 2, SITE_A_FULL = 3, SITE_B_FULL = 4, SITE_ACC_EMPTY = 5, SITE_ACC_FULL = 6,
    SITE_RAW_EMPTY = 7, SITE_RAW_FULL = 8, SITE_BAND = 9
};

constexpr int TC_THREADS = 256;
constexpr int TC_THREADS_FUSED = 384;    // + 4 transposer warps
constexpr int RAW_PX = 32;               // pixels per row of a raw box (64 bytes), starting 8 pixels left of the tile
constexpr int TC_MAX_STAGES = 12;
constexpr int TC_BIAS_SMEM = 512;

struct TcShared {  // placed after the rings
    uint64_t full_a[TC_MAX_STAGES], empty_a[TC_MAX_STAGES];
    uint64_t full_b[TC_MAX_STAGES], empty_b[TC_MAX_STAGES];
    uint64_t acc_full[4], acc_empty[4];   // (the convolution kernel uses two, the 1x1x1 streaming kernel up to four)
    uint64_t raw_full[2], raw_empty[2];
    uint64_t stg_full[STAGER_MAX_SLOTS];  // cooperative staging: a task's raw boxes have landed
    StagerRec stg_rec[STAGER_MAX_SLOTS];
    uint32_t tmem_base;
    volatile int abort_flag;
    alignas(16) float bias_s[TC_BIAS_SMEM];   // the layer's padded bias when it fits (the epilogue reads it once per element)
};

// Work item u of a launch as a tile.  Items below main_tiles (all of them when main_tiles == 0) are tiles of the
// launch's own output-channel width; the others enumerate the remaining tiles at half that width (the mechanism of
// split_n, per tile): full-width tile f = halves 2f and 2f+1, so item u >= main_tiles is half-width tile u + main_tiles.
struct TileView {
    int tile, NT, NPAD, split;
    uint32_t b_tap;       // bytes of one tap of this CTA's weight tile
    bool half;
};
template <bool TAIL>      // TAIL = false: kernels that never see half-width items (everything folds to the launch's values)
__device__ __forceinline__ TileView tile_view(const TcParams& p, int u) {
    TileView v;
    v.half = TAIL && p.main_tiles > 0 && u >= p.main_tiles;
    v.tile = v.half ? u + p.main_tiles : u;
    v.NT = v.half ? 2 * p.NT : p.NT;
    v.NPAD = v.half ? p.NPAD >> 1 : p.NPAD;
    v.split = v.half ? 1 : p.split_n;
    v.b_tap = v.half ? p.b_tap >> 1 : p.b_tap;
    return v;
}

// Bounded wait.  Returns false when the limit expired or another role of this CTA aborted.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, TcShared* sh, const TcParams& p, uint32_t site) {
    const uint32_t b = smem_u32(bar);
#ifdef CCV3D_DEV_TRACE
    // dev builds: cycles CTA 0 spends in waits, summed per wait site (words 16.. of the trace buffer); the first try is
    // inside the measured span, since the hardware may hold a try_wait for a while before it answers
    const long long tw0 = clock64();
    struct Acc { const TcParams& p; uint32_t site; long long t; __device__ ~Acc() {
        if (p.trace && blockIdx.x == 0 && (threadIdx.x & 31) == 0) atomicAdd(p.trace + 16 + site, (unsigned long long)(clock64() - t)); } } acc_{p, site, tw0};
#endif
    if (mbar_try_wait(b, parity)) return true;
    long long t0 = 0;
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(b, parity)) return true;
        if ((it & 63u) == 0u) {
            if (sh->abort_flag) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > p.wait_limit_clk) {
                sh->abort_flag = 1;
                atomicCAS(p.status, 0u, (blockIdx.x << 8) | site);
                return false;
            }
        }
    }
}

// After an abort: give copies in flight a bounded time to land before the CTA goes away.
__device__ __forceinline__ void drain_delay() {
    const long long t0 = clock64();
    while (clock64() - t0 < 400000) __nanosleep(1000);
}

__device__ __forceinline__ uint32_t make_desc_hi(uint32_t sbo_bytes, uint32_t layout_type) {
    // upper word of a shared-memory matrix descriptor: bits 32-45 stride-dimension byte offset >> 4,
    // bits 46-47 descriptor version 1, bits 61-63 swizzle mode
    return ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (layout_type << 29);
}
__device__ __forceinline__ uint32_t make_desc_lo(uint32_t addr) {
    // lower word: bits 0-13 start address >> 4, bits 16-29 leading-dimension byte offset >> 4 (unused for
    // swizzled K-major operands; canonical value 1)
    return ((addr & 0x3FFFFu) >> 4) | (1u << 16);
}

// Residual of one pixel: 32 consecutive channels (64 bytes) starting at channel co0 of a frame ring, as 16 BF16
// pairs.  res_row addresses channel block 0 of the pixel's image row; zeros when there is no residual or the
// pixel lies outside the image.
__device__ __forceinline__ void load_res32(const __nv_bfloat16* res_row, bool valid, int w, int co0, const TcParams& p,
                                           int64_t HW, uint32_t (&rr)[16]) {
    if (res_row && valid) {
        const uint4* src = reinterpret_cast<const uint4*>(res_row + ((int64_t)(co0 / p.res_KB) * HW + w) * p.res_KB +
                                                          (co0 % p.res_KB));
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const uint4 u = __ldg(src + c);
            rr[4 * c] = u.x; rr[4 * c + 1] = u.y; rr[4 * c + 2] = u.z; rr[4 * c + 3] = u.w;
        }
    } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) rr[j] = 0u;
    }
}

// Two neighbouring output channels: round conv + bias to BF16 once; with a residual, add it to that rounded value
// in FP32 and round again (the result of a BF16 convolution followed by a BF16 addition).
__device__ __forceinline__ float silu_f32(float v) { return __fdividef(v, 1.f + __expf(-v)); }

__device__ __forceinline__ uint32_t epi_pair(float a0, float a1, uint32_t res_pair, bool has_res) {
    __nv_bfloat162 o = __floats2bfloat162_rn(a0, a1);
    if (has_res) {
        const float2 of = __bfloat1622float2(o);
        const float2 rf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&res_pair));
        o = __floats2bfloat162_rn(of.x + rf.x, of.y + rf.y);
    }
    return *reinterpret_cast<const uint32_t*>(&o);
}

// The stager warps of the cooperative schedule (warps 8..11 of a CTA): the staging pass - same tile move as
// stage_frames_kernel, cache update included - band by band of 16 image rows; every finished band is signalled with a
// fence and one atomic per CTA.
// Inside a band the tasks ([KB channels][SPX pixels] of one image row of one Z frame, 8 or 16 KB) are ordered (sample, frame,
// channel block, row, chunk of the row) and CTA k takes the k-th of gridDim.x contiguous runs, so that the next task is an
// odometer step away (a team of four warps is bound by its own instruction stream: decoding every task with divisions
// cost more than moving it).  Thread 0 of the team keeps p.stg_slots tasks in flight: it leaves a task's record in
// shared memory and fetches its raw boxes by TMA; the team waits for a task's boxes, transposes them with
// ldmatrix.trans (each lane ends up with 8 consecutive channels of one pixel) and writes them channels-last.  Frames
// of the updated cache leave the same raw boxes by TMA store.  One barrier per task: it shares the outcome of the wait
// and tells thread 0 that everybody has finished reading the previous task's slot.
// PH2: the copy is the phase-decomposed one of a stride-2 layer (four phase images per channel block, pixel (h, w) in
// image (h mod 2) * 2 + w mod 2 at (h / 2, w / 2); H and W even): a task's pixels go alternately to two images.
template <int KB, int NBX, bool PH2 = false>     // NBX: raw boxes of 4 KB per task (2 or 4)
__device__ __forceinline__ void run_stagers(const TcParams& p, const StageParams& sp, const StagerMaps* maps, uint32_t raw0,
                                            TcShared* sh) {
    const int tid = threadIdx.x - 256;
    const int lane = tid & 31, swp = tid >> 5;
    constexpr int SPX = StagerGeom<KB>::PX * (NBX >> 1);    // pixels of an image row per task
    constexpr uint32_t slot_bytes = (uint32_t)NBX * 4096u;
    const int nchunks = (sp.W + SPX - 1) / SPX;
    // box j of a task: 64 pixels x 32 channels at pixel offset box_px(j), channel offset box_ch(j)
    auto box_px = [&](int j) { return KB == 64 ? 64 * (j >> 1) : 64 * j; };
    auto box_ch = [&](int j) { return KB == 64 ? 32 * (j & 1) : 0; };
    const int nf = sp.tc + sp.T - sp.f_begin;
    const int R = p.stg_slots;
    const int64_t HW = (int64_t)sp.H * sp.W;
    const int64_t HWp = PH2 ? (int64_t)sp.ph_Hp * sp.ph_Wp : 0;    // pixels of a phase image
    auto px_off = [&](int px) { return PH2 ? ((int64_t)(px & 1) * HWp + (px >> 1)) * KB : (int64_t)px * KB; };   // (w0 is even)
    // this CTA's run of tasks in band b: [first, last)
    auto band_run = [&](int b, int& first, int& last, int& rows) {
        rows = (sp.H - 16 * b < 16) ? sp.H - 16 * b : 16;
        const int64_t ntask = (int64_t)sp.N * nf * sp.CB * rows * nchunks;
        first = (int)(ntask * blockIdx.x / gridDim.x);
        last = (int)(ntask * (blockIdx.x + 1) / gridDim.x);
    };
    // ldmatrix roles: lane l addresses row l%8 of matrix l/8; a row is one channel's 8 pixels.  Matrix j takes, from
    // each of the four channel octets, the channel pair (octet + j) mod 4, so that its eight rows fall on eight
    // different 16-byte columns of the swizzled box (no bank conflict) and lane (pixel, octet q) receives the four
    // pairs of octet q, rotated by q.
    const int mj = lane >> 3, qq = (lane & 7) >> 1;
    const int cl = 8 * qq + 2 * ((qq + mj) & 3) + (lane & 1);
    const uint32_t lane_off = (uint32_t)cl * 128u, c7 = (uint32_t)(cl & 7);
    const int pq = lane & 3, pp = lane >> 2;

    // thread 0: a cursor over this CTA's tasks
    struct Cursor { int b, left, wc, hr, cb, fi, n, rows; };
    auto open_band = [&](Cursor& c) {
        while (c.b < p.nbands) {
            int first, last;
            band_run(c.b, first, last, c.rows);
            if (last > first) {
                int r = first;
                c.wc = r % nchunks; r /= nchunks;
                c.hr = r % c.rows; r /= c.rows;
                c.cb = r % sp.CB; r /= sp.CB;
                c.fi = r % nf;
                c.n = r / nf;
                c.left = last - first;
                return;
            }
            ++c.b;
        }
        c.left = 0;
    };
    auto advance = [&](Cursor& c) {
        if (--c.left == 0) { ++c.b; open_band(c); return; }
        if (++c.wc == nchunks) {
            c.wc = 0;
            if (++c.hr == c.rows) {
                c.hr = 0;
                if (++c.cb == sp.CB) {
                    c.cb = 0;
                    if (++c.fi == nf) { c.fi = 0; ++c.n; }
                }
            }
        }
    };
    struct Src { const CUtensorMap* tm; int fr; bool present; };
    auto source = [&](int f) {                             // Z frame f: x, or the cache (oldest first), or absent history
        Src s;
        s.tm = &maps->x; s.fr = f - sp.tc;
        if (f < sp.tc) { s.tm = &maps->cache; s.fr = f - (sp.tc - sp.cf); }
        s.present = f >= sp.tc || (sp.cache && s.fr >= 0);
        return s;
    };
    Cursor it = {p.band_first, 0, 0, 0, 0, 0, 0, 0};
    auto issue = [&](int slot) {
        if (it.left == 0) return;
        const int f = sp.f_begin + it.fi, h = 16 * it.b + it.hr, n = it.n;
        const Src s = source(f);
        StagerRec rec;
        rec.w0 = it.wc * SPX; rec.h = h; rec.n = n; rec.c0 = it.cb * KB;
        if (PH2)
            rec.dst = sp.zs + (((((int64_t)n * (sp.tc + sp.T) + f) * sp.CB + it.cb) * 4 + (h & 1) * 2) * HWp +
                               (int64_t)(h >> 1) * sp.ph_Wp + (rec.w0 >> 1)) * KB;
        else
        rec.dst = sp.zs + ((((int64_t)n * (sp.tc + sp.T) + f) * sp.CB + it.cb) * HW + (int64_t)h * sp.W + rec.w0) * KB;
        const int jc = f - sp.T;                           // new_cache[j] = Z[T + j]
        rec.fr_nc = (sp.new_cache && jc >= 0 && jc < sp.tc) ? jc : -1;
        rec.present = s.present ? 1 : 0;
        sh->stg_rec[slot] = rec;
        const uint32_t bar = smem_u32(&sh->stg_full[slot]);
        if (s.present) {
            // (boxes that lie beyond the row are left out)
            const uint32_t dst = raw0 + (uint32_t)slot * slot_bytes;
            int nb = 0;
#pragma unroll
            for (int j = 0; j < NBX; ++j) nb += rec.w0 + box_px(j) < sp.W;
            mbar_expect_tx(bar, (uint32_t)nb * 4096u);
#pragma unroll
            for (int j = 0; j < NBX; ++j)
                if (rec.w0 + box_px(j) < sp.W) tma_load_5d(dst + (uint32_t)j * 4096u, s.tm, bar, rec.w0 + box_px(j), h, s.fr, rec.c0 + box_ch(j), n);
        } else {
            mbar_arrive(bar);
        }
        advance(it);
    };
    if (tid == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&maps->x) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&maps->cache) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&maps->nc) : "memory");
        open_band(it);
        for (int s = 0; s < R; ++s) issue(s);
    }
    int slot = 0, prev = R - 1;
    uint32_t par = 0;
    bool first_task = true, ok = true;
    for (int b = p.band_first; ok && b < p.nbands; ++b) {
        int first, last, rows;
        band_run(b, first, last, rows);
        for (int task = first; task < last; ++task) {
            ok = stager_bar_and(mbar_wait(&sh->stg_full[slot], par, sh, p, SITE_RAW_FULL));
            if (!ok) break;
            if (tid == 0 && !first_task) {
                bulk_wait_read<0>();                       // (a cache frame's stores out of the previous slot)
                issue(prev);
            }
            first_task = false;
            const StagerRec rec = sh->stg_rec[slot];
            const uint32_t src = raw0 + (uint32_t)slot * slot_bytes;
            if (rec.present) {
                if (tid == 0 && rec.fr_nc >= 0) {
#pragma unroll
                    for (int j = 0; j < NBX; ++j)
                        if (rec.w0 + box_px(j) < sp.W)
                            tma_store_5d(&maps->nc, src + (uint32_t)j * 4096u, rec.w0 + box_px(j), rec.h, rec.fr_nc, rec.c0 + box_ch(j), rec.n);
                    bulk_commit();
                }
                // A box is eight units of 8 pixels x 32 channels.  The warp of thread 0, which also decodes and fetches the
                // tasks, takes few of a task's units and the other three warps share the rest: the team moves at the pace
                // of its slowest warp.
                auto units = [&](auto cnt, int first) {
#pragma unroll
                    for (int i = 0; i < decltype(cnt)::value; ++i) {
                        const int u = first + i, o = u & 7, hb = u >> 3;       // pixel octet, box of the slot
                        uint32_t f[4];
                        ldmatrix_x4_trans(src + (uint32_t)hb * 4096u + lane_off + ((((uint32_t)o) ^ c7) << 4), f);
                        // f[j] = channel pair (pq + j) mod 4 of octet pq: rotate into channel order
                        uint32_t g0 = (pq & 1) ? f[3] : f[0], g1 = (pq & 1) ? f[0] : f[1], g2 = (pq & 1) ? f[1] : f[2],
                                 g3 = (pq & 1) ? f[2] : f[3];
                        if (pq & 2) { const uint32_t t0 = g0, t1 = g1; g0 = g2; g1 = g3; g2 = t0; g3 = t1; }
                        const int px = box_px(hb) + 8 * o + pp;
                        const int ch = box_ch(hb) + 8 * pq;
                        if (rec.w0 + px < sp.W) *reinterpret_cast<uint4*>(rec.dst + px_off(px) + ch) = make_uint4(g0, g1, g2, g3);
                    }
                };
                constexpr int U0 = NBX / 2, U1 = (8 * NBX - U0) / 3;           // 1 + 3 x 5 of 16 units, 2 + 3 x 10 of 32
                static_assert(U0 + 3 * U1 == 8 * NBX, "the units of a task are dealt out completely");
                if (swp == 0) units(std::integral_constant<int, U0>{}, 0);
                else units(std::integral_constant<int, U1>{}, U0 + (swp - 1) * U1);
            } else {
                // absent history: zeros, also into the updated cache when the frame belongs to it
                const uint4 z = make_uint4(0u, 0u, 0u, 0u);
                for (int i = tid; i < SPX * (KB / 8); i += 128) {
                    const int px = i / (KB / 8), oc = i % (KB / 8);
                    if (rec.w0 + px < sp.W) *reinterpret_cast<uint4*>(rec.dst + px_off(px) + oc * 8) = z;
                }
                if (rec.fr_nc >= 0)
                    for (int i = tid; i < KB * (SPX / 8); i += 128) {
                        const int c = rec.c0 + i / (SPX / 8), w = rec.w0 + (i % (SPX / 8)) * 8;
                        if (c < sp.Cin && w < sp.W)
                            *reinterpret_cast<uint4*>(sp.new_cache + (((int64_t)rec.n * sp.Cin + c) * sp.tc + rec.fr_nc) * HW +
                                                      (int64_t)rec.h * sp.W + w) = z;
                    }
            }
            prev = slot;
            if (++slot == R) { slot = 0; par ^= 1; }
        }
        if (!ok) break;
        __threadfence();                                   // this thread's stores are visible GPU-wide ...
        stager_bar();                                      // ... for all 128 stager threads, before the band is signalled
        if (tid == 0) atomicAdd(p.band_ctr + b, 1u);
    }
    // the stores of cache frames must have finished READING shared memory before the CTA exits; their writes complete
    // with the grid
    if (tid == 0) bulk_wait_read<0>();
    if (!ok && tid == 0) drain_delay();
#ifdef CCV3D_DEV_TRACE
    if (tid == 0 && p.trace && blockIdx.x == 0) p.trace[12] = clock64();
#endif
}

// KB: input channels per K block (64 -> 128-byte swizzle, 32 -> 64-byte swizzle).  NB: 128-pixel blocks per tile.
// KS/TPBC: compile-time spatial kernel size (kh = kw = KS) and taps per weight stage, which turn the tap loop
// into straight-line code with immediate descriptor offsets; KS = 0 keeps everything run-time (any odd kh, kw,
// and the per-tap A mode).
// FUSED: no staging copy; tm_a is x as (w, h, t, c, n), tm_c the cache as (w, h, frame, c, n); needs KB = 32.
// COOP: cooperative staging - there is no separate staging kernel; four extra warps of every CTA move the
// channels-last copy of [cache ; x] (and the cache update) band by band of 16 image rows, ahead of the tiles that
// read it, so that this HBM-bound work hides under the tensor-core work of the same kernel.  A band is usable
// when every CTA has signalled it (release: fence + atomic; acquire: polled load + proxy fence before the TMA
// loads).  All CTAs are co-resident (grid <= SM count, 1 CTA per SM) and stagers never wait on consumers, so the
// dependency is acyclic; the wait is bounded like every other.
// TF32 (FP32 layers, "3xTF32"): KB = 64 then means 128-byte rows of 32 FP32 channels.  An FP32 product a*w is
// evaluated as hi(a)*lo(w) + lo(a)*hi(w) + hi(a)*hi(w) with hi = the TF32 truncation the tensor core applies by
// itself and lo = the FP32 remainder, staged and packed explicitly: the staging copy holds two blocks per channel
// block (a, a - hi(a)), the packed weights three images (lo(w), w, w).  The whole K loop runs three times, one
// pass per term, the two small correction terms first: the tensor core's FP32 accumulation truncates, which
// costs a fraction of the accumulator's last bit per step, so the long chain of full-size terms is kept as short
// as it can be and the corrections are summed while the accumulator is still 2^-11 of its final size.
// PAIR (cta_group::2): launched in clusters of two CTAs.  A tile is 16 rows x 16*NB pixels; CTA r of the pair loads
// the halo tile of pixel columns 8*NB*r .. and rows r*NPAD/2.. of every weight tile (tm_c is then a 2-D map over the
// packed weights); the leader issues MMAs with M = 256 that read both CTAs' shared memory and fill both CTAs'
// tensor memory, so that per SM and MMA only half of the weight tile crosses L2 -> shared memory and the
// shared-memory read port.  Loads of both CTAs are counted on the leader's "full" barriers; the leader's commits
// arrive on the "empty" and "accumulator full" barriers of both CTAs; both epilogues arrive on the leader's
// "accumulator empty" barrier.
// DIL = TAPS_STRIDE2: the straight-line tap loop of a 3x3 kernel with spatial stride 2 and padding 1 over the four phase
// images of the staged copy (see the host side): per (dt, ci-block) four halo tiles of 17 x (8 NB + 1) pixels, one per
// phase, holding 1, 2, 2 and 4 taps; the nine taps run in phase order, their offsets compile-time constants.
// DIL: spatial dilation of the straight-line tap loop (1, or 2 for 3x3 kernels with d_h = d_w = 2: the tap offsets
// into the halo tile double and stay compile-time constants).
constexpr int TAPS_STRIDE2 = -2;
template <int KB, int NB, int KS, int TPBC, bool FUSED, bool COOP, bool TF32 = false, bool PAIR = false, bool TAIL = false, int DIL = 1>
__global__ void __launch_bounds__((FUSED || COOP) ? TC_THREADS_FUSED : TC_THREADS, 1)
conv3d_tcgen05_kernel(const __grid_constant__ CUtensorMap tm_a,   // staged activations (c, w, h, cb, n*F+f), or x
                      const __grid_constant__ CUtensorMap tm_c,   // fused mode: the cache; PAIR: the packed weights
                      const __grid_constant__ CUtensorMap tm_o,   // out (w, h, t, co, n); used when p.epi_tma
                      const TcParams p, const StageParams sp,
                      const __grid_constant__ StagerMaps smaps) {  // COOP: raw views of x, the cache and the new cache
    static_assert(!(FUSED && COOP), "one or the other");
    static_assert(!FUSED || KB == 32, "the fused mode transposes 32-channel blocks");
    static_assert(!TF32 || (KB == 64 && !FUSED && !COOP), "FP32 layers: 128-byte rows, plain variant");
    static_assert(!PAIR || (KS > 0 && !FUSED), "CTA pairs: straight-line taps");
    static_assert(DIL != TAPS_STRIDE2 || (KS == 3 && PAIR && !TF32 && !TAIL && (TPBC == 1 || TPBC == 3)), "stride-2 straight-line taps: 3x3, CTA pairs");
    static_assert(DIL == 1 || DIL == TAPS_STRIDE2 || (DIL == 2 && KS == 3 && PAIR && !TF32 && !TAIL), "dilated straight-line taps: 3x3, d = 2, CTA pairs");
    // (TF32 layers always write FP32 through the direct-store epilogue, which is where the two accumulators of the
    // last pass are added)
    constexpr uint32_t ROWB = KB * 2;                       // bytes per pixel row (one swizzle span)
    constexpr uint32_t LAYOUT = (KB == 64) ? 2u : 4u;       // 128-byte / 64-byte swizzle
    constexpr uint32_t B_SBO = 8 * ROWB;                    // 8-row group pitch of the weight tile
    constexpr int KSTEPS = KB / 16;
    constexpr int TW = 8 * NB;                              // tile width in pixels; tile height is 16
    constexpr int NI = (NB >= 2) ? 2 : 1;                   // MMA-issuing warps (2 and 3), each owning NB/NI pixel blocks
    constexpr int NBW = NB / NI;
    constexpr int ASETS = TF32 ? 2 : 1;                     // accumulators per tile buffer (TF32: the last pass uses two)
    constexpr int TWT = PAIR ? 2 * TW : TW;                 // tile width in the tile index space (a pair shares a tile)
    const uint32_t rank = PAIR ? cluster_rank() : 0u;       // 0 = leader
    const int cta_lin = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;   // tiles are dealt to clusters
    const int cta_cnt = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    const int wofs = PAIR ? TW * (int)rank : 0;             // this CTA's pixel columns inside the tile

#ifdef CCV3D_DEV_TRACE
#define TC_STAMP(k) do { if (p.trace && blockIdx.x == 0) p.trace[(k)] = clock64(); } while (0)
#else
#define TC_STAMP(k) do { } while (0)
#endif
    if (threadIdx.x == 0) TC_STAMP(0);
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* ring_a = smem;
    uint8_t* ring_b = ring_a + (size_t)p.SA * p.a_slot;
    uint8_t* epi_buf = ring_b + (size_t)p.SB * p.b_slot;
    uint8_t* ring_raw = epi_buf + (p.epi_tma ? 2 * (size_t)p.e_slot : 0);
    uint8_t* dummy = ring_raw + (FUSED ? 2 * (size_t)p.raw_slot : 0);   // 2 KB sink for the unused rows of edge blocks
    // (COOP: ring_raw holds the stagers' raw slots, p.stg_slots of STAGER_BOXES<NB> * 4 KB, 1024-byte aligned like every ring)
    TcShared* sh = reinterpret_cast<TcShared*>(dummy + (FUSED ? 2048 : 0) + (COOP ? (size_t)p.stg_slots * STAGER_BOXES<NB>::value * 4096 : 0));

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);  // provably warp-uniform
    const int lane = threadIdx.x & 31;
    const int ph = p.general ? p.pad_h : (p.kh - 1) / 2, pw = p.general ? p.pad_w : (p.kw - 1) / 2;
    const int dlh = p.general ? p.dil_h : 1, dlw = p.general ? p.dil_w : 1, dlt = p.general ? p.dil_t : 1;
    const int sth = p.general ? p.str_h : 1, stw = p.general ? p.str_w : 1;      // > 1 only in the per-tap mode
    const int stt = p.general ? p.str_t : 1;                // temporal stride: output frame t reads Z frames t*stt + dt*dlt
    const int BW = p.phased ? TW + p.ph_bw : (p.per_tap_a ? TW : TW + (p.kw - 1) * dlw);        // pixels per smem image row
    const int BH = p.phased ? 16 + p.ph_bh : (p.per_tap_a ? 16 : 16 + (p.kh - 1) * dlh);
    const int spatial = p.kh * p.kw;

    if (threadIdx.x == 0) {
        for (int i = 0; i < p.SA; ++i) { mbar_init(smem_u32(&sh->full_a[i]), FUSED ? 4 : 1); mbar_init(smem_u32(&sh->empty_a[i]), NI); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&sh->raw_full[i]), 1); mbar_init(smem_u32(&sh->raw_empty[i]), 4); }
        if (COOP) for (int i = 0; i < STAGER_MAX_SLOTS; ++i) mbar_init(smem_u32(&sh->stg_full[i]), 1);
        for (int i = 0; i < p.SB; ++i) { mbar_init(smem_u32(&sh->full_b[i]), 1); mbar_init(smem_u32(&sh->empty_b[i]), NI); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&sh->acc_full[i]), NI); mbar_init(smem_u32(&sh->acc_empty[i]), PAIR ? 8 : 4); }
        sh->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (PAIR) cluster_sync_all();   // both CTAs' barriers exist before anything of the peer can arrive on them
    if (warp == 3) {
        if (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)),
                         "r"(p.tmem_cols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)),
                         "r"(p.tmem_cols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;
    if (threadIdx.x == 0) TC_STAMP(1);
    // Programmatic dependent launch: everything above (barriers, tensor memory) touched no global data, so it may
    // run while the previous kernel of the stream is still finishing.  From here on the kernel reads what that
    // kernel wrote: wait for it (returns at once when the launch carried no such dependency), and let the next
    // kernel of the stream start its own set-up as soon as CTAs of this one retire.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 0) TC_STAMP(2);

    // ---------------------------------------------------------------- A producer
    if (warp == 0) {
        if (lane == 0 && FUSED) {
            // raw boxes [32 ch][BH rows][32 px] straight from x or the cache: tap dt of output frame t reads frame
            // t+dt of Z = [cache ; x]; columns start 8 pixels left of the tile so that the start is 16-byte aligned
            asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_a) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_c) : "memory");
            const uint32_t raw_bytes = (uint32_t)KB * BH * RAW_PX * 2;
            int s = 0;
            uint32_t phase = 1;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x) {
                int r = tile / p.NT;
                const int t = r % p.T; r /= p.T;
                const int tx = r % p.tiles_w; r /= p.tiles_w;
                const int ty = p.ty_begin + r % p.tiles_h;
                const int n = r / p.tiles_h;
                const int h0 = ty * 16, w0 = tx * TW;
                const int dt0 = (p.first_frame - t * stt > 0) ? (p.first_frame - t * stt + dlt - 1) / dlt : 0;   // first tap whose frame exists
                for (int dt = dt0; ok && dt < p.kt; ++dt)
                    for (int cb = 0; ok && cb < p.CB; ++cb) {
                        if (!(ok = mbar_wait(&sh->raw_empty[s], phase, sh, p, SITE_RAW_EMPTY))) break;
                        const uint32_t bar = smem_u32(&sh->raw_full[s]);
                        mbar_expect_tx(bar, raw_bytes);
                        const int fz = t + dt;
                        const uint32_t dst = smem_u32(ring_raw + (size_t)s * p.raw_slot);
                        if (fz < p.tc) tma_load_5d(dst, &tm_c, bar, w0 - 8, h0 - ph, fz - (p.tc - p.cf), cb * KB, n);
                        else tma_load_5d(dst, &tm_a, bar, w0 - 8, h0 - ph, fz - p.tc, cb * KB, n);
                        s ^= 1;
                        if (s == 0) phase ^= 1;
                    }
            }
            if (!ok) drain_delay();
        } else if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_a) : "memory");
            const uint32_t a_bytes = (uint32_t)BW * BH * ROWB;
            int s = 0;
            uint32_t phase = 1;
            bool ok = true;
            int bands_ready = COOP ? p.band_first : 0;   // COOP: bands [0, bands_ready) are known to be staged
            for (int item = cta_lin; ok && item < p.total_tiles; item += cta_cnt) {
                const TileView tv = tile_view<TAIL>(p, item);
                int r = tv.tile / tv.NT;
                const int t = r % p.T; r /= p.T;
                const int tx = r % p.tiles_w; r /= p.tiles_w;
                const int ty = p.ty_begin + r % p.tiles_h;
                const int n = r / p.tiles_h;
                const int h0 = ty * 16, w0 = tx * TWT + wofs;
                if (COOP) {
                    // the halo of tile row ty ends at input row 16 ty + 15 + (kh-1) d_h - pad_h (bands ty-1 .. ty+1 of
                    // a size-preserving 3-tap layer); bands are bands of INPUT rows
                    // (stride 2, padding 1: output row h reads input rows 2h - 1 .. 2h + 1)
                    const int last_band = DIL == TAPS_STRIDE2 ? (2 * h0 + 31) >> 4 : (h0 + 15 + (p.kh - 1) * dlh - ph) >> 4;
                    const int need = (last_band + 1 < p.nbands) ? last_band + 1 : p.nbands;
                    if (bands_ready < need) {
                        const long long t0 = clock64();
                        while (ok && bands_ready < need) {
                            unsigned int v;
                            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p.band_ctr + bands_ready) : "memory");
                            if (v >= gridDim.x) { ++bands_ready; continue; }
                            if (sh->abort_flag) ok = false;
                            else if (clock64() - t0 > p.wait_limit_clk) {
                                sh->abort_flag = 1;
                                atomicCAS(p.status, 0u, (blockIdx.x << 8) | SITE_BAND);
                                ok = false;
                            } else __nanosleep(200);
                        }
                        if (!ok) break;
#ifdef CCV3D_DEV_TRACE
                        if (p.trace && blockIdx.x == 0) atomicAdd(p.trace + 16 + SITE_BAND, (unsigned long long)(clock64() - t0));
#endif
                        asm volatile("fence.proxy.async;" ::: "memory");   // other SMs' generic writes -> this SM's TMA reads
                    }
                }
                const int dt0 = (p.first_frame - t * stt > 0) ? (p.first_frame - t * stt + dlt - 1) / dlt : 0;   // first tap whose frame exists
                for (int pass = 0; pass < (TF32 ? 3 : 1); ++pass)
                for (int dt = dt0; ok && dt < p.kt; ++dt)
                    for (int cb = 0; ok && cb < p.CB; ++cb) {
                        int fr = p.f0 + t * stt + dt * dlt;       // ring slot of Z frame t s_t + dt d_t (f0 = 0: the frame itself)
                        if (fr >= p.F) fr -= p.F;
                        const int fz = n * p.F + fr;
                        if ((KS == 0 || DIL == TAPS_STRIDE2) && p.phased) {       // one halo tile per phase image that has taps
                            for (int q = 0; ok && q < p.S2; ++q) {
                                if (p.ph_first[q + 1] == p.ph_first[q]) continue;
                                if (!(ok = mbar_wait(&sh->empty_a[s], phase, sh, p, SITE_A_EMPTY))) break;
                                const uint32_t bar = smem_u32(&sh->full_a[s]);
                                if (PAIR) {                       // (both CTAs' tiles are counted on the leader's barrier)
                                    if (rank == 0) mbar_expect_tx(bar, 2 * a_bytes);
                                    tma_load_5d_pair(smem_u32(ring_a + (size_t)s * p.a_slot), &tm_a, bar, 0, w0 + p.ph_w0[q],
                                                     h0 + p.ph_h0[q], cb * p.S2 + q, fz);
                                } else {
                                    mbar_expect_tx(bar, a_bytes);
                                    tma_load_5d(smem_u32(ring_a + (size_t)s * p.a_slot), &tm_a, bar, 0, w0 + p.ph_w0[q], h0 + p.ph_h0[q],
                                                cb * p.S2 + q, fz);
                                }
                                if (++s == p.SA) { s = 0; phase ^= 1; }
                            }
                            continue;
                        }
                        const int ntap = p.per_tap_a ? spatial : 1;
                        for (int tp = 0; tp < ntap; ++tp) {
                            if (!(ok = mbar_wait(&sh->empty_a[s], phase, sh, p, SITE_A_EMPTY))) break;
                            const uint32_t bar = smem_u32(&sh->full_a[s]);
                            const int dh = p.per_tap_a ? tp / p.kw : 0, dw = p.per_tap_a ? tp % p.kw : 0;
                            if (PAIR) {
                                // both CTAs' boxes are counted on the leader's barrier, which the leader arms for both
                                if (rank == 0) mbar_expect_tx(bar, 2 * a_bytes);
                                tma_load_5d_pair(smem_u32(ring_a + (size_t)s * p.a_slot), &tm_a, bar, 0, w0 - pw, h0 - ph,
                                                 TF32 ? 2 * cb + (pass == 1) : cb, fz);
                                if (item == cta_lin && dt == dt0 && cb == 0) TC_STAMP(3);
                            } else {
                                mbar_expect_tx(bar, a_bytes);
                                tma_load_5d(smem_u32(ring_a + (size_t)s * p.a_slot), &tm_a, bar, 0, w0 * stw - pw + dw * dlw,
                                            h0 * sth - ph + dh * dlh, TF32 ? 2 * cb + (pass == 1) : cb, fz);
                            }
                            if (++s == p.SA) { s = 0; phase ^= 1; }
                        }
                    }
            }
            if (!ok) drain_delay();
        }
    }
    // ---------------------------------------------------------------- B producer
    else if (warp == 1) {
        if (lane == 0) {
            int s = 0;
            uint32_t phase = 1;
            bool ok = true;
            if (PAIR) asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_c) : "memory");
            for (int item = cta_lin; ok && item < p.total_tiles; item += cta_cnt) {
                const TileView tv = tile_view<TAIL>(p, item);
                const int nt = tv.tile % tv.NT;
                const int t = (tv.tile / tv.NT) % p.T;
                const uint32_t b_bytes = tv.b_tap * p.TPB;
                // bytes between taps in the packed weights (half-width tiles: those of the full-width tile)
                const uint32_t src_tap = tv.half ? p.b_tap : (p.b_src_tap ? p.b_src_tap : p.b_tap);
                const int dt0 = (p.first_frame - t * stt > 0) ? (p.first_frame - t * stt + dlt - 1) / dlt : 0;   // first tap whose frame exists
                for (int pass = 0; pass < (TF32 ? 3 : 1); ++pass)
                for (int dt = dt0; ok && dt < p.kt; ++dt)
                    for (int cb = 0; ok && cb < p.CB; ++cb) {
                        if (PAIR) {
                            // this CTA's half (rows rank*NPAD/2 ..) of every tap's weight tile, as boxes of the 2-D map
                            // over the packed weights; both CTAs' boxes are counted on the leader's barrier
                            // (split_n: NT and NPAD describe half-width tiles of a layer packed at full width; the rows of
                            // a tap's full-width tile are then [half 0 | half 1], each again split between the two CTAs)
                            const int npw = tv.NPAD << tv.split;                      // rows of a packed (full-width) tile
                            const int row0 = ((((pass * p.kt + dt) * p.CB + cb) * (tv.NT >> tv.split) + (nt >> tv.split)) * spatial) * npw +
                                             (nt & tv.split) * tv.NPAD + (int)rank * (tv.NPAD >> 1);
                            for (int tp = 0; tp < spatial; tp += p.TPB) {
                                if (!(ok = mbar_wait(&sh->empty_b[s], phase, sh, p, SITE_B_EMPTY))) break;
                                const uint32_t bar = smem_u32(&sh->full_b[s]);
                                if (rank == 0) mbar_expect_tx(bar, 2 * b_bytes);
                                const uint32_t dst = smem_u32(ring_b + (size_t)s * p.b_slot);
                                // (a launch with half-width items carries the weight map of those: its box is a quarter of
                                // a full tile's rows, and a CTA's half of a full-width tile arrives as two boxes)
                                const int parts = (TAIL && p.main_tiles > 0 && !tv.half) ? 2 : 1;
                                for (int u = 0; u < p.TPB; ++u)
                                    for (int q = 0; q < parts; ++q)
                                        // (the map's rows are 512 bytes = 256 / KB rows of the packed image; every offset here is a
                                        // multiple of eight image rows)
                                        tma_load_2d_pair(dst + u * tv.b_tap + q * (tv.b_tap >> 1), &tm_c, bar, 0,
                                                         (row0 + (DIL == TAPS_STRIDE2 ? (int)p.ph_tap[tp + u] : tp + u) * npw + q * (tv.NPAD >> 2)) / (256 / KB));   // (stride 2: taps in phase order)
                                if (++s == p.SB) { s = 0; phase ^= 1; }
                            }
                            continue;
                        }
                        // split_n: this launch runs half-width output-channel tiles; the packed image of a full tile
                        // holds its two halves back to back (the swizzle repeats every 8 rows), so a half tile of a
                        // tap is a contiguous piece of it and only the distance between taps differs
                        const uint8_t* src = p.wq + (size_t)(((pass * p.kt + dt) * p.CB + cb) * (tv.NT >> tv.split) + (nt >> tv.split)) * spatial * src_tap +
                                             (size_t)(nt & tv.split) * tv.b_tap;
                        for (int tp = 0; tp < spatial; tp += p.TPB) {
                            if (!(ok = mbar_wait(&sh->empty_b[s], phase, sh, p, SITE_B_EMPTY))) break;
                            const uint32_t bar = smem_u32(&sh->full_b[s]);
                            mbar_expect_tx(bar, b_bytes);
                            const uint32_t dst = smem_u32(ring_b + (size_t)s * p.b_slot);
                            if (KS == 0 && p.phased) bulk_load(dst, src + (size_t)p.ph_tap[tp] * src_tap, b_bytes, bar);   // taps in phase order (TPB = 1)
                            else
                            if (src_tap == tv.b_tap) bulk_load(dst, src + (size_t)tp * src_tap, b_bytes, bar);
                            else
                                for (int u = 0; u < p.TPB; ++u) bulk_load(dst + u * tv.b_tap, src + (size_t)(tp + u) * src_tap, tv.b_tap, bar);
                            if (++s == p.SB) { s = 0; phase ^= 1; }
                        }
                    }
            }
            if (!ok) drain_delay();
        }
    }
    // ---------------------------------------------------------------- MMA issuers
    // Warp 2 (and warp 3 when NB >= 2) issues the MMAs of its own pixel blocks.  A commit
    // only tracks the MMAs of the committing thread, so the "slot free" and "accumulator full" barriers
    // count one arrival per issuer.
    else if ((warp == 2 || (warp == 3 && NI == 2)) && rank == 0) {     // (of a CTA pair only the leader issues MMAs)
        // The whole warp runs the loop (warp-uniform control flow); one elected lane issues.
        const int iss = warp - 2;
        // instruction descriptor: D=F32, A=B=BF16, both K-major, N = NPAD, M = 128
        // (operand formats: 1 = BF16, 2 = TF32)
        constexpr uint32_t FMT = TF32 ? 2u : 1u;
        const uint32_t idesc_full = (1u << 4) | (FMT << 7) | (FMT << 10) | ((uint32_t)(p.NPAD >> 3) << 17) | (((PAIR ? 256u : 128u) >> 4) << 24);
        const uint32_t idesc_half = (1u << 4) | (FMT << 7) | (FMT << 10) | ((uint32_t)(p.NPAD >> 4) << 17) | (((PAIR ? 256u : 128u) >> 4) << 24);
        const uint32_t idesc = idesc_full;                // (the run-time tap loop below never sees half-width items)
        const uint32_t a_hi = make_desc_hi((uint32_t)BW * ROWB, LAYOUT);  // 8-pixel groups are one image row apart
        const uint32_t b_hi = make_desc_hi(B_SBO, LAYOUT);
        const uint32_t a_blk = (uint32_t)(iss * NBW) * ((8 * ROWB) >> 4);  // descriptor offset of this issuer's first block
        const uint32_t a_rowstep = ((uint32_t)(BW * dlh) * ROWB) >> 4;   // descriptor step between kernel rows
        const uint32_t b_tapstep = p.b_tap >> 4;
        int sa = 0, sb = 0, acc = 0;
        uint32_t pa = 0, pb = 0, pacc = 1;
        bool ok = true;
        if constexpr (KS > 0) {
            constexpr bool STR2 = DIL == TAPS_STRIDE2;
            // one kernel row down the halo tile (stride 2: one row down a phase's tile of 8 NB + 1 pixels per row)
            constexpr uint32_t A_ROWSTEP = STR2 ? ((uint32_t)(TW + 1) * ROWB) >> 4 : ((uint32_t)(TW + (KS - 1) * DIL) * DIL * ROWB) >> 4;
            constexpr int STAGES = KS * KS / TPBC;
            uint32_t a_ring = make_desc_lo(smem_u32(ring_a)) + a_blk, b_ring = make_desc_lo(smem_u32(ring_b));
            const uint32_t a_slotstep = p.a_slot >> 4, b_slotstep = p.b_slot >> 4;
            const uint32_t a_ring0 = a_ring, b_ring0 = b_ring;
            for (int item = cta_lin; ok && item < p.total_tiles; item += cta_cnt) {
                const TileView tv = tile_view<TAIL>(p, item);
                const int t = (tv.tile / tv.NT) % p.T;
                // N of the instruction and the tap distance in a weight slot follow the tile's width; the accumulators
                // keep the launch's column layout
                const uint32_t idesc = tv.half ? idesc_half : idesc_full;
                const uint32_t b_tapstep = tv.b_tap >> 4;
                const int dt0 = (p.first_frame - t * stt > 0) ? (p.first_frame - t * stt + dlt - 1) / dlt : 0;   // first tap whose frame exists
                if (!(ok = mbar_wait(&sh->acc_empty[acc], pacc, sh, p, SITE_ACC_EMPTY))) break;
                tc_fence_after();
                const uint32_t d_first = tmem_base + (uint32_t)(acc * ASETS * NB + iss * NBW) * p.NPAD;
                uint32_t accumulate = 0, accumulate2 = 0;
                const int nst = (p.kt - dt0) * p.CB;                          // (dt, ci-block) stages per pass
                for (int st = 0; ok && st < (TF32 ? 3 : 1) * nst; ++st) {     // (pass, dt, ci-block) stages
                    // TF32: the stages of the last (full-size) pass alternate between two accumulators, which halves
                    // the length of either truncating chain; the epilogue adds the two
                    const bool second = TF32 && st >= 2 * nst && ((st - 2 * nst) & 1);
                    const uint32_t d0 = d_first + (second ? (uint32_t)NB * p.NPAD : 0u);
                    const uint32_t acc_in = second ? accumulate2 : accumulate;
                    // Stride 2: position i of the phase order (taps 4 | 3 5 | 1 7 | 0 2 6 8 of the 3x3 kernel) reads phase
                    // str2_q(i)'s tile, which sits in activation slot (sa + str2_q(i)) mod SA (SA >= 4: a fifth slot already lets
                    // the producer request the four-tap phase's next tile ten taps ahead instead of five),
                    // at row offset (i == 4 || i >= 7) and pixel offset (i == 2 || i == 6 || i == 8).
                    auto str2_q = [](int i) { return i == 0 ? 0 : i < 3 ? 1 : i < 5 ? 2 : 3; };
                    int qs[4];                                     // slot of each phase's tile
                    uint32_t qp[4];                                // ... and the parity to wait for
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const bool wrap = STR2 && sa + q >= p.SA;
                        qs[q] = wrap ? sa + q - p.SA : sa + q;
                        qp[q] = wrap ? pa ^ 1u : pa;
                    }
                    if (!STR2 && !(ok = mbar_wait(&sh->full_a[sa], pa, sh, p, SITE_A_FULL))) break;
                    if (item == cta_lin && st == 0 && lane == 0 && iss == 0) TC_STAMP(4);
#pragma unroll
                    for (int g = 0; g < STAGES; ++g) {
                        if (STR2) {
#pragma unroll
                            for (int u = 0; u < TPBC; ++u) {
                                const int i = g * TPBC + u;
                                if (i == 0 || i == 1 || i == 3 || i == 5)      // a phase's first tap
                                    ok = ok && mbar_wait(&sh->full_a[qs[str2_q(i)]], qp[str2_q(i)], sh, p, SITE_A_FULL);
                            }
                            if (!ok) break;
                        }
                        if (!(ok = mbar_wait(&sh->full_b[sb], pb, sh, p, SITE_B_FULL))) break;
                        if (item == cta_lin && st == 0 && g == 0 && lane == 0 && iss == 0) TC_STAMP(5);
                        tc_fence_after();
                        if (elect_one()) {
#pragma unroll
                            for (int u = 0; u < TPBC; ++u) {
                                const int tap = g * TPBC + u;
                                // tap (dh, dw) = a descriptor offset into the one halo tile.  The start address is only
                                // 16-byte granular and need not sit on the swizzle period: the swizzle is a function of
                                // the absolute shared-memory address (as the TMA unit applied it), so the descriptor's
                                // base-offset field stays 0.
                                const uint32_t a_lo = STR2 ? a_ring0 + (uint32_t)qs[str2_q(tap)] * a_slotstep +
                                                                 (uint32_t)(tap == 4 || tap >= 7) * A_ROWSTEP +
                                                                 (uint32_t)(tap == 2 || tap == 6 || tap == 8) * (ROWB >> 4)
                                                           : a_ring + (uint32_t)(tap / KS) * A_ROWSTEP + (uint32_t)(tap % KS) * DIL * (ROWB >> 4);
                                const uint32_t b_lo = b_ring + (uint32_t)u * b_tapstep;
#pragma unroll
                                for (int j = 0; j < NBW; ++j) {
#pragma unroll
                                    for (int k = 0; k < KSTEPS; ++k)
                                        if (PAIR && TF32)
                                            tc_mma_tf32_pair(d0 + j * p.NPAD, a_lo + j * ((8 * ROWB) >> 4) + 2 * k, a_hi, b_lo + 2 * k, b_hi,
                                                             idesc, (tap == 0 && k == 0) ? acc_in : 1u);
                                        else if (PAIR)
                                            tc_mma_bf16_pair(d0 + j * p.NPAD, a_lo + j * ((8 * ROWB) >> 4) + 2 * k, a_hi, b_lo + 2 * k, b_hi,
                                                             idesc, (tap == 0 && k == 0) ? acc_in : 1u);
                                        else
                                            tc_mma<TF32>(d0 + j * p.NPAD, a_lo + j * ((8 * ROWB) >> 4) + 2 * k, a_hi, b_lo + 2 * k, b_hi,
                                                         idesc, (tap == 0 && k == 0) ? acc_in : 1u);
                                }
                                // (stride 2: a phase's slot is free after its last tap; the commit covers everything issued so far)
                                if (STR2 && (tap == 0 || tap == 2 || tap == 4)) tc_commit_pair(smem_u32(&sh->empty_a[qs[str2_q(tap)]]));
                            }
                            if (PAIR) tc_commit_pair(smem_u32(&sh->empty_b[sb])); else tc_commit(smem_u32(&sh->empty_b[sb]));
                        }
                        __syncwarp();
                        b_ring += b_slotstep;
                        if (++sb == p.SB) { sb = 0; pb ^= 1; b_ring = b_ring0; }
                    }
                    if (!ok) break;
                    if (second) accumulate2 = 1; else accumulate = 1;
                    if (elect_one()) { if (PAIR) tc_commit_pair(smem_u32(&sh->empty_a[STR2 ? qs[3] : sa])); else tc_commit(smem_u32(&sh->empty_a[sa])); }
                    __syncwarp();
                    if (STR2) {
                        sa += 4;
                        if (sa >= p.SA) { sa -= p.SA; pa ^= 1; }
                    } else {
                        a_ring += a_slotstep;
                        if (++sa == p.SA) { sa = 0; pa ^= 1; a_ring = a_ring0; }
                    }
                }
                if (!ok) break;
                if (elect_one()) { if (PAIR) tc_commit_pair(smem_u32(&sh->acc_full[acc])); else tc_commit(smem_u32(&sh->acc_full[acc])); }
                __syncwarp();
                if (item == cta_lin && lane == 0 && iss == 0) TC_STAMP(6);
                if (++acc == p.ACC) { acc = 0; pacc ^= 1; }
            }
        } else
        for (int tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x) {
            const int t = (tile / p.NT) % p.T;
            const int dt0 = (p.first_frame - t * stt > 0) ? (p.first_frame - t * stt + dlt - 1) / dlt : 0;   // first tap whose frame exists
            if (!(ok = mbar_wait(&sh->acc_empty[acc], pacc, sh, p, SITE_ACC_EMPTY))) break;
            tc_fence_after();
            const uint32_t d_first = tmem_base + (uint32_t)(acc * ASETS * NB + iss * NBW) * p.NPAD;
            uint32_t accumulate1 = 0, accumulate2 = 0;
            int st2 = 0;                                       // stage counter of the last pass
            for (int pass = 0; pass < (TF32 ? 3 : 1); ++pass)
            for (int dt = dt0; ok && dt < p.kt; ++dt)
                for (int cb = 0; ok && cb < p.CB; ++cb) {
                    const bool second = TF32 && pass == 2 && (st2++ & 1);   // see the straight-line variant
                    const uint32_t d0 = d_first + (second ? (uint32_t)NB * p.NPAD : 0u);
                    uint32_t accumulate = second ? accumulate2 : accumulate1;
                    if (p.phased) {
                        // phase images: one halo tile per phase, its taps are (row, column) offsets into it
                        const uint32_t row1 = ((uint32_t)BW * ROWB) >> 4;
                        for (int q = 0; ok && q < p.S2; ++q) {
                            const int i0 = p.ph_first[q], i1 = p.ph_first[q + 1];
                            if (i0 == i1) continue;
                            if (!(ok = mbar_wait(&sh->full_a[sa], pa, sh, p, SITE_A_FULL))) break;
                            const uint32_t a_base = make_desc_lo(smem_u32(ring_a + (size_t)sa * p.a_slot)) + a_blk;
                            for (int i = i0; i < i1; ++i) {
                                if (!(ok = mbar_wait(&sh->full_b[sb], pb, sh, p, SITE_B_FULL))) break;
                                tc_fence_after();
                                const uint32_t b_lo = make_desc_lo(smem_u32(ring_b + (size_t)sb * p.b_slot));
                                const uint32_t a_lo = a_base + (uint32_t)p.ph_roff[i] * row1 + (uint32_t)p.ph_coff[i] * (ROWB >> 4);
                                if (elect_one()) {
#pragma unroll
                                    for (int j = 0; j < NBW; ++j) {
#pragma unroll
                                        for (int k = 0; k < KSTEPS; ++k)
                                            tc_mma<TF32>(d0 + j * p.NPAD, a_lo + j * ((8 * ROWB) >> 4) + 2 * k, a_hi, b_lo + 2 * k, b_hi,
                                                        idesc, (k == 0) ? accumulate : 1u);
                                    }
                                    tc_commit(smem_u32(&sh->empty_b[sb]));
                                }
                                __syncwarp();
                                accumulate = 1;
                                if (++sb == p.SB) { sb = 0; pb ^= 1; }
                            }
                            if (!ok) break;
                            if (elect_one()) tc_commit(smem_u32(&sh->empty_a[sa]));
                            __syncwarp();
                            if (++sa == p.SA) { sa = 0; pa ^= 1; }
                        }
                        if (second) accumulate2 = accumulate; else accumulate1 = accumulate;
                        continue;
                    }
                    uint32_t a_row = 0;  // descriptor low word of the halo row of the current tap row
                    if (!p.per_tap_a) {
                        if (!(ok = mbar_wait(&sh->full_a[sa], pa, sh, p, SITE_A_FULL))) break;
                        a_row = make_desc_lo(smem_u32(ring_a + (size_t)sa * p.a_slot)) + a_blk;
                    }
                    for (int tp = 0, dw = 0; tp < spatial; tp += p.TPB) {
                        if (!(ok = mbar_wait(&sh->full_b[sb], pb, sh, p, SITE_B_FULL))) break;
                        tc_fence_after();
                        uint32_t b_lo = make_desc_lo(smem_u32(ring_b + (size_t)sb * p.b_slot));
                        for (int u = 0; u < p.TPB; ++u) {
                            uint32_t a_lo;
                            if (p.per_tap_a) {
                                if (!(ok = mbar_wait(&sh->full_a[sa], pa, sh, p, SITE_A_FULL))) break;
                                tc_fence_after();
                                a_lo = make_desc_lo(smem_u32(ring_a + (size_t)sa * p.a_slot)) + a_blk;
                            } else {
                                // The start address is only 16-byte granular and need not sit on the swizzle
                                // period: the swizzle is a function of the absolute shared-memory address (as
                                // the TMA unit applied it), so the descriptor's base-offset field stays 0.
                                a_lo = a_row + (uint32_t)(dw * dlw) * (ROWB >> 4);
                            }
                            if (elect_one()) {
#pragma unroll
                                for (int j = 0; j < NBW; ++j) {
#pragma unroll
                                    for (int k = 0; k < KSTEPS; ++k)
                                        tc_mma<TF32>(d0 + j * p.NPAD, a_lo + j * ((8 * ROWB) >> 4) + 2 * k, a_hi, b_lo + 2 * k, b_hi,
                                                    idesc, (k == 0) ? accumulate : 1u);
                                }
                                if (p.per_tap_a) tc_commit(smem_u32(&sh->empty_a[sa]));
                            }
                            __syncwarp();
                            accumulate = 1;
                            b_lo += b_tapstep;
                            if (p.per_tap_a) {
                                if (++sa == p.SA) { sa = 0; pa ^= 1; }
                            }
                            if (++dw == p.kw) { dw = 0; a_row += a_rowstep; }
                        }
                        if (!ok) break;
                        if (elect_one()) tc_commit(smem_u32(&sh->empty_b[sb]));
                        __syncwarp();
                        if (++sb == p.SB) { sb = 0; pb ^= 1; }
                    }
                    if (ok && !p.per_tap_a) {
                        if (elect_one()) tc_commit(smem_u32(&sh->empty_a[sa]));
                        __syncwarp();
                        if (++sa == p.SA) { sa = 0; pa ^= 1; }
                    }
                    if (second) accumulate2 = accumulate; else accumulate1 = accumulate;
                }
            if (!ok) break;
            if (elect_one()) tc_commit(smem_u32(&sh->acc_full[acc]));
            __syncwarp();
            if (++acc == p.ACC) { acc = 0; pacc ^= 1; }
        }
    }
    // ---------------------------------------------------------------- epilogue (warps 4..7)
    else if (warp >= 4 && warp < 8) {
        const int q = warp & 3;  // TMEM lane quarter this warp may read
        int acc = 0;
        uint32_t pacc = 0;
        bool ok = true;
        const int64_t HW = (int64_t)p.H * p.W;
        const int m = q * 32 + lane;  // accumulator row = pixel m of a 128-pixel block: image row m/8, pixel m%8
        const bool elected = (threadIdx.x == 4 * 32);
        constexpr bool RING = !FUSED && !COOP;                 // frame-ring output and residual: plain variant only
        const bool has_res = RING && p.res != nullptr;
        int ebuf = 0;
        // bias: a shared-memory copy when the padded channel count fits.  A global load per element costs little
        // while the next tile's MMAs run, but its latency sits in the exposed tail of a CTA's last tile: 11 us
        // against 5 us for a 192-channel tile.
        const bool bias_smem = p.NT * p.NPAD <= TC_BIAS_SMEM;
        if (bias_smem)
            for (int i = threadIdx.x - 128; i < p.NT * p.NPAD; i += 128) sh->bias_s[i] = __ldg(p.bias + i);
        epi_bar_sync();
        const float* bias = bias_smem ? sh->bias_s : p.bias;
        // the tile loop exists twice, with and without the optional SiLU, so that the plain epilogue carries no trace of it
        auto run_tiles = [&](auto act_c) {
            constexpr bool ACT = decltype(act_c)::value;
            for (int item = cta_lin; ok && item < p.total_tiles; item += cta_cnt) {
                const TileView tv = tile_view<TAIL>(p, item);
                const int nt = tv.tile % tv.NT;
                int r = tv.tile / tv.NT;
                const int t = r % p.T; r /= p.T;
                const int tx = r % p.tiles_w; r /= p.tiles_w;
                const int ty = p.ty_begin + r % p.tiles_h;
                const int n = r / p.tiles_h;
                const int h = ty * 16 + (m >> 3);
                const int wt = tx * TWT + wofs;                  // first pixel column of this CTA's part of the tile
                // residual: pixel (h, w) of frame t holds its Cout channels in blocks of res_KB (64 bytes per 32 channels)
                const __nv_bfloat16* res_row = nullptr;
                if (has_res && h < p.H) {
                    int rs = p.res_f0 + t;
                    if (rs >= p.res_F) rs -= p.res_F;
                    res_row = p.res + (((int64_t)n * p.res_F + rs) * p.res_CB * HW + (int64_t)h * p.W) * p.res_KB;
                }
                // the residual of the first chunk is fetched while the MMAs of this tile still run; every later chunk's
                // residual is fetched one chunk ahead
                uint32_t rr_next[16];
                if (p.epi_tma) load_res32(res_row, wt + (m & 7) < p.W, wt + (m & 7), nt * tv.NPAD, p, HW, rr_next);
                ok = mbar_wait(&sh->acc_full[acc], pacc, sh, p, SITE_ACC_FULL);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (item == cta_lin && elected) TC_STAMP(7);
                tc_fence_after();
                const uint32_t t_acc = tmem_base + (uint32_t)(acc * ASETS * NB) * p.NPAD + ((uint32_t)(q * 32) << 16);
                // TF32: was the second accumulator of the last pass used (at least two stages per pass)?
                const int dt0e = (p.first_frame - t * stt > 0) ? (p.first_frame - t * stt + dlt - 1) / dlt : 0;
                const bool two_acc = TF32 && (p.kt - dt0e) * p.CB >= 2;
                if (p.epi_tma) {
                    // BF16 tile chunks -> shared memory -> one TMA store per chunk.  NCTHW output: [ECH channels][16 rows]
                    // [TW pixels]; ring output: [16 rows][TW pixels][32 channels] with the 64-byte swizzle of the tensor map.
                    for (int c0 = 0; c0 < tv.NPAD; c0 += p.ECH) {
                        if (elected) bulk_wait_read<1>();   // the store that last read this buffer has finished reading
                        epi_bar_sync();
                        uint8_t* stg = epi_buf + (size_t)ebuf * p.e_slot;
                        const int co0 = nt * tv.NPAD + c0;
    #pragma unroll
                        for (int blk = 0; blk < NB; ++blk) {
                            uint32_t rr[16];
    #pragma unroll
                            for (int j = 0; j < 16; ++j) rr[j] = rr_next[j];
                            if (has_res) {
                                const int wn = wt + ((blk + 1 < NB) ? blk + 1 : 0) * 8 + (m & 7);
                                const int con = (blk + 1 < NB) ? co0 : co0 + p.ECH;
                                load_res32(res_row, wn < p.W && con < (nt + 1) * tv.NPAD, wn, con, p, HW, rr_next);
                            }
                            uint32_t v[32];
                            if (p.ECH == 32) tc_ld32(t_acc + blk * p.NPAD + c0, v); else tc_ld16(t_acc + blk * p.NPAD + c0, v);
                            tc_wait_ld();
                            uint32_t pk[16];
                            float bb[32];                       // the chunk's bias: eight 16-byte reads (co0 is a multiple of 16)
    #pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const float4 b4 = (4 * j < p.ECH) ? *reinterpret_cast<const float4*>(bias + co0 + 4 * j)
                                                                  : make_float4(0.f, 0.f, 0.f, 0.f);
                                bb[4 * j] = b4.x; bb[4 * j + 1] = b4.y; bb[4 * j + 2] = b4.z; bb[4 * j + 3] = b4.w;
                            }
    #pragma unroll
                            for (int j = 0; j < 32; ++j) bb[j] += __uint_as_float(v[j]);
                            if (ACT) {      // optional SiLU on conv + bias, in FP32, before the one rounding: one uniform branch per chunk
    #pragma unroll
                                for (int j = 0; j < 32; ++j) bb[j] = silu_f32(bb[j]);
                            }
    #pragma unroll
                            for (int j = 0; j < 16; ++j)
                                pk[j] = (2 * j < p.ECH) ? epi_pair(bb[2 * j], bb[2 * j + 1], rr[j], has_res) : 0u;
                            const uint32_t px = (uint32_t)((m >> 3) * TW + blk * 8 + (m & 7));   // pixel of the tile, row-major
                            if (RING && p.epi_tma == 2) {
                                uint4* row = reinterpret_cast<uint4*>(stg + (size_t)px * 64);
                                const uint32_t sw = (px >> 1) & 3u;
    #pragma unroll
                                for (int c = 0; c < 4; ++c)
                                    row[c ^ sw] = make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
                            } else {
                                unsigned short* dst = reinterpret_cast<unsigned short*>(stg) + px;
    #pragma unroll
                                for (int j = 0; j < 16; ++j)
                                    if (2 * j < p.ECH) {
                                        dst[(2 * j) * 16 * TW] = (unsigned short)(pk[j] & 0xFFFFu);
                                        dst[(2 * j + 1) * 16 * TW] = (unsigned short)(pk[j] >> 16);
                                    }
                            }
                        }
                        fence_async_smem();
                        epi_bar_sync();
                        if (elected) {
                            if (RING && p.epi_tma == 2 && p.up_rt > 0) {
                                // fused nearest-neighbour upsample: the tensor map walks the 2H x 2W ring with a traversal
                                // stride of 2 pixels, so one store drops the tile onto every second pixel from (b, a)
                                for (int j = 0; j < p.up_rt; ++j) {
                                    const int os = (p.out_f0 + t * p.up_rt + j) % p.out_F;
                                    for (int ab = 0; ab < 4; ++ab)
                                        tma_store_5d(&tm_o, smem_u32(stg), co0 % p.out_KB, 2 * wt + (ab & 1), 2 * ty * 16 + (ab >> 1),
                                                     co0 / p.out_KB, n * p.out_F + os);
                                }
                            } else if (RING && p.epi_tma == 2) {
                                int os = p.out_f0 + t;
                                if (os >= p.out_F) os -= p.out_F;
                                tma_store_5d(&tm_o, smem_u32(stg), co0 % p.out_KB, wt, ty * 16, co0 / p.out_KB, n * p.out_F + os);
                            } else {
                                tma_store_5d(&tm_o, smem_u32(stg), wt, ty * 16, t, co0, n);
                            }
                            bulk_commit();
                        }
                        ebuf ^= 1;
                    }
                } else {
    #pragma unroll 1
                    for (int blk = 0; blk < NB; ++blk) {
                        const int w = wt + blk * 8 + (m & 7);
                        const bool valid = h < p.H && w < p.W;
                        const int64_t pix = (int64_t)t * HW + (int64_t)h * p.W + w;
    #pragma unroll 1
                        for (int c0 = 0; c0 < tv.NPAD; c0 += 32) {
                            const int co0 = nt * tv.NPAD + c0;
                            uint32_t rr[16];
                            load_res32(res_row, valid, w, co0, p, HW, rr);
                            uint32_t v[32];
                            const int nc = (tv.NPAD - c0 >= 32) ? 32 : 16;
                            if (nc == 32) tc_ld32(t_acc + blk * p.NPAD + c0, v); else tc_ld16(t_acc + blk * p.NPAD + c0, v);
                            tc_wait_ld();
                            if (two_acc) {
                                uint32_t v2[32];
                                if (nc == 32) tc_ld32(t_acc + (NB + blk) * p.NPAD + c0, v2); else tc_ld16(t_acc + (NB + blk) * p.NPAD + c0, v2);
                                tc_wait_ld();
    #pragma unroll
                                for (int j = 0; j < 32; ++j)
                                    if (j < nc) v[j] = __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(v2[j]));
                            }
                            if (valid) {
                                float a[32];
    #pragma unroll
                                for (int j = 0; j < 32; ++j) a[j] = (j < nc) ? __uint_as_float(v[j]) + bias[co0 + j] : 0.f;
                                if (ACT) {      // optional SiLU on conv + bias: one uniform branch per chunk
    #pragma unroll
                                    for (int j = 0; j < 32; ++j) a[j] = silu_f32(a[j]);
                                }
                                if (p.out_f32) {
    #pragma unroll
                                    for (int j = 0; j < 32; ++j) {
                                        const int co = co0 + j;
                                        if (j < nc && co < p.Cout)
                                            reinterpret_cast<float*>(p.out)[((int64_t)n * p.Cout + co) * p.T * HW + pix] = a[j];
                                    }
                                } else {
    #pragma unroll
                                    for (int j = 0; j < 16; ++j) {
                                        const int co = co0 + 2 * j;
                                        if (2 * j < nc) {
                                            const uint32_t pr = epi_pair(a[2 * j], a[2 * j + 1], rr[j], has_res);
                                            unsigned short* o = reinterpret_cast<unsigned short*>(p.out) +
                                                                ((int64_t)n * p.Cout + co) * p.T * HW + pix;
                                            if (co < p.Cout) o[0] = (unsigned short)(pr & 0xFFFFu);
                                            if (co + 1 < p.Cout) o[(int64_t)p.T * HW] = (unsigned short)(pr >> 16);
                                        }
                                    }
                                }
                            }
                        }
                    }
                }
                if (item == cta_lin && elected) TC_STAMP(8);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) { if (PAIR) mbar_arrive_leader(smem_u32(&sh->acc_empty[acc])); else mbar_arrive(smem_u32(&sh->acc_empty[acc])); }
                if (++acc == p.ACC) { acc = 0; pacc ^= 1; }
            }
        };
        if (p.act) run_tiles(std::true_type{}); else run_tiles(std::false_type{});
        // Before the CTA exits the stores must have finished READING its shared memory; their writes complete with
        // the grid (which is what a dependent kernel waits for), so nothing here waits for them (0.8 us per launch).
        if (p.epi_tma && elected) bulk_wait_read<0>();
        if (elected) TC_STAMP(9);
    }

    // ---------------------------------------------------------------- stagers (cooperative staging, warps 8..11)
    if (COOP && warp >= 8) run_stagers<KB, STAGER_BOXES<NB>::value, DIL == TAPS_STRIDE2>(p, sp, &smaps, smem_u32(ring_raw), sh);

    // ---------------------------------------------------------------- transposers (fused mode, warps 8..11)
    if (FUSED && warp >= 8) {
        // raw [c][row][32 px] (64-byte rows, 64-byte swizzle as TMA wrote it) -> halo tile [pixel][32 ch] (64-byte
        // rows, 64-byte swizzle: the K-major operand).  Per step a warp moves 8 pixels x 32 channels: ldmatrix.trans
        // reads four 8x8 blocks (one per channel octet, rows = channels), stmatrix writes them with rows = pixels.
        const int tw = warp - 8;
        const int colshift = 8 - pw;                       // raw column of halo column 0
        const int mi = lane >> 3, mj = lane & 7;           // this lane addresses row mj of matrix (channel octet) mi
        const uint32_t src_lane = (uint32_t)(mi * 8 + mj) * (uint32_t)(BH * RAW_PX * 2);
        const uint32_t dummy_addr = smem_u32(dummy) + (uint32_t)(tw * 32 + lane) * 16;
        int rs = 0, sa = 0;
        uint32_t pr = 0, pea = 1;
        bool ok = true;
        for (int tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x) {
            const int t = (tile / p.NT) % p.T;
            const int dt0 = (p.first_frame - t * stt > 0) ? (p.first_frame - t * stt + dlt - 1) / dlt : 0;   // first tap whose frame exists
            for (int kb = (p.kt - dt0) * p.CB; ok && kb > 0; --kb) {
                ok = mbar_wait(&sh->raw_full[rs], pr, sh, p, SITE_RAW_FULL) && mbar_wait(&sh->empty_a[sa], pea, sh, p, SITE_A_EMPTY);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const uint32_t raw_base = smem_u32(ring_raw + (size_t)rs * p.raw_slot);
                const uint32_t a_base = smem_u32(ring_a + (size_t)sa * p.a_slot);
                // warp tw owns column block tw of every halo row; rows go in batches of TR so that the loads of a
                // batch are in flight together before its stores
                constexpr int TR = 6;
                const int col = 8 * tw + mj - colshift;
                const bool col_ok = col >= 0 && col < BW;
                uint32_t so0 = src_lane + (uint32_t)tw * 16;
                for (int hb = 0; hb < BH; hb += TR) {
                    uint32_t frag[TR][4];
#pragma unroll
                    for (int u = 0; u < TR; ++u) {
                        if (hb + u < BH) {
                            uint32_t so = so0 + (uint32_t)(hb + u) * (RAW_PX * 2);
                            so ^= ((so >> 7) & 3u) << 4;             // the 64-byte swizzle TMA applied to the raw box
                            ldmatrix_x4_trans(raw_base + so, frag[u]);
                        }
                    }
#pragma unroll
                    for (int u = 0; u < TR; ++u) {
                        if (hb + u < BH) {
                            const uint32_t r = (uint32_t)((hb + u) * BW + col);
                            const uint32_t dst = col_ok ? a_base + r * 64 + (((uint32_t)mi ^ ((r >> 1) & 3u)) << 4) : dummy_addr;
                            stmatrix_x4(dst, frag[u]);
                        }
                    }
                }
                fence_async_smem();                        // generic-proxy writes -> visible to the tensor core's reads
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(smem_u32(&sh->full_a[sa]));
                    mbar_arrive(smem_u32(&sh->raw_empty[rs]));
                }
                rs ^= 1;
                if (rs == 0) pr ^= 1;
                if (++sa == p.SA) { sa = 0; pea ^= 1; }
            }
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) TC_STAMP(10);
    if (PAIR) cluster_sync_all();   // the leader's MMAs read the peer's shared memory and write its tensor memory
    if (threadIdx.x == 0) TC_STAMP(11);
    if (warp == 3) {
        tc_fence_after();
        if (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
        else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
    }
}

// ------------------------------------------------------------------------------------------------
// Self-test of the bounded-wait path: one CTA waits on an mbarrier phase that nothing ever completes.
// The wait gives up after limit_clk clocks, records (block << 8) | site in the status word and the kernel
// returns normally - the same code path a lost TMA completion would take in the convolution kernels.
// ------------------------------------------------------------------------------------------------
__global__ void wait_timeout_selftest_kernel(unsigned int* status, long long limit_clk) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t b = smem_u32(&bar);
        const long long t0 = clock64();
        for (uint32_t it = 1;; ++it) {
            if (mbar_try_wait(b, 0)) break;                       // phase 0 never completes: nobody arrives
            if ((it & 63u) == 0u && clock64() - t0 > limit_clk) {
                atomicCAS(status, 0u, (blockIdx.x << 8) | 0x7Fu);  // site 0x7F: the self-test
                break;
            }
        }
    }
    __syncthreads();
}

}  // namespace ccv3d
