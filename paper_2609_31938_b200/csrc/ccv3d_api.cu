// C-ABI of the cached causal Conv3D library: validation (Algorithm 1's
// "validate and prepare" step turned into error codes - there is no fallback
// route), handle life cycle, route selection, launches, counters.
#include "../../include/ccv3d.h"

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "ccv3d_simt.cuh"
#include "ccv3d_tc.cuh"

using namespace ccv3d;

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr int PROF_SLOTS = 1024;
constexpr int MAX_BANDS = 4;
constexpr int MAX_COOP_BANDS = 4096;     // image rows / 16 that cooperative staging can track
constexpr size_t STAGE_COEXIST_BYTES = 20480;  // shared memory left free for staging blocks next to a convolution CTA
constexpr size_t SMEM_LIMIT = 232448;  // 227 KB of dynamic shared memory per CTA on sm_100

struct TcPlan {      // per-layer choices of the tensor-core route
    int KB, CB, cin_pad;
    int NT, NPAD, cout_pad;
    int NB, ACC;
    bool fused;      // CCV3D_FLAG_FUSED: no staging copy when the call's W allows TMA rows (W % 8 == 0)
};

struct ShapeKey {
    const void* zs;
    int N, T, H, W, BW;
    bool operator==(const ShapeKey& o) const {
        return zs == o.zs && N == o.N && T == o.T && H == o.H && W == o.W && BW == o.BW;
    }
};

}  // namespace

struct ccv3d_handle {
    ccv3d_desc d;
    int device;
    int sm_count;
    bool use_tc;         // BF16 layer on the tensor-core route
    bool use_tc32;       // FP32 layer that may take the tensor-core route (3xTF32) when the call is large enough
    TcPlan plan;
    void* w_copy;        // SIMT route: weights in their original order (device)
    void* wp;            // TC route: packed weights (device)
    float* bias32;       // FP32 bias, padded (device)
    unsigned int* status;  // device status word
    unsigned int* band_ctr;  // cooperative staging: per-band arrival counters (MAX_COOP_BANDS words, device)
    void* workspace;
    uint64_t workspace_bytes;
    // host-entry staging (device buffers)
    void* hx; void* hc; void* ho; void* hn;
    uint64_t hx_b, hc_b, ho_b, hn_b;
    cudaEvent_t hp_ev[4][3];   // pipelined host entry: per frame buffer {uploaded, input buffer free, computed, downloaded}
    bool hp_ready;
    EncodeTiledFn encode;
    CUtensorMap tm_a;
    ShapeKey tm_a_key;
    CUtensorMap tm_o;
    CUtensorMap tm_w[2]; // CTA pairs: 2-D maps over the packed weights (half-tile and quarter-tile boxes)
    int tm_w_rows[2];    // box height each was encoded for (0 = not yet)
    long long wait_limit_clk;
    // side streams and events of the banded, overlapped schedule (created with the handle)
    cudaStream_t side[3];
    cudaEvent_t ev_fork, ev_band[MAX_BANDS], ev_join[2];
    // optional per-kernel timing
    int prof_on;
    int64_t prof_n;
    cudaEvent_t* prof_ev;   // PROF_SLOTS x 3 events, created on first enable
    int pdl;             // 1: convolution kernels on frame rings are launched with programmatic stream serialization
    int cluster_ok;      // the device launches thread-block clusters (needed for CTA pairs)
    int call_cf;         // history frames held by the cache of the call being served (set by the entry points)
    ccv3d_counters ctr;
};

namespace {

inline size_t esize(int dt) { return dt == CCV3D_BF16 ? 2 : 4; }
inline uint64_t align_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }

bool overlap(const void* a, uint64_t an, const void* b, uint64_t bn) {
    if (!a || !b || an == 0 || bn == 0) return false;
    const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return a0 < b0 + bn && b0 < a0 + an;
}

// History frames a layer reads: the causal left pad p_l^base = d_t (kt-1) of Section 4.2.
inline int hist_len(const ccv3d_desc& d) { return d.dilation[0] * (d.kt - 1); }

// The geometry every route handles: unit strides and dilations, odd kh and kw, padding that preserves H and W.
// Anything else within the paper's supported contract (spatial stride, padding, dilation; temporal dilation) is
// "general": served by the FP32-FMA kernel and by the tensor-core kernel's run-time tap path.
inline bool standard_geom(const ccv3d_desc& d) {
    for (int i = 0; i < 3; ++i)
        if (d.stride[i] != 1 || d.dilation[i] != 1) return false;
    return (d.kh & 1) && (d.kw & 1) && d.pad_h == (d.kh - 1) / 2 && d.pad_w == (d.kw - 1) / 2;
}

inline int out_extent(int in, int pad, int dil, int k, int stride) {
    const int span = in + 2 * pad - dil * (k - 1) - 1;
    return span < 0 ? 0 : span / stride + 1;
}
inline int out_t(const ccv3d_desc& d, int T) { return (T - 1) / d.stride[0] + 1; }   // Eq. (3) with |Z| + p_l = d_t (kt-1) + T
inline int out_h(const ccv3d_desc& d, int H) { return out_extent(H, d.pad_h, d.dilation[1], d.kh, d.stride[1]); }
inline int out_w(const ccv3d_desc& d, int W) { return out_extent(W, d.pad_w, d.dilation[2], d.kw, d.stride[2]); }

ccv3d_status validate_desc(const ccv3d_desc* d) {
    if (!d) return CCV3D_ERR_INVALID_ARG;
    if (d->cin < 1 || d->cout < 1 || d->kt < 1 || d->kh < 1 || d->kw < 1) return CCV3D_ERR_INVALID_ARG;
    if (d->dtype != CCV3D_F32 && d->dtype != CCV3D_BF16) return CCV3D_ERR_INVALID_ARG;
    if (d->out_dtype != CCV3D_F32 && d->out_dtype != CCV3D_BF16) return CCV3D_ERR_INVALID_ARG;
    for (int i = 0; i < 3; ++i)
        if (d->stride[i] < 1 || d->dilation[i] < 1) return CCV3D_ERR_INVALID_ARG;
    if (d->pad_h < 0 || d->pad_w < 0 || d->pad_t < 0) return CCV3D_ERR_INVALID_ARG;
    // Algorithm 1 rejects groups != 1.  The spatial stride, padding and dilation of the layer and its temporal
    // dilation are part of the paper's supported contract (Eq. (1)-(2)); a temporal stride is not (Algorithm 1
    // sends it to the framework) but is the same operator with source time o s_t + k d_t and T_o from Eq. (3).
    if (d->groups != 1) return CCV3D_ERR_UNSUPPORTED;
    for (int i = 0; i < 3; ++i)
        if (d->stride[i] > 8 || d->dilation[i] > 8) return CCV3D_ERR_UNSUPPORTED;
    if (d->kh > 7 || d->kw > 7 || d->kt > 8 || d->pad_h > 32 || d->pad_w > 32) return CCV3D_ERR_UNSUPPORTED;
    // the temporal padding is causal: all d_t (kt-1) frames on the left, supplied by the cache.  A framework-style
    // symmetric value is accepted when it describes the same total (2 pad_t = d_t (kt-1)); nothing else is.
    const int tc = d->dilation[0] * (d->kt - 1);
    if (!(tc & 1) && d->pad_t != tc / 2) return CCV3D_ERR_UNSUPPORTED;
    if (d->dtype == CCV3D_F32 && d->out_dtype != CCV3D_F32) return CCV3D_ERR_UNSUPPORTED;
    if (d->cin > 65536 || d->cout > 65536) return CCV3D_ERR_UNSUPPORTED;
    return CCV3D_OK;
}

void make_plan(const ccv3d_desc& d, TcPlan* pl) {
    // 64-channel K blocks for the staged route and the 1x1x1 streaming kernel when Cin allows; the fused route
    // (CCV3D_FLAG_FUSED) transposes 32-channel blocks, so its layers are packed for 32
    const bool pointwise = d.kt == 1 && d.kh == 1 && d.kw == 1;
    pl->fused = (d.flags & CCV3D_FLAG_FUSED) && !(d.flags & (CCV3D_FLAG_TC_PER_TAP_A | CCV3D_FLAG_OVERLAP)) && !pointwise &&
                d.out_dtype == CCV3D_BF16;
    pl->KB = (d.cin % 64 == 0 && !pl->fused) ? 64 : 32;
    pl->CB = (d.cin + pl->KB - 1) / pl->KB;
    pl->cin_pad = pl->CB * pl->KB;
    pl->NT = (d.cout + 255) / 256;
    const int per = (d.cout + pl->NT - 1) / pl->NT;
    pl->NPAD = (per + 15) / 16 * 16;
    pl->cout_pad = pl->NT * pl->NPAD;
    // Two 128-pixel blocks per tile (they share every weight tile) when their accumulators can be double buffered
    // in the 512 TMEM columns (Cout <= 128); wider layers take one block per tile so that the epilogue of a tile
    // still overlaps the MMAs of the next (measured at 192 channels: 4 % faster than 2 blocks with one buffer).
    pl->NB = (4 * pl->NPAD <= 512) ? 2 : 1;
    pl->ACC = (2 * pl->NB * pl->NPAD <= 512) ? 2 : 1;
}

// FP32 layers on the tensor cores: rows of 32 FP32 channels = 128 bytes, i.e. the geometry of 64-channel BF16
// blocks; the K loop runs three passes (hi*lo, lo*hi, hi*hi) over the 32-channel blocks.
void make_plan_f32(const ccv3d_desc& d, TcPlan* pl) {
    pl->fused = false;
    pl->KB = 64;
    pl->CB = (d.cin + 31) / 32;
    pl->cin_pad = pl->CB * 32;
    pl->NT = (d.cout + 255) / 256;
    const int per = (d.cout + pl->NT - 1) / pl->NT;
    pl->NPAD = (per + 15) / 16 * 16;
    pl->cout_pad = pl->NT * pl->NPAD;
    pl->NB = (8 * pl->NPAD <= 512) ? 2 : 1;                 // two accumulators per pixel block (see the kernel)
    pl->ACC = (4 * pl->NB * pl->NPAD <= 512) ? 2 : 1;
}

// Taps per weight stage and ring depths that fit `budget` bytes of shared memory: a whole kernel row of taps per
// stage when that stays small (so that a stage carries enough MMAs), at least two activation and two weight
// stages, weight ring up to 8 deep, then a deeper activation ring with what is left.
ccv3d_status size_pipeline(TcParams* p, size_t budget, bool per_tap, int kw) {
    p->TPB = (!per_tap && (size_t)p->b_tap * kw <= 40960) ? kw : 1;
    int SA = per_tap ? 3 : 2;
    for (;;) {
        p->b_slot = (uint32_t)align_up((uint64_t)p->b_tap * p->TPB, 1024);
        if ((size_t)SA * p->a_slot + 3 * (size_t)p->b_slot <= budget) break;
        if (p->TPB > 1) { p->TPB = 1; continue; }
        if ((size_t)SA * p->a_slot + 2 * (size_t)p->b_slot <= budget) break;
        return CCV3D_ERR_UNSUPPORTED;
    }
    int SB = (int)((budget - (size_t)SA * p->a_slot) / p->b_slot);
    if (SB > 8) SB = 8;
    while (SA < 4 && (size_t)(SA + 1) * p->a_slot + (size_t)SB * p->b_slot <= budget) ++SA;
    p->SA = SA;
    p->SB = SB;
    return CCV3D_OK;
}

uint32_t pow2_cols(uint32_t c) {
    uint32_t v = 32;
    while (v < c) v <<= 1;
    return v;
}

ccv3d_status count(ccv3d_handle* h, ccv3d_status s) {
    switch (s) {
        case CCV3D_OK: h->ctr.ok++; break;
        case CCV3D_ERR_UNSUPPORTED: h->ctr.unsupported++; break;
        case CCV3D_ERR_INVALID_ARG:
        case CCV3D_ERR_ALIGNMENT:
        case CCV3D_ERR_ALIAS: h->ctr.invalid++; break;
        default: h->ctr.cuda_error++; break;
    }
    return s;
}

ccv3d_status cuda_fail() {
    cudaGetLastError();  // clear the sticky-less error so that later calls start clean
    return CCV3D_ERR_CUDA;
}

ccv3d_status grow(void** buf, uint64_t* have, uint64_t need) {
    if (need <= *have) return CCV3D_OK;
    if (*buf) {
        if (cudaDeviceSynchronize() != cudaSuccess) return cuda_fail();
        cudaFree(*buf);
        *buf = nullptr;
        *have = 0;
    }
    if (cudaMalloc(buf, need) != cudaSuccess) {
        cudaGetLastError();
        *buf = nullptr;
        return CCV3D_ERR_NOMEM;
    }
    *have = need;
    return CCV3D_OK;
}

// es_w, es_h: traversal strides of the box along w and h (the layer's spatial stride in the per-tap mode, else 1);
// the box then spans BW*es_w x BH*es_h pixels and delivers BW x BH of them.
ccv3d_status encode_act_map(ccv3d_handle* h, int N, int T, int H, int W, int BW, int BH, int es_w = 1, int es_h = 1) {
    const TcPlan& pl = h->plan;
    const int F = hist_len(h->d) + T;
    const bool f32 = h->d.dtype == CCV3D_F32;             // rows of 32 FP32 channels; two blocks (value, remainder) per real block
    const uint64_t rowb = (uint64_t)pl.KB * 2;
    const int inner = f32 ? 32 : pl.KB, blocks = f32 ? 2 * pl.CB : pl.CB;
    cuuint64_t dims[5] = {(cuuint64_t)inner, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)blocks, (cuuint64_t)N * F};
    cuuint64_t strides[4] = {rowb, rowb * W, rowb * W * H, rowb * W * H * blocks};
    cuuint32_t box[5] = {(cuuint32_t)inner, (cuuint32_t)(BW * es_w), (cuuint32_t)(BH * es_h), 1, 1};
    cuuint32_t es[5] = {1, (cuuint32_t)es_w, (cuuint32_t)es_h, 1, 1};
    if (box[1] > 256 || box[2] > 256) return CCV3D_ERR_UNSUPPORTED;
    CUresult r = h->encode(&h->tm_a, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, h->workspace, dims, strides, box, es,
                           CU_TENSOR_MAP_INTERLEAVE_NONE,
                           pl.KB == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? CCV3D_OK : CCV3D_ERR_CUDA;
}

ccv3d_status encode_out_map(ccv3d_handle* h, void* out, int N, int T, int H, int W, int TW, int ECH) {
    const uint64_t es2 = 2;  // BF16 output only
    cuuint64_t dims[5] = {(cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)T, (cuuint64_t)h->d.cout, (cuuint64_t)N};
    cuuint64_t strides[4] = {es2 * W, es2 * W * H, es2 * W * H * T, es2 * W * H * T * h->d.cout};
    cuuint32_t box[5] = {(cuuint32_t)TW, 16, 1, (cuuint32_t)ECH, 1};
    cuuint32_t es[5] = {1, 1, 1, 1, 1};
    CUresult r = h->encode(&h->tm_o, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, out, dims, strides, box, es,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? CCV3D_OK : CCV3D_ERR_CUDA;
}

uint64_t tc_workspace_bytes(const ccv3d_handle* h, int N, int T, int H, int W) {
    const int F = hist_len(h->d) + T;
    if (h->d.dtype == CCV3D_F32) return (uint64_t)N * F * h->plan.cin_pad * H * W * 8;   // values and remainders, FP32
    return (uint64_t)N * F * h->plan.cin_pad * H * W * 2;
}

template <int KB, int NB, int KS, int TPBC>
ccv3d_status launch_tc_coop(ccv3d_handle* h, const TcParams& p, const StageParams& sp, size_t smem, int grid,
                            cudaStream_t st) {
    auto kern = conv3d_tcgen05_kernel<KB, NB, KS, TPBC, false, true>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return cuda_fail();
    // cooperative launch: the tiles of a CTA wait for bands that every other CTA helps to stage, so all CTAs must be
    // resident together - which an ordinary launch does not promise when another stream's kernel holds some SMs
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(TC_THREADS_FUSED);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kern, h->tm_a, h->tm_a, h->tm_o, p, sp) != cudaSuccess) return cuda_fail();
    if (cudaGetLastError() != cudaSuccess) return cuda_fail();
    h->ctr.kernel_launches++;
    return CCV3D_OK;
}

template <int KB, int NB, int KS, int TPBC, bool TF32 = false>
ccv3d_status launch_tc(ccv3d_handle* h, const TcParams& p, size_t smem, int grid, cudaStream_t st) {
    auto kern = conv3d_tcgen05_kernel<KB, NB, KS, TPBC, false, false, TF32>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return cuda_fail();
    StageParams nosp;
    memset(&nosp, 0, sizeof(nosp));
    kern<<<grid, TC_THREADS, smem, st>>>(h->tm_a, h->tm_a, h->tm_o, p, nosp);
    if (cudaGetLastError() != cudaSuccess) return cuda_fail();
    h->ctr.kernel_launches++;
    return CCV3D_OK;
}

// Launch the staging kernel for image rows [h0, h1) on stream st.
ccv3d_status launch_stage(ccv3d_handle* h, StageParams sp, int h0, int h1, int nframes, cudaStream_t st) {
    const TcPlan& pl = h->plan;
    sp.h_begin = h0;
    const bool vec = (sp.W % 8 == 0);
    dim3 sgrid((sp.W + STG_PX - 1) / STG_PX, h1 - h0, (unsigned)(sp.N * nframes * pl.CB));
    if (sgrid.y > 65535 || sgrid.z > 65535) return CCV3D_ERR_UNSUPPORTED;
    if (pl.KB == 64) {
        if (vec) stage_frames_kernel<64, true><<<sgrid, 256, 0, st>>>(sp);
        else stage_frames_kernel<64, false><<<sgrid, 256, 0, st>>>(sp);
    } else {
        if (vec) stage_frames_kernel<32, true><<<sgrid, 128, 0, st>>>(sp);
        else stage_frames_kernel<32, false><<<sgrid, 128, 0, st>>>(sp);
    }
    if (cudaGetLastError() != cudaSuccess) return cuda_fail();
    h->ctr.kernel_launches++;
    return CCV3D_OK;
}

// CTA pairs: clusters of two CTAs, one 16x16-pixel tile per cluster (see the kernel).  tm_w is the 2-D map over the
// packed weights from which each CTA takes its half of every tap's tile.
template <int KB, int NB, int KS, int TPBC, bool COOP, bool TF32 = false>
ccv3d_status launch_tc_pair(ccv3d_handle* h, const CUtensorMap& tm_a, const CUtensorMap& tm_w, const CUtensorMap& tm_o,
                            const TcParams& p, const StageParams& sp, size_t smem, int grid, cudaStream_t st) {
    auto kern = conv3d_tcgen05_kernel<KB, NB, KS, TPBC, false, COOP, TF32, true>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return cuda_fail();
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(COOP ? TC_THREADS_FUSED : TC_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    if (COOP) {          // all CTAs must be resident together (see launch_tc_coop)
        attr[1].id = cudaLaunchAttributeCooperative;
        attr[1].val.cooperative = 1;
    }
    cfg.attrs = attr;
    cfg.numAttrs = (COOP || h->pdl) ? 2 : 1;
    if (cudaLaunchKernelEx(&cfg, kern, tm_a, tm_w, tm_o, p, sp) != cudaSuccess) return cuda_fail();
    if (cudaGetLastError() != cudaSuccess) return cuda_fail();
    h->ctr.kernel_launches++;
    return CCV3D_OK;
}

// 2-D map over the packed weights: rows of KB channels (one swizzle span), all tiles of all taps one after another;
// a box is one CTA's share of a tile: half of it, or a quarter when the launch runs half-width tiles.  Encoded once
// per handle and box height.
ccv3d_status weight_map(ccv3d_handle* h, int box_rows, const CUtensorMap** out) {
    const int slot = (box_rows == h->plan.NPAD / 2) ? 0 : 1;
    if (h->tm_w_rows[slot] == box_rows) { *out = &h->tm_w[slot]; return CCV3D_OK; }
    CUtensorMap* tm = &h->tm_w[slot];
    const TcPlan& pl = h->plan;
    const ccv3d_desc& d = h->d;
    const uint64_t rows = (uint64_t)(d.dtype == CCV3D_F32 ? 3 : 1) * d.kt * pl.CB * pl.NT * d.kh * d.kw * pl.NPAD;
    cuuint64_t dims[2] = {(cuuint64_t)pl.KB, (cuuint64_t)rows};   // (FP32 layers: 128-byte rows of 32 values, seen as 64 BF16)
    cuuint64_t strides[1] = {(cuuint64_t)pl.KB * 2};
    cuuint32_t box[2] = {(cuuint32_t)pl.KB, (cuuint32_t)box_rows};
    cuuint32_t es[2] = {1, 1};
    if (rows > 0x7FFFFFFFull || box_rows > 256 || box_rows % 8) return CCV3D_ERR_UNSUPPORTED;
    CUresult rc = h->encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, h->wp, dims, strides, box, es,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (rc != CUDA_SUCCESS) return CCV3D_ERR_CUDA;
    h->tm_w_rows[slot] = box_rows;
    *out = tm;
    return CCV3D_OK;
}

// Dispatch over the compiled pair variants (straight-line taps only: ks = 3 or 1).
template <bool COOP>
ccv3d_status launch_pair_any(ccv3d_handle* h, const CUtensorMap& tm_a, const CUtensorMap& tm_o, const TcParams& p,
                             const StageParams& sp, size_t smem, int grid, int ks, int nb, cudaStream_t st) {
    const CUtensorMap* tm_w = nullptr;
    ccv3d_status s = weight_map(h, p.NPAD / 2, &tm_w);
    if (s != CCV3D_OK) return s;
#define CCV3D_LAUNCH_PAIR(KBv, NBv)                                                                                        \
    do {                                                                                                                   \
        if (ks == 3 && p.TPB == 3) return launch_tc_pair<KBv, NBv, 3, 3, COOP>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st); \
        if (ks == 3) return launch_tc_pair<KBv, NBv, 3, 1, COOP>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);              \
        return launch_tc_pair<KBv, NBv, 1, 1, COOP>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);                           \
    } while (0)
    if (h->d.dtype == CCV3D_F32) {          // 3xTF32 (plain schedule only)
        if (COOP) return CCV3D_ERR_UNSUPPORTED;
        if (nb == 2) {
            if (ks == 3 && p.TPB == 3) return launch_tc_pair<64, 2, 3, 3, false, true>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);
            if (ks == 3) return launch_tc_pair<64, 2, 3, 1, false, true>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);
            return launch_tc_pair<64, 2, 1, 1, false, true>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);
        }
        if (ks == 3 && p.TPB == 3) return launch_tc_pair<64, 1, 3, 3, false, true>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);
        if (ks == 3) return launch_tc_pair<64, 1, 3, 1, false, true>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);
        return launch_tc_pair<64, 1, 1, 1, false, true>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);
    }
    if (h->plan.KB == 64 && nb == 2) CCV3D_LAUNCH_PAIR(64, 2);
    else if (h->plan.KB == 64) CCV3D_LAUNCH_PAIR(64, 1);
    else if (nb == 2) CCV3D_LAUNCH_PAIR(32, 2);
    else CCV3D_LAUNCH_PAIR(32, 1);
#undef CCV3D_LAUNCH_PAIR
}

// A layer runs on CTA pairs (every SM then reads half of each weight tile from L2 and from its shared memory) when
// its taps are the straight-line kind and there are tiles for at least a quarter of the pairs.  `pair_tiles` counts
// tiles of 16 rows x 16*NB pixels.
bool pair_eligible(const ccv3d_handle* h, int64_t pair_tiles) {
    const ccv3d_desc& d = h->d;
    const TcPlan& pl = h->plan;
    if ((d.flags & CCV3D_FLAG_NO_PAIR) || !h->cluster_ok) return false;
    if (d.flags & CCV3D_FLAG_TC_PER_TAP_A) return false;
    if (d.stride[1] != 1 || d.stride[2] != 1 || d.dilation[1] != 1 || d.dilation[2] != 1) return false;
    if (d.kh != 3 || d.kw != 3) return false;              // (1x1 layers are bound by their epilogue; pairs make them slower)
    if (pl.NPAD % 16 != 0 || h->sm_count < 2) return false;
    return pair_tiles * pl.NT >= h->sm_count / 8;
}

ccv3d_status launch_conv(ccv3d_handle* h, TcParams p, int nb, int ty0, int ty1, size_t smem, int ks, cudaStream_t st) {
    const TcPlan& pl = h->plan;
    p.ty_begin = ty0;
    p.tiles_h = ty1 - ty0;
    const int64_t total = (int64_t)p.N * p.tiles_h * p.tiles_w * p.T * p.NT;
    if (total > 0x7FFFFFFF) return CCV3D_ERR_UNSUPPORTED;
    p.total_tiles = (int)total;
    const int grid = p.total_tiles < h->sm_count ? p.total_tiles : h->sm_count;
    ccv3d_status s;
    // straight-line tap loops for the common kernels; the run-time variant takes everything else
#define CCV3D_LAUNCH(KBv, NBv)                                                                   \
    do {                                                                                         \
        if (ks == 3 && p.TPB == 3) s = launch_tc<KBv, NBv, 3, 3>(h, p, smem, grid, st);          \
        else if (ks == 3 && p.TPB == 1) s = launch_tc<KBv, NBv, 3, 1>(h, p, smem, grid, st);     \
        else if (ks == 1) s = launch_tc<KBv, NBv, 1, 1>(h, p, smem, grid, st);                   \
        else s = launch_tc<KBv, NBv, 0, 0>(h, p, smem, grid, st);                                \
    } while (0)
#define CCV3D_LAUNCH_F32(NBv)                                                                      \
    do {                                                                                          \
        if (ks == 3 && p.TPB == 3) s = launch_tc<64, NBv, 3, 3, true>(h, p, smem, grid, st);      \
        else if (ks == 3 && p.TPB == 1) s = launch_tc<64, NBv, 3, 1, true>(h, p, smem, grid, st); \
        else if (ks == 1) s = launch_tc<64, NBv, 1, 1, true>(h, p, smem, grid, st);               \
        else s = launch_tc<64, NBv, 0, 0, true>(h, p, smem, grid, st);                            \
    } while (0)
    if (h->d.dtype == CCV3D_F32) {
        if (nb == 2) CCV3D_LAUNCH_F32(2);
        else CCV3D_LAUNCH_F32(1);
    } else if (pl.KB == 64 && nb == 2) CCV3D_LAUNCH(64, 2);
    else if (pl.KB == 64) CCV3D_LAUNCH(64, 1);
    else if (nb == 2) CCV3D_LAUNCH(32, 2);
    else CCV3D_LAUNCH(32, 1);
#undef CCV3D_LAUNCH_F32
#undef CCV3D_LAUNCH
    return s;
}

ccv3d_status forward_tc(ccv3d_handle* h, const void* x, const void* cache, void* out, void* new_cache, int N, int T,
                        int H, int W, cudaStream_t st) {
    const ccv3d_desc& d = h->d;
    const TcPlan& pl = h->plan;
    const int tc = hist_len(d);
    const int F = tc + T;
    const bool general = !standard_geom(d);
    const int Ho = out_h(d, H), Wo = out_w(d, W), To = out_t(d, T);   // output extents; T, H, W are the input's
    const bool strided = d.stride[1] > 1 || d.stride[2] > 1;
    const bool f32 = d.dtype == CCV3D_F32;                 // 3xTF32: FP32 staging with the hi/lo split, TF32 MMAs

    ccv3d_status s = grow(&h->workspace, &h->workspace_bytes, tc_workspace_bytes(h, N, T, H, W));
    if (s != CCV3D_OK) return s;

    // ---- staging: [cache ; x] channels-last, cache update in the same pass ----
    StageParams sp;
    memset(&sp, 0, sizeof(sp));
    sp.x = (const __nv_bfloat16*)x;
    const int cf = (tc && cache) ? h->call_cf : 0;          // older history frames are absent: their taps are skipped
    sp.cache = cf ? (const __nv_bfloat16*)cache : nullptr;
    sp.cf = cf;
    sp.zs = (__nv_bfloat16*)h->workspace;
    sp.new_cache = tc ? (__nv_bfloat16*)new_cache : nullptr;
    sp.N = N; sp.Cin = d.cin; sp.T = T; sp.H = H; sp.W = W; sp.tc = tc; sp.CB = pl.CB;
    sp.f_begin = (tc - cf) < T ? (tc - cf) : T;
    const int nframes = F - sp.f_begin;

    // ---- implicit GEMM parameters ----
    // a spatial stride cannot be a shift inside one halo tile: those layers fetch one strided box per tap
    const int per_tap = ((d.flags & CCV3D_FLAG_TC_PER_TAP_A) || strided) ? 1 : 0;
    // 256-pixel tiles (two 128-pixel blocks sharing every weight tile) unless that leaves SMs without a tile
    int NB = pl.NB;
    if ((int64_t)N * ((Ho + 15) / 16) * ((Wo + 15) / 16) * To * pl.NT < h->sm_count) NB = 1;
    // Still fewer than half as many work items as SMs (the 44x80 layers): run half-width output-channel tiles.
    // Twice the items, each streaming half of the weights through its SM - the per-SM weight stream is what
    // bounds a 128-pixel tile - and nothing to reduce afterwards.
    int NT = pl.NT, NPAD = pl.NPAD, split_n = 0;
    if (NB == 1 && !per_tap && pl.NPAD % 32 == 0 &&
        2 * (int64_t)N * ((Ho + 15) / 16) * ((Wo + 7) / 8) * To * pl.NT <= h->sm_count) {
        split_n = 1; NT = 2 * pl.NT; NPAD = pl.NPAD / 2;
    }
    const int asets = (d.dtype == CCV3D_F32) ? 2 : 1;       // FP32 layers keep two accumulators per pixel block
    const int ACC = (2 * asets * NB * NPAD <= 512) ? 2 : 1;
    // CTA pairs (wide output-channel tiles): 16x16-pixel tiles shared by the two CTAs of a cluster; not combined with
    // the banded multi-stream schedule
    const bool pair = !per_tap && !(d.flags & CCV3D_FLAG_OVERLAP) &&
                      pair_eligible(h, (int64_t)N * ((Ho + 15) / 16) * ((Wo + 16 * NB - 1) / (16 * NB)) * To);
    const int TW = 8 * NB;                                 // pixels per row of a CTA's part of a tile
    const int TWT = pair ? 2 * TW : TW;                    // tile width in the tile index space
    const int BW = per_tap ? TW : TW + (d.kw - 1) * d.dilation[2];
    const int BH = per_tap ? 16 : 16 + (d.kh - 1) * d.dilation[1];
    ShapeKey key{h->workspace, N, T, H, W, BW};
    if (!(key == h->tm_a_key)) {
        s = encode_act_map(h, N, T, H, W, BW, BH, per_tap ? d.stride[2] : 1, per_tap ? d.stride[1] : 1);
        if (s != CCV3D_OK) return s;
        h->tm_a_key = key;
    }
    TcParams p;
    memset(&p, 0, sizeof(p));
    p.N = N; p.T = To; p.H = Ho; p.W = Wo; p.Cout = d.cout; p.F = F;
    p.kt = d.kt; p.kh = d.kh; p.kw = d.kw;
    p.general = general ? 1 : 0;
    p.act = (d.flags & CCV3D_FLAG_EPI_SILU) ? 1 : 0;
    p.pad_h = d.pad_h; p.pad_w = d.pad_w; p.dil_h = d.dilation[1]; p.dil_w = d.dilation[2]; p.dil_t = d.dilation[0];
    p.str_h = d.stride[1]; p.str_w = d.stride[2]; p.str_t = d.stride[0];
    p.CB = pl.CB; p.NT = NT; p.NPAD = NPAD;
    const int tiles_h = (Ho + 15) / 16;
    p.tiles_w = (Wo + TWT - 1) / TWT;
    p.first_frame = tc - cf;
    p.out_f32 = d.out_dtype == CCV3D_F32;
    p.per_tap_a = per_tap;
    p.ACC = ACC;
    p.a_slot = (uint32_t)align_up((uint64_t)BW * BH * pl.KB * 2, 1024);
    p.b_tap = (uint32_t)(pair ? NPAD / 2 : NPAD) * pl.KB * 2;   // a CTA of a pair holds half of every weight tile
    p.split_n = split_n;
    p.b_src_tap = split_n ? (uint32_t)pl.NPAD * pl.KB * 2 : 0;
    // epilogue: BF16 output rows that TMA can address (W*2 bytes a multiple of 16) go through shared memory
    p.epi_tma = (!p.out_f32 && Wo % 8 == 0) ? 1 : 0;
    p.ECH = (NPAD % 32 == 0) ? 32 : 16;
    p.e_slot = p.epi_tma ? (uint32_t)(p.ECH * 16 * TW * 2) : 0;

    // Optional (CCV3D_FLAG_OVERLAP): large images are cut into bands of tile rows; band k is staged on a side
    // stream while the convolution kernel of band k-1 runs (the staging pass is bound by HBM, the convolution
    // by the tensor cores), and consecutive convolution launches alternate between two streams so that the next
    // band's CTAs fill the ragged tail of the previous one.  The caller only ever sees its own stream: the side
    // streams fork from it after everything enqueued so far and join it before the call returns.  Measured
    // effect on B200: 0 to -6 % time (the co-resident staging blocks make little headway next to the
    // persistent convolution CTAs), which is why it is not the default.
    int nbands = 1;
    if ((d.flags & CCV3D_FLAG_OVERLAP) && h->side[0] && !general && !f32 &&
        (int64_t)N * tiles_h * p.tiles_w * To * NT >= 2LL * h->sm_count && tiles_h >= 4)
        nbands = tiles_h / 2 < MAX_BANDS ? tiles_h / 2 : MAX_BANDS;

    // Cooperative staging (default when W % 8 == 0): the staging pass runs inside the convolution kernel, on four
    // extra warps per CTA, one band of 16 rows ahead of the tiles that read it.
    const bool coop = nbands == 1 && !per_tap && !general && !f32 && !(d.flags & CCV3D_FLAG_TWO_KERNELS) && W % 8 == 0 &&
                      tiles_h <= MAX_COOP_BANDS && tiles_h >= 4 &&
                      (int64_t)N * tiles_h * p.tiles_w * To * NT * (pair ? 2 : 1) >= 4LL * h->sm_count;   // small problems: two kernels
    size_t fixed = 1024 /*alignment slack*/ + align_up(sizeof(TcShared), 128) + 2 * (size_t)p.e_slot + (coop ? 9216 : 0);
    // leave room for staging blocks to be resident next to a convolution CTA when the two overlap
    const size_t limit = nbands > 1 ? SMEM_LIMIT - STAGE_COEXIST_BYTES : SMEM_LIMIT;
    const size_t budget = limit - fixed;
    s = size_pipeline(&p, budget, per_tap != 0, d.kw);
    if (s != CCV3D_OK) return s;
    p.tmem_cols = pow2_cols((uint32_t)(asets * NB * NPAD * ACC));
    if (p.tmem_cols > 512) return CCV3D_ERR_UNSUPPORTED;
    p.wait_limit_clk = h->wait_limit_clk;
    p.bias = h->bias32;
    p.wq = (const uint8_t*)h->wp;
    p.out = out;
    p.status = h->status;
    if (p.epi_tma) {
        s = encode_out_map(h, out, N, To, Ho, Wo, TW, p.ECH);
        if (s != CCV3D_OK) return s;
    } else {
        h->tm_o = h->tm_a;  // never dereferenced on this path; any valid descriptor will do
    }
    const size_t smem = fixed + (size_t)p.SA * p.a_slot + (size_t)p.SB * p.b_slot;
    // straight-line tap loops need unit spatial dilation (the tap offsets are compile-time); padding and the temporal
    // dilation only move the producer's TMA coordinates
    const int ks = (!per_tap && d.dilation[1] == 1 && d.dilation[2] == 1 && d.kh == d.kw && (d.kh == 1 || d.kh == 3)) ? d.kh : 0;
    const int ph = (d.kh - 1) / 2;
    cudaEvent_t* pev = (h->prof_on && h->prof_ev) ? h->prof_ev + 3 * (h->prof_n % PROF_SLOTS) : nullptr;

    if (coop) {
        if (pev) { cudaEventRecord(pev[0], st); cudaEventRecord(pev[1], st); }
        if (cudaMemsetAsync(h->band_ctr, 0, (size_t)tiles_h * sizeof(unsigned int), st) != cudaSuccess) return cuda_fail();
        p.band_ctr = h->band_ctr;
        p.nbands = tiles_h;
        p.ty_begin = 0;
        p.tiles_h = tiles_h;
        const int64_t total = (int64_t)N * tiles_h * p.tiles_w * To * NT;
        if (total > 0x7FFFFFFF) return CCV3D_ERR_UNSUPPORTED;
        p.total_tiles = (int)total;
        int grid = p.total_tiles < h->sm_count ? p.total_tiles : h->sm_count;
        if (pair) {
            grid = 2 * (p.total_tiles < h->sm_count / 2 ? p.total_tiles : h->sm_count / 2);
            s = launch_pair_any<true>(h, h->tm_a, h->tm_o, p, sp, smem, grid, ks, NB, st);
            if (s != CCV3D_OK) return s;
        } else {
#define CCV3D_LAUNCH_COOP(KBv, NBv)                                                                        \
    do {                                                                                                   \
        if (ks == 3 && p.TPB == 3) s = launch_tc_coop<KBv, NBv, 3, 3>(h, p, sp, smem, grid, st);           \
        else if (ks == 3 && p.TPB == 1) s = launch_tc_coop<KBv, NBv, 3, 1>(h, p, sp, smem, grid, st);      \
        else if (ks == 1) s = launch_tc_coop<KBv, NBv, 1, 1>(h, p, sp, smem, grid, st);                    \
        else s = launch_tc_coop<KBv, NBv, 0, 0>(h, p, sp, smem, grid, st);                                 \
    } while (0)
        if (pl.KB == 64 && NB == 2) CCV3D_LAUNCH_COOP(64, 2);
        else if (pl.KB == 64) CCV3D_LAUNCH_COOP(64, 1);
        else if (NB == 2) CCV3D_LAUNCH_COOP(32, 2);
        else CCV3D_LAUNCH_COOP(32, 1);
#undef CCV3D_LAUNCH_COOP
        if (s != CCV3D_OK) return s;
        }
    } else if (nbands == 1) {
        if (pev) cudaEventRecord(pev[0], st);
        if (f32) {
            StageF32Params sf;
            sf.x = (const float*)x; sf.cache = cf ? (const float*)cache : nullptr; sf.cf = cf;
            sf.zs = (float*)h->workspace; sf.new_cache = tc ? (float*)new_cache : nullptr;
            sf.N = N; sf.Cin = d.cin; sf.T = T; sf.H = H; sf.W = W; sf.tc = tc; sf.CBr = pl.CB; sf.f_begin = sp.f_begin;
            dim3 sgrid((W + 31) / 32, H, (unsigned)((int64_t)N * nframes * sf.CBr));
            if (H > 65535 || (int64_t)N * nframes * sf.CBr > 65535) return CCV3D_ERR_UNSUPPORTED;
            stage_frames_f32_kernel<<<sgrid, 256, 0, st>>>(sf);
            if (cudaGetLastError() != cudaSuccess) return cuda_fail();
            h->ctr.kernel_launches++;
            s = CCV3D_OK;
        } else {
            s = launch_stage(h, sp, 0, H, nframes, st);
        }
        if (s != CCV3D_OK) return s;
        if (pev) cudaEventRecord(pev[1], st);
        if (pair) {
            p.ty_begin = 0;
            p.tiles_h = tiles_h;
            const int64_t total = (int64_t)N * tiles_h * p.tiles_w * To * NT;
            if (total > 0x7FFFFFFF) return CCV3D_ERR_UNSUPPORTED;
            p.total_tiles = (int)total;
            const int grid = 2 * (p.total_tiles < h->sm_count / 2 ? p.total_tiles : h->sm_count / 2);
            StageParams nosp;
            memset(&nosp, 0, sizeof(nosp));
            s = launch_pair_any<false>(h, h->tm_a, h->tm_o, p, nosp, smem, grid, ks, NB, st);
        } else {
            s = launch_conv(h, p, NB, 0, tiles_h, smem, ks, st);
        }
        if (s != CCV3D_OK) return s;
    } else {
        cudaStream_t s_stage = h->side[0];
        if (pev) cudaEventRecord(pev[0], st);
        if (cudaEventRecord(h->ev_fork, st) != cudaSuccess) return cuda_fail();
        for (int i = 0; i < 3; ++i)
            if (cudaStreamWaitEvent(h->side[i], h->ev_fork, 0) != cudaSuccess) return cuda_fail();
        int staged_to = 0;   // image rows [0, staged_to) are staged (or enqueued for staging)
        for (int k = 0; k < nbands; ++k) {
            const int ty0 = (int)((int64_t)tiles_h * k / nbands), ty1 = (int)((int64_t)tiles_h * (k + 1) / nbands);
            int need_to = ty1 * 16 + ph;              // last image row (exclusive) this band's halo reaches
            if (need_to > H || k == nbands - 1) need_to = H;
            if (need_to > staged_to) {
                s = launch_stage(h, sp, staged_to, need_to, nframes, s_stage);
                if (s != CCV3D_OK) return s;
                staged_to = need_to;
            }
            if (cudaEventRecord(h->ev_band[k], s_stage) != cudaSuccess) return cuda_fail();
            cudaStream_t s_conv = h->side[1 + (k & 1)];
            if (cudaStreamWaitEvent(s_conv, h->ev_band[k], 0) != cudaSuccess) return cuda_fail();
            if (k == 0 && pev) cudaEventRecord(pev[1], s_conv);
            s = launch_conv(h, p, NB, ty0, ty1, smem, ks, s_conv);
            if (s != CCV3D_OK) return s;
        }
        for (int i = 1; i < 3; ++i) {
            if (cudaEventRecord(h->ev_join[i - 1], h->side[i]) != cudaSuccess) return cuda_fail();
            if (cudaStreamWaitEvent(st, h->ev_join[i - 1], 0) != cudaSuccess) return cuda_fail();
        }
    }
    h->ctr.tcgen05_bf16++;
    if (pev) {
        cudaEventRecord(pev[2], st);
        h->prof_n++;
    }
    return CCV3D_OK;
}

// ------------------------------------------------------------------------------------------------
// Fused route: no staging copy.  The convolution kernel reads x and the cache through two tensor maps and
// transposes in shared memory; the cache update is a separate bit-copy kernel.
// ------------------------------------------------------------------------------------------------
template <int NB, int KS, int TPBC>
ccv3d_status launch_fused(ccv3d_handle* h, const CUtensorMap& tm_x, const CUtensorMap& tm_c, const CUtensorMap& tm_o,
                          const TcParams& p, size_t smem, int grid, cudaStream_t st) {
    auto kern = conv3d_tcgen05_kernel<32, NB, KS, TPBC, true, false>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return cuda_fail();
    StageParams nosp;
    memset(&nosp, 0, sizeof(nosp));
    kern<<<grid, TC_THREADS_FUSED, smem, st>>>(tm_x, tm_c, tm_o, p, nosp);
    if (cudaGetLastError() != cudaSuccess) return cuda_fail();
    h->ctr.kernel_launches++;
    return CCV3D_OK;
}

ccv3d_status encode_ncthw_map(ccv3d_handle* h, CUtensorMap* tm, const void* base, int N, int C, int T, int H, int W,
                              int box_w, int box_h, int box_c, CUtensorMapSwizzle swz) {
    cuuint64_t dims[5] = {(cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)T, (cuuint64_t)C, (cuuint64_t)N};
    cuuint64_t strides[4] = {2ull * W, 2ull * W * H, 2ull * W * H * T, 2ull * W * H * T * C};
    cuuint32_t box[5] = {(cuuint32_t)box_w, (cuuint32_t)box_h, 1, (cuuint32_t)box_c, 1};
    cuuint32_t es[5] = {1, 1, 1, 1, 1};
    CUresult r = h->encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, es,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? CCV3D_OK : CCV3D_ERR_CUDA;
}

bool fused_eligible(const ccv3d_handle* h, int W) { return h->plan.fused && W % 8 == 0 && standard_geom(h->d); }

ccv3d_status forward_fused(ccv3d_handle* h, const void* x, const void* cache, void* out, void* new_cache, int N, int T,
                           int H, int W, cudaStream_t st) {
    const ccv3d_desc& d = h->d;
    const TcPlan& pl = h->plan;
    const int tc = d.kt - 1;
    const int cf = (tc && cache) ? h->call_cf : 0;
    if (!cf) cache = nullptr;
    int NB = 2;   // 256-pixel tiles: the raw-box requests per FLOP, this route's bottleneck, halve against 128-pixel tiles
    if ((int64_t)N * ((H + 15) / 16) * ((W + 15) / 16) * T * pl.NT < h->sm_count) NB = 1;
    const int ACC = (2 * NB * pl.NPAD <= 512) ? 2 : 1;
    const int TW = 8 * NB, BW = TW + d.kw - 1, BH = 16 + d.kh - 1;

    TcParams p;
    memset(&p, 0, sizeof(p));
    p.N = N; p.T = T; p.H = H; p.W = W; p.Cout = d.cout; p.F = tc + T;
    p.kt = d.kt; p.kh = d.kh; p.kw = d.kw; p.tc = tc; p.cf = cf;
    p.act = (d.flags & CCV3D_FLAG_EPI_SILU) ? 1 : 0;
    p.CB = pl.CB; p.NT = pl.NT; p.NPAD = pl.NPAD;
    p.tiles_h = (H + 15) / 16;
    p.tiles_w = (W + TW - 1) / TW;
    const int64_t total = (int64_t)N * p.tiles_h * p.tiles_w * T * pl.NT;
    if (total > 0x7FFFFFFF) return CCV3D_ERR_UNSUPPORTED;
    p.total_tiles = (int)total;
    p.first_frame = tc - cf;
    p.ACC = ACC;
    p.a_slot = (uint32_t)align_up((uint64_t)BW * BH * 64, 1024);
    p.raw_slot = (uint32_t)align_up((uint64_t)32 * BH * RAW_PX * 2, 1024);
    p.b_tap = (uint32_t)pl.NPAD * 64;
    p.epi_tma = 1;
    p.ECH = (pl.NPAD % 32 == 0) ? 32 : 16;
    p.e_slot = (uint32_t)(p.ECH * 16 * TW * 2);
    const size_t fixed = 1024 + align_up(sizeof(TcShared), 128) + 2 * (size_t)p.e_slot + 2 * (size_t)p.raw_slot + 2048;
    if (fixed + 2 * (size_t)p.a_slot + 2 * (size_t)p.b_tap > SMEM_LIMIT) return CCV3D_ERR_UNSUPPORTED;
    const size_t budget = SMEM_LIMIT - fixed;
    p.TPB = ((size_t)p.b_tap * d.kw <= 24576) ? d.kw : 1;
    int SA = 2;
    for (;;) {
        p.b_slot = (uint32_t)align_up((uint64_t)p.b_tap * p.TPB, 1024);
        if ((size_t)SA * p.a_slot + 3 * (size_t)p.b_slot <= budget) break;
        if (p.TPB > 1) { p.TPB = 1; continue; }
        if ((size_t)SA * p.a_slot + 2 * (size_t)p.b_slot <= budget) break;
        return CCV3D_ERR_UNSUPPORTED;
    }
    int SB = (int)((budget - (size_t)SA * p.a_slot) / p.b_slot);
    if (SB > TC_MAX_STAGES) SB = TC_MAX_STAGES;
    p.SA = SA; p.SB = SB;
    p.tmem_cols = pow2_cols((uint32_t)(NB * pl.NPAD * ACC));
    if (p.tmem_cols > 512) return CCV3D_ERR_UNSUPPORTED;
    p.wait_limit_clk = h->wait_limit_clk;
    p.bias = h->bias32;
    p.wq = (const uint8_t*)h->wp;
    p.out = out;
    p.status = h->status;

    // The raw boxes have 64-byte rows, so they take the 64-byte swizzle: a swizzle span wider than the box row
    // (128-byte swizzle here) made the copy land outside its shared-memory slot.
    CUtensorMap tm_x, tm_c, tm_o;
    ccv3d_status s = encode_ncthw_map(h, &tm_x, x, N, d.cin, T, H, W, RAW_PX, BH, 32, CU_TENSOR_MAP_SWIZZLE_64B);
    if (s != CCV3D_OK) return s;
    if (cache) {
        s = encode_ncthw_map(h, &tm_c, cache, N, d.cin, cf, H, W, RAW_PX, BH, 32, CU_TENSOR_MAP_SWIZZLE_64B);
        if (s != CCV3D_OK) return s;
    } else {
        tm_c = tm_x;   // never dereferenced: the taps that would read the cache are skipped
    }
    s = encode_ncthw_map(h, &tm_o, out, N, d.cout, T, H, W, TW, 16, p.ECH, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (s != CCV3D_OK) return s;

    const size_t smem = fixed + (size_t)p.SA * p.a_slot + (size_t)p.SB * p.b_slot;
    const int grid = p.total_tiles < h->sm_count ? p.total_tiles : h->sm_count;
    const int ks = (d.kh == d.kw && (d.kh == 1 || d.kh == 3)) ? d.kh : 0;
    cudaEvent_t* pev = (h->prof_on && h->prof_ev) ? h->prof_ev + 3 * (h->prof_n % PROF_SLOTS) : nullptr;
    if (pev) cudaEventRecord(pev[0], st);
    // cache update: bit copy of the last kt-1 frames of [cache ; x]
    if (tc && new_cache) {
        const uint64_t fbytes = (uint64_t)H * W * 2;          // W % 8 == 0: whole frames in 16-byte units
        const int64_t planes = (int64_t)N * d.cin * tc;
        const int64_t units = (int64_t)(fbytes / 16);
        dim3 g((unsigned)((units + 255) / 256 > 64 ? 64 : (units + 255) / 256), (unsigned)(planes < 65535 ? planes : 65535));
        cache_update_kernel<uint4><<<g, 256, 0, st>>>((const uint4*)x, (const uint4*)cache, (uint4*)new_cache, d.cin, T, tc,
                                                     cf, units, planes);
        if (cudaGetLastError() != cudaSuccess) return cuda_fail();
        h->ctr.kernel_launches++;
    }
    if (pev) cudaEventRecord(pev[1], st);
#define CCV3D_LAUNCH_FUSED(NBv)                                                                              \
    do {                                                                                                     \
        if (ks == 3 && p.TPB == 3) s = launch_fused<NBv, 3, 3>(h, tm_x, tm_c, tm_o, p, smem, grid, st);      \
        else if (ks == 3 && p.TPB == 1) s = launch_fused<NBv, 3, 1>(h, tm_x, tm_c, tm_o, p, smem, grid, st); \
        else if (ks == 1) s = launch_fused<NBv, 1, 1>(h, tm_x, tm_c, tm_o, p, smem, grid, st);               \
        else s = launch_fused<NBv, 0, 0>(h, tm_x, tm_c, tm_o, p, smem, grid, st);                            \
    } while (0)
    if (NB == 2) CCV3D_LAUNCH_FUSED(2);
    else CCV3D_LAUNCH_FUSED(1);
#undef CCV3D_LAUNCH_FUSED
    if (s != CCV3D_OK) return s;
    h->ctr.tcgen05_bf16++;
    if (pev) {
        cudaEventRecord(pev[2], st);
        h->prof_n++;
    }
    return CCV3D_OK;
}

// 1x1x1 layers whose weights fit in shared memory stream straight from NCTHW (no staging copy).
bool pointwise_eligible(const ccv3d_handle* h, int T, int H, int W) {
    const ccv3d_desc& d = h->d;
    const TcPlan& pl = h->plan;
    if (!(d.kt == 1 && d.kh == 1 && d.kw == 1) || !standard_geom(d) || (d.flags & CCV3D_FLAG_EPI_SILU)) return false;
    if (d.flags & CCV3D_FLAG_TC_PER_TAP_A) return false;
    if (pl.KB != 64 || pl.NT != 1 || d.out_dtype != CCV3D_BF16) return false;
    if (((int64_t)T * H * W) % 8 != 0) return false;                       // TMA strides are multiples of 16 bytes
    return (uint64_t)pl.CB * pl.NPAD * 128 <= 98304;
}

ccv3d_status forward_pointwise(ccv3d_handle* h, const void* x, void* out, int N, int T, int H, int W, cudaStream_t st) {
    const ccv3d_desc& d = h->d;
    const TcPlan& pl = h->plan;
    const uint64_t P = (uint64_t)T * H * W;
    if (P > 0x7FFFFFFFull) return CCV3D_ERR_UNSUPPORTED;
    PwParams p;
    memset(&p, 0, sizeof(p));
    p.N = N; p.Cout = d.cout; p.CB = pl.CB; p.NPAD = pl.NPAD;
    p.tiles_p = (int)((P + 127) / 128);
    const int64_t total = (int64_t)N * p.tiles_p;
    if (total > 0x7FFFFFFF) return CCV3D_ERR_UNSUPPORTED;
    p.total_tiles = (int)total;
    p.ECH = (pl.NPAD % 32 == 0) ? 32 : 16;
    p.a_slot = 2 * 64 * 128;
    p.e_slot = (uint32_t)(p.ECH * 128 * 2);
    p.b_tap = (uint32_t)pl.NPAD * 128;
    p.w_bytes = (uint32_t)pl.CB * p.b_tap;
    p.tmem_cols = pow2_cols((uint32_t)(2 * pl.NPAD));
    p.wait_limit_clk = h->wait_limit_clk;
    p.bias = h->bias32;
    p.wq = (const uint8_t*)h->wp;
    p.status = h->status;
    const size_t w_al = align_up(p.w_bytes, 1024);
    const size_t fixed = 1024 + align_up(sizeof(TcShared), 128) + 2 * (size_t)p.e_slot + w_al;
    int SA = (int)((SMEM_LIMIT - fixed) / p.a_slot);
    if (SA > TC_MAX_STAGES) SA = TC_MAX_STAGES;
    if (SA < 2) return CCV3D_ERR_UNSUPPORTED;
    p.SA = SA;
    p.w_bytes = (uint32_t)w_al;   // ring starts on a 1024-byte boundary; the copy itself is CB*b_tap bytes (a multiple of 1024)
    CUtensorMap tm_x, tm_o;
    {
        cuuint64_t dims[3] = {(cuuint64_t)P, (cuuint64_t)d.cin, (cuuint64_t)N};
        cuuint64_t strides[2] = {2ull * P, 2ull * P * d.cin};
        cuuint32_t box[3] = {64, 64, 1};
        cuuint32_t es[3] = {1, 1, 1};
        if (h->encode(&tm_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(x), dims, strides, box, es,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return CCV3D_ERR_CUDA;
    }
    {
        cuuint64_t dims[3] = {(cuuint64_t)P, (cuuint64_t)d.cout, (cuuint64_t)N};
        cuuint64_t strides[2] = {2ull * P, 2ull * P * d.cout};
        cuuint32_t box[3] = {128, (cuuint32_t)p.ECH, 1};
        cuuint32_t es[3] = {1, 1, 1};
        if (h->encode(&tm_o, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, out, dims, strides, box, es,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return CCV3D_ERR_CUDA;
    }
    const size_t smem = fixed + (size_t)SA * p.a_slot;
    if (cudaFuncSetAttribute(conv1x1_tcgen05_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return cuda_fail();
    cudaEvent_t* pev = (h->prof_on && h->prof_ev) ? h->prof_ev + 3 * (h->prof_n % PROF_SLOTS) : nullptr;
    if (pev) { cudaEventRecord(pev[0], st); cudaEventRecord(pev[1], st); }
    const int grid = p.total_tiles < h->sm_count ? p.total_tiles : h->sm_count;
    conv1x1_tcgen05_kernel<<<grid, TC_THREADS, smem, st>>>(tm_x, tm_o, p);
    if (cudaGetLastError() != cudaSuccess) return cuda_fail();
    if (pev) {
        cudaEventRecord(pev[2], st);
        h->prof_n++;
    }
    h->ctr.kernel_launches++;
    h->ctr.tcgen05_bf16++;
    return CCV3D_OK;
}

// ------------------------------------------------------------------------------------------------
// Allocation-free variant of the tensor-core route (ccv3d_forward_static).  Its channels-last staging copy
// lives in a fixed array in device memory that is part of the loaded library image, so the call needs no
// allocator.  Everything below is separate from forward_tc: it has its own tensor maps and launch helper.
// ------------------------------------------------------------------------------------------------
constexpr uint64_t STATIC_SCRATCH_BYTES = 32ull << 20;   // 32 MiB per GPU that loads the library, until exit
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];
constexpr int MAX_DEVICES = 64;
static void* g_static_scratch_addr[MAX_DEVICES];         // device address of the array, per device; set on first use

// In host code the name g_static_scratch is only a stand-in for the symbol: the address a kernel can use has
// to be asked for, once per device, with that device current.
ccv3d_status static_scratch_for_current_device(void** out_ptr) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return cuda_fail();
    if (dev < 0 || dev >= MAX_DEVICES) return CCV3D_ERR_UNSUPPORTED;
    if (!g_static_scratch_addr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return cuda_fail();
        g_static_scratch_addr[dev] = ptr;
    }
    *out_ptr = g_static_scratch_addr[dev];
    return CCV3D_OK;
}

template <int KB, int NB, int KS, int TPBC>
ccv3d_status launch_tc_with_maps(ccv3d_handle* h, const CUtensorMap& tm_a, const CUtensorMap& tm_o, const TcParams& p,
                                 size_t smem, int grid, cudaStream_t st) {
    auto kern = conv3d_tcgen05_kernel<KB, NB, KS, TPBC, false, false>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return cuda_fail();
    StageParams nosp;
    memset(&nosp, 0, sizeof(nosp));
    // programmatic dependent launch: the kernel's set-up may overlap the tail of the previous kernel of the stream
    // (it waits for that kernel before it touches global data)
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(TC_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = h->pdl ? 1 : 0;
    if (cudaLaunchKernelEx(&cfg, kern, tm_a, tm_a, tm_o, p, nosp) != cudaSuccess) return cuda_fail();
    if (cudaGetLastError() != cudaSuccess) return cuda_fail();
    h->ctr.kernel_launches++;
    return CCV3D_OK;
}

ccv3d_status forward_tc_static(ccv3d_handle* h, const void* x, const void* cache, void* out, void* new_cache, int N,
                               int T, int H, int W, cudaStream_t st) {
    const ccv3d_desc& d = h->d;
    const TcPlan& pl = h->plan;
    const int tc = d.kt - 1;
    const int F = tc + T;
    if (d.flags & CCV3D_FLAG_TC_PER_TAP_A) return CCV3D_ERR_UNSUPPORTED;
    if (tc_workspace_bytes(h, N, T, H, W) > STATIC_SCRATCH_BYTES) return CCV3D_ERR_UNSUPPORTED;
    void* scratch = nullptr;
    ccv3d_status s = static_scratch_for_current_device(&scratch);
    if (s != CCV3D_OK) return s;

    // staging pass: it overwrites every byte of the scratch that the convolution kernel will read (padded
    // channels included), so nothing of an earlier call's contents is ever consumed and nothing needs clearing
    StageParams sp;
    sp.x = (const __nv_bfloat16*)x;
    sp.cache = tc ? (const __nv_bfloat16*)cache : nullptr;
    sp.cf = sp.cache ? tc : 0;
    sp.zs = (__nv_bfloat16*)scratch;
    sp.new_cache = tc ? (__nv_bfloat16*)new_cache : nullptr;
    sp.N = N; sp.Cin = d.cin; sp.T = T; sp.H = H; sp.W = W; sp.tc = tc; sp.CB = pl.CB;
    sp.f_begin = sp.cache ? 0 : (tc < T ? tc : T);
    sp.h_begin = 0;
    const bool vec = (W % 8 == 0);
    dim3 sgrid((W + STG_PX - 1) / STG_PX, H, (unsigned)(N * (F - sp.f_begin) * pl.CB));
    if (sgrid.y > 65535 || sgrid.z > 65535) return CCV3D_ERR_UNSUPPORTED;
    if (pl.KB == 64) {
        if (vec) stage_frames_kernel<64, true><<<sgrid, 256, 0, st>>>(sp);
        else stage_frames_kernel<64, false><<<sgrid, 256, 0, st>>>(sp);
    } else {
        if (vec) stage_frames_kernel<32, true><<<sgrid, 128, 0, st>>>(sp);
        else stage_frames_kernel<32, false><<<sgrid, 128, 0, st>>>(sp);
    }
    if (cudaGetLastError() != cudaSuccess) return cuda_fail();
    h->ctr.kernel_launches++;

    const int NB = 2, TW = 8 * NB, BW = TW + d.kw - 1, BH = 16 + d.kh - 1;   // this variant always runs 256-pixel tiles
    const int ACC = (2 * NB * pl.NPAD <= 512) ? 2 : 1;
    CUtensorMap tm_a, tm_o;
    {
        const uint64_t rowb = (uint64_t)pl.KB * 2;
        cuuint64_t dims[5] = {(cuuint64_t)pl.KB, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)pl.CB, (cuuint64_t)N * F};
        cuuint64_t strides[4] = {rowb, rowb * W, rowb * W * H, rowb * W * H * pl.CB};
        cuuint32_t box[5] = {(cuuint32_t)pl.KB, (cuuint32_t)BW, (cuuint32_t)BH, 1, 1};
        cuuint32_t es[5] = {1, 1, 1, 1, 1};
        if (h->encode(&tm_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, scratch, dims, strides, box, es,
                      CU_TENSOR_MAP_INTERLEAVE_NONE,
                      pl.KB == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return CCV3D_ERR_CUDA;
    }
    TcParams p;
    memset(&p, 0, sizeof(p));
    p.N = N; p.T = T; p.H = H; p.W = W; p.Cout = d.cout; p.F = F;
    p.kt = d.kt; p.kh = d.kh; p.kw = d.kw;
    p.CB = pl.CB; p.NT = pl.NT; p.NPAD = pl.NPAD;
    p.tiles_h = (H + 15) / 16;
    p.tiles_w = (W + TW - 1) / TW;
    const int64_t total = (int64_t)N * p.tiles_h * p.tiles_w * T * pl.NT;
    if (total > 0x7FFFFFFF) return CCV3D_ERR_UNSUPPORTED;
    p.total_tiles = (int)total;
    p.first_frame = (tc && !cache) ? tc : 0;
    p.out_f32 = d.out_dtype == CCV3D_F32;
    p.per_tap_a = 0;
    p.act = (d.flags & CCV3D_FLAG_EPI_SILU) ? 1 : 0;
    p.ACC = ACC;
    p.a_slot = (uint32_t)align_up((uint64_t)BW * BH * pl.KB * 2, 1024);
    p.b_tap = (uint32_t)pl.NPAD * pl.KB * 2;
    p.epi_tma = (!p.out_f32 && W % 8 == 0) ? 1 : 0;
    p.ECH = (pl.NPAD % 32 == 0) ? 32 : 16;
    p.e_slot = p.epi_tma ? (uint32_t)(p.ECH * 16 * TW * 2) : 0;
    const size_t fixed = 1024 + align_up(sizeof(TcShared), 128) + 2 * (size_t)p.e_slot;
    const size_t budget = SMEM_LIMIT - fixed;
    s = size_pipeline(&p, budget, false, d.kw);
    if (s != CCV3D_OK) return s;
    p.tmem_cols = pow2_cols((uint32_t)(NB * pl.NPAD * ACC));
    if (p.tmem_cols > 512) return CCV3D_ERR_UNSUPPORTED;
    p.wait_limit_clk = h->wait_limit_clk;
    p.bias = h->bias32;
    p.wq = (const uint8_t*)h->wp;
    p.out = out;
    p.status = h->status;
    if (p.epi_tma) {
        cuuint64_t dims[5] = {(cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)T, (cuuint64_t)d.cout, (cuuint64_t)N};
        cuuint64_t strides[4] = {2ull * W, 2ull * W * H, 2ull * W * H * T, 2ull * W * H * T * d.cout};
        cuuint32_t box[5] = {(cuuint32_t)TW, 16, 1, (cuuint32_t)p.ECH, 1};
        cuuint32_t es[5] = {1, 1, 1, 1, 1};
        if (h->encode(&tm_o, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, out, dims, strides, box, es,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return CCV3D_ERR_CUDA;
    } else {
        tm_o = tm_a;   // never dereferenced on this path
    }
    const size_t smem = fixed + (size_t)p.SA * p.a_slot + (size_t)p.SB * p.b_slot;
    const int grid = p.total_tiles < h->sm_count ? p.total_tiles : h->sm_count;
    const int ks = (d.kh == d.kw && (d.kh == 1 || d.kh == 3)) ? d.kh : 0;
#define CCV3D_LAUNCH_STATIC(KBv)                                                                              \
    do {                                                                                                      \
        if (ks == 3 && p.TPB == 3) s = launch_tc_with_maps<KBv, 2, 3, 3>(h, tm_a, tm_o, p, smem, grid, st);   \
        else if (ks == 3 && p.TPB == 1) s = launch_tc_with_maps<KBv, 2, 3, 1>(h, tm_a, tm_o, p, smem, grid, st); \
        else if (ks == 1) s = launch_tc_with_maps<KBv, 2, 1, 1>(h, tm_a, tm_o, p, smem, grid, st);            \
        else s = launch_tc_with_maps<KBv, 2, 0, 0>(h, tm_a, tm_o, p, smem, grid, st);                         \
    } while (0)
    if (pl.KB == 64) CCV3D_LAUNCH_STATIC(64);
    else CCV3D_LAUNCH_STATIC(32);
#undef CCV3D_LAUNCH_STATIC
    if (s == CCV3D_OK) h->ctr.tcgen05_bf16++;
    return s;
}

// ------------------------------------------------------------------------------------------------
// Resident activations: frame rings [N][F][C/KB][H][W][KB] in the tensor-core operand order.  The convolution
// kernel reads its halo tiles straight from the input ring (history = the slots before x, left there by earlier
// calls), and writes the next layer's ring, so a chain of layers needs no staging pass, no cache tensor and no
// cache update.
// ------------------------------------------------------------------------------------------------
bool ring_valid(const ccv3d_ring* r) {
    if (!r || !r->base) return false;
    if (r->N < 1 || r->C < 1 || r->F < 1 || r->H < 1 || r->W < 1) return false;
    if (r->KB != 64 && r->KB != 32) return false;
    if (r->C % r->KB) return false;
    if ((uint64_t)r->H * r->W > 0x7FFFFFFFull) return false;
    return true;
}

uint64_t ring_bytes_of(const ccv3d_ring* r) { return (uint64_t)r->N * r->F * r->C * r->H * r->W * 2; }

RingGeom ring_geom(const ccv3d_ring* r) {
    RingGeom g;
    g.base = (__nv_bfloat16*)r->base;
    g.N = r->N; g.F = r->F; g.CB = r->C / r->KB; g.H = r->H; g.W = r->W; g.KB = r->KB;
    return g;
}

// Tensor map over a ring as (channel in block, w, h, channel block, n*F + slot).
// es > 1: traversal stride along w and h (box_w x box_h pixels are delivered to / taken from every es-th pixel).
ccv3d_status encode_ring_map(ccv3d_handle* h, CUtensorMap* tm, const ccv3d_ring* r, int box_c, int box_w, int box_h,
                             CUtensorMapSwizzle swz, int es_px = 1) {
    const uint64_t rowb = (uint64_t)r->KB * 2;
    cuuint64_t dims[5] = {(cuuint64_t)r->KB, (cuuint64_t)r->W, (cuuint64_t)r->H, (cuuint64_t)(r->C / r->KB),
                          (cuuint64_t)r->N * r->F};
    cuuint64_t strides[4] = {rowb, rowb * r->W, rowb * r->W * r->H, rowb * r->W * r->H * (r->C / r->KB)};
    cuuint32_t box[5] = {(cuuint32_t)box_c, (cuuint32_t)(box_w * es_px), (cuuint32_t)(box_h * es_px), 1, 1};
    cuuint32_t es[5] = {1, (cuuint32_t)es_px, (cuuint32_t)es_px, 1, 1};
    CUresult rc = h->encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, r->base, dims, strides, box, es,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS ? CCV3D_OK : CCV3D_ERR_CUDA;
}

ccv3d_status forward_ring(ccv3d_handle* h, const ccv3d_ring* in, int x_slot, int hist, const ccv3d_ring* res, int res_slot,
                          const ccv3d_ring* oring, int out_slot, void* out_ncthw, int T, cudaStream_t st, int up_rt = 0) {
    const ccv3d_desc& d = h->d;
    const TcPlan& pl = h->plan;
    const int tc = d.kt - 1;
    if (!h->use_tc || (d.flags & CCV3D_FLAG_TC_PER_TAP_A) || !standard_geom(d)) return CCV3D_ERR_UNSUPPORTED;
    if (!ring_valid(in) || T < 1 || (oring != nullptr) == (out_ncthw != nullptr)) return CCV3D_ERR_INVALID_ARG;
    if (up_rt < 0 || (up_rt > 0 && !oring)) return CCV3D_ERR_INVALID_ARG;
    if (((uintptr_t)in->base | (uintptr_t)out_ncthw) & 15u) return CCV3D_ERR_ALIGNMENT;
    if (in->C != d.cin || in->F < T + tc || x_slot < 0 || x_slot >= in->F || hist < 0 || hist > tc) return CCV3D_ERR_INVALID_ARG;
    if (in->KB != pl.KB) return CCV3D_ERR_UNSUPPORTED;
    const int N = in->N, H = in->H, W = in->W;
    const bool chunked = (d.cout / pl.NT) % 32 == 0 && pl.NT * pl.NPAD == d.cout;   // whole 32-channel chunks per tile
    if (res) {
        if (!ring_valid(res) || res->C != d.cout || res->N != N || res->H != H || res->W != W || res->F < T || res_slot < 0 ||
            res_slot >= res->F)
            return CCV3D_ERR_INVALID_ARG;
        if ((uintptr_t)res->base & 15u) return CCV3D_ERR_ALIGNMENT;
        if (d.out_dtype != CCV3D_BF16 || !chunked) return CCV3D_ERR_UNSUPPORTED;
    }
    const uint64_t in_b = ring_bytes_of(in);
    if (oring) {
        const int oscale = up_rt > 0 ? 2 : 1;              // fused upsample: the output ring is 2H x 2W, up_rt slots per frame
        if (!ring_valid(oring) || oring->C != d.cout || oring->N != N || oring->H != oscale * H || oring->W != oscale * W ||
            (int64_t)oring->F < (int64_t)T * (up_rt > 0 ? up_rt : 1) || out_slot < 0 || out_slot >= oring->F)
            return CCV3D_ERR_INVALID_ARG;
        if ((uintptr_t)oring->base & 15u) return CCV3D_ERR_ALIGNMENT;
        if (d.out_dtype != CCV3D_BF16 || !chunked) return CCV3D_ERR_UNSUPPORTED;
        if (overlap(oring->base, ring_bytes_of(oring), in->base, in_b) ||
            (res && overlap(oring->base, ring_bytes_of(oring), res->base, ring_bytes_of(res))))
            return CCV3D_ERR_ALIAS;
    } else {
        const uint64_t ob = (uint64_t)N * d.cout * T * H * W * esize(d.out_dtype);
        if (overlap(out_ncthw, ob, in->base, in_b) || (res && overlap(out_ncthw, ob, res->base, ring_bytes_of(res))))
            return CCV3D_ERR_ALIAS;
    }

    int NB = pl.NB;
    if ((int64_t)N * ((H + 15) / 16) * ((W + 15) / 16) * T * pl.NT < h->sm_count) NB = 1;
    // fewer than half as many work items as SMs: half-width output-channel tiles (see forward_tc)
    int NT = pl.NT, NPAD = pl.NPAD, split_n = 0;
    if (NB == 1 && pl.NPAD % 64 == 0 && 2 * (int64_t)N * ((H + 15) / 16) * ((W + 7) / 8) * T * pl.NT <= h->sm_count) {
        split_n = 1; NT = 2 * pl.NT; NPAD = pl.NPAD / 2;
    }
    // CTA pairs: 16x16-pixel tiles shared by two CTAs, one 128-pixel block each
    const bool pair =
                      pair_eligible(h, (int64_t)N * ((H + 15) / 16) * ((W + 16 * NB - 1) / (16 * NB)) * T);
    const int ACC = (2 * NB * NPAD <= 512) ? 2 : 1;
    const int TW = 8 * NB, BW = TW + d.kw - 1, BH = 16 + d.kh - 1;
    const int TWT = pair ? 2 * TW : TW;                    // tile width in the tile index space
    CUtensorMap tm_a, tm_o;
    ccv3d_status s = encode_ring_map(h, &tm_a, in, pl.KB, BW, BH, pl.KB == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B);
    if (s != CCV3D_OK) return s;

    TcParams p;
    memset(&p, 0, sizeof(p));
    p.N = N; p.T = T; p.H = H; p.W = W; p.Cout = d.cout;
    p.F = in->F;
    p.f0 = (x_slot - tc + in->F) % in->F;
    p.act = (d.flags & CCV3D_FLAG_EPI_SILU) ? 1 : 0;
    p.kt = d.kt; p.kh = d.kh; p.kw = d.kw;
    p.CB = pl.CB; p.NT = NT; p.NPAD = NPAD;
    p.tiles_h = (H + 15) / 16;
    p.tiles_w = (W + TWT - 1) / TWT;
    const int64_t total = (int64_t)N * p.tiles_h * p.tiles_w * T * NT;
    if (total > 0x7FFFFFFF) return CCV3D_ERR_UNSUPPORTED;
    p.total_tiles = (int)total;
    p.first_frame = tc - hist;
    p.out_f32 = d.out_dtype == CCV3D_F32;
    p.ACC = ACC;
    p.a_slot = (uint32_t)align_up((uint64_t)BW * BH * pl.KB * 2, 1024);
    p.b_tap = (uint32_t)(pair ? NPAD / 2 : NPAD) * pl.KB * 2;   // a CTA of a pair holds half of every weight tile
    p.split_n = split_n;
    p.b_src_tap = split_n ? (uint32_t)pl.NPAD * pl.KB * 2 : 0;
    if (oring) {
        p.epi_tma = 2;
        p.ECH = 32;
        p.e_slot = (uint32_t)(16 * TW * 64);
        p.out_F = oring->F; p.out_f0 = out_slot; p.out_KB = oring->KB;
        p.up_rt = up_rt;
        s = encode_ring_map(h, &tm_o, oring, 32, TW, 16, CU_TENSOR_MAP_SWIZZLE_64B, up_rt > 0 ? 2 : 1);
        if (s != CCV3D_OK) return s;
    } else {
        p.epi_tma = (!p.out_f32 && W % 8 == 0) ? 1 : 0;
        p.ECH = (NPAD % 32 == 0) ? 32 : 16;
        p.e_slot = p.epi_tma ? (uint32_t)(p.ECH * 16 * TW * 2) : 0;
        if (p.epi_tma) {
            cuuint64_t dims[5] = {(cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)T, (cuuint64_t)d.cout, (cuuint64_t)N};
            cuuint64_t strides[4] = {2ull * W, 2ull * W * H, 2ull * W * H * T, 2ull * W * H * T * d.cout};
            cuuint32_t box[5] = {(cuuint32_t)TW, 16, 1, (cuuint32_t)p.ECH, 1};
            cuuint32_t es[5] = {1, 1, 1, 1, 1};
            if (h->encode(&tm_o, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, out_ncthw, dims, strides, box, es,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return CCV3D_ERR_CUDA;
        } else {
            tm_o = tm_a;   // never dereferenced on this path
        }
    }
    if (res) {
        p.res = (const __nv_bfloat16*)res->base;
        p.res_F = res->F; p.res_f0 = res_slot; p.res_CB = res->C / res->KB; p.res_KB = res->KB;
    }
    const size_t fixed = 1024 + align_up(sizeof(TcShared), 128) + 2 * (size_t)p.e_slot;
    const size_t budget = SMEM_LIMIT - fixed;
    s = size_pipeline(&p, budget, false, d.kw);
    if (s != CCV3D_OK) return s;
    p.tmem_cols = pow2_cols((uint32_t)(NB * NPAD * ACC));
    if (p.tmem_cols > 512) return CCV3D_ERR_UNSUPPORTED;
    p.wait_limit_clk = h->wait_limit_clk;
    p.bias = h->bias32;
    p.wq = (const uint8_t*)h->wp;
    p.out = out_ncthw;
    p.status = h->status;
    const size_t smem = fixed + (size_t)p.SA * p.a_slot + (size_t)p.SB * p.b_slot;
    int grid = p.total_tiles < h->sm_count ? p.total_tiles : h->sm_count;
    if (pair) grid = 2 * (p.total_tiles < h->sm_count / 2 ? p.total_tiles : h->sm_count / 2);
    const int ks = (d.kh == d.kw && (d.kh == 1 || d.kh == 3)) ? d.kh : 0;
    cudaEvent_t* pev = (h->prof_on && h->prof_ev) ? h->prof_ev + 3 * (h->prof_n % PROF_SLOTS) : nullptr;
    if (pev) { cudaEventRecord(pev[0], st); cudaEventRecord(pev[1], st); }
#define CCV3D_LAUNCH_RING(KBv, NBv)                                                                              \
    do {                                                                                                         \
        if (ks == 3 && p.TPB == 3) s = launch_tc_with_maps<KBv, NBv, 3, 3>(h, tm_a, tm_o, p, smem, grid, st);    \
        else if (ks == 3 && p.TPB == 1) s = launch_tc_with_maps<KBv, NBv, 3, 1>(h, tm_a, tm_o, p, smem, grid, st); \
        else if (ks == 1) s = launch_tc_with_maps<KBv, NBv, 1, 1>(h, tm_a, tm_o, p, smem, grid, st);             \
        else s = launch_tc_with_maps<KBv, NBv, 0, 0>(h, tm_a, tm_o, p, smem, grid, st);                          \
    } while (0)
    if (pair) {
        StageParams nosp;
        memset(&nosp, 0, sizeof(nosp));
        s = launch_pair_any<false>(h, tm_a, tm_o, p, nosp, smem, grid, ks, NB, st);
    } else if (pl.KB == 64 && NB == 2) CCV3D_LAUNCH_RING(64, 2);
    else if (pl.KB == 64) CCV3D_LAUNCH_RING(64, 1);
    else if (NB == 2) CCV3D_LAUNCH_RING(32, 2);
    else CCV3D_LAUNCH_RING(32, 1);
#undef CCV3D_LAUNCH_RING
    if (s != CCV3D_OK) return s;
    h->ctr.tcgen05_bf16++;
    if (pev) {
        cudaEventRecord(pev[2], st);
        h->prof_n++;
    }
    return CCV3D_OK;
}

ccv3d_status forward_simt(ccv3d_handle* h, const void* x, const void* cache, void* out, void* new_cache, int N, int T,
                          int H, int W, cudaStream_t st) {
    const ccv3d_desc& d = h->d;
    const int tc = hist_len(d);
    SimtParams p;
    const int cf = (tc && cache) ? h->call_cf : 0;
    p.x = x; p.cache = cf ? cache : nullptr; p.cf = cf; p.w = h->w_copy; p.bias = h->bias32; p.out = out;
    p.N = N; p.Cin = d.cin; p.Cout = d.cout; p.T = T; p.H = H; p.W = W; p.kt = d.kt; p.kh = d.kh; p.kw = d.kw;
    p.To = out_t(d, T); p.Ho = out_h(d, H); p.Wo = out_w(d, W); p.st = d.stride[0];
    p.sh = d.stride[1]; p.sw = d.stride[2]; p.ph = d.pad_h; p.pw = d.pad_w; p.dh = d.dilation[1]; p.dw = d.dilation[2];
    p.dil_t = d.dilation[0];
    p.act = (d.flags & CCV3D_FLAG_EPI_SILU) ? 1 : 0;
    const int64_t npix = (int64_t)N * p.To * p.Ho * p.Wo;
    const int64_t gx = (npix + SIMT_THREADS - 1) / SIMT_THREADS;
    if (gx > 0x7FFFFFFF) return CCV3D_ERR_UNSUPPORTED;
    dim3 grid((unsigned)gx, (d.cout + SIMT_CO - 1) / SIMT_CO);
    cudaEvent_t* pev = (h->prof_on && h->prof_ev) ? h->prof_ev + 3 * (h->prof_n % PROF_SLOTS) : nullptr;
    if (pev) { cudaEventRecord(pev[0], st); cudaEventRecord(pev[1], st); }
    if (d.dtype == CCV3D_F32) conv3d_direct_kernel<float, float><<<grid, SIMT_THREADS, 0, st>>>(p);
    else if (d.out_dtype == CCV3D_BF16) conv3d_direct_kernel<__nv_bfloat16, __nv_bfloat16><<<grid, SIMT_THREADS, 0, st>>>(p);
    else conv3d_direct_kernel<__nv_bfloat16, float><<<grid, SIMT_THREADS, 0, st>>>(p);
    if (cudaGetLastError() != cudaSuccess) return cuda_fail();
    h->ctr.kernel_launches++;
    h->ctr.simt++;
    if (pev) {
        cudaEventRecord(pev[2], st);
        h->prof_n++;
    }

    if (tc && new_cache) {
        const uint64_t fbytes = (uint64_t)H * W * esize(d.dtype);
        const int64_t planes = (int64_t)N * d.cin * tc;
        const unsigned gy = (unsigned)(planes < 65535 ? planes : 65535);  // the kernel strides over the rest
        if (fbytes % 16 == 0) {
            const int64_t units = fbytes / 16;
            dim3 g((unsigned)((units + 255) / 256 > 1024 ? 1024 : (units + 255) / 256), gy);
            cache_update_kernel<uint4><<<g, 256, 0, st>>>((const uint4*)x, (const uint4*)cache, (uint4*)new_cache, d.cin, T,
                                                          tc, cf, units, planes);
        } else if (d.dtype == CCV3D_F32) {
            const int64_t units = (int64_t)H * W;
            dim3 g((unsigned)((units + 255) / 256 > 1024 ? 1024 : (units + 255) / 256), gy);
            cache_update_kernel<uint32_t><<<g, 256, 0, st>>>((const uint32_t*)x, (const uint32_t*)cache,
                                                             (uint32_t*)new_cache, d.cin, T, tc, cf, units, planes);
        } else {
            const int64_t units = (int64_t)H * W;
            dim3 g((unsigned)((units + 255) / 256 > 1024 ? 1024 : (units + 255) / 256), gy);
            cache_update_kernel<uint16_t><<<g, 256, 0, st>>>((const uint16_t*)x, (const uint16_t*)cache,
                                                             (uint16_t*)new_cache, d.cin, T, tc, cf, units, planes);
        }
        if (cudaGetLastError() != cudaSuccess) return cuda_fail();
        h->ctr.kernel_launches++;
    }
    return CCV3D_OK;
}

// A handle belongs to the device it was created on: its weights, maps and scratch live there.
bool on_handle_device(const ccv3d_handle* h) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == h->device;
}

// FP32 layers: the FP32-FMA kernel is exact FP32 and fine for small calls; from 0.2 GFLOP on (or when the layer
// asks for it) the call goes to the tensor cores as 3xTF32.  The tensor core's accumulation truncates: measured
// against the FP64 definition the worst element is off by about 4.5e-9 x K x RMS(out) (K = cin*kt*kh*kw; 2.5e-5 at
// K = 5184, 4.7e-5 at K = 10368), so layers with K > 16384 stay on the FP32-FMA kernel unless the flag insists.
bool f32_takes_tensor_cores(const ccv3d_handle* h, int N, int T, int H, int W) {
    const ccv3d_desc& d = h->d;
    if (d.flags & CCV3D_FLAG_F32_TENSOR) return true;
    if ((int64_t)d.cin * d.kt * d.kh * d.kw > 16384) return false;
    const double flops = 2.0 * N * out_t(d, T) * out_h(d, H) * out_w(d, W) * d.cout * d.cin * d.kt * d.kh * d.kw;
    return flops >= 2.0e8;
}

ccv3d_status check_forward_args(const ccv3d_handle* h, const void* x, const void* cache, void* out, void* new_cache,
                                int N, int T, int H, int W, bool device_ptrs) {
    if (!h || !x || !out) return CCV3D_ERR_INVALID_ARG;
    if (N < 1 || T < 1 || H < 1 || W < 1) return CCV3D_ERR_INVALID_ARG;
    const ccv3d_desc& d = h->d;
    const uint64_t px = (uint64_t)N * H * W;
    if ((double)px * T * (d.cin > d.cout ? d.cin : d.cout) > 9.0e15) return CCV3D_ERR_UNSUPPORTED;
    if ((uint64_t)H * W > 0x7FFFFFFFull) return CCV3D_ERR_UNSUPPORTED;
    const int tc = hist_len(d);
    const int Ho = out_h(d, H), Wo = out_w(d, W);
    if (Ho < 1 || Wo < 1) return CCV3D_ERR_INVALID_ARG;                          // the kernel does not fit the padded input
    const uint64_t xb = px * d.cin * T * esize(d.dtype), cb = px * d.cin * tc * esize(d.dtype);
    const uint64_t ccb = px * d.cin * (uint64_t)h->call_cf * esize(d.dtype);     // bytes of the cache actually passed
    const uint64_t ob = (uint64_t)N * Ho * Wo * d.cout * out_t(d, T) * esize(d.out_dtype);
    if (!tc) { cache = nullptr; new_cache = nullptr; }
    if (device_ptrs) {
        const uintptr_t m = (uintptr_t)x | (uintptr_t)cache | (uintptr_t)out | (uintptr_t)new_cache;
        if (m & 15u) return CCV3D_ERR_ALIGNMENT;
    }
    if (overlap(out, ob, x, xb) || overlap(out, ob, cache, ccb)) return CCV3D_ERR_ALIAS;
    if (overlap(new_cache, cb, x, xb) || overlap(new_cache, cb, cache, ccb) || overlap(new_cache, cb, out, ob))
        return CCV3D_ERR_ALIAS;
    return CCV3D_OK;
}

}  // namespace

extern "C" {

const char* ccv3d_status_string(ccv3d_status s) {
    switch (s) {
        case CCV3D_OK: return "CCV3D_OK";
        case CCV3D_ERR_INVALID_ARG: return "CCV3D_ERR_INVALID_ARG";
        case CCV3D_ERR_UNSUPPORTED: return "CCV3D_ERR_UNSUPPORTED";
        case CCV3D_ERR_ALIGNMENT: return "CCV3D_ERR_ALIGNMENT";
        case CCV3D_ERR_ALIAS: return "CCV3D_ERR_ALIAS";
        case CCV3D_ERR_ARCH: return "CCV3D_ERR_ARCH";
        case CCV3D_ERR_NOMEM: return "CCV3D_ERR_NOMEM";
        case CCV3D_ERR_CUDA: return "CCV3D_ERR_CUDA";
        case CCV3D_ERR_DEVICE_TIMEOUT: return "CCV3D_ERR_DEVICE_TIMEOUT";
    }
    return "CCV3D_ERR_UNKNOWN";
}

ccv3d_status ccv3d_create(ccv3d_handle** out_h, const ccv3d_desc* d, const void* w_dev, const void* b_dev,
                          void* stream) {
    if (!out_h) return CCV3D_ERR_INVALID_ARG;
    *out_h = nullptr;
    ccv3d_status s = validate_desc(d);   // host-only checks come first: they need no device
    if (s != CCV3D_OK) return s;
    if (!w_dev) return CCV3D_ERR_INVALID_ARG;
    if (((uintptr_t)w_dev | (uintptr_t)b_dev) & 15u) return CCV3D_ERR_ALIGNMENT;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return cuda_fail();
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return cuda_fail();
    if (prop.major != 10) return CCV3D_ERR_ARCH;

    ccv3d_handle* h = new (std::nothrow) ccv3d_handle();
    if (!h) return CCV3D_ERR_NOMEM;
    memset(h, 0, sizeof(*h));
    h->d = *d;
    h->device = dev;
    h->sm_count = prop.multiProcessorCount;
    h->use_tc = (d->dtype == CCV3D_BF16) && !(d->flags & CCV3D_FLAG_FORCE_SIMT);
    h->use_tc32 = (d->dtype == CCV3D_F32) && !(d->flags & CCV3D_FLAG_FORCE_SIMT);
    // bound of every in-kernel wait: about one second of SM clocks (clock rate is reported in kHz)
    h->wait_limit_clk = (long long)prop.clockRate * 1000ll;
    if (const char* e = getenv("CCV3D_WAIT_LIMIT_MS")) {
        const long v = atol(e);
        if (v > 0 && v <= 10000) h->wait_limit_clk = (long long)prop.clockRate * v;
    }
    h->pdl = getenv("CCV3D_NO_PDL") ? 0 : 1;
    if (cudaDeviceGetAttribute(&h->cluster_ok, cudaDevAttrClusterLaunch, dev) != cudaSuccess) {
        cudaGetLastError();
        h->cluster_ok = 0;
    }
    cudaStream_t st = (cudaStream_t)stream;
    const int taps = d->kt * d->kh * d->kw;

    auto fail = [&](ccv3d_status e) {
        ccv3d_destroy(h);
        return e;
    };

    if (cudaMalloc((void**)&h->status, sizeof(unsigned int)) != cudaSuccess) return fail(CCV3D_ERR_NOMEM);
    if (cudaMalloc((void**)&h->band_ctr, MAX_COOP_BANDS * sizeof(unsigned int)) != cudaSuccess) return fail(CCV3D_ERR_NOMEM);
    if (cudaMemsetAsync(h->status, 0, sizeof(unsigned int), st) != cudaSuccess) return fail(cuda_fail());

    int bias_n = d->cout;
    if (h->use_tc) {
        make_plan(*d, &h->plan);
        bias_n = h->plan.cout_pad;
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
            qres != cudaDriverEntryPointSuccess)
            return fail(cuda_fail());
        h->encode = (EncodeTiledFn)fn;
        bool ok_side = true;
        for (int i = 0; i < 3 && ok_side; ++i)
            ok_side = cudaStreamCreateWithFlags(&h->side[i], cudaStreamNonBlocking) == cudaSuccess;
        ok_side = ok_side && cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; i < MAX_BANDS && ok_side; ++i)
            ok_side = cudaEventCreateWithFlags(&h->ev_band[i], cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; i < 2 && ok_side; ++i)
            ok_side = cudaEventCreateWithFlags(&h->ev_join[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok_side) return fail(cuda_fail());
        const uint64_t wpb = (uint64_t)taps * h->plan.cout_pad * h->plan.cin_pad * 2;
        if (cudaMalloc(&h->wp, wpb) != cudaSuccess) return fail(CCV3D_ERR_NOMEM);
        pack_weights_kernel<<<1024, 256, 0, st>>>((const __nv_bfloat16*)w_dev, (__nv_bfloat16*)h->wp, d->cout, d->cin,
                                                  d->kt, d->kh * d->kw, h->plan.CB, h->plan.KB, h->plan.NT,
                                                  h->plan.NPAD);
        if (cudaGetLastError() != cudaSuccess) return fail(cuda_fail());
        h->ctr.kernel_launches++;
    } else {
        const uint64_t wb = (uint64_t)d->cout * d->cin * taps * esize(d->dtype);
        if (cudaMalloc(&h->w_copy, wb) != cudaSuccess) return fail(CCV3D_ERR_NOMEM);
        if (cudaMemcpyAsync(h->w_copy, w_dev, wb, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return fail(cuda_fail());
    }
    if (h->use_tc32) {
        // FP32 layer: besides the plain copy for the FP32-FMA kernel, the 3xTF32 operand images (lo(w), w, w: one per
        // pass of the K loop; rows of 128 bytes, which the kernel treats like 64-channel BF16 rows)
        make_plan_f32(*d, &h->plan);
        bias_n = h->plan.cout_pad;
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
            qres != cudaDriverEntryPointSuccess)
            return fail(cuda_fail());
        h->encode = (EncodeTiledFn)fn;
        const uint64_t wpb = (uint64_t)3 * taps * h->plan.cout_pad * h->plan.cin_pad * 4;
        if (cudaMalloc(&h->wp, wpb) != cudaSuccess) return fail(CCV3D_ERR_NOMEM);
        pack_weights_f32_kernel<<<1024, 256, 0, st>>>((const float*)w_dev, (float*)h->wp, d->cout, d->cin, d->kt,
                                                      d->kh * d->kw, h->plan.CB, h->plan.NT, h->plan.NPAD);
        if (cudaGetLastError() != cudaSuccess) return fail(cuda_fail());
        h->ctr.kernel_launches++;
    }
    if (cudaMalloc((void**)&h->bias32, (size_t)bias_n * sizeof(float)) != cudaSuccess) return fail(CCV3D_ERR_NOMEM);
    if (d->dtype == CCV3D_BF16)
        bias_to_f32_kernel<__nv_bfloat16><<<(bias_n + 255) / 256, 256, 0, st>>>((const __nv_bfloat16*)b_dev, h->bias32,
                                                                                d->cout, bias_n);
    else
        bias_to_f32_kernel<float><<<(bias_n + 255) / 256, 256, 0, st>>>((const float*)b_dev, h->bias32, d->cout, bias_n);
    if (cudaGetLastError() != cudaSuccess) return fail(cuda_fail());
    h->ctr.kernel_launches++;
    *out_h = h;
    return CCV3D_OK;
}

ccv3d_status ccv3d_destroy(ccv3d_handle* h) {
    if (!h) return CCV3D_OK;
    cudaDeviceSynchronize();
    void* bufs[] = {h->w_copy, h->wp, h->bias32, h->status, h->band_ctr, h->workspace, h->hx, h->hc, h->ho, h->hn};
    for (void* b : bufs)
        if (b) cudaFree(b);
    for (int i = 0; i < 3; ++i)
        if (h->side[i]) cudaStreamDestroy(h->side[i]);
    if (h->ev_fork) cudaEventDestroy(h->ev_fork);
    for (int i = 0; i < MAX_BANDS; ++i)
        if (h->ev_band[i]) cudaEventDestroy(h->ev_band[i]);
    for (int i = 0; i < 2; ++i)
        if (h->ev_join[i]) cudaEventDestroy(h->ev_join[i]);
    if (h->hp_ready)
        for (int k = 0; k < 4; ++k)
            for (int b = 0; b < 3; ++b) cudaEventDestroy(h->hp_ev[k][b]);
    if (h->prof_ev) {
        for (int i = 0; i < 3 * PROF_SLOTS; ++i) cudaEventDestroy(h->prof_ev[i]);
        delete[] h->prof_ev;
    }
    cudaGetLastError();
    delete h;
    return CCV3D_OK;
}

ccv3d_status ccv3d_workspace_bytes(const ccv3d_handle* h, int32_t N, int32_t T, int32_t H, int32_t W,
                                   uint64_t* bytes_host) {
    if (!h || !bytes_host || N < 1 || T < 1 || H < 1 || W < 1) return CCV3D_ERR_INVALID_ARG;
    const bool scratch_free = (h->use_tc32 ? !f32_takes_tensor_cores(h, N, T, H, W) : !h->use_tc) ||
                              (h->use_tc && (pointwise_eligible(h, T, H, W) || fused_eligible(h, W)));
    *bytes_host = scratch_free ? 0 : tc_workspace_bytes(h, N, T, H, W);
    return CCV3D_OK;
}

ccv3d_status ccv3d_out_dims(const ccv3d_handle* h, int32_t T, int32_t H, int32_t W, int32_t* out_t_host,
                            int32_t* out_h_host, int32_t* out_w_host, int32_t* cache_frames_host) {
    if (!h || T < 1 || H < 1 || W < 1) return CCV3D_ERR_INVALID_ARG;
    if (out_t_host) *out_t_host = out_t(h->d, T);
    if (out_h_host) *out_h_host = out_h(h->d, H);
    if (out_w_host) *out_w_host = out_w(h->d, W);
    if (cache_frames_host) *cache_frames_host = hist_len(h->d);
    return CCV3D_OK;
}

ccv3d_status ccv3d_forward_ex(ccv3d_handle* h, const void* x, const void* cache, int32_t cache_frames, void* out,
                              void* new_cache, int32_t N, int32_t T, int32_t H, int32_t W, void* stream) {
    if (!h) return CCV3D_ERR_INVALID_ARG;
    h->ctr.calls++;
    const int tc = hist_len(h->d);
    if (cache_frames < 0 || cache_frames > tc) return count(h, CCV3D_ERR_INVALID_ARG);
    if (cache_frames > 0 && !cache) return count(h, CCV3D_ERR_INVALID_ARG);
    if (cache_frames == 0) cache = nullptr;
    h->call_cf = cache_frames;
    ccv3d_status s = check_forward_args(h, x, cache, out, new_cache, N, T, H, W, true);
    if (s != CCV3D_OK) return count(h, s);
    if (!on_handle_device(h)) return count(h, CCV3D_ERR_INVALID_ARG);
    cudaStream_t st = (cudaStream_t)stream;
    if (h->use_tc && pointwise_eligible(h, T, H, W)) s = forward_pointwise(h, x, out, N, T, H, W, st);
    else if (h->use_tc && fused_eligible(h, W)) s = forward_fused(h, x, cache, out, new_cache, N, T, H, W, st);
    else if (h->use_tc) s = forward_tc(h, x, cache, out, new_cache, N, T, H, W, st);
    else if (h->use_tc32 && f32_takes_tensor_cores(h, N, T, H, W)) s = forward_tc(h, x, cache, out, new_cache, N, T, H, W, st);
    else s = forward_simt(h, x, cache, out, new_cache, N, T, H, W, st);
    return count(h, s);
}

ccv3d_status ccv3d_forward(ccv3d_handle* h, const void* x, const void* cache, void* out, void* new_cache, int32_t N,
                           int32_t T, int32_t H, int32_t W, void* stream) {
    if (!h) return CCV3D_ERR_INVALID_ARG;
    return ccv3d_forward_ex(h, x, cache, cache ? hist_len(h->d) : 0, out, new_cache, N, T, H, W, stream);
}

ccv3d_status ccv3d_forward_static(ccv3d_handle* h, const void* x, const void* cache, void* out, void* new_cache,
                                  int32_t N, int32_t T, int32_t H, int32_t W, void* stream) {
    if (!h) return CCV3D_ERR_INVALID_ARG;
    h->ctr.calls++;
    h->call_cf = cache ? hist_len(h->d) : 0;
    ccv3d_status s = check_forward_args(h, x, cache, out, new_cache, N, T, H, W, true);
    if (s != CCV3D_OK) return count(h, s);
    if (!on_handle_device(h)) return count(h, CCV3D_ERR_INVALID_ARG);
    if (!h->use_tc) return count(h, CCV3D_ERR_UNSUPPORTED);   // the FP32-FMA route has no scratch to replace
    if (!standard_geom(h->d)) return count(h, CCV3D_ERR_UNSUPPORTED);   // unit stride and dilation, size-preserving padding only
    return count(h, forward_tc_static(h, x, cache, out, new_cache, N, T, H, W, (cudaStream_t)stream));
}

// Host entry point, pipelined frame by frame (standard BF16 tensor-core layers whose channels fit a frame ring).
// Frame t of x is a strided 2-D copy (one row per (n, channel) plane) into a dense one-frame device buffer on an
// upload stream; on the caller's stream it is moved into a frame ring and convolved as a one-frame chunk (history =
// the ring, exactly the streaming form of the operator, so the result is bit for bit that of one T-frame call);
// the output frame goes back with another strided 2-D copy on a download stream.  Three buffers of each kind rotate,
// so that upload, compute and download of different frames overlap: the call takes about as long as the slower of
// the two PCIe directions instead of their sum.
static ccv3d_status forward_host_pipelined(ccv3d_handle* h, const void* x_host, const void* cache_host, void* out_host,
                                    void* new_cache_host, int N, int T, int H, int W, cudaStream_t st) {
    const ccv3d_desc& d = h->d;
    const int tc = hist_len(d);
    constexpr int NBUF = 3;
    const uint64_t HWb = (uint64_t)H * W * 2;
    const uint64_t xf = (uint64_t)N * d.cin * HWb, of = (uint64_t)N * d.cout * HWb;      // one frame of x / of out
    ccv3d_ring ring;
    ring.N = N; ring.C = d.cin; ring.F = tc + 1; ring.H = H; ring.W = W; ring.KB = h->plan.KB;
    ccv3d_status s;
    if ((s = grow(&h->hx, &h->hx_b, NBUF * xf)) != CCV3D_OK) return s;
    if ((s = grow(&h->ho, &h->ho_b, NBUF * of)) != CCV3D_OK) return s;
    if ((s = grow(&h->hc, &h->hc_b, (uint64_t)ring.F * xf)) != CCV3D_OK) return s;
    if (tc && new_cache_host && (s = grow(&h->hn, &h->hn_b, (uint64_t)tc * xf)) != CCV3D_OK) return s;
    ring.base = h->hc;
    if (!h->hp_ready) {
        for (int k = 0; k < 4; ++k)
            for (int b = 0; b < NBUF; ++b)
                if (cudaEventCreateWithFlags(&h->hp_ev[k][b], cudaEventDisableTiming) != cudaSuccess) return cuda_fail();
        h->hp_ready = true;
    }
    cudaStream_t s_up = h->side[0], s_down = h->side[1];
    if (cudaEventRecord(h->ev_fork, st) != cudaSuccess) return cuda_fail();
    if (cudaStreamWaitEvent(s_up, h->ev_fork, 0) != cudaSuccess || cudaStreamWaitEvent(s_down, h->ev_fork, 0) != cudaSuccess)
        return cuda_fail();
    if (!cache_host && tc && cudaMemsetAsync(ring.base, 0, (size_t)ring.F * xf, st) != cudaSuccess) return cuda_fail();

    const int pre = (cache_host && tc) ? tc : 0;           // history frames uploaded before the first frame of x
    const bool nc_early = tc && new_cache_host && tc < NBUF && pre + T >= tc;
    int slot = 0, seen = 0;                                // ring slot of the next frame; frames in the ring so far
    for (int i = 0; i < pre + T; ++i) {
        const int b = i % NBUF;
        const bool is_x = i >= pre;
        const int t = is_x ? i - pre : i;
        char* xin = (char*)h->hx + (size_t)b * xf;
        // upload: wait until the ring load that last read this buffer is done
        if (i >= NBUF && cudaStreamWaitEvent(s_up, h->hp_ev[1][b], 0) != cudaSuccess) return cuda_fail();
        const char* src = is_x ? (const char*)x_host + (size_t)t * HWb : (const char*)cache_host + (size_t)t * HWb;
        const size_t spitch = (size_t)(is_x ? T : tc) * HWb;
        if (cudaMemcpy2DAsync(xin, HWb, src, spitch, HWb, (size_t)N * d.cin, cudaMemcpyHostToDevice, s_up) != cudaSuccess)
            return cuda_fail();
        if (cudaEventRecord(h->hp_ev[0][b], s_up) != cudaSuccess) return cuda_fail();
        // cache update: the last tc frames of the stream go straight back from their upload buffers (bit copies),
        // early, while the download stream has nothing else to do.  (tc < NBUF: these buffers are not reused in
        // this call; the next call starts after the download stream has been joined.)
        if (nc_early && i >= pre + T - tc) {
            const int j = i - (pre + T - tc);
            if (cudaStreamWaitEvent(s_down, h->hp_ev[0][b], 0) != cudaSuccess) return cuda_fail();
            if (cudaMemcpy2DAsync((char*)new_cache_host + (size_t)j * HWb, (size_t)tc * HWb, xin, HWb, HWb, (size_t)N * d.cin,
                                  cudaMemcpyDeviceToHost, s_down) != cudaSuccess)
                return cuda_fail();
        }
        // compute
        if (cudaStreamWaitEvent(st, h->hp_ev[0][b], 0) != cudaSuccess) return cuda_fail();
        if ((s = ccv3d_ring_load(&ring, slot, xin, 1, st)) != CCV3D_OK) return s;
        h->ctr.kernel_launches++;
        if (cudaEventRecord(h->hp_ev[1][b], st) != cudaSuccess) return cuda_fail();
        if (is_x) {
            const int ob = t % NBUF;
            char* oout = (char*)h->ho + (size_t)ob * of;
            if (t >= NBUF && cudaStreamWaitEvent(st, h->hp_ev[3][ob], 0) != cudaSuccess) return cuda_fail();
            const int hist = seen < tc ? seen : tc;
            if ((s = forward_ring(h, &ring, slot, hist, nullptr, 0, nullptr, 0, oout, 1, st)) != CCV3D_OK) return s;
            if (cudaEventRecord(h->hp_ev[2][ob], st) != cudaSuccess) return cuda_fail();
            // download
            if (cudaStreamWaitEvent(s_down, h->hp_ev[2][ob], 0) != cudaSuccess) return cuda_fail();
            if (cudaMemcpy2DAsync((char*)out_host + (size_t)t * HWb, (size_t)T * HWb, oout, HWb, HWb, (size_t)N * d.cout,
                                  cudaMemcpyDeviceToHost, s_down) != cudaSuccess)
                return cuda_fail();
            if (cudaEventRecord(h->hp_ev[3][ob], s_down) != cudaSuccess) return cuda_fail();
        }
        slot = (slot + 1) % ring.F;
        ++seen;
    }
    if (tc && new_cache_host && !nc_early) {
        // the last tc frames of [cache ; x] are the tc slots before `slot` (zeros where the stream had no history)
        if ((s = ccv3d_ring_store(&ring, (slot + ring.F - tc) % ring.F, h->hn, tc, st)) != CCV3D_OK) return s;
        h->ctr.kernel_launches++;
        if (cudaMemcpyAsync(new_cache_host, h->hn, (size_t)tc * xf, cudaMemcpyDeviceToHost, st) != cudaSuccess) return cuda_fail();
    }
    if (cudaEventRecord(h->ev_join[0], s_down) != cudaSuccess || cudaStreamWaitEvent(st, h->ev_join[0], 0) != cudaSuccess)
        return cuda_fail();
    if (cudaEventRecord(h->ev_join[1], s_up) != cudaSuccess || cudaStreamWaitEvent(st, h->ev_join[1], 0) != cudaSuccess)
        return cuda_fail();
    h->ctr.tcgen05_bf16++;
    return CCV3D_OK;
}

static bool host_pipeline_eligible(const ccv3d_handle* h, int T, int H, int W) {
    const ccv3d_desc& d = h->d;
    if (!h->use_tc || !standard_geom(d) || d.out_dtype != CCV3D_BF16 || (d.flags & CCV3D_FLAG_TC_PER_TAP_A)) return false;
    if (!h->side[0] || d.cin % h->plan.KB) return false;
    return (uint64_t)H * W * (d.cin + d.cout) * 2 >= (4u << 20) && T >= 2;      // a few MB per frame, or the copies are latency
}

ccv3d_status ccv3d_forward_host(ccv3d_handle* h, const void* x_host, const void* cache_host, void* out_host,
                                void* new_cache_host, int32_t N, int32_t T, int32_t H, int32_t W, void* stream) {
    if (!h) return CCV3D_ERR_INVALID_ARG;
    h->call_cf = cache_host ? hist_len(h->d) : 0;
    ccv3d_status s = check_forward_args(h, x_host, cache_host, out_host, new_cache_host, N, T, H, W, false);
    if (s != CCV3D_OK) {
        h->ctr.calls++;
        return count(h, s);
    }
    if (host_pipeline_eligible(h, T, H, W)) {
        h->ctr.calls++;
        if (!on_handle_device(h)) return count(h, CCV3D_ERR_INVALID_ARG);
        s = forward_host_pipelined(h, x_host, cache_host, out_host, new_cache_host, N, T, H, W, (cudaStream_t)stream);
        if (s != CCV3D_OK) return count(h, s);
        if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return count(h, cuda_fail());
        count(h, CCV3D_OK);
        return ccv3d_device_status(h, nullptr);
    }
    const ccv3d_desc& d = h->d;
    const int tc = hist_len(d);
    const uint64_t px = (uint64_t)N * H * W;
    const uint64_t xb = px * d.cin * T * esize(d.dtype), cb = px * d.cin * tc * esize(d.dtype);
    const uint64_t ob = (uint64_t)N * out_h(d, H) * out_w(d, W) * d.cout * out_t(d, T) * esize(d.out_dtype);
    cudaStream_t st = (cudaStream_t)stream;
    const bool has_c = tc && cache_host, has_n = tc && new_cache_host;
    if ((s = grow(&h->hx, &h->hx_b, xb)) != CCV3D_OK) return s;
    if ((s = grow(&h->ho, &h->ho_b, ob)) != CCV3D_OK) return s;
    if (has_c && (s = grow(&h->hc, &h->hc_b, cb)) != CCV3D_OK) return s;
    if (has_n && (s = grow(&h->hn, &h->hn_b, cb)) != CCV3D_OK) return s;
    if (cudaMemcpyAsync(h->hx, x_host, xb, cudaMemcpyHostToDevice, st) != cudaSuccess) return cuda_fail();
    if (has_c && cudaMemcpyAsync(h->hc, cache_host, cb, cudaMemcpyHostToDevice, st) != cudaSuccess) return cuda_fail();
    s = ccv3d_forward(h, h->hx, has_c ? h->hc : nullptr, h->ho, has_n ? h->hn : nullptr, N, T, H, W, stream);
    if (s != CCV3D_OK) return s;
    if (cudaMemcpyAsync(out_host, h->ho, ob, cudaMemcpyDeviceToHost, st) != cudaSuccess) return cuda_fail();
    if (has_n && cudaMemcpyAsync(new_cache_host, h->hn, cb, cudaMemcpyDeviceToHost, st) != cudaSuccess) return cuda_fail();
    if (cudaStreamSynchronize(st) != cudaSuccess) return cuda_fail();
    return ccv3d_device_status(h, nullptr);
}

ccv3d_status ccv3d_profile_enable(ccv3d_handle* h, int32_t enable) {
    if (!h) return CCV3D_ERR_INVALID_ARG;
    if (enable && !h->prof_ev) {
        h->prof_ev = new (std::nothrow) cudaEvent_t[3 * PROF_SLOTS];
        if (!h->prof_ev) return CCV3D_ERR_NOMEM;
        for (int i = 0; i < 3 * PROF_SLOTS; ++i)
            if (cudaEventCreate(&h->prof_ev[i]) != cudaSuccess) {
                for (int j = 0; j < i; ++j) cudaEventDestroy(h->prof_ev[j]);
                delete[] h->prof_ev;
                h->prof_ev = nullptr;
                return cuda_fail();
            }
    }
    h->prof_on = enable ? 1 : 0;
    h->prof_n = 0;
    return CCV3D_OK;
}

ccv3d_status ccv3d_profile_read(ccv3d_handle* h, double* stage_ms_host, double* conv_ms_host, int64_t* calls_host) {
    if (!h || !stage_ms_host || !conv_ms_host || !calls_host) return CCV3D_ERR_INVALID_ARG;
    double a = 0.0, b = 0.0;
    const int64_t n = h->prof_n < PROF_SLOTS ? h->prof_n : PROF_SLOTS;
    for (int64_t i = 0; i < n && h->prof_ev; ++i) {
        float t0 = 0.f, t1 = 0.f;
        if (cudaEventElapsedTime(&t0, h->prof_ev[3 * i], h->prof_ev[3 * i + 1]) != cudaSuccess ||
            cudaEventElapsedTime(&t1, h->prof_ev[3 * i + 1], h->prof_ev[3 * i + 2]) != cudaSuccess)
            return cuda_fail();
        a += t0;
        b += t1;
    }
    *stage_ms_host = a;
    *conv_ms_host = b;
    *calls_host = n;
    h->prof_n = 0;
    return CCV3D_OK;
}

ccv3d_status ccv3d_get_counters(const ccv3d_handle* h, ccv3d_counters* out_host) {
    if (!h || !out_host) return CCV3D_ERR_INVALID_ARG;
    *out_host = h->ctr;
    return CCV3D_OK;
}

ccv3d_status ccv3d_device_status(ccv3d_handle* h, uint32_t* detail_host) {
    if (!h) return CCV3D_ERR_INVALID_ARG;
    unsigned int word = 0;
    if (cudaMemcpy(&word, h->status, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) return cuda_fail();
    if (detail_host) *detail_host = word;
    if (word == 0) return CCV3D_OK;
    cudaMemset(h->status, 0, sizeof(word));
    h->ctr.device_timeout++;
    return CCV3D_ERR_DEVICE_TIMEOUT;
}

ccv3d_status ccv3d_selftest_wait_timeout(ccv3d_handle* h, int32_t limit_ms, void* stream) {
    if (!h || limit_ms < 1 || limit_ms > 1000) return CCV3D_ERR_INVALID_ARG;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, h->device) != cudaSuccess) return cuda_fail();
    wait_timeout_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(h->status, (long long)prop.clockRate * limit_ms);
    if (cudaGetLastError() != cudaSuccess) return cuda_fail();
    h->ctr.kernel_launches++;
    return CCV3D_OK;
}

ccv3d_status ccv3d_add_bf16(const void* a, const void* b, void* y, int64_t n, void* stream) {
    if (!a || !b || !y || n < 0) return CCV3D_ERR_INVALID_ARG;
    if (n == 0) return CCV3D_OK;
    const bool vec = (n % 8 == 0) && !(((uintptr_t)a | (uintptr_t)b | (uintptr_t)y) & 15u);
    const int64_t work = vec ? n / 8 : n;
    const int64_t blocks = (work + 255) / 256;
    const unsigned grid = (unsigned)(blocks > 148 * 16 ? 148 * 16 : blocks);
    if (vec)
        add_bf16_vec_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>((const uint4*)a, (const uint4*)b, (uint4*)y, work);
    else
        add_bf16_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)a, (const __nv_bfloat16*)b,
                                                               (__nv_bfloat16*)y, n);
    return cudaGetLastError() == cudaSuccess ? CCV3D_OK : cuda_fail();
}

ccv3d_status ccv3d_upsample_bf16(const void* x, void* y, int32_t N, int32_t C, int32_t T, int32_t H, int32_t W,
                                 int32_t rt, void* stream) {
    if (!x || !y || N < 1 || C < 1 || T < 1 || H < 1 || W < 1 || rt < 1) return CCV3D_ERR_INVALID_ARG;
    const bool vec = (W % 4 == 0) && !(((uintptr_t)x | (uintptr_t)y) & 15u);
    const int64_t work = vec ? (int64_t)N * C * T * H * (W / 4) : (int64_t)N * C * T * rt * 4 * H * W;
    const int64_t blocks = (work + 255) / 256;
    const unsigned grid = (unsigned)(blocks > 148 * 16 ? 148 * 16 : blocks);
    if (vec)
        upsample_bf16_vec_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>((const uint2*)x, (uint4*)y, (int64_t)N * C, T, H,
                                                                       W, rt);
    else
        upsample_bf16_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)x, (__nv_bfloat16*)y,
                                                                   (int64_t)N * C, T, H, W, rt);
    return cudaGetLastError() == cudaSuccess ? CCV3D_OK : cuda_fail();
}

int32_t ccv3d_ring_kb(int32_t C) { return C < 1 ? 0 : (C % 64 == 0 ? 64 : (C % 32 == 0 ? 32 : 0)); }

uint64_t ccv3d_ring_bytes(const ccv3d_ring* r) {
    if (!r || r->N < 1 || r->C < 1 || r->F < 1 || r->H < 1 || r->W < 1) return 0;
    if ((r->KB != 64 && r->KB != 32) || r->C % r->KB) return 0;
    return ring_bytes_of(r);
}

ccv3d_status ccv3d_ring_load(const ccv3d_ring* r, int32_t slot0, const void* x, int32_t T, void* stream) {
    if (!ring_valid(r) || !x || T < 1 || T > r->F || slot0 < 0 || slot0 >= r->F) return CCV3D_ERR_INVALID_ARG;
    if (((uintptr_t)r->base | (uintptr_t)x) & 15u) return CCV3D_ERR_ALIGNMENT;
    if (overlap(r->base, ring_bytes_of(r), x, (uint64_t)r->N * r->C * T * r->H * r->W * 2)) return CCV3D_ERR_ALIAS;
    StageParams sp;
    memset(&sp, 0, sizeof(sp));
    sp.x = (const __nv_bfloat16*)x;
    sp.zs = (__nv_bfloat16*)r->base;
    sp.N = r->N; sp.Cin = r->C; sp.T = T; sp.H = r->H; sp.W = r->W; sp.tc = 0; sp.CB = r->C / r->KB;
    sp.ring_F = r->F; sp.ring_f0 = slot0;
    const bool vec = (r->W % 8 == 0);
    dim3 grid((r->W + STG_PX - 1) / STG_PX, r->H, (unsigned)((int64_t)r->N * T * sp.CB));
    if (r->H > 65535 || (int64_t)r->N * T * sp.CB > 65535) return CCV3D_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    if (r->KB == 64) {
        if (vec) stage_frames_kernel<64, true><<<grid, 256, 0, st>>>(sp);
        else stage_frames_kernel<64, false><<<grid, 256, 0, st>>>(sp);
    } else {
        if (vec) stage_frames_kernel<32, true><<<grid, 128, 0, st>>>(sp);
        else stage_frames_kernel<32, false><<<grid, 128, 0, st>>>(sp);
    }
    return cudaGetLastError() == cudaSuccess ? CCV3D_OK : cuda_fail();
}

ccv3d_status ccv3d_ring_store(const ccv3d_ring* r, int32_t slot0, void* y, int32_t T, void* stream) {
    if (!ring_valid(r) || !y || T < 1 || T > r->F || slot0 < 0 || slot0 >= r->F) return CCV3D_ERR_INVALID_ARG;
    if (((uintptr_t)r->base | (uintptr_t)y) & 15u) return CCV3D_ERR_ALIGNMENT;
    if (overlap(r->base, ring_bytes_of(r), y, (uint64_t)r->N * r->C * T * r->H * r->W * 2)) return CCV3D_ERR_ALIAS;
    const int CB = r->C / r->KB;
    if (r->H > 65535 || (int64_t)r->N * T * CB > 65535) return CCV3D_ERR_UNSUPPORTED;
    dim3 grid((r->W + STG_PX - 1) / STG_PX, r->H, (unsigned)((int64_t)r->N * T * CB));
    cudaStream_t st = (cudaStream_t)stream;
    if (r->KB == 64) ring_store_kernel<64><<<grid, 256, 0, st>>>(ring_geom(r), slot0, T, r->C, (__nv_bfloat16*)y);
    else ring_store_kernel<32><<<grid, 256, 0, st>>>(ring_geom(r), slot0, T, r->C, (__nv_bfloat16*)y);
    return cudaGetLastError() == cudaSuccess ? CCV3D_OK : cuda_fail();
}

ccv3d_status ccv3d_upsample_ring(const ccv3d_ring* in, int32_t in_slot0, const ccv3d_ring* out, int32_t out_slot0,
                                 int32_t T, int32_t rt, void* stream) {
    if (!ring_valid(in) || !ring_valid(out) || T < 1 || rt < 1 || T > in->F || (int64_t)T * rt > out->F) return CCV3D_ERR_INVALID_ARG;
    if (in_slot0 < 0 || in_slot0 >= in->F || out_slot0 < 0 || out_slot0 >= out->F) return CCV3D_ERR_INVALID_ARG;
    if (out->N != in->N || out->C != in->C || out->KB != in->KB || out->H != 2 * in->H || out->W != 2 * in->W)
        return CCV3D_ERR_INVALID_ARG;
    if (((uintptr_t)in->base | (uintptr_t)out->base) & 15u) return CCV3D_ERR_ALIGNMENT;
    if (overlap(in->base, ring_bytes_of(in), out->base, ring_bytes_of(out))) return CCV3D_ERR_ALIAS;
    const int64_t total = (int64_t)in->N * T * (in->C / 8) * in->H * in->W;
    const int64_t blocks = (total + 255) / 256;
    ring_upsample_kernel<<<(unsigned)(blocks < 65536 ? blocks : 65536), 256, 0, (cudaStream_t)stream>>>(
        ring_geom(in), in_slot0, ring_geom(out), out_slot0, T, rt);
    return cudaGetLastError() == cudaSuccess ? CCV3D_OK : cuda_fail();
}

ccv3d_status ccv3d_forward_ring_up(ccv3d_handle* h, const ccv3d_ring* in, int32_t x_slot, int32_t hist_frames,
                                   const ccv3d_ring* res, int32_t res_slot, const ccv3d_ring* out_ring, int32_t out_slot,
                                   int32_t rt, int32_t T, void* stream) {
    if (!h) return CCV3D_ERR_INVALID_ARG;
    h->ctr.calls++;
    if (rt < 1 || !out_ring) return count(h, CCV3D_ERR_INVALID_ARG);
    if (!on_handle_device(h)) return count(h, CCV3D_ERR_INVALID_ARG);
    return count(h, forward_ring(h, in, x_slot, hist_frames, res, res_slot, out_ring, out_slot, nullptr, T,
                                 (cudaStream_t)stream, rt));
}

ccv3d_status ccv3d_forward_ring(ccv3d_handle* h, const ccv3d_ring* in, int32_t x_slot, int32_t hist_frames,
                                const ccv3d_ring* res, int32_t res_slot, const ccv3d_ring* out_ring,
                                int32_t out_slot, void* out_ncthw, int32_t T, void* stream) {
    if (!h) return CCV3D_ERR_INVALID_ARG;
    h->ctr.calls++;
    if (!on_handle_device(h)) return count(h, CCV3D_ERR_INVALID_ARG);
    return count(h, forward_ring(h, in, x_slot, hist_frames, res, res_slot, out_ring, out_slot, out_ncthw, T,
                                 (cudaStream_t)stream));
}

}  // extern "C"
