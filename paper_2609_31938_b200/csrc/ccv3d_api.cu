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
#include <atomic>
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
    void* workspace;     // staging copy owned by the handle (allocated on demand) ...
    uint64_t workspace_bytes;
    void* ext_ws;        // ... or lent by the caller (ccv3d_set_workspace): then nothing is ever allocated by a forward call
    uint64_t ext_ws_bytes;
    void* ws_cur;        // the one the call in progress uses
    // host-entry staging (device buffers)
    void* hx; void* hc; void* ho; void* hn;
    uint64_t hx_b, hc_b, ho_b, hn_b;
    cudaEvent_t hp_ev[5][3];   // pipelined host entry: per buffer {uploaded, input buffer free, computed, downloaded, cache piece read}
    bool hp_ready;
    EncodeTiledFn encode;
    CUtensorMap tm_a;
    ShapeKey tm_a_key;
    CUtensorMap tm_o;
    StagerMaps stg_maps; // cooperative staging: raw NCTHW views of x, the cache and the new cache (per call)
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
    int coop_launch;     // 1: cooperative-staging kernels are launched with the cooperative attribute
    int log;             // CCV3D_LOG: one line per call on stderr (entry point, shape, status, route counters)
    const char* call_name;   // entry point and shape of the call in progress, for that line
    int call_dims[4];
    bool hs_valid;       // host stream (ccv3d_forward_host_stream): the device ring holds the history of hs_geom
    int hs_state[2];     //   ring slot of the next frame, history frames present
    int hs_geom[3];      //   N, H, W of the stream
    int cluster_ok;      // the device launches thread-block clusters (needed for CTA pairs)
    int call_cf;         // history frames held by the cache of the call being served (set by the entry points)
    ccv3d_counters ctr;
};

namespace {

#include "ccv3d_host_common.cuh"
#include "ccv3d_host_tc.cuh"
#include "ccv3d_host_ring.cuh"

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
    // eight output channels per thread amortise the activation loads; a call with fewer threads than that gives the
    // device (configuration 1: 512 pixels x 2 channel groups) runs one channel per thread instead
    const bool thin = gx * ((d.cout + SIMT_CO - 1) / SIMT_CO) < 4LL * h->sm_count;
    const int co_per_thread = thin ? 1 : SIMT_CO;
    dim3 grid((unsigned)gx, (d.cout + co_per_thread - 1) / co_per_thread);
    cudaEvent_t* pev = (h->prof_on && h->prof_ev) ? h->prof_ev + 3 * (h->prof_n % PROF_SLOTS) : nullptr;
    if (pev) { cudaEventRecord(pev[0], st); cudaEventRecord(pev[1], st); }
    if (thin) {
        if (d.dtype == CCV3D_F32) conv3d_direct_kernel<float, float, 1><<<grid, SIMT_THREADS, 0, st>>>(p);
        else if (d.out_dtype == CCV3D_BF16) conv3d_direct_kernel<__nv_bfloat16, __nv_bfloat16, 1><<<grid, SIMT_THREADS, 0, st>>>(p);
        else conv3d_direct_kernel<__nv_bfloat16, float, 1><<<grid, SIMT_THREADS, 0, st>>>(p);
    } else if (d.dtype == CCV3D_F32) conv3d_direct_kernel<float, float><<<grid, SIMT_THREADS, 0, st>>>(p);
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
// K = 5184, 4.7e-5 at K = 10368) and the error depends on the data (inputs of one sign keep the accumulator at full
// size along the whole chain), so the automatic route stops at K = 8192 - a third of the 1e-4 tolerance by that model -
// and longer layers stay on the FP32-FMA kernel unless the flag insists.
constexpr int64_t F32_TENSOR_MAX_K = 8192;
bool f32_takes_tensor_cores(const ccv3d_handle* h, int N, int T, int H, int W) {
    const ccv3d_desc& d = h->d;
    if (d.flags & CCV3D_FLAG_F32_TENSOR) return true;
    const int64_t K = (int64_t)d.cin * d.kt * d.kh * d.kw;
    if (K > F32_TENSOR_MAX_K) return false;
    // Large calls for the throughput; small ones whenever the FMA kernel's serial walk over K (one thread per output
    // element, ~0.2 us per tap row) would outlast the two short launches of this route (~20 us together):
    // configuration 1 (K = 432) runs 21 us here against 80 us there.
    const double flops = 2.0 * N * out_t(d, T) * out_h(d, H) * out_w(d, W) * d.cout * K;
    return flops >= 2.0e8 || K >= 256;
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
    h->log = (getenv("CCV3D_LOG") && atoi(getenv("CCV3D_LOG")) > 0) ? 1 : 0;
    // a kernel-replaying profiler (it announces itself through NV_COMPUTE_PROFILER_PERFWORKS_DIR) refuses
    // cooperative launches of clusters: ordinary launches there, on a device the profiled process has to itself
    h->coop_launch = (getenv("CCV3D_NO_COOP_LAUNCH") || getenv("NV_COMPUTE_PROFILER_PERFWORKS_DIR")) ? 0 : 1;
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
        for (int k = 0; k < 5; ++k)
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

ccv3d_status ccv3d_set_workspace(ccv3d_handle* h, void* ws_dev, uint64_t bytes) {
    if (!h) return CCV3D_ERR_INVALID_ARG;
    if (!ws_dev || bytes == 0) {                            // back to a workspace the handle allocates on demand
        h->ext_ws = nullptr;
        h->ext_ws_bytes = 0;
        return CCV3D_OK;
    }
    if ((uintptr_t)ws_dev & 255u) return CCV3D_ERR_ALIGNMENT;
    h->ext_ws = ws_dev;
    h->ext_ws_bytes = bytes;
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
    begin_call(h, "ccv3d_forward_ex", N, T, H, W);
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
    begin_call(h, "ccv3d_forward_static", N, T, H, W);
    h->call_cf = cache ? hist_len(h->d) : 0;
    ccv3d_status s = check_forward_args(h, x, cache, out, new_cache, N, T, H, W, true);
    if (s != CCV3D_OK) return count(h, s);
    if (!on_handle_device(h)) return count(h, CCV3D_ERR_INVALID_ARG);
    if (!h->use_tc) return count(h, CCV3D_ERR_UNSUPPORTED);   // the FP32-FMA route has no scratch to replace
    if (!standard_geom(h->d)) return count(h, CCV3D_ERR_UNSUPPORTED);   // unit stride and dilation, size-preserving padding only
    return count(h, forward_tc_static(h, x, cache, out, new_cache, N, T, H, W, (cudaStream_t)stream));
}

// Host entry point, pipelined (standard BF16 tensor-core layers whose channels fit a frame ring).
// The image is cut into bands of rows, and a band into frames.  Band rows [h0, h1) of frame t of x, with the p_h halo
// rows above and below that exist, are a strided 2-D copy (one piece per (n, channel) plane) into a dense device buffer
// on an upload stream; on the caller's stream that slab frame is moved into a frame ring of slab height and convolved as
// a one-frame chunk (history = the ring, exactly the streaming form of the operator); the band's rows of the output
// frame go back with another strided 2-D copy on a download stream.  A slab is convolved as an image of its own: its
// first and last output rows see zero padding where the neighbouring band's rows belong and are not downloaded, every
// other row sees what it sees in the whole image, in the same order of accumulation, so the result is bit for bit that
// of one call on the whole image.  Three buffers of each kind rotate, so that upload, compute and download of different
// pieces overlap: the call takes about as long as the slower of the two PCIe directions - plus the time until the first
// output piece exists, which is why the pieces are bands and not whole frames (kt-1 + 1 whole frames are a third of
// configuration 3's upload).
// stream_state != nullptr: streaming form - {ring slot of the next frame, frames seen so far} carried in the handle from
// call to call; the history is whatever the previous call left in the rings (cache_host and new_cache_host are null).
static int host_bands(const ccv3d_handle* h, int N, int H, int W) {
    // pieces of at least 16 MB on the larger side (PCIe efficiency) and bands of at least 32 rows; at most 8 bands
    const uint64_t frame = (uint64_t)N * (h->d.cin > h->d.cout ? h->d.cin : h->d.cout) * H * W * 2;
    int nb = (int)(frame / (16u << 20));
    if (nb > H / 32) nb = H / 32;
    if (nb > 8) nb = 8;
    return nb < 1 ? 1 : nb;
}

static ccv3d_status forward_host_pipelined(ccv3d_handle* h, const void* x_host, const void* cache_host, void* out_host,
                                    void* new_cache_host, int N, int T, int H, int W, cudaStream_t st,
                                    int* stream_state = nullptr) {
    const ccv3d_desc& d = h->d;
    const int tc = hist_len(d);
    const int ph = (d.kh - 1) / 2;                         // (standard geometry: size-preserving padding)
    constexpr int NBUF = 3;
    const int nbands = host_bands(h, N, H, W);
    const int Hs_max = (H + nbands - 1) / nbands + 2 * ph; // rows of the tallest slab
    const uint64_t Wb = (uint64_t)W * 2;                   // bytes of an image row
    const uint64_t HWb = (uint64_t)H * Wb;                 // bytes of a plane of the whole image
    const uint64_t xf = (uint64_t)N * d.cin * Hs_max * Wb, of = (uint64_t)N * d.cout * Hs_max * Wb;   // one slab frame of x / of out
    const int F = tc + 1;
    ccv3d_status s;
    if ((s = grow(&h->hx, &h->hx_b, NBUF * xf)) != CCV3D_OK) return s;
    if ((s = grow(&h->ho, &h->ho_b, NBUF * of)) != CCV3D_OK) return s;
    if ((s = grow(&h->hc, &h->hc_b, (uint64_t)nbands * F * xf)) != CCV3D_OK) return s;
    if (tc && new_cache_host && (s = grow(&h->hn, &h->hn_b, (uint64_t)tc * xf)) != CCV3D_OK) return s;
    if (!h->hp_ready) {
        for (int k = 0; k < 5; ++k)
            for (int b = 0; b < NBUF; ++b)
                if (cudaEventCreateWithFlags(&h->hp_ev[k][b], cudaEventDisableTiming) != cudaSuccess) return cuda_fail();
        h->hp_ready = true;
    }
    cudaStream_t s_up = h->side[0], s_down = h->side[1];
    if (cudaEventRecord(h->ev_fork, st) != cudaSuccess) return cuda_fail();
    if (cudaStreamWaitEvent(s_up, h->ev_fork, 0) != cudaSuccess || cudaStreamWaitEvent(s_down, h->ev_fork, 0) != cudaSuccess)
        return cuda_fail();
    if (!stream_state && !cache_host && tc && cudaMemsetAsync(h->hc, 0, (size_t)nbands * F * xf, st) != cudaSuccess)
        return cuda_fail();

    const int pre = (cache_host && tc) ? tc : 0;           // history frames uploaded before the first frame of x
    const bool nc_early = tc && new_cache_host && pre + T >= tc;
    int slot0 = 0, seen0 = 0;                              // ring slot of the next frame; frames in the ring so far
    if (stream_state) { slot0 = stream_state[0]; seen0 = stream_state[1]; }
    int slot = slot0, seen = seen0;
    int g = 0, go = 0;                                     // pieces uploaded / downloaded so far (buffers rotate over all bands)
    bool nc_pending[NBUF] = {false, false, false};         // a cache piece is still being read out of this upload buffer
    for (int band = 0; band < nbands; ++band) {
        const int h0 = (int)((int64_t)H * band / nbands), h1 = (int)((int64_t)H * (band + 1) / nbands);
        const int hs0 = h0 - ph > 0 ? h0 - ph : 0, hs1 = h1 + ph < H ? h1 + ph : H;
        const int Hs = hs1 - hs0, top = h0 - hs0, rows = h1 - h0;
        const uint64_t HWs = (uint64_t)Hs * Wb;            // bytes of a plane of the slab
        ccv3d_ring ring;
        ring.N = N; ring.C = d.cin; ring.F = F; ring.H = Hs; ring.W = W; ring.KB = h->plan.KB;
        ring.base = (char*)h->hc + (size_t)band * F * xf;
        slot = slot0; seen = seen0;
        for (int i = 0; i < pre + T; ++i, ++g) {
            const int b = g % NBUF;
            const bool is_x = i >= pre;
            const int t = is_x ? i - pre : i;
            char* xin = (char*)h->hx + (size_t)b * xf;
            // upload: wait until the ring load (and the cache piece, if any) that last read this buffer is done
            if (g >= NBUF && cudaStreamWaitEvent(s_up, h->hp_ev[1][b], 0) != cudaSuccess) return cuda_fail();
            if (nc_pending[b]) {
                if (cudaStreamWaitEvent(s_up, h->hp_ev[4][b], 0) != cudaSuccess) return cuda_fail();
                nc_pending[b] = false;
            }
            const char* src = (is_x ? (const char*)x_host : (const char*)cache_host) + (size_t)t * HWb + (size_t)hs0 * Wb;
            const size_t spitch = (size_t)(is_x ? T : tc) * HWb;
            if (cudaMemcpy2DAsync(xin, HWs, src, spitch, HWs, (size_t)N * d.cin, cudaMemcpyHostToDevice, s_up) != cudaSuccess)
                return cuda_fail();
            if (cudaEventRecord(h->hp_ev[0][b], s_up) != cudaSuccess) return cuda_fail();
            // cache update: the band's rows of the last tc frames of the stream go straight back from their upload
            // buffers (bit copies), in between the output pieces
            if (nc_early && i >= pre + T - tc) {
                const int j = i - (pre + T - tc);
                if (cudaStreamWaitEvent(s_down, h->hp_ev[0][b], 0) != cudaSuccess) return cuda_fail();
                if (cudaMemcpy2DAsync((char*)new_cache_host + (size_t)j * HWb + (size_t)h0 * Wb, (size_t)tc * HWb,
                                      xin + (size_t)top * Wb, HWs, (size_t)rows * Wb, (size_t)N * d.cin, cudaMemcpyDeviceToHost,
                                      s_down) != cudaSuccess)
                    return cuda_fail();
                if (cudaEventRecord(h->hp_ev[4][b], s_down) != cudaSuccess) return cuda_fail();
                nc_pending[b] = true;
            }
            // compute
            if (cudaStreamWaitEvent(st, h->hp_ev[0][b], 0) != cudaSuccess) return cuda_fail();
            if ((s = ccv3d_ring_load(&ring, slot, xin, 1, st)) != CCV3D_OK) return s;
            h->ctr.kernel_launches++;
            if (cudaEventRecord(h->hp_ev[1][b], st) != cudaSuccess) return cuda_fail();
            if (is_x) {
                const int ob = go % NBUF;
                char* oout = (char*)h->ho + (size_t)ob * of;
                if (go >= NBUF && cudaStreamWaitEvent(st, h->hp_ev[3][ob], 0) != cudaSuccess) return cuda_fail();
                const int hist = seen < tc ? seen : tc;
                if ((s = forward_ring(h, &ring, slot, hist, nullptr, 0, nullptr, 0, oout, 1, st)) != CCV3D_OK) return s;
                if (cudaEventRecord(h->hp_ev[2][ob], st) != cudaSuccess) return cuda_fail();
                // download the band's own rows of the slab's output frame
                if (cudaStreamWaitEvent(s_down, h->hp_ev[2][ob], 0) != cudaSuccess) return cuda_fail();
                if (cudaMemcpy2DAsync((char*)out_host + (size_t)t * HWb + (size_t)h0 * Wb, (size_t)T * HWb, oout + (size_t)top * Wb,
                                      HWs, (size_t)rows * Wb, (size_t)N * d.cout, cudaMemcpyDeviceToHost, s_down) != cudaSuccess)
                    return cuda_fail();
                if (cudaEventRecord(h->hp_ev[3][ob], s_down) != cudaSuccess) return cuda_fail();
                ++go;
            }
            slot = (slot + 1) % F;
            ++seen;
        }
        if (tc && new_cache_host && !nc_early) {
            // (T + history shorter than tc frames.)  The last tc frames of [cache ; x] are the tc slots before `slot`
            // (zeros where the stream had no history): back to NCTHW on the device, then the band's rows to the host
            if ((s = ccv3d_ring_store(&ring, (slot + F - tc) % F, h->hn, tc, st)) != CCV3D_OK) return s;
            h->ctr.kernel_launches++;
            if (cudaMemcpy2DAsync((char*)new_cache_host + (size_t)h0 * Wb, HWb, (char*)h->hn + (size_t)top * Wb, HWs, (size_t)rows * Wb,
                                  (size_t)N * d.cin * tc, cudaMemcpyDeviceToHost, st) != cudaSuccess)
                return cuda_fail();
        }
    }
    if (cudaEventRecord(h->ev_join[0], s_down) != cudaSuccess || cudaStreamWaitEvent(st, h->ev_join[0], 0) != cudaSuccess)
        return cuda_fail();
    if (cudaEventRecord(h->ev_join[1], s_up) != cudaSuccess || cudaStreamWaitEvent(st, h->ev_join[1], 0) != cudaSuccess)
        return cuda_fail();
    if (stream_state) { stream_state[0] = slot; stream_state[1] = seen < tc ? seen : tc; }
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
        begin_call(h, "ccv3d_forward_host", N, T, H, W);
        return count(h, s);
    }
    h->hs_valid = false;                                   // this call reuses the device buffers of a host stream
    if (host_pipeline_eligible(h, T, H, W)) {
        begin_call(h, "ccv3d_forward_host", N, T, H, W);
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

ccv3d_status ccv3d_forward_host_stream(ccv3d_handle* h, const void* x_host, void* out_host, int32_t reset, int32_t N,
                                       int32_t T, int32_t H, int32_t W, void* stream) {
    if (!h) return CCV3D_ERR_INVALID_ARG;
    begin_call(h, "ccv3d_forward_host_stream", N, T, H, W);
    h->call_cf = 0;
    ccv3d_status s = check_forward_args(h, x_host, nullptr, out_host, nullptr, N, T, H, W, false);
    if (s != CCV3D_OK) return count(h, s);
    if (!host_pipeline_eligible(h, 2, H, W)) return count(h, CCV3D_ERR_UNSUPPORTED);
    if (!on_handle_device(h)) return count(h, CCV3D_ERR_INVALID_ARG);
    if (reset || !h->hs_valid || h->hs_geom[0] != N || h->hs_geom[1] != H || h->hs_geom[2] != W) {
        h->hs_state[0] = h->hs_state[1] = 0;               // first chunk: no history (its taps are skipped, nothing is zeroed)
        h->hs_geom[0] = N; h->hs_geom[1] = H; h->hs_geom[2] = W;
    }
    h->hs_valid = false;                                   // stays false if anything below fails
    s = forward_host_pipelined(h, x_host, nullptr, out_host, nullptr, N, T, H, W, (cudaStream_t)stream, h->hs_state);
    if (s != CCV3D_OK) return count(h, s);
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return count(h, cuda_fail());
    s = ccv3d_device_status(h, nullptr);
    h->hs_valid = (s == CCV3D_OK);
    return count(h, s);
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

ccv3d_status ccv3d_rows_copy(void* dst, int32_t dst_H, int32_t dst_row0, const void* src, int32_t src_H,
                             int32_t src_row0, int64_t planes, int32_t rows, int64_t row_bytes, void* stream) {
    if (!dst || planes < 1 || rows < 1 || row_bytes < 1 || dst_row0 < 0 || dst_row0 + rows > dst_H)
        return CCV3D_ERR_INVALID_ARG;
    if (src && (src_row0 < 0 || src_row0 + rows > src_H)) return CCV3D_ERR_INVALID_ARG;
    unsigned char* d = (unsigned char*)dst + (int64_t)dst_row0 * row_bytes;
    const unsigned char* s = src ? (const unsigned char*)src + (int64_t)src_row0 * row_bytes : nullptr;
    const bool vec = row_bytes % 16 == 0 && !(((uintptr_t)d | (uintptr_t)s) & 15u);
    const int64_t unit = vec ? 16 : 1;
    const int64_t chunk = rows * row_bytes / unit, total = planes * chunk;
    const int64_t blocks = (total + 255) / 256;
    const unsigned grid = (unsigned)(blocks > 148 * 16 ? 148 * 16 : blocks);
    const int64_t dp = dst_H * row_bytes / unit, sp = src ? src_H * row_bytes / unit : 0;
    if (vec)
        rows_copy_kernel<uint4><<<grid, 256, 0, (cudaStream_t)stream>>>((uint4*)d, dp, (const uint4*)s, sp, planes, chunk);
    else
        rows_copy_kernel<unsigned char><<<grid, 256, 0, (cudaStream_t)stream>>>(d, dp, s, sp, planes, chunk);
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
    begin_call(h, "ccv3d_forward_ring_up", in ? in->N : 0, T, in ? in->H : 0, in ? in->W : 0);
    if (rt < 1 || !out_ring) return count(h, CCV3D_ERR_INVALID_ARG);
    if (!on_handle_device(h)) return count(h, CCV3D_ERR_INVALID_ARG);
    return count(h, forward_ring(h, in, x_slot, hist_frames, res, res_slot, out_ring, out_slot, nullptr, T,
                                 (cudaStream_t)stream, rt));
}

ccv3d_status ccv3d_forward_ring(ccv3d_handle* h, const ccv3d_ring* in, int32_t x_slot, int32_t hist_frames,
                                const ccv3d_ring* res, int32_t res_slot, const ccv3d_ring* out_ring,
                                int32_t out_slot, void* out_ncthw, int32_t T, void* stream) {
    if (!h) return CCV3D_ERR_INVALID_ARG;
    begin_call(h, "ccv3d_forward_ring", in ? in->N : 0, T, in ? in->H : 0, in ? in->W : 0);
    if (!on_handle_device(h)) return count(h, CCV3D_ERR_INVALID_ARG);
    return count(h, forward_ring(h, in, x_slot, hist_frames, res, res_slot, out_ring, out_slot, out_ncthw, T,
                                 (cudaStream_t)stream));
}

}  // extern "C"
