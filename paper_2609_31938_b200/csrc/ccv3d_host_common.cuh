// Host helpers: geometry rules, validation, per-layer plans, pipeline sizing, tensor maps of the staged copy.
// Part of the single translation unit ccv3d_api.cu (included inside its anonymous namespace).
#pragma once

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
// whole_kernel > 0: all kh*kw taps in one weight stage when that fits in 28 KB (narrow tiles of 32-channel blocks on CTA
// pairs: a stage of one kernel row would carry only 6 MMAs per issuing warp).
ccv3d_status size_pipeline(TcParams* p, size_t budget, bool per_tap, int kw, int whole_kernel = 0) {
    p->TPB = (!per_tap && (size_t)p->b_tap * kw <= 40960) ? kw : 1;
    if (whole_kernel > 0 && !per_tap && (size_t)p->b_tap * whole_kernel <= 28672) p->TPB = whole_kernel;
    int SA = per_tap ? 3 : 2;
    for (;;) {
        p->b_slot = (uint32_t)align_up((uint64_t)p->b_tap * p->TPB, 1024);
        if ((size_t)SA * p->a_slot + 3 * (size_t)p->b_slot <= budget) break;
        if (p->TPB > kw && kw > 1) { p->TPB = kw; continue; }
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

// Every entry point that counts as a call starts here ...
void begin_call(ccv3d_handle* h, const char* name, int N, int T, int H, int W) {
    h->ctr.calls++;
    h->call_name = name;
    h->call_dims[0] = N; h->call_dims[1] = T; h->call_dims[2] = H; h->call_dims[3] = W;
}

// ... and ends here: the status is counted (Algorithm 1's route counters) and, with CCV3D_LOG=1, reported.
ccv3d_status count(ccv3d_handle* h, ccv3d_status s) {
    if (h->log)
        fprintf(stderr, "ccv3d %p %s N=%d T=%d H=%d W=%d %d->%d k=%dx%dx%d: %s (calls %llu tcgen05 %llu 3xtf32 %llu 1x1x1 %llu fma %llu launches %llu)\n",
                (void*)h, h->call_name ? h->call_name : "?", h->call_dims[0], h->call_dims[1], h->call_dims[2], h->call_dims[3],
                h->d.cin, h->d.cout, h->d.kt, h->d.kh, h->d.kw, ccv3d_status_string(s), (unsigned long long)h->ctr.calls,
                (unsigned long long)h->ctr.tcgen05_bf16, (unsigned long long)h->ctr.tcgen05_f32,
                (unsigned long long)h->ctr.pointwise, (unsigned long long)h->ctr.simt,
                (unsigned long long)h->ctr.kernel_launches);
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
// phases > 1: H and W are the extents of one phase image and every channel block holds `phases` of them.
ccv3d_status encode_act_map(ccv3d_handle* h, int N, int T, int H, int W, int BW, int BH, int es_w = 1, int es_h = 1,
                            int phases = 1) {
    const TcPlan& pl = h->plan;
    const int F = hist_len(h->d) + T;
    const bool f32 = h->d.dtype == CCV3D_F32;             // rows of 32 FP32 channels; two blocks (value, remainder) per real block
    const uint64_t rowb = (uint64_t)pl.KB * 2;
    const int inner = f32 ? 32 : pl.KB, blocks = (f32 ? 2 * pl.CB : pl.CB) * phases;
    cuuint64_t dims[5] = {(cuuint64_t)inner, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)blocks, (cuuint64_t)N * F};
    cuuint64_t strides[4] = {rowb, rowb * W, rowb * W * H, rowb * W * H * blocks};
    cuuint32_t box[5] = {(cuuint32_t)inner, (cuuint32_t)(BW * es_w), (cuuint32_t)(BH * es_h), 1, 1};
    cuuint32_t es[5] = {1, (cuuint32_t)es_w, (cuuint32_t)es_h, 1, 1};
    if (box[1] > 256 || box[2] > 256) return CCV3D_ERR_UNSUPPORTED;
    CUresult r = h->encode(&h->tm_a, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, h->ws_cur, dims, strides, box, es,
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

// Raw view of an NCTHW tensor [N, C, Fr, H, W] (BF16) for the stager warps of the cooperative schedule: boxes of
// [32 channels][64 pixels] of one image row, 128-byte swizzle.  Needs W % 8 == 0 and a 16-byte aligned base.
ccv3d_status encode_raw_map(ccv3d_handle* h, CUtensorMap* tm, const void* base, int N, int C, int Fr, int H, int W) {
    const uint64_t row = 2ull * W;
    cuuint64_t dims[5] = {(cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)Fr, (cuuint64_t)C, (cuuint64_t)N};
    cuuint64_t strides[4] = {row, row * H, row * H * Fr, row * H * Fr * C};
    cuuint32_t box[5] = {64, 1, 1, 32, 1};
    cuuint32_t es[5] = {1, 1, 1, 1, 1};
    CUresult r = h->encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, es,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? CCV3D_OK : CCV3D_ERR_CUDA;
}

// The three raw views of a cooperative call (absent tensors get a copy of x's view: never used for a transfer).
ccv3d_status encode_stager_maps(ccv3d_handle* h, const void* x, const void* cache, int cf, void* new_cache, int N, int T, int H,
                                int W) {
    const int tc = hist_len(h->d);
    ccv3d_status s = encode_raw_map(h, &h->stg_maps.x, x, N, h->d.cin, T, H, W);
    if (s == CCV3D_OK && cf) s = encode_raw_map(h, &h->stg_maps.cache, cache, N, h->d.cin, cf, H, W);
    if (s == CCV3D_OK && new_cache && tc) s = encode_raw_map(h, &h->stg_maps.nc, new_cache, N, h->d.cin, tc, H, W);
    if (s != CCV3D_OK) return s;
    if (!cf) h->stg_maps.cache = h->stg_maps.x;
    if (!(new_cache && tc)) h->stg_maps.nc = h->stg_maps.x;
    return CCV3D_OK;
}

// Can the stager warps fetch these tensors by TMA?  16-byte aligned bases, rows of whole 16-byte pieces, strides that fit.
inline bool raw_maps_ok(const ccv3d_handle* h, const void* x, const void* cache, const void* new_cache, int T, int H, int W) {
    const int tc = hist_len(h->d);
    return W % 8 == 0 && ((uintptr_t)x & 15) == 0 && ((uintptr_t)cache & 15) == 0 && ((uintptr_t)new_cache & 15) == 0 &&
           2ull * W * H * (uint64_t)(T > tc ? T : tc) * h->d.cin < (1ull << 40);
}

uint64_t tc_workspace_bytes(const ccv3d_handle* h, int N, int T, int H, int W) {
    const int F = hist_len(h->d) + T;
    if (h->d.dtype == CCV3D_F32) return (uint64_t)N * F * h->plan.cin_pad * H * W * 8;   // values and remainders, FP32
    // (layers with a spatial stride: whole phase images, i.e. extents rounded up to multiples of the stride)
    const int sh = h->d.stride[1], sw = h->d.stride[2];
    return (uint64_t)N * F * h->plan.cin_pad * ((H + sh - 1) / sh * sh) * ((W + sw - 1) / sw * sw) * 2;
}
