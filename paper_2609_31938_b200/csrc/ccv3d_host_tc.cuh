// Host side of the tensor-core route through the NCTHW boundary: launchers (single CTAs, CTA pairs, cooperative),
// forward_tc, the fused route, the 1x1x1 streaming kernel, the allocation-free variant.
// Part of the single translation unit ccv3d_api.cu (included inside its anonymous namespace).
#pragma once

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
    cfg.numAttrs = h->coop_launch ? 1 : 0;
    if (cudaLaunchKernelEx(&cfg, kern, h->tm_a, h->tm_a, h->tm_o, p, sp, h->stg_maps) != cudaSuccess) return cuda_fail();
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
    kern<<<grid, TC_THREADS, smem, st>>>(h->tm_a, h->tm_a, h->tm_o, p, nosp, h->stg_maps);
    if (cudaGetLastError() != cudaSuccess) return cuda_fail();
    h->ctr.kernel_launches++;
    return CCV3D_OK;
}

// Launch the staging kernel for image rows [h0, h1) on stream st.
ccv3d_status launch_stage(ccv3d_handle* h, StageParams sp, int h0, int h1, int nframes, cudaStream_t st) {
    const TcPlan& pl = h->plan;
    sp.h_begin = h0;
    const bool vec = (sp.W % 8 == 0);
    const int wcols = sp.ph_sh > 0 ? sp.ph_Wp * sp.ph_sw : sp.W;   // (phase-decomposed copy: columns up to a whole number of phases)
    dim3 sgrid((wcols + STG_PX - 1) / STG_PX, h1 - h0, (unsigned)(sp.N * nframes * pl.CB));
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
template <int KB, int NB, int KS, int TPBC, bool COOP, bool TF32 = false, bool TAIL = false, int DIL = 1>
ccv3d_status launch_tc_pair(ccv3d_handle* h, const CUtensorMap& tm_a, const CUtensorMap& tm_w, const CUtensorMap& tm_o,
                            const TcParams& p, const StageParams& sp, size_t smem, int grid, cudaStream_t st) {
    auto kern = conv3d_tcgen05_kernel<KB, NB, KS, TPBC, false, COOP, TF32, true, TAIL, DIL>;
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
    cfg.numAttrs = ((COOP && h->coop_launch) || (!COOP && h->pdl)) ? 2 : 1;
    if (cudaLaunchKernelEx(&cfg, kern, tm_a, tm_w, tm_o, p, sp, h->stg_maps) != cudaSuccess) return cuda_fail();
    if (cudaGetLastError() != cudaSuccess) return cuda_fail();
    h->ctr.kernel_launches++;
    return CCV3D_OK;
}

// 2-D map over the packed weights, all tiles of all taps one after another, seen as rows of 512 bytes (four or eight of
// the image's rows of KB channels: the image is packed with its swizzle applied, so the copy is a plain one, and a
// row is one request of the TMA unit - with 64-byte rows a 32-channel layer spent more requests on its weights than
// on anything else); a box is one CTA's share of a tile: half of it, or a quarter when the launch runs half-width
// tiles.  Encoded once per handle and box height.
ccv3d_status weight_map(ccv3d_handle* h, int box_rows, const CUtensorMap** out) {
    const int slot = (box_rows == h->plan.NPAD / 2) ? 0 : 1;
    if (h->tm_w_rows[slot] == box_rows) { *out = &h->tm_w[slot]; return CCV3D_OK; }
    CUtensorMap* tm = &h->tm_w[slot];
    const TcPlan& pl = h->plan;
    const ccv3d_desc& d = h->d;
    const uint64_t rows = (uint64_t)(d.dtype == CCV3D_F32 ? 3 : 1) * d.kt * pl.CB * pl.NT * d.kh * d.kw * pl.NPAD;
    const uint64_t rpb = 256 / pl.KB;                              // image rows per 512-byte row of the map (FP32 layers: KB = 64)
    cuuint64_t dims[2] = {256, (cuuint64_t)(rows / rpb)};
    cuuint64_t strides[1] = {512};
    cuuint32_t box[2] = {256, (cuuint32_t)(box_rows / rpb)};
    cuuint32_t es[2] = {1, 1};
    if (rows > 0x7FFFFFFFull || box_rows > 256 || box_rows % 8 || rows % rpb) return CCV3D_ERR_UNSUPPORTED;
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
                             const StageParams& sp, size_t smem, int grid, int ks, int nb, cudaStream_t st, int dil = 1) {
    const CUtensorMap* tm_w = nullptr;
    // (a launch that ends in half-width items carries the weight map of those, see the kernel's B producer)
    ccv3d_status s = weight_map(h, p.main_tiles > 0 ? p.NPAD / 4 : p.NPAD / 2, &tm_w);
    if (s != CCV3D_OK) return s;
    if (dil == TAPS_STRIDE2) {              // 3x3 taps at stride 2 over the four phase images: three taps per weight stage
        if (ks != 3 || !p.phased || p.TPB != 3 || p.SA < 4 || p.main_tiles > 0 || h->d.dtype == CCV3D_F32) return CCV3D_ERR_UNSUPPORTED;
        if (h->plan.KB == 64 && nb == 2) return launch_tc_pair<64, 2, 3, 3, COOP, false, false, TAPS_STRIDE2>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);
        if (h->plan.KB == 64) return launch_tc_pair<64, 1, 3, 3, COOP, false, false, TAPS_STRIDE2>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);
        if (nb == 2) return launch_tc_pair<32, 2, 3, 3, COOP, false, false, TAPS_STRIDE2>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);
        return launch_tc_pair<32, 1, 3, 3, COOP, false, false, TAPS_STRIDE2>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);
    }
    if (p.TPB == 9) {                       // all nine taps per weight stage: 32-channel blocks, narrow tiles
        if (ks != 3 || dil != 1 || p.main_tiles > 0 || h->d.dtype == CCV3D_F32 || h->plan.KB != 32) return CCV3D_ERR_UNSUPPORTED;
        if (nb == 2) return launch_tc_pair<32, 2, 3, 9, COOP>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);
        return launch_tc_pair<32, 1, 3, 9, COOP>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);
    }
#define CCV3D_LAUNCH_PAIR(KBv, NBv)                                                                                        \
    do {                                                                                                                   \
        if (ks == 3 && p.TPB == 3) return launch_tc_pair<KBv, NBv, 3, 3, COOP>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st); \
        if (ks == 3) return launch_tc_pair<KBv, NBv, 3, 1, COOP>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);              \
        return launch_tc_pair<KBv, NBv, 1, 1, COOP>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);                           \
    } while (0)
    if (dil == 2) {                         // 3x3 taps two pixels apart: straight-line taps with the doubled offsets
        if (ks != 3 || p.main_tiles > 0 || h->d.dtype == CCV3D_F32) return CCV3D_ERR_UNSUPPORTED;
#define CCV3D_LAUNCH_PAIR_D2(KBv, NBv)                                                                                              \
    do {                                                                                                                            \
        if (p.TPB == 3) return launch_tc_pair<KBv, NBv, 3, 3, COOP, false, false, 2>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);   \
        return launch_tc_pair<KBv, NBv, 3, 1, COOP, false, false, 2>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);                   \
    } while (0)
        if (h->plan.KB == 64 && nb == 2) CCV3D_LAUNCH_PAIR_D2(64, 2);
        else if (h->plan.KB == 64) CCV3D_LAUNCH_PAIR_D2(64, 1);
        else if (nb == 2) CCV3D_LAUNCH_PAIR_D2(32, 2);
        else CCV3D_LAUNCH_PAIR_D2(32, 1);
#undef CCV3D_LAUNCH_PAIR_D2
    }
    if (p.main_tiles > 0) {                 // launches ending in half-width items: 64-channel blocks, one pixel block, 3x3 taps
        if (COOP || h->d.dtype == CCV3D_F32 || h->plan.KB != 64 || nb != 1 || ks != 3) return CCV3D_ERR_UNSUPPORTED;
        if (p.TPB == 3) return launch_tc_pair<64, 1, 3, 3, false, false, true>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);
        return launch_tc_pair<64, 1, 3, 1, false, false, true>(h, tm_a, *tm_w, tm_o, p, sp, smem, grid, st);
    }
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
bool pair_eligible(const ccv3d_handle* h, int64_t pair_tiles, bool phased = false) {
    const ccv3d_desc& d = h->d;
    const TcPlan& pl = h->plan;
    if ((d.flags & CCV3D_FLAG_NO_PAIR) || !h->cluster_ok) return false;
    if (d.flags & CCV3D_FLAG_TC_PER_TAP_A) return false;
    // (strided layers: stride 2 with padding 1 over phase images has a straight-line tap loop of its own; kh = kw = 3 below)
    if ((d.stride[1] != 1 || d.stride[2] != 1) &&
        !(phased && d.stride[1] == 2 && d.stride[2] == 2 && d.pad_h == 1 && d.pad_w == 1 && d.dilation[1] == 1 && d.dilation[2] == 1 &&
          (size_t)(pl.NPAD / 2) * pl.KB * 2 * 3 <= 40960))
        return false;
    if (d.kh != 3 || d.kw != 3) return false;              // (1x1 layers are bound by their epilogue; pairs make them slower)
    // unit spatial dilation, or dilation 2 in both directions (its own straight-line variant of the tap loop)
    const bool dil1 = d.dilation[1] == 1 && d.dilation[2] == 1, dil2 = d.dilation[1] == 2 && d.dilation[2] == 2;
    if (!(dil1 || (dil2 && d.dtype == CCV3D_BF16))) return false;
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

    // the staging copy: in the caller's workspace when one was lent (never allocates; too small = an error before
    // any launch), else in the handle's own, which grows on demand
    ccv3d_status s = CCV3D_OK;
    if (h->ext_ws) {
        if (tc_workspace_bytes(h, N, T, H, W) > h->ext_ws_bytes) return CCV3D_ERR_NOMEM;
        h->ws_cur = h->ext_ws;
    } else {
        s = grow(&h->workspace, &h->workspace_bytes, tc_workspace_bytes(h, N, T, H, W));
        if (s != CCV3D_OK) return s;
        h->ws_cur = h->workspace;
    }

    // ---- staging: [cache ; x] channels-last, cache update in the same pass ----
    StageParams sp;
    memset(&sp, 0, sizeof(sp));
    sp.x = (const __nv_bfloat16*)x;
    const int cf = (tc && cache) ? h->call_cf : 0;          // older history frames are absent: their taps are skipped
    sp.cache = cf ? (const __nv_bfloat16*)cache : nullptr;
    sp.cf = cf;
    sp.zs = (__nv_bfloat16*)h->ws_cur;
    sp.new_cache = tc ? (__nv_bfloat16*)new_cache : nullptr;
    sp.N = N; sp.Cin = d.cin; sp.T = T; sp.H = H; sp.W = W; sp.tc = tc; sp.CB = pl.CB;
    sp.f_begin = (tc - cf) < T ? (tc - cf) : T;
    const int nframes = F - sp.f_begin;

    // ---- implicit GEMM parameters ----
    // A spatial stride cannot be a shift inside one halo tile of the image.  BF16 layers stage a phase-decomposed copy
    // instead (s_h * s_w phase images, in which consecutive output pixels are consecutive again: one halo tile per phase,
    // its taps descriptor offsets); FP32 layers and strides of more than 16 phases fetch one strided box per tap.
    const int S2 = d.stride[1] * d.stride[2];
    const bool phased = strided && !f32 && !(d.flags & CCV3D_FLAG_TC_PER_TAP_A) && S2 <= 16 && d.kh * d.kw <= 49;
    const int per_tap = ((d.flags & CCV3D_FLAG_TC_PER_TAP_A) || (strided && !phased)) ? 1 : 0;
    const int Hp = phased ? (H + d.stride[1] - 1) / d.stride[1] : H, Wp = phased ? (W + d.stride[2] - 1) / d.stride[2] : W;
    // 256-pixel tiles (two 128-pixel blocks sharing every weight tile) unless that leaves SMs without a tile
    int NB = pl.NB;
    // (phase-decomposed layers on single CTAs run one tap per weight stage, where the weight stream from L2 is
    // what limits a 128-pixel tile: two pixel blocks per weight tile even when that leaves one accumulator buffer.
    // The stride-2 layers that run on CTA pairs keep their own tile width.)
    bool phased_pair = phased && !(d.flags & CCV3D_FLAG_OVERLAP) &&
                       pair_eligible(h, (int64_t)N * ((Ho + 15) / 16) * ((Wo + 16 * NB - 1) / (16 * NB)) * To, true);
    if (phased_pair) {
        // that variant holds four halo tiles (one per phase) per activation stage group and three taps per weight stage
        auto fits = [&](int nb) {
            const size_t a_slot = align_up((uint64_t)(8 * nb + 1) * 17 * pl.KB * 2, 1024);
            const size_t b_slot = align_up((uint64_t)(pl.NPAD / 2) * pl.KB * 2 * 3, 1024);
            const size_t e_slot = (d.out_dtype != CCV3D_F32 && Wo % 8 == 0) ? (size_t)32 * 16 * 8 * nb * 2 : 0;
            // (four activation slots and two weight stages to run; two and three for size_pipeline to keep three taps per stage)
            const size_t rings = 4 * a_slot + 2 * b_slot > 2 * a_slot + 3 * b_slot ? 4 * a_slot + 2 * b_slot : 2 * a_slot + 3 * b_slot;
            return 1024 + align_up(sizeof(TcShared), 128) + 2 * e_slot + rings <= SMEM_LIMIT;
        };
        // 32-channel blocks: two pixel blocks per CTA even with one accumulator buffer (96->192 from 704x1280: 0.95 ms
        // against 1.03 ms with one block; 96->96: 0.75 against 0.92 ms).  Two blocks of 64 channels do not fit: one block
        // (128->128 from 352x640: 0.31 ms against 0.32 ms on single CTAs with two blocks).
        if (pl.KB == 32 && 2 * pl.NPAD <= 512 && fits(2)) NB = 2;
        if (!fits(NB)) {
            if (NB == 2 && fits(1)) NB = 1;
            else phased_pair = false;
        }
    }
    if (phased && !phased_pair && 2 * pl.NPAD <= 512) NB = 2;
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
    const bool pair = !per_tap && !(d.flags & CCV3D_FLAG_OVERLAP) && (!phased || phased_pair) &&
                      pair_eligible(h, (int64_t)N * ((Ho + 15) / 16) * ((Wo + 16 * NB - 1) / (16 * NB)) * To, phased);
    const int TW = 8 * NB;                                 // pixels per row of a CTA's part of a tile
    const int TWT = pair ? 2 * TW : TW;                    // tile width in the tile index space
    TcParams p;
    memset(&p, 0, sizeof(p));
    if (phased) {
        // tap (a, c) of output pixel (oh, ow) reads input (oh s_h + a d_h - p_h, ...) = phase ((a d_h - p_h) mod s_h, ...)
        // at phase-image pixel (oh + floor((a d_h - p_h) / s_h), ...)
        auto fdiv = [](int v, int m) { return v >= 0 ? v / m : -((-v + m - 1) / m); };
        int offh[49], offw[49], phq[49], minh[16], minw[16], maxh[16], maxw[16];
        for (int q = 0; q < S2; ++q) { minh[q] = minw[q] = 1 << 20; maxh[q] = maxw[q] = -(1 << 20); }
        for (int a = 0; a < d.kh; ++a)
            for (int c = 0; c < d.kw; ++c) {
                const int i = a * d.kw + c;
                const int eh = a * d.dilation[1] - d.pad_h, ew = c * d.dilation[2] - d.pad_w;
                offh[i] = fdiv(eh, d.stride[1]); offw[i] = fdiv(ew, d.stride[2]);
                phq[i] = (eh - offh[i] * d.stride[1]) * d.stride[2] + (ew - offw[i] * d.stride[2]);
                const int q = phq[i];
                if (offh[i] < minh[q]) minh[q] = offh[i];
                if (offh[i] > maxh[q]) maxh[q] = offh[i];
                if (offw[i] < minw[q]) minw[q] = offw[i];
                if (offw[i] > maxw[q]) maxw[q] = offw[i];
            }
        int n = 0;
        p.phased = 1; p.S2 = S2;
        for (int q = 0; q < S2; ++q) {
            p.ph_first[q] = (unsigned char)n;
            for (int i = 0; i < d.kh * d.kw; ++i)
                if (phq[i] == q) {
                    p.ph_tap[n] = (unsigned char)i;
                    p.ph_roff[n] = (unsigned char)(offh[i] - minh[q]);
                    p.ph_coff[n] = (unsigned char)(offw[i] - minw[q]);
                    ++n;
                }
            if (n > p.ph_first[q]) {
                p.ph_h0[q] = (signed char)minh[q]; p.ph_w0[q] = (signed char)minw[q];
                if (maxh[q] - minh[q] > p.ph_bh) p.ph_bh = maxh[q] - minh[q];
                if (maxw[q] - minw[q] > p.ph_bw) p.ph_bw = maxw[q] - minw[q];
            }
        }
        for (int q = S2; q <= 16; ++q) p.ph_first[q] = (unsigned char)n;
        sp.ph_sh = d.stride[1]; sp.ph_sw = d.stride[2]; sp.ph_Hp = Hp; sp.ph_Wp = Wp;
    }
    const int BW = phased ? TW + p.ph_bw : (per_tap ? TW : TW + (d.kw - 1) * d.dilation[2]);
    const int BH = phased ? 16 + p.ph_bh : (per_tap ? 16 : 16 + (d.kh - 1) * d.dilation[1]);
    ShapeKey key{h->ws_cur, N, T, H, W, BW};
    if (!(key == h->tm_a_key)) {
        s = encode_act_map(h, N, T, Hp, Wp, BW, BH, per_tap ? d.stride[2] : 1, per_tap ? d.stride[1] : 1, phased ? S2 : 1);
        if (s != CCV3D_OK) return s;
        h->tm_a_key = key;
    }
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
    // (with the layer's own padding and dilation too, at unit strides: the bands are bands of input rows)
    const int in_bands = (H + 15) / 16;
    // (of the phase-decomposed copies of strided layers only those of the stride-2 layers on CTA pairs, with even H and W.
    // The single-CTA kernel with its run-time tap loop and one tap per weight stage lost more to the stagers' traffic than
    // the hidden staging pass returned: 1.41 ms against 1.24 ms for the two kernels at 96->192, stride 2, from 704x1280)
    const bool str2 = phased && pair;                      // (pair_eligible admits one kind of strided layer)
    const int str2_slots = NB == 2 ? 3 : 4;                // stager slots of such a layer (16 KB / 8 KB each)
    const size_t str2_b = align_up((uint64_t)p.b_tap * 3, 1024);
    const size_t str2_rings = 4 * (size_t)p.a_slot + 2 * str2_b > 2 * (size_t)p.a_slot + 3 * str2_b ? 4 * (size_t)p.a_slot + 2 * str2_b
                                                                                                  : 2 * (size_t)p.a_slot + 3 * str2_b;
    const bool str2_coop = str2 && H % 2 == 0 && W % 2 == 0 &&
                           1024 + align_up(sizeof(TcShared), 128) + 2 * (size_t)p.e_slot + (size_t)str2_slots * (NB == 2 ? 4 : 2) * 4096 +
                                   str2_rings <= SMEM_LIMIT;
    // (a temporal stride only moves the frame a tap reads: the downsampling layers in time, stride (2, 1, 1), and in time
    // and space, stride (2, 2, 2), included - with nine or more spatial taps: 192->192, T = 8, at 352x640 with a 3x1x1
    // kernel stages two input frames per output frame for three taps of work and lost 5 % to its stagers)
    const bool coop = nbands == 1 && !per_tap && (!phased || str2_coop) && (d.stride[0] == 1 || d.kh * d.kw >= 9) && !f32 &&
                      !(d.flags & CCV3D_FLAG_TWO_KERNELS) && raw_maps_ok(h, x, cache, new_cache, T, H, W) &&
                      in_bands <= MAX_COOP_BANDS && tiles_h >= 4 &&
                      // too few waves of tiles: two kernels.  Measured with the stager warps on TMA: wide tiles (one pixel block
                      // per CTA) and two or more output frames are ahead from four waves (192->192 at 128x160, T = 4: 2 %;
                      // 176x160: 4 %; 256->256 at 128x160: 11 %; at three waves 3 % behind); narrow tiles and one-frame calls
                      // are 10-20 % behind at six waves and level from eight or nine
                      (int64_t)N * tiles_h * p.tiles_w * To * NT * (pair ? 2 : 1) >= ((NB == 1 && To >= 2) ? 4LL : 8LL) * h->sm_count;
    // Cooperative staging: the stager team keeps stg_slots tasks in flight, two, and a third only when that costs the
    // rings nothing (192->192 at 352x640 loses 3 % when a third slot takes the fourth weight slot's place).  A task is
    // 8 KB next to wide tiles and 16 KB next to narrow ones (two pixel blocks per CTA, at most 128 output channels:
    // STAGER_BOXES), which stage twice as many input bytes per MMA cycle: the team is bound by its per-task instructions
    // (a barrier, the odometer, the TMA issue), and with tasks of twice the pixels 96->96 at 704x1280 went from 1.80 M to
    // 1.66 M cycles, the figure of the same layer on frame rings (three slots of 8 KB before; with two the team, then
    // bound by the latency of its fetches, finished last: 4.34 M cycles against 3.35 M at 192->96).
    // Calls that stage three or more frames per output frame (one frame on top of a two-frame history) are bound by the
    // stager team, which is bound by the latency of its fetches: they get two more slots of 8 KB, or one more of 16 KB,
    // at the cost of a weight slot (192->192, T = 1, 352x640: 596 k -> 466 k cycles; 192->96, T = 1, 704x1280: 1.57 M ->
    // 1.27 M; with two output frames the weight slot is worth more).
    const bool stage_heavy = coop && (F >= 3 * T || str2);    // (stride 2: four input pixels per output pixel)
    p.stg_slots = coop ? (stage_heavy ? (NB == 2 ? 3 : 4) : 2) : 0;
    const size_t stg_slot = (size_t)(NB == 2 ? 4 : 2) * 4096;       // (STAGER_BOXES<NB>)
    size_t fixed = 1024 /*alignment slack*/ + align_up(sizeof(TcShared), 128) + 2 * (size_t)p.e_slot +
                   (size_t)p.stg_slots * stg_slot;
    // leave room for staging blocks to be resident next to a convolution CTA when the two overlap
    const size_t limit = nbands > 1 ? SMEM_LIMIT - STAGE_COEXIST_BYTES : SMEM_LIMIT;
    const size_t budget = limit - fixed;
    const bool tpb9 = pair && !f32 && !phased && pl.KB == 32 && d.kh == 3 && d.kw == 3 && d.dilation[1] == 1 && d.dilation[2] == 1;
    s = size_pipeline(&p, budget, per_tap != 0 || (phased && !str2), (phased && !str2) ? 1 : d.kw, tpb9 ? 9 : 0);   // (run-time phase order: one tap per weight stage)
    if (s != CCV3D_OK) return s;
    if (str2) {
        // four halo tiles (one per phase) per (dt, ci-block): the activation ring holds whole groups of four
        static const unsigned char order[9] = {4, 3, 5, 1, 7, 0, 2, 6, 8}, roff[9] = {0, 0, 0, 0, 1, 0, 0, 1, 1}, coff[9] = {0, 0, 1, 0, 0, 0, 1, 0, 1};
        bool same = p.TPB == 3 && p.S2 == 4 && p.ph_bh == 1 && p.ph_bw == 1 && p.ph_first[1] == 1 && p.ph_first[2] == 3 && p.ph_first[3] == 5;
        for (int i = 0; i < 9; ++i) same = same && p.ph_tap[i] == order[i] && p.ph_roff[i] == roff[i] && p.ph_coff[i] == coff[i];
        if (!same) return CCV3D_ERR_UNSUPPORTED;           // (the kernel's compile-time tap table is this one)
        while (p.SB > 2 && 4 * (size_t)p.a_slot + (size_t)p.SB * p.b_slot > budget) --p.SB;
        if (4 * (size_t)p.a_slot + (size_t)p.SB * p.b_slot > budget) return CCV3D_ERR_UNSUPPORTED;
        p.SA = 4;
        while (p.SA < 8 && (size_t)(p.SA + 1) * p.a_slot + (size_t)p.SB * p.b_slot <= budget) ++p.SA;
        // more activation slots are worth weight stages down to four of those (a fifth slot lets the producer request the
        // four-tap phase's next tile ten taps ahead instead of five: 96->192 from 352x640 on two kernels 314 -> 296 us;
        // down to two weight stages 331 us; the cooperative schedule has three stages and keeps them)
        while (p.SB > 4 && p.SA < 8 && (size_t)(p.SA + 1) * p.a_slot + (size_t)(p.SB - 1) * p.b_slot <= budget) { ++p.SA; --p.SB; }
    }
    if (coop && !stage_heavy && p.stg_slots < 3 && (size_t)p.SA * p.a_slot + (size_t)p.SB * p.b_slot + stg_slot <= budget) {
        ++p.stg_slots;
        fixed += stg_slot;
    }
    // ... and with narrow tiles a third activation slot is worth a weight slot when four or more of those are left: next to
    // the stagers' traffic it is the halo tiles that arrive late (96->96 at 704x1280: 1.95 M cycles with 2 + 4 slots,
    // 1.86 M with 3 + 3)
    if (coop && NB == 2 && p.SA == 2 && p.SB >= 4 && 3 * (size_t)p.a_slot + (size_t)(p.SB - 1) * p.b_slot <= limit - fixed) {
        p.SA = 3;
        --p.SB;
    }
    p.tmem_cols = pow2_cols((uint32_t)(asets * NB * NPAD * ACC));
    if (p.tmem_cols > 512) return CCV3D_ERR_UNSUPPORTED;
    p.wait_limit_clk = h->wait_limit_clk;
    p.bias = h->bias32;
    p.wq = (const uint8_t*)h->wp;
    p.out = out;
    p.status = h->status;
#ifdef CCV3D_DEV_TRACE
    p.trace = getenv("CCV3D_TC_TRACE") ? (unsigned long long*)strtoull(getenv("CCV3D_TC_TRACE"), nullptr, 0) : nullptr;
#endif
    if (p.epi_tma) {
        s = encode_out_map(h, out, N, To, Ho, Wo, TW, p.ECH);
        if (s != CCV3D_OK) return s;
    } else {
        h->tm_o = h->tm_a;  // never dereferenced on this path; any valid descriptor will do
    }
    const size_t smem = fixed + (size_t)p.SA * p.a_slot + (size_t)p.SB * p.b_slot;
    // straight-line tap loops need unit spatial dilation (the tap offsets are compile-time); padding and the temporal
    // dilation only move the producer's TMA coordinates
    // (spatial dilation 2 of a 3x3 kernel has such a variant too, on CTA pairs)
    const int dil = str2 ? TAPS_STRIDE2 : (pair && !f32 && d.dilation[1] == 2 && d.dilation[2] == 2) ? 2 : 1;
    const int ks = (!per_tap && (!phased || str2) && ((d.dilation[1] == 1 && d.dilation[2] == 1) || dil == 2) && d.kh == d.kw && (d.kh == 1 || d.kh == 3)) ? d.kh : 0;
    const int ph = (d.kh - 1) / 2;
    cudaEvent_t* pev = (h->prof_on && h->prof_ev) ? h->prof_ev + 3 * (h->prof_n % PROF_SLOTS) : nullptr;

    if (coop) {
        if (pev) { cudaEventRecord(pev[0], st); cudaEventRecord(pev[1], st); }
        if (cudaMemsetAsync(h->band_ctr, 0, (size_t)in_bands * sizeof(unsigned int), st) != cudaSuccess) return cuda_fail();
        p.band_ctr = h->band_ctr;
        p.nbands = in_bands;
        // The first tiles of every CTA read bands 0 and 1 (of all frames), and until those are staged nothing else can run:
        // with four stager warps per SM that took 113 k of the 1620 k cycles of 192->192 at 352x640.  Those two bands go
        // through the staging kernel instead (all warps of all SMs, about 20 us), the stagers take over from band 2.
        p.band_first = in_bands < 2 ? in_bands : 2;
        s = launch_stage(h, sp, 0, H < 16 * p.band_first ? H : 16 * p.band_first, nframes, st);
        if (s != CCV3D_OK) return s;
        s = encode_stager_maps(h, x, cache, cf, sp.new_cache, N, T, H, W);
        if (s != CCV3D_OK) return s;
        p.ty_begin = 0;
        p.tiles_h = tiles_h;
        const int64_t total = (int64_t)N * tiles_h * p.tiles_w * To * NT;
        if (total > 0x7FFFFFFF) return CCV3D_ERR_UNSUPPORTED;
        p.total_tiles = (int)total;
        int grid = p.total_tiles < h->sm_count ? p.total_tiles : h->sm_count;
        if (pair) {
            grid = 2 * (p.total_tiles < h->sm_count / 2 ? p.total_tiles : h->sm_count / 2);
            s = launch_pair_any<true>(h, h->tm_a, h->tm_o, p, sp, smem, grid, ks, NB, st, dil);
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
            sf.zs = (float*)h->ws_cur; sf.new_cache = tc ? (float*)new_cache : nullptr;
            sf.N = N; sf.Cin = d.cin; sf.T = T; sf.H = H; sf.W = W; sf.tc = tc; sf.CBr = pl.CB; sf.f_begin = sp.f_begin;
            dim3 sgrid((W + 31) / 32, H, (unsigned)((int64_t)N * nframes * sf.CBr));
            if (H > 65535 || (int64_t)N * nframes * sf.CBr > 65535) return CCV3D_ERR_UNSUPPORTED;
            stage_frames_f32_kernel<<<sgrid, 256, 0, st>>>(sf);
            if (cudaGetLastError() != cudaSuccess) return cuda_fail();
            h->ctr.kernel_launches++;
            s = CCV3D_OK;
        } else {
            s = launch_stage(h, sp, 0, phased ? Hp * d.stride[1] : H, nframes, st);
        }
        if (s != CCV3D_OK) return s;
        if (pev) cudaEventRecord(pev[1], st);
        if (pair) {
            p.ty_begin = 0;
            p.tiles_h = tiles_h;
            const int64_t total = (int64_t)N * tiles_h * p.tiles_w * To * NT;
            if (total > 0x3FFFFFFF) return CCV3D_ERR_UNSUPPORTED;
            p.total_tiles = (int)total;
            // a last wave that is at most half full runs at half width (see forward_ring)
            const int64_t slots = h->sm_count / 2, frac = total % slots;
            if (!split_n && NB == 1 && pl.KB == 64 && pl.NPAD % 64 == 0 && ks == 3 && dil == 1 && !f32 &&
                !(d.flags & CCV3D_FLAG_NO_TAIL_SPLIT) && total > slots && total / slots <= 12 && frac > 0 && 2 * frac <= slots) {
                p.main_tiles = (int)(total - frac);
                p.total_tiles = (int)(total + frac);
            }
            const int grid = 2 * (p.total_tiles < h->sm_count / 2 ? p.total_tiles : h->sm_count / 2);
            StageParams nosp;
            memset(&nosp, 0, sizeof(nosp));
            s = launch_pair_any<false>(h, h->tm_a, h->tm_o, p, nosp, smem, grid, ks, NB, st, dil);
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
    if (f32) h->ctr.tcgen05_f32++; else h->ctr.tcgen05_bf16++;
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
    kern<<<grid, TC_THREADS_FUSED, smem, st>>>(tm_x, tm_c, tm_o, p, nosp, h->stg_maps);
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
    p.NACC = 2;               // (four buffers, where they fit, measured no better: 170 against 174 us at 64->64, 4x704x1280)
    p.tmem_cols = pow2_cols((uint32_t)(p.NACC * pl.NPAD));
    p.wait_limit_clk = h->wait_limit_clk;
    p.bias = h->bias32;
    p.wq = (const uint8_t*)h->wp;
    p.status = h->status;
    p.EG = 2;                 // two epilogue groups: with one, layers of as many output as input channels are bound by it
    const size_t w_al = align_up(p.w_bytes, 1024);
    const size_t fixed = 1024 + align_up(sizeof(TcShared), 128) + 2 * (size_t)p.EG * p.e_slot + w_al;
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
    conv1x1_tcgen05_kernel<<<grid, PW_THREADS, smem, st>>>(tm_x, tm_o, p);
    if (cudaGetLastError() != cudaSuccess) return cuda_fail();
    if (pev) {
        cudaEventRecord(pev[2], st);
        h->prof_n++;
    }
    h->ctr.kernel_launches++;
    h->ctr.pointwise++;
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
static std::atomic<void*> g_static_scratch_addr[MAX_DEVICES];   // device address of the array, per device; set on first use

// In host code the name g_static_scratch is only a stand-in for the symbol: the address a kernel can use has
// to be asked for, once per device, with that device current.
ccv3d_status static_scratch_for_current_device(void** out_ptr) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return cuda_fail();
    if (dev < 0 || dev >= MAX_DEVICES) return CCV3D_ERR_UNSUPPORTED;
    // Threads of different handles may arrive here together: the table is atomic, and every thread that finds
    // the entry empty looks the address up itself and stores the same value.
    void* ptr = g_static_scratch_addr[dev].load(std::memory_order_acquire);
    if (!ptr) {
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return cuda_fail();
        g_static_scratch_addr[dev].store(ptr, std::memory_order_release);
    }
    *out_ptr = ptr;
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
    if (cudaLaunchKernelEx(&cfg, kern, tm_a, tm_a, tm_o, p, nosp, h->stg_maps) != cudaSuccess) return cuda_fail();
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
