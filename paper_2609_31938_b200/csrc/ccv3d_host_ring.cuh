// Host side of the frame-ring boundary (resident activations): ring checks, tensor maps, forward_ring.
// Part of the single translation unit ccv3d_api.cu (included inside its anonymous namespace).
#pragma once

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
    if (total > 0x3FFFFFFF) return CCV3D_ERR_UNSUPPORTED;
    p.total_tiles = (int)total;
    // A last wave of tiles that is at most half full runs at half width: twice the items, each half as long, so the
    // call ends half a wave earlier (192 channels at 88x160: 240 pair tiles on 74 pairs, 4 waves -> 3.5).  CTA pairs with
    // 64-channel blocks and 3x3 taps only (a kernel variant of its own); the few-waves limit keeps the two-box weight
    // loads of the full-width tiles (see the kernel) away from long launches, where half a wave is nothing.
    {
        const int64_t slots = pair ? h->sm_count / 2 : h->sm_count;
        const int64_t frac = total % slots;
        if (pair && !split_n && NB == 1 && pl.KB == 64 && pl.NPAD % 64 == 0 && d.kh == 3 && d.kw == 3 &&
            d.dtype == CCV3D_BF16 && !(d.flags & CCV3D_FLAG_NO_TAIL_SPLIT) &&
            total > slots && total / slots <= 12 && frac > 0 && 2 * frac <= slots) {
            p.main_tiles = (int)(total - frac);
            p.total_tiles = (int)(total + frac);
        }
    }
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
    s = size_pipeline(&p, budget, false, d.kw, (pair && pl.KB == 32 && d.kh == 3 && d.kw == 3 && p.main_tiles == 0) ? 9 : 0);
    if (s != CCV3D_OK) return s;
    p.tmem_cols = pow2_cols((uint32_t)(NB * NPAD * ACC));
    if (p.tmem_cols > 512) return CCV3D_ERR_UNSUPPORTED;
    p.wait_limit_clk = h->wait_limit_clk;
    p.bias = h->bias32;
    p.wq = (const uint8_t*)h->wp;
    p.out = out_ncthw;
    p.status = h->status;
#ifdef CCV3D_DEV_TRACE
    p.trace = getenv("CCV3D_TC_TRACE") ? (unsigned long long*)strtoull(getenv("CCV3D_TC_TRACE"), nullptr, 0) : nullptr;
#endif
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
