// The 1x1x1 streaming kernel (conv1x1_tcgen05_kernel).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ccv3d {

// ------------------------------------------------------------------------------------------------
// 1x1x1 kernels (per-pixel matmul, no cache, no halo): streaming kernel straight from NCTHW
// ------------------------------------------------------------------------------------------------
// With one tap there is no shift to express, so the activations can be used as they lie in memory: for a
// fixed channel the P = T*H*W pixels of a sample are contiguous, i.e. the A operand is "MN-major".  A TMA box
// of {64 pixels, 64 channels} with 128-byte swizzle lands as 64 K-rows of 128 bytes = the canonical MN-major
// layout (8-row groups 1024 bytes apart); a 128-pixel M tile is two such boxes.  The whole weight matrix
// (Cin_pad x NPAD, packed as for the general kernel) stays resident in shared memory; the kernel is bound by
// HBM (read x once, write out once) and the tensor core is mostly idle.
struct PwParams {
    int N, Cout, CB, NPAD;
    int tiles_p;              // 128-pixel tiles per sample
    int total_tiles;
    int SA;                   // activation ring depth
    int ECH;                  // channels per epilogue chunk (32 or 16)
    int EG;                   // epilogue warp groups (1 or 2): group g drains the accumulators of this CTA's tiles g, g+EG, ...
    int NACC;                 // accumulator buffers in tensor memory (2..4): tile i of a CTA uses buffer i % NACC
    uint32_t a_slot, e_slot, w_bytes, b_tap;
    uint32_t tmem_cols;
    long long wait_limit_clk;
    const float* bias;
    const uint8_t* wq;
    unsigned int* status;
};

__device__ __forceinline__ bool pw_wait(uint64_t* bar, uint32_t parity, TcShared* sh, const PwParams& p, uint32_t site) {
    const uint32_t b = smem_u32(bar);
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

constexpr int PW_THREADS = 384;       // producer, weights, MMA, allocator warps + two epilogue groups of four warps

__global__ void __launch_bounds__(PW_THREADS, 1)
conv1x1_tcgen05_kernel(const __grid_constant__ CUtensorMap tm_x,   // x as (pixel, channel, sample)
                       const __grid_constant__ CUtensorMap tm_o,   // out as (pixel, channel, sample)
                       const PwParams p) {
    constexpr int KB = 64;
    constexpr uint32_t HALF = 64 * 128;                     // bytes of one {64 px, 64 ch} box
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* w_smem = smem;
    uint8_t* ring_a = w_smem + p.w_bytes;
    uint8_t* epi_buf = ring_a + (size_t)p.SA * p.a_slot;
    TcShared* sh = reinterpret_cast<TcShared*>(epi_buf + 2 * (size_t)p.EG * p.e_slot);

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int i = 0; i < p.SA; ++i) { mbar_init(smem_u32(&sh->full_a[i]), 1); mbar_init(smem_u32(&sh->empty_a[i]), 1); }
        mbar_init(smem_u32(&sh->full_b[0]), 1);
        for (int i = 0; i < p.NACC; ++i) { mbar_init(smem_u32(&sh->acc_full[i]), 1); mbar_init(smem_u32(&sh->acc_empty[i]), 4); }
        sh->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 3) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)),
                     "r"(p.tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    for (int i = threadIdx.x; i < p.NPAD; i += blockDim.x) sh->bias_s[i] = __ldg(p.bias + i);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;
    const int t_first = (int)blockIdx.x, t_end = p.total_tiles, t_step = (int)gridDim.x;   // this CTA's tiles

    if (warp == 0) {                      // activation producer
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_x) : "memory");
            int s = 0;
            uint32_t phase = 1;
            bool ok = true;
            for (int tile = t_first; ok && tile < t_end; tile += t_step) {
                const int n = tile / p.tiles_p, p0 = (tile % p.tiles_p) * 128;
                for (int cb = 0; cb < p.CB; ++cb) {
                    if (!(ok = pw_wait(&sh->empty_a[s], phase, sh, p, SITE_A_EMPTY))) break;
                    const uint32_t bar = smem_u32(&sh->full_a[s]);
                    const uint32_t dst = smem_u32(ring_a + (size_t)s * p.a_slot);
                    mbar_expect_tx(bar, 2 * HALF);
                    tma_load_3d(dst, &tm_x, bar, p0, cb * KB, n);
                    tma_load_3d(dst + HALF, &tm_x, bar, p0 + 64, cb * KB, n);
                    if (++s == p.SA) { s = 0; phase ^= 1; }
                }
            }
            if (!ok) drain_delay();
        }
    } else if (warp == 1) {               // weights: loaded once, resident for the whole kernel
        if (lane == 0) {
            const uint32_t bar = smem_u32(&sh->full_b[0]);
            mbar_expect_tx(bar, p.w_bytes);
            bulk_load(smem_u32(w_smem), p.wq, p.w_bytes, bar);
        }
    } else if (warp == 2) {               // MMA issuer (warp-uniform; one elected lane issues)
        // instruction descriptor: D=F32, A=B=BF16, A MN-major (bit 15), B K-major, N = NPAD, M = 128
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | ((uint32_t)(p.NPAD >> 3) << 17) | ((128u >> 4) << 24);
        const uint32_t a_hi = make_desc_hi(1024, 2u);       // MN-major: 8-channel groups 1024 bytes apart
        const uint32_t b_hi = make_desc_hi(8 * 128, 2u);
        const uint32_t a_lbo = (HALF >> 4) << 16;           // next 64 pixels: the second box
        const uint32_t w_lo = make_desc_lo(smem_u32(w_smem));
        int sa = 0, acc = 0;
        uint32_t pa = 0, pacc = 1;
        bool ok = pw_wait(&sh->full_b[0], 0, sh, p, SITE_B_FULL);
        for (int tile = t_first; ok && tile < t_end; tile += t_step) {
            if (!(ok = pw_wait(&sh->acc_empty[acc], pacc, sh, p, SITE_ACC_EMPTY))) break;   // (first use of a buffer: passes at once)
            tc_fence_after();
            const uint32_t d0 = tmem_base + (uint32_t)acc * p.NPAD;
            for (int cb = 0; cb < p.CB; ++cb) {
                if (!(ok = pw_wait(&sh->full_a[sa], pa, sh, p, SITE_A_FULL))) break;
                tc_fence_after();
                const uint32_t a_lo = (((smem_u32(ring_a + (size_t)sa * p.a_slot)) & 0x3FFFFu) >> 4) | a_lbo;
                const uint32_t b_lo = w_lo + (uint32_t)cb * (p.b_tap >> 4);
                if (elect_one()) {
#pragma unroll
                    for (int k = 0; k < KB / 16; ++k)     // 16 channels = two 8-row groups = 2048 bytes of A, 32 bytes of B
                        tc_mma_bf16(d0, a_lo + k * (2048 >> 4), a_hi, b_lo + 2 * k, b_hi, idesc, (cb | k) ? 1u : 0u);
                    tc_commit(smem_u32(&sh->empty_a[sa]));
                }
                __syncwarp();
                if (++sa == p.SA) { sa = 0; pa ^= 1; }
            }
            if (!ok) break;
            if (elect_one()) tc_commit(smem_u32(&sh->acc_full[acc]));
            __syncwarp();
            if (++acc == p.NACC) { acc = 0; pacc ^= 1; }
        }
    } else if (warp >= 4 && warp < 4 + 4 * p.EG) {   // epilogue: +bias, RNE to BF16, [channel][128 px] tile, TMA store
        // One group of four warps drains both accumulator buffers in turn, or two groups drain one buffer each (tile
        // i of this CTA uses buffer i & 1), each with its own staging buffers, named barrier and store groups.
        const int g = (warp - 4) >> 2;
        const int q = warp & 3;
        const int m = q * 32 + lane;
        const bool elected = (q == 0 && lane == 0);
        const uint32_t bar_id = 1u + 2u * (uint32_t)g;
        uint8_t* my_buf = epi_buf + (size_t)g * 2 * p.e_slot;
        int ebuf = 0, it = 0;
        bool ok = true;
        for (int tile = t_first; ok && tile < t_end; tile += t_step, ++it) {
            if (p.EG == 2 && (it & 1) != g) continue;
            const int acc = it % p.NACC;
            const uint32_t pacc = (uint32_t)(it / p.NACC) & 1u;      // the k-th use of a buffer completes its phase k
            const int n = tile / p.tiles_p, p0 = (tile % p.tiles_p) * 128;
            ok = pw_wait(&sh->acc_full[acc], pacc, sh, p, SITE_ACC_FULL);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_acc = tmem_base + (uint32_t)acc * p.NPAD + ((uint32_t)(q * 32) << 16);
            for (int c0 = 0; c0 < p.NPAD; c0 += p.ECH) {
                if (elected) bulk_wait_read<1>();   // the store that last read this buffer has finished reading
                asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
                __nv_bfloat16* stg = reinterpret_cast<__nv_bfloat16*>(my_buf + (size_t)ebuf * p.e_slot);
                uint32_t v[32];
                if (p.ECH == 32) tc_ld32(t_acc + c0, v); else tc_ld16(t_acc + c0, v);
                tc_wait_ld();
                // +bias, two neighbouring channels per (packed) conversion, their halves to two rows of the
                // [channel][128 px] tile; one straight-line body per chunk width
                auto convert_store = [&](auto ech_c) {
                    constexpr int E = decltype(ech_c)::value;
                    unsigned short* st16 = reinterpret_cast<unsigned short*>(stg) + m;
                    float bb[E];
#pragma unroll
                    for (int j4 = 0; j4 < E / 4; ++j4) {
                        const float4 b4 = *reinterpret_cast<const float4*>(sh->bias_s + c0 + 4 * j4);
                        bb[4 * j4] = b4.x; bb[4 * j4 + 1] = b4.y; bb[4 * j4 + 2] = b4.z; bb[4 * j4 + 3] = b4.w;
                    }
#pragma unroll
                    for (int j = 0; j < E / 2; ++j) {
                        const __nv_bfloat162 pr = __floats2bfloat162_rn(__uint_as_float(v[2 * j]) + bb[2 * j],
                                                                        __uint_as_float(v[2 * j + 1]) + bb[2 * j + 1]);
                        const uint32_t u = *reinterpret_cast<const uint32_t*>(&pr);
                        st16[(2 * j) * 128] = (unsigned short)(u & 0xFFFFu);
                        st16[(2 * j + 1) * 128] = (unsigned short)(u >> 16);
                    }
                };
                if (p.ECH == 32) convert_store(std::integral_constant<int, 32>{});
                else convert_store(std::integral_constant<int, 16>{});
                fence_async_smem();
                asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
                if (elected) {
                    tma_store_3d(&tm_o, smem_u32(stg), p0, c0, n);
                    bulk_commit();
                }
                ebuf ^= 1;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->acc_empty[acc]));
        }
        if (elected) bulk_wait_read<0>();     // (the stores have read the staging buffers; their writes complete with the grid)
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 3) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
    }
}

}  // namespace ccv3d
