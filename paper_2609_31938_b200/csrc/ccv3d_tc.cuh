// Tensor-core route for BF16 layers on sm_100a.
//
//   pack_weights_kernel   once per layer: w[Cout,Cin,kt,kh,kw] -> per (tap, ci-block, co-tile) tiles stored
//                         as the swizzled shared-memory image of the K-major B operand.
//   stage_frames_kernel   per call: Z = [cache ; x] (NCTHW) -> channels-last blocks
//                         Zs[n][frame][cb][h][w][KB], and in the same pass the
//                         bit-exact cache update new_cache = last kt-1 frames of Z.
//   (fused mode)          no staging pass: a producer thread fetches raw [channel][row][32 pixels] boxes by TMA
//                         straight from x or from the cache (whichever holds the tap's frame), and four
//                         transposer warps turn each into the channels-last halo tile in shared memory
//                         (ldmatrix.trans + stmatrix); the cache update is then a separate copy kernel.
//   conv3d_tcgen05_kernel per call: persistent implicit GEMM.  For an output tile of
//                         16 rows x 8*NB pixels of one frame t, D[pixel, co] =
//                         sum over (dt, ci-block, dh, dw) of A_tap[pixel, ci] * Wp[tap][co, ci]
//                         (Eq. (2) with all taps folded into one K loop).  One TMA load
//                         brings the (16+kh-1) x (8*NB+kw-1) pixel halo of a (frame, ci-block)
//                         into shared memory (out-of-image pixels arrive as zeros = the
//                         spatial padding); the kh*kw spatial taps are shared-memory
//                         descriptor offsets into that one halo tile.  Accumulation is FP32
//                         in tensor memory; the epilogue adds the bias once, rounds once
//                         and stores NCTHW.
//
// Every wait on an mbarrier is bounded: when a limit expires the CTA records the
// wait site in a global status word, raises a shared abort flag so that its other
// roles stop too, releases its tensor memory and returns.
//
// Files: ccv3d_tc_layout.cuh (packing, staging, ring moves), ccv3d_tc_ptx.cuh (PTX wrappers), ccv3d_tc_conv.cuh (the
// implicit-GEMM kernel), ccv3d_tc_pointwise.cuh (the 1x1x1 streaming kernel).
#pragma once
#include "ccv3d_tc_layout.cuh"
#include "ccv3d_tc_ptx.cuh"
#include "ccv3d_tc_conv.cuh"
#include "ccv3d_tc_pointwise.cuh"
