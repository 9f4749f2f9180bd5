/*
 * ccv3d - cached causal Conv3D forward pass for NVIDIA B200 (sm_100a).
 *
 * C ABI.  Plain pointers and sizes only; every tensor pointer says whether it
 * is a DEVICE or a HOST address.  All tensors are dense and contiguous in the
 * stated index order (last index fastest).  Functions return a ccv3d_status;
 * nothing throws, aborts or traps.  A handle is not thread-safe; distinct
 * handles are independent.
 *
 * The operation (paper Section 4.1-4.2, Eq. (1) source time, Eq. (2) conv3d):
 * with Z = [cache ; x] concatenated along time (cache = the previous chunk's
 * last kt-1 input frames, oldest first; all zeros on the first chunk),
 *
 *   out[n,co,t,h,w] = b[co] + sum_{ci,dt,dh,dw} w[co,ci,dt,dh,dw]
 *                                * Z[n,ci,t+dt,h+dh-pad_h,w+dw-pad_w]      0 <= t < T
 *
 * (cross-correlation, unit stride and dilation, one group, zero spatial
 * padding pad_h=(kh-1)/2, pad_w=(kw-1)/2 so that H and W are preserved, causal
 * temporal padding of kt-1 frames supplied by the cache; the bias is added
 * exactly once), and
 *
 *   new_cache[n,ci,j,h,w] = Z[n,ci,T+j,h,w]                               0 <= j < kt-1
 *
 * i.e. the last kt-1 frames of the running input stream (for T < kt-1 this
 * keeps the newest frames of the old cache in front of x).
 */
#ifndef CCV3D_H_
#define CCV3D_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ccv3d_handle ccv3d_handle; /* opaque; one per convolution layer */

typedef enum { CCV3D_F32 = 0, CCV3D_BF16 = 1 } ccv3d_dtype;

typedef enum {
    CCV3D_OK = 0,
    CCV3D_ERR_INVALID_ARG = 1,    /* NULL pointer, non-positive size, bad enum */
    CCV3D_ERR_UNSUPPORTED = 2,    /* groups != 1 (Algorithm 1's reject list), extents beyond the limits stated at ccv3d_desc, a
                                     temporal padding that is not the causal one, or an entry point that does not take this layer */
    CCV3D_ERR_ALIGNMENT = 3,      /* a tensor pointer is not 16-byte aligned */
    CCV3D_ERR_ALIAS = 4,          /* out or new_cache overlaps an input (or each other) */
    CCV3D_ERR_ARCH = 5,           /* current device is not compute capability 10.x */
    CCV3D_ERR_NOMEM = 6,          /* device or host allocation failed */
    CCV3D_ERR_CUDA = 7,           /* a CUDA runtime/driver call or a launch failed */
    CCV3D_ERR_DEVICE_TIMEOUT = 8  /* a bounded wait inside a kernel gave up (see ccv3d_device_status) */
} ccv3d_status;

/* ccv3d_desc.flags */
#define CCV3D_FLAG_FORCE_SIMT 0x1u      /* BF16 layers: use the plain FP32-FMA kernel instead of the tensor-core kernel */
#define CCV3D_FLAG_OVERLAP 0x4u          /* tensor-core route: process large images in bands, staging band k+1 on a side stream while band k is convolved */
#define CCV3D_FLAG_TWO_KERNELS 0x10u     /* tensor-core route: run the staging pass as its own kernel before the convolution kernel instead of
                                            inside it (cooperative staging, the default for large calls with W % 8 == 0: four warps of
                                            every CTA stage a band of rows ahead of the tiles; only the first two bands go through
                                            the staging kernel) */
#define CCV3D_FLAG_FUSED 0x8u            /* tensor-core route without scratch memory: no channels-last staging copy; the kernel reads x and the cache
                                            by TMA and transposes in shared memory (needs W % 8 == 0, else the staged route is taken). Some 10 % slower
                                            than the default route; for callers that cannot afford the workspace. */
#define CCV3D_FLAG_F32_TENSOR 0x20u       /* FP32 layers: always use the tensor cores (3xTF32: each FP32 product as hi*hi + hi*lo + lo*hi of TF32
                                            operands, FP32 accumulate); the default sends layers with K = cin*kt*kh*kw > 8192, and calls that are
                                            both under 0.2 GFLOP and of K < 256, to the FP32-FMA kernel */
#define CCV3D_FLAG_NO_PAIR 0x40u          /* tensor-core route: never run tiles on pairs of CTAs (cta_group::2 MMAs with M = 256, each SM
                                            streaming half of every weight tile) - the default for layers with more than 128 output
                                            channels per tile and 3x3 or 1x1 spatial kernels */
#define CCV3D_FLAG_EPI_SILU 0x80u         /* epilogue activation (not part of the paper's operator): out = silu(conv + b), v / (1 + exp(-v)) in
                                            FP32 before the one output rounding; a residual (frame rings) is added after it */
#define CCV3D_FLAG_NO_TAIL_SPLIT 0x100u   /* never finish a launch with half-width output-channel tiles (the default on CTA pairs
                                            when the last wave of tiles would be at most half full) */
#define CCV3D_FLAG_TC_PER_TAP_A 0x2u    /* tensor-core kernel: fetch the activation tile once per tap (no halo reuse in shared memory) */

/* Layer description, fixed at create time (Algorithm 1's Require line: W, b, p, s, d, g).
 * The supported contract is the paper's (Section 4.1): any spatial stride, padding and dilation of the layer
 * inside each temporal tap (Eq. (2)), a temporal dilation d_t in the source time (Eq. (1)), one group - plus a
 * temporal stride s_t, which the paper's Algorithm 1 hands back to the framework (the encoder's temporal
 * downsampling layers) and which is here the same operator with source time t s_t + k d_t.  The output extents are
 *   H_o = floor((H + 2 pad_h - dilation[1] (kh-1) - 1) / stride[1]) + 1,   W_o likewise,
 *   T_o = floor((T - 1) / stride[0]) + 1                 (Eq. (3) with the causal pad supplied in full),
 * the history a call reads is dilation[0]*(kt-1) frames (the cache length; ccv3d_out_dims reports all four),
 * and out[n,co,t,ho,wo] = b + sum w[co,ci,k,a,c] * Z[n,ci, t s_t + k d_t, ho s_h + a d_h - pad_h, wo s_w + c d_w - pad_w].
 * Streaming with s_t > 1: chunk lengths that are multiples of s_t keep the phase of the output frames.
 * Layers with unit strides and dilations, odd kh and kw and size-preserving padding (pad = (k-1)/2) are the
 * "standard" geometry of the header comment; only they can use the fused, 1x1x1-streaming, allocation-free and
 * frame-ring paths.  Other geometries run on the tensor-core kernel too - BF16 layers always, FP32 layers as 3xTF32
 * under the rule stated at CCV3D_FLAG_F32_TENSOR, else on the FP32-FMA kernel: unit spatial strides through the same
 * staged copy and schedules (cooperative staging included; 3x3 kernels with dilation 2 keep the straight-line tap
 * loop), spatial strides through a phase-decomposed staged copy (BF16; s_h * s_w phase images in which neighbouring
 * output pixels are neighbours again; a 3x3 kernel with stride 2 and padding 1 runs on CTA pairs and under
 * cooperative staging like a standard layer) or, for FP32 layers and more than 16 phases, one strided TMA box per tap. */
typedef struct {
    int32_t cin, cout;            /* channels */
    int32_t kt, kh, kw;           /* kernel extent; 1 <= kt <= 8, 1 <= kh,kw <= 7 */
    int32_t pad_t, pad_h, pad_w;  /* pad_h, pad_w: symmetric spatial zero padding, 0..32.  pad_t: the temporal padding is causal - all
                                     dilation[0]*(kt-1) frames on the left, supplied by the cache, never zeros on the right; the
                                     framework-style value must describe the same total (2 pad_t = dilation[0]*(kt-1)) when that
                                     is even and is ignored otherwise. */
    int32_t stride[3];            /* {s_t, s_h, s_w}, 1..8 */
    int32_t dilation[3];          /* {d_t, d_h, d_w}, 1..8 */
    int32_t groups;               /* must be 1 */
    int32_t dtype;                /* ccv3d_dtype of x, cache, w, b and new_cache */
    int32_t out_dtype;            /* ccv3d_dtype of out: F32 layers -> F32; BF16 layers -> BF16 or F32 */
    uint32_t flags;               /* CCV3D_FLAG_* */
} ccv3d_desc;

/* Route counters (the paper's rho: calls, fast-path hits, rejected calls), per handle. */
typedef struct {
    uint64_t calls;           /* ccv3d_forward* calls */
    uint64_t ok;              /* calls that enqueued all their work */
    uint64_t tcgen05_bf16;    /* calls served by the BF16 tensor-core convolution kernel (NCTHW, host and frame-ring entry points) */
    uint64_t tcgen05_f32;     /* FP32 calls served by the tensor-core kernel as 3xTF32 */
    uint64_t pointwise;       /* 1x1x1 calls served by the streaming kernel that reads NCTHW directly */
    uint64_t simt;            /* calls served by the FP32-FMA kernel (FP32 layers, and BF16 layers on request) */
    uint64_t unsupported;     /* rejected: unsupported */
    uint64_t invalid;         /* rejected: invalid argument / alignment / alias */
    uint64_t cuda_error;      /* failed in a CUDA call */
    uint64_t device_timeout;  /* ccv3d_device_status reports that counted a kernel-side timeout */
    uint64_t kernel_launches; /* kernels launched by this handle since create */
} ccv3d_counters;

/*
 * Create a layer (Algorithm 1's derived-weight caching, done once: the
 * weights are repacked per tap into the tensor-core operand order and the
 * bias is widened to FP32 here, never per call).
 *   out_h   HOST   receives the handle.
 *   d       HOST   layer description; validated (CCV3D_ERR_UNSUPPORTED / INVALID_ARG).
 *   w_dev   DEVICE [cout,cin,kt,kh,kw] in d->dtype.  Read during the call (stream-ordered);
 *                  may be released after the stream has passed this point.
 *   b_dev   DEVICE [cout] in d->dtype, or NULL for a zero bias.
 *   stream  a cudaStream_t (NULL = default stream).
 * The handle owns: packed weights, FP32 bias, a status word, an optional
 * workspace (see ccv3d_forward).  The caller owns everything else.
 * A few environment variables are read here, for diagnosis only: CCV3D_LOG=1 prints one line per call on stderr
 * (entry point, shape, status, cumulative route counters); CCV3D_WAIT_LIMIT_MS (1..10000, default about one
 * second of SM clocks) bounds every wait inside the kernels; CCV3D_NO_PDL (any value) launches the frame-ring
 * kernels without programmatic stream serialization; CCV3D_NO_COOP_LAUNCH (any value; implied when the
 * process runs under Nsight Compute, which sets NV_COMPUTE_PROFILER_PERFWORKS_DIR) launches the
 * cooperative-staging kernels as ordinary launches (a profiler that replays kernels refuses cooperative launches of
 * clusters; only safe while nothing else runs on the device, since the CTAs of such a kernel wait for one another,
 * within the bound of every wait).
 */
ccv3d_status ccv3d_create(ccv3d_handle** out_h, const ccv3d_desc* d, const void* w_dev, const void* b_dev,
                          void* stream);

/*
 * One forward call on DEVICE buffers: Eq. (2) plus the cache update, all
 * enqueued on `stream` (asynchronous; no host synchronisation).
 *   x          DEVICE [N,cin,T,H,W]
 *   cache      DEVICE [N,cin,kt-1,H,W], or NULL = first chunk (all-zero history;
 *              the taps that would read it are skipped).  Ignored when kt == 1.
 *   out        DEVICE [N,cout,T,H,W] in out_dtype; fully overwritten.
 *   new_cache  DEVICE [N,cin,kt-1,H,W], or NULL to skip the update; fully overwritten,
 *              bit-exact copy of the last kt-1 frames of [cache ; x].  Ignored when kt == 1.
 *   (General geometry: out is [N,cout,T_o,H_o,W_o] and both caches hold dilation[0]*(kt-1) frames; T, H and W
 *   are always the INPUT extents.  See ccv3d_out_dims.)
 * out must not overlap x or cache; new_cache must not overlap x, cache or out
 * (CCV3D_ERR_ALIAS): ping-pong two cache buffers.  All pointers must be 16-byte aligned.
 * The current CUDA device must be the one the handle was created on (else CCV3D_ERR_INVALID_ARG).
 * With CCV3D_FLAG_OVERLAP large images are processed in bands of rows on three side streams owned by the handle
 * (staging of the next band overlaps the convolution of the current one); they fork from `stream` after
 * everything enqueued on it so far and join it before the call returns, so the caller only ever needs to order
 * against `stream`.
 * The tensor-core path keeps a channels-last staging copy of [cache ; x] in a
 * workspace: the caller's when one was lent with ccv3d_set_workspace (then no call
 * ever allocates), else one owned by the handle, (re)allocated when a call needs
 * more than the handle holds (that call synchronises the device), so steady-state
 * calls of one shape allocate nothing.  ccv3d_workspace_bytes tells the size in advance.
 */
ccv3d_status ccv3d_forward(ccv3d_handle* h, const void* x, const void* cache, void* out, void* new_cache,
                           int32_t N, int32_t T, int32_t H, int32_t W, void* stream);

/* Output extents and history length of a layer for an input of T x H x W (HOST outputs, each may be NULL). */
ccv3d_status ccv3d_out_dims(const ccv3d_handle* h, int32_t T, int32_t H, int32_t W, int32_t* out_t_host,
                            int32_t* out_h_host, int32_t* out_w_host, int32_t* cache_frames_host);

/*
 * ccv3d_forward with a history shorter than kt-1 frames (the paper's Table 1 lists such calls: T_c = 1 with
 * a temporal kernel of 3).  cache is DEVICE [N,cin,cache_frames,H,W] with 0 <= cache_frames <= kt-1 (NULL allowed
 * only with cache_frames = 0); the kt-1-cache_frames frames before it do not exist and contribute zero, exactly as
 * Eq. (1)-(3) prescribe with p_l = kt-1-cache_frames (their taps are skipped).  new_cache still receives kt-1
 * frames, zero where the stream has no history yet.  Everything else as ccv3d_forward, which is this call with
 * cache_frames = kt-1 (or 0 for a NULL cache).
 */
ccv3d_status ccv3d_forward_ex(ccv3d_handle* h, const void* x, const void* cache, int32_t cache_frames, void* out,
                              void* new_cache, int32_t N, int32_t T, int32_t H, int32_t W, void* stream);

/*
 * ccv3d_forward without any allocation.  (The paper has no counterpart: its route runs inside a framework
 * that allocates freely.)
 *
 * Who needs it: code that must not, or cannot, call the device allocator when it runs the layer - a real-time
 * loop that may not block on cudaMalloc, a callback running where allocation is forbidden, an embedding
 * runtime that owns all device memory and hands this library none.  ccv3d_forward keeps its channels-last
 * staging copy in a workspace it allocates on demand; this entry point keeps it instead in a fixed 32 MiB
 * array that is part of the library's device image, so it calls neither cudaMalloc nor cudaFree nor any other
 * allocating routine.  Every GPU whose context loads the library holds those 32 MiB until the process exits.
 *
 * Same arguments, meaning, aliasing and alignment rules as ccv3d_forward (x, cache, out, new_cache are DEVICE
 * pointers owned by the caller).  Differences:
 *   - BF16 tensor-core layers only (a handle created with CCV3D_FLAG_FORCE_SIMT or with FP32 data, and the
 *     CCV3D_FLAG_TC_PER_TAP_A mode, return CCV3D_ERR_UNSUPPORTED);
 *   - the staging copy must fit the 32 MiB array, otherwise the call returns CCV3D_ERR_UNSUPPORTED and launches
 *     nothing.  Its size is N * (kt-1+T) * cin_pad * H * W * 2 bytes, cin_pad = cin rounded up to a multiple of 32
 *     (this entry point always stages, so the bound holds also for the layers for which ccv3d_workspace_bytes
 *     reports 0 because ccv3d_forward would not stage them: 1x1x1 layers and CCV3D_FLAG_FUSED handles);
 *   - the first call on each device looks up the array's device address (a one-time set-up with that device
 *     current); make that first call outside any stream capture;
 *   - all handles and all calls on one GPU share the one array.  Calls that may overlap on the GPU (different
 *     streams, no ordering between them) race on it and corrupt each other's results: order them.  The array
 *     keeps the previous call's bytes; each call overwrites everything it later reads, so stale contents are
 *     never consumed and nothing has to be cleared.
 */
ccv3d_status ccv3d_forward_static(ccv3d_handle* h, const void* x, const void* cache, void* out, void* new_cache,
                                  int32_t N, int32_t T, int32_t H, int32_t W, void* stream);

/*
 * The same call on HOST buffers (same shapes and meaning as above): copies x
 * and cache to device staging owned by the handle, runs ccv3d_forward, copies
 * out and new_cache back, and returns after the stream has completed.  Pinned
 * host memory makes the copies asynchronous with respect to each other.
 * Standard BF16 tensor-core layers with cin % 32 == 0 and frames of a few MB run
 * piece by piece instead (upload of piece k+1, convolution of piece k on a frame
 * ring and download of piece k-1 overlap on three streams; a piece is a frame, or -
 * frames of tens of MB - a band of rows of a frame with its halo rows; same bits,
 * since the operator streams exactly in time and is local in space): the call then
 * takes about as long as the slower PCIe direction alone.
 */
ccv3d_status ccv3d_forward_host(ccv3d_handle* h, const void* x_host, const void* cache_host, void* out_host,
                                void* new_cache_host, int32_t N, int32_t T, int32_t H, int32_t W, void* stream);

/*
 * Streaming form of ccv3d_forward_host: the temporal history (the cache of Eq. (1)'s Z = [C ; X]) stays on the
 * device between calls, in a frame ring the handle owns, so a call moves only x (HOST [N,cin,T,H,W]) up and out
 * (HOST [N,cout,T,H,W]) down - the cache never crosses the bus.  reset != 0 starts a new stream (first chunk: no
 * history); a change of N, H or W, or any other host entry point used on the handle in between, starts a new
 * stream as well.  Same piece-by-piece pipeline (one history ring per band of rows), same results bit for bit as ccv3d_forward_host with the cache
 * carried by the caller.  Synchronous like ccv3d_forward_host.  Layers and sizes the pipelined path does not take
 * (see ccv3d_forward_host: standard geometry, BF16, cin a multiple of the channel block, a few MB per frame)
 * return CCV3D_ERR_UNSUPPORTED; any T >= 1.
 */
ccv3d_status ccv3d_forward_host_stream(ccv3d_handle* h, const void* x_host, void* out_host, int32_t reset, int32_t N,
                                       int32_t T, int32_t H, int32_t W, void* stream);

/* Bytes of workspace a ccv3d_forward / ccv3d_forward_ex call of this shape needs (0 for the FP32-FMA route, the
 * 1x1x1 streaming kernel and the fused route). */
ccv3d_status ccv3d_workspace_bytes(const ccv3d_handle* h, int32_t N, int32_t T, int32_t H, int32_t W,
                                   uint64_t* bytes_host);

/*
 * Lend the handle a workspace (the lowering's extra memory - Section 7.2 of the paper lists its temporaries as
 * the overhead that is left - made the caller's to place).  From now on ccv3d_forward / ccv3d_forward_ex keep the
 * staging copy in ws_dev (DEVICE, 256-byte aligned, `bytes` long, owned by the caller, who keeps it alive while
 * the handle may use it) and never allocate, free or synchronise: a call that needs more than `bytes` returns
 * CCV3D_ERR_NOMEM before it launches anything.  Such calls are legal inside a stream capture.
 * Several handles may be lent the same buffer - a decoder of many layers needs one workspace of the largest
 * single need (the maximum of ccv3d_workspace_bytes over its calls), not one per layer: the buffer only holds
 * data between the kernels of one call.  Calls that share a workspace must be ordered on the GPU (same stream,
 * or events); calls that may overlap race on it.  ws_dev = NULL or bytes = 0 returns the handle to a workspace
 * of its own, allocated on demand.  CCV3D_ERR_ALIGNMENT for a misaligned pointer.  The host entry points and
 * ccv3d_forward_static do not use this workspace.
 */
ccv3d_status ccv3d_set_workspace(ccv3d_handle* h, void* ws_dev, uint64_t bytes);

/* Destroy a handle and free what it owns.  NULL is accepted. */
ccv3d_status ccv3d_destroy(ccv3d_handle* h);

/* Copy the counters (HOST struct). */
ccv3d_status ccv3d_get_counters(const ccv3d_handle* h, ccv3d_counters* out_host);

/*
 * After the caller has synchronised the stream: CCV3D_OK, or
 * CCV3D_ERR_DEVICE_TIMEOUT if a kernel gave up on a bounded wait since the
 * last query (the outputs of that call are then undefined).  Reading clears
 * the word.  detail_host (may be NULL) receives the raw word:
 * bits 0-7 wait site, bits 8-31 block index.
 */
ccv3d_status ccv3d_device_status(ccv3d_handle* h, uint32_t* detail_host);

/*
 * Optional per-kernel timing for benchmarks.  While enabled, every ccv3d_forward records CUDA events on the
 * caller's stream before the staging kernel, between the two kernels and after the convolution kernel (up to
 * 1024 calls are kept; later calls overwrite the oldest).  ccv3d_profile_read must be called after the stream
 * has been synchronised; it returns the summed device time of the staging (or FP32-FMA route: zero) and of the
 * convolution kernel over the calls recorded since the last read, and their number, then clears the record.
 * All three outputs are HOST pointers.
 */
ccv3d_status ccv3d_profile_enable(ccv3d_handle* h, int32_t enable);
ccv3d_status ccv3d_profile_read(ccv3d_handle* h, double* stage_ms_host, double* conv_ms_host, int64_t* calls_host);

/*
 * Self-test of the bounded-wait mechanism (no counterpart in the paper).  Enqueues a one-block kernel that waits
 * on a barrier nothing will ever signal, with the given limit (1..1000 ms).  The wait gives up, the kernel
 * returns normally and the handle's status word is set, so that after synchronising the stream
 * ccv3d_device_status returns CCV3D_ERR_DEVICE_TIMEOUT with detail 0x7F in its low byte.  Nothing faults,
 * traps or hangs; the handle stays usable.
 */
ccv3d_status ccv3d_selftest_wait_timeout(ccv3d_handle* h, int32_t limit_ms, void* stream);

/* Static, human-readable name of a status code. */
const char* ccv3d_status_string(ccv3d_status s);

/*
 * Element-wise glue of a streamed decoder chain (not part of the paper's
 * operator; provided so that a chain of layers runs entirely in this library).
 * All tensors DEVICE, BF16, contiguous.
 *   ccv3d_add_bf16:        y[i] = bf16(float(a[i]) + float(b[i])),  n elements (round to nearest even).
 *   ccv3d_upsample_bf16:   y[N,C,T*rt,H*2,W*2] = nearest-neighbour repeat of x[N,C,T,H,W]
 *                          (each pixel 2x2, each frame rt times, rt >= 1).
 */
ccv3d_status ccv3d_add_bf16(const void* a, const void* b, void* y, int64_t n, void* stream);
ccv3d_status ccv3d_upsample_bf16(const void* x, void* y, int32_t N, int32_t C, int32_t T, int32_t H, int32_t W,
                                 int32_t rt, void* stream);

/*
 * Image-row slabs, the data movement of a height-split layer (each GPU owns a band of image rows and needs
 * the kernel's halo rows of its neighbours, the per-tap 2-D correlation of Eq. (2) being local in h):
 * for every one of `planes` planes (a plane = one (n, c, t) image of rows of row_bytes bytes)
 *     dst plane p, rows dst_row0 .. dst_row0+rows-1   <-   src plane p, rows src_row0 .. src_row0+rows-1,
 * dst planes dst_H rows high, src planes src_H rows high (DEVICE, any element type).  src == NULL writes zeros
 * (the image edge, where the halo is the layer's zero padding).  Packs halo rows into a contiguous send buffer
 * (dst_H = rows), unpacks a received one, and places a band inside its slab.  16-byte vector copies when
 * row_bytes and both row addresses are multiples of 16, byte copies otherwise.  Stream-ordered.
 * CCV3D_ERR_INVALID_ARG for NULL dst, non-positive sizes or row ranges outside their planes.
 */
ccv3d_status ccv3d_rows_copy(void* dst, int32_t dst_H, int32_t dst_row0, const void* src, int32_t src_H,
                             int32_t src_row0, int64_t planes, int32_t rows, int64_t row_bytes, void* stream);

/*
 * ------------------------------------------------------------------------------------------------
 * Resident activations: frame rings in the tensor-core operand order
 * ------------------------------------------------------------------------------------------------
 * Algorithm 1 ends every call by restoring the framework layout and returning a contiguous tensor, and
 * Section 7.2 names the temporaries around the call (folded inputs, the cache concatenation, accumulation
 * buffers) as the overhead that is left.  Between two layers of one decoder nobody needs the framework layout,
 * so this library can keep the activations in the order its tensor-core kernel consumes, and keep the temporal
 * history in place instead of copying a cache:
 *
 *   a frame ring is a DEVICE BF16 buffer  [N][F][C/KB][H][W][KB]  (KB = 64 or 32 channels innermost),
 *   F >= T + kt - 1 frame slots used modulo F.
 *
 * A layer reads its input x from slots x_slot .. x_slot+T-1 (mod F) of its input ring and its history from the
 * kt-1 slots before x_slot - the frames a previous call left there, so Eq. (1)'s source frame of tap dt for
 * output t is simply slot x_slot + t + dt - (kt-1), and there is no cache tensor, no concatenation and no cache
 * update.  It writes its output either into the next layer's ring (channels-last, by TMA store) or as NCTHW.
 * An optional residual (a ring holding cout channels) is added in the epilogue with the chain's rounding:
 *   out = bf16( float(bf16(conv + b)) + float(res) ),
 * i.e. bit-identical to ccv3d_forward followed by ccv3d_add_bf16.
 * Results are those of ccv3d_forward on the same values (same accumulation order per output element).
 * Rings have no width restriction (any W; the NCTHW TMA paths need W % 8 == 0).
 */
typedef struct {
    void*   base;        /* DEVICE, 16-byte aligned, ccv3d_ring_bytes() bytes; owned by the caller */
    int32_t N, C, F, H, W;
    int32_t KB;          /* channels per innermost block: 64 or 32; C % KB == 0.  A ring read by a layer must use
                            KB = 64 if cin % 64 == 0 else 32 (ccv3d_ring_kb(cin)). */
} ccv3d_ring;

/* 64 if C % 64 == 0, 32 if C % 32 == 0, else 0 (such a tensor cannot live in a ring). */
int32_t ccv3d_ring_kb(int32_t C);
/* N*F*C*H*W*2, or 0 for an invalid geometry. */
uint64_t ccv3d_ring_bytes(const ccv3d_ring* r);

/* x DEVICE [N,C,T,H,W] BF16 -> ring slots (slot0 + t) mod F, t < T <= F.  Stream-ordered. */
ccv3d_status ccv3d_ring_load(const ccv3d_ring* r, int32_t slot0, const void* x, int32_t T, void* stream);
/* ring slots (slot0 + t) mod F -> y DEVICE [N,C,T,H,W] BF16 (bit-exact inverse of ccv3d_ring_load). */
ccv3d_status ccv3d_ring_store(const ccv3d_ring* r, int32_t slot0, void* y, int32_t T, void* stream);
/* Nearest-neighbour 2x2 spatial upsample with frame repeat rt between rings of equal C and KB:
 * out slot (out_slot0 + t*rt + j) mod F_out <- in slot (in_slot0 + t) mod F_in, j < rt; out->H = 2*in->H,
 * out->W = 2*in->W. */
ccv3d_status ccv3d_upsample_ring(const ccv3d_ring* in, int32_t in_slot0, const ccv3d_ring* out, int32_t out_slot0,
                                 int32_t T, int32_t rt, void* stream);

/*
 * One forward call on resident activations (BF16 tensor-core layers only; others: CCV3D_ERR_UNSUPPORTED).
 *   in          ring with C = cin, KB = ccv3d_ring_kb(cin), F >= T + kt - 1; x frame t is slot (x_slot + t) mod F.
 *   hist_frames how many of the kt-1 slots before x_slot hold history (0..kt-1); older ones do not exist and
 *               contribute zero (first chunks).  The caller advances x_slot by T per call, so the history is
 *               whatever the previous calls wrote; nothing is copied.
 *   res         optional ring with C = cout (any KB), same N, H, W: residual frame t is slot (res_slot + t) mod F.
 *               May be the input ring itself.  Requires out_dtype BF16.
 *   out_ring    ring with C = cout, same N, H, W; output frame t goes to slot (out_slot + t) mod F (only those
 *               slots are written).  Must not overlap `in` or `res`.  Requires cout/ceil(cout/256) % 32 == 0.
 *   out_ncthw   DEVICE [N,cout,T,H,W] in out_dtype.  Exactly one of out_ring / out_ncthw is non-NULL.
 * All ring structs are HOST pointers read during the call.  Stream-ordered, allocates nothing.
 */
ccv3d_status ccv3d_forward_ring(ccv3d_handle* h, const ccv3d_ring* in, int32_t x_slot, int32_t hist_frames,
                                const ccv3d_ring* res, int32_t res_slot, const ccv3d_ring* out_ring,
                                int32_t out_slot, void* out_ncthw, int32_t T, void* stream);

/*
 * ccv3d_forward_ring with a nearest-neighbour upsample fused into the store: out_ring has 2H x 2W pixels and
 * F >= T*rt slots; output frame t is written to the rt slots (out_slot + t*rt + j) mod F, every pixel 2x2 times
 * (the epilogue issues 4*rt strided TMA stores of the same shared-memory tile).  Bit-identical to
 * ccv3d_forward_ring into an H x W ring followed by ccv3d_upsample_ring.  rt >= 1; everything else as
 * ccv3d_forward_ring with a ring output.
 */
ccv3d_status ccv3d_forward_ring_up(ccv3d_handle* h, const ccv3d_ring* in, int32_t x_slot, int32_t hist_frames,
                                   const ccv3d_ring* res, int32_t res_slot, const ccv3d_ring* out_ring, int32_t out_slot,
                                   int32_t rt, int32_t T, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* CCV3D_H_ */
