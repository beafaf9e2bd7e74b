/*
 * rt3d.h - C ABI of the B200 library for the inference hot path of RT3D
 * (arXiv 2007.09835): forward 3-D convolution over NDHWC video activations with weights
 * pruned to the paper's kernel-group-structured (KGS) or vanilla structured sparsity.
 *
 * Conventions
 *   - Plain C linkage, no exceptions; every call returns an rt3d_status.
 *   - "host" / "device" on a pointer says where the memory must live.  Activations,
 *     bias and outputs are DEVICE memory owned by the caller; dense weights and masks
 *     handed to the packers are HOST memory owned by the caller.  The library owns an
 *     rt3d_packed handle (host canonical arrays + per-device weight blobs) until
 *     rt3d_packed_free.
 *   - Compute calls enqueue work on the given CUDA stream (a cudaStream_t passed as
 *     void*, NULL = default stream) and return without synchronising.  The first compute
 *     call that uses a handle on a device uploads the handle's device blobs (allocation +
 *     copy), and the first call of a shape that splits K grows the handle's scratch buffer;
 *     later calls allocate nothing.  rt3d_packed_prepare does the upload ahead of time.
 *     That scratch belongs to the handle: two calls on the SAME handle whose kernels may overlap
 *     on the GPU (different streams) must be serialised by the caller.
 *   - Kernels are launched with programmatic stream serialisation: a kernel's set-up may overlap
 *     the tail of the previous kernel on its stream, but it reads and writes global memory only
 *     after that kernel has completed (environment RT3D_PDL=0 turns the attribute off).
 *   - Argument errors are detected on the host before anything is launched.
 *   - Activation layout: NDHWC = [n][t][h][w][c] with a channel pitch c_stride >= c
 *     (elements between consecutive voxels).  An output tensor's padding channels c .. c_stride-1 are left as
 *     they are, except those that share the last 16-byte unit of a voxel row with real channels (bf16:
 *     channels c .. 8*ceil(c/8)-1): the tensor-core kernels' bulk stores move whole 16-byte units and write
 *     zeros there.  (A channel slice of a wider tensor that is followed by another slice starts that slice
 *     on a 16-byte boundary anyway, so only a row's last slice can have such channels.)  Weight layout handed to the packers:
 *     [M][N][Kt][Kh][Kw], M filters, N input channels (Section 3; the paper's kernel depth
 *     K_d is the temporal extent Kt).  Kernel location index kpos = (kt*Kh + kh)*Kw + kw.
 *   - Convolution is cross-correlation with zero padding, no dilation; output extent
 *     floor((in + 2*pad - K)/stride) + 1 per axis.
 */
#ifndef RT3D_H_
#define RT3D_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  RT3D_OK = 0,
  RT3D_ERR_INVALID_ARG = 1,            /* NULL pointer, non-positive extent, bad enum            */
  RT3D_ERR_SHAPE = 2,                  /* tensor extents / dtypes do not fit the weights/params  */
  RT3D_ERR_MASK_NOT_GROUP_UNIFORM = 3, /* mask differs inside one (kernel group, location)       */
  RT3D_ERR_UNSUPPORTED = 4,            /* valid request this build cannot run                    */
  RT3D_ERR_ALLOC = 5,                  /* host or device allocation failed                       */
  RT3D_ERR_CUDA = 6,                   /* a CUDA runtime / driver call failed                    */
  RT3D_ERR_TIMEOUT = 7,                /* a bounded device-side wait gave up (see rt3d_last_device_status) */
  RT3D_ERR_WORKSPACE = 8,              /* rt3d_conv3d_sparse_noalloc: the call needs more than the fixed workspace */
  RT3D_ERR_NOT_PREPARED = 9            /* rt3d_conv3d_sparse_noalloc: handle was not prepared on this device */
} rt3d_status;

typedef enum { RT3D_F32 = 0, RT3D_BF16 = 1 } rt3d_dtype;

/* Kernel family selection for the convolution calls. */
typedef enum {
  RT3D_ALGO_AUTO = 0,   /* tensor-core kernel when the shape allows it, else the CUDA-core kernel */
  RT3D_ALGO_SIMT = 1,   /* CUDA-core kernel driven by the canonical packed index (any shape)      */
  RT3D_ALGO_UMMA = 2,   /* tcgen05 tensor-core kernel, one CTA per tile; RT3D_ERR_UNSUPPORTED if not applicable */
  RT3D_ALGO_UMMA_PAIR = 3, /* tcgen05 kernel on CTA pairs (two tiles per MMA, weight tile shared by the
                             pair); RT3D_ERR_UNSUPPORTED if not applicable                        */
  RT3D_ALGO_UMMA_HALO = 4, /* tcgen05 kernel on CTA pairs for thin stride-1 layers: the layer's packed weights
                             stay in shared memory and each output tile's input block (with halo) is
                             staged once for all kernel locations; RT3D_ERR_UNSUPPORTED if the weights
                             plus two input blocks do not fit, M > 256, or a stride is not 1      */
  RT3D_ALGO_UMMA_SUB = 5   /* tcgen05 kernel that skips pruned kernel locations per block of 16 output x 16
                             input channels (input tiles held in tensor memory, eight issuing warps).
                             Never chosen by RT3D_ALGO_AUTO: on B200 it is slower than multiplying the
                             zero-filled tiles (see the kernel's header comment); kept as the measured
                             answer to "can skipping at the paper's group sizes pay on this hardware".
                             RT3D_ERR_UNSUPPORTED for dense handles, fused pooling and fp32         */
} rt3d_algo;

/* NDHWC activation tensor in DEVICE memory (HOST memory for the *_host entry point), caller-owned. */
typedef struct {
  void*   data;          /* 16-byte aligned                                                      */
  int32_t n, t, h, w, c; /* logical extents                                                      */
  int32_t c_stride;      /* elements between voxels, >= c                                        */
  int32_t dtype;         /* rt3d_dtype                                                           */
} rt3d_tensor;

typedef struct {
  int32_t st, sh, sw;    /* strides  (>= 1)                                                      */
  int32_t pt, ph, pw;    /* zero padding on both sides of each axis (>= 0)                       */
  int32_t relu;          /* nonzero: y = max(y, 0) fused after the bias                          */
  int32_t algo;          /* rt3d_algo                                                            */
  int32_t x_pad_zero;    /* nonzero: the caller guarantees that the padding channels c..c_stride-1 of x
                            hold zeros.  Never needed for correctness (by default no kernel lets them
                            reach the result); it lets the small-C_in kernel fetch whole image rows in
                            one request instead of one voxel at a time                              */
  int32_t concurrent;    /* nonzero: other kernels may run on the device while this call does (parallel
                            streams).  The library then avoids plans whose CTAs wait for one another (the
                            tail split of the CTA-pair kernel), which need the whole grid resident at once */
} rt3d_conv_params;

typedef struct rt3d_packed rt3d_packed;   /* opaque; immutable after creation */

/* Host pointers into a handle's canonical arrays; valid until rt3d_packed_free. */
typedef struct {
  int32_t M, N, Kt, Kh, Kw, g_m, g_n, P, Q, Ks;
  int32_t dtype;               /* rt3d_dtype of `tiles`                                          */
  int32_t is_vanilla;          /* every group keeps all or none of its locations                 */
  int32_t is_dense;            /* created by rt3d_pack_dense                                     */
  int64_t nnz;                 /* kept (group, location) entries                                 */
  const int32_t*  group_ptr;   /* [P*Q + 1] CSR offsets, group id = p*Q + q                      */
  const uint16_t* pos_idx;     /* [nnz] kpos, strictly ascending inside a group                  */
  const void*     tiles;       /* [nnz][g_m][g_n] float or bf16 bits (round-to-nearest-even);
                                  tiles[e][i][j] = W[p*g_m+i][q*g_n+j][kpos(e)], 0 where the
                                  kernel does not exist (ragged last groups)                     */
} rt3d_packed_view;

/*
 * rt3d_pack_kgs - weight reorganisation for KGS / vanilla sparsity.
 * Section 3: the weight tensor is partitioned into aligned groups of g_m x g_n kernels
 * (P = ceil(M/g_m), Q = ceil(N/g_n), Section 4); inside a group every kernel location
 * (kt,kh,kw) is kept or pruned for all kernels together, which is whole-column removal in
 * the group's weight matrix.  The pack keeps, per group, the list of kept locations and one
 * compact g_m x g_n tile per kept location (the compile-time weight reordering step of
 * Section 5.2).  Vanilla sparsity (whole groups removed) is the special case where each
 * group keeps all or no locations.
 *   w     host, [M][N][Kt][Kh][Kw] float
 *   mask  host, same shape, uint8, nonzero = keep; NULL = keep everything.  The mask is
 *         authoritative: kept weights are stored even if zero, pruned ones dropped even if not.
 *   g_m, g_n  group size, 1..256 each (the paper prefers g_n = 4, g_m = 4 or 8; groups wider than 8
 *             run on the tensor-core kernels only);  Kt*Kh*Kw <= 65535
 *   compute_dtype  storage/compute precision of the tiles (RT3D_F32, or RT3D_BF16 = RNE-rounded)
 *   out   receives the new handle
 * Errors: INVALID_ARG, MASK_NOT_GROUP_UNIFORM (mask is not a KGS mask), ALLOC.
 * Pure host work: usable without a GPU.
 */
rt3d_status rt3d_pack_kgs(const float* w, const uint8_t* mask, int M, int N, int Kt, int Kh, int Kw,
                          int g_m, int g_n, int compute_dtype, rt3d_packed** out);

/* rt3d_pack_dense - handle for the unpruned layer (the "RT3D (Dense)" path of Table 2):
 * every location of every kernel kept.  Same argument rules as rt3d_pack_kgs. */
rt3d_status rt3d_pack_dense(const float* w, int M, int N, int Kt, int Kh, int Kw,
                            int compute_dtype, rt3d_packed** out);

/* Read-only view of the canonical arrays (for bit-exact checks of the pack). */
rt3d_status rt3d_packed_view_get(const rt3d_packed* p, rt3d_packed_view* view);

/* Inverse of the pack: w_out host [M][N][Kt][Kh][Kw] float, zeros at pruned locations
 * (bf16 handles return the rounded values widened to float). */
rt3d_status rt3d_unpack_to_dense(const rt3d_packed* p, float* w_out);

/* Inverse of the tensor-core weight layout the handle would upload for bundles of
 * `n_tile` output channels (0 = the library's choice): w_out as above.  Lets a host-only
 * test check that derived layout against the canonical one. */
rt3d_status rt3d_unpack_device_layout(const rt3d_packed* p, int n_tile, float* w_out);
/* The same for the t-grouped order of that layout (steps ordered by (kh, kw), channel chunk, kt; the runs that
 * differ only in kt are the groups whose steps share one staged input tile in the CTA-pair kernel).  Also checks
 * the group tables: RT3D_ERR_INVALID_ARG if the groups do not tile every bundle's list or a group mixes
 * locations other than along kt. */
rt3d_status rt3d_unpack_device_layout_tgroups(const rt3d_packed* p, int n_tile, float* w_out);

/* The same check for the layout of the sub-tile kernel (RT3D_ALGO_UMMA_SUB): w_out is rebuilt from the
 * 16 x 16 weight blocks and the step headers; RT3D_ERR_INVALID_ARG if they are inconsistent (a non-zero
 * weight outside the tensor, a block index out of range, a first step that does not start every range of
 * its bundle).  Pure host work. */
rt3d_status rt3d_unpack_sub_layout(const rt3d_packed* p, int n_tile, float* w_out);

/* Upload the handle's device blobs to the current CUDA device now (otherwise done by the
 * first compute call), and look up, once per device, the device address of the fixed workspace of
 * rt3d_conv3d_sparse_noalloc (that look-up may make the CUDA runtime load this library's module on the
 * device, which is when the driver sets the workspace's memory aside).  Call it before any stream capture.
 * Synchronises the device. */
rt3d_status rt3d_packed_prepare(rt3d_packed* p);

void rt3d_packed_free(rt3d_packed* p);

/*
 * rt3d_conv3d_sparse - the hot path: y = act(bias + conv3d(x, W (.) mask)), iterating only
 * the kept (group, location) entries of the packed index (Section 3: pruning a location in a group removes
 * a whole column of the group's weight matrix, and what is left is again a dense, only smaller, product).
 *   x, y   device tensors; x.c == N, y.c == M, y extents = output extents of (x, params);
 *          dtypes equal the handle's compute dtype.  bf16: c_stride multiple of 8, fp32:
 *          multiple of 4; data 16-byte aligned.  x and y must not overlap.
 *   w      handle from rt3d_pack_kgs (or rt3d_pack_dense)
 *   bias   device, [M] float, or NULL
 *   p      strides, padding, fused ReLU, kernel family
 *   stream cudaStream_t as void*
 * Accumulation is fp32; bf16 outputs are rounded once after bias and ReLU.
 * Errors: INVALID_ARG, SHAPE, UNSUPPORTED, ALLOC/CUDA (first-use upload), and nothing is
 * launched on error.  A bounded device-side wait that gives up is reported later by
 * rt3d_last_device_status.
 */
rt3d_status rt3d_conv3d_sparse(const rt3d_tensor* x, const rt3d_packed* w, const float* bias,
                               const rt3d_conv_params* p, rt3d_tensor* y, void* stream);

/* rt3d_conv3d_dense - same operation for a handle from rt3d_pack_dense: all locations
 * iterated, no index lookups (the dense baseline the paper compares its sparse path with). */
rt3d_status rt3d_conv3d_dense(const rt3d_tensor* x, const rt3d_packed* w, const float* bias,
                              const rt3d_conv_params* p, rt3d_tensor* y, void* stream);

/*
 * Fused layer boundaries (Section 5.2 says the paper's framework optimises the computation graph
 * without detailing how; these two fusions are the ones its models need).
 *   residual  device tensor with the extents, dtype and alignment rules of the un-pooled output
 *             (c == M), added to conv + bias BEFORE the ReLU of p->relu; NULL = none.  Must not
 *             overlap y.  (R(2+1)D block end: y = relu(conv(x) + shortcut).)
 *   pool_t/h/w  max-pool window applied AFTER the activation, window = stride, no padding, each
 *             1 or 2 (1,1,1 = none); y then has extents floor(To/pool_t) x floor(Ho/pool_h) x
 *             floor(Wo/pool_w).  (C3D: conv + ReLU + 1x2x2 or 2x2x2 pool.)
 */
typedef struct {
  const rt3d_tensor* residual;
  int32_t pool_t, pool_h, pool_w;
} rt3d_fusion;

/* rt3d_conv3d_sparse_fused - rt3d_conv3d_sparse (or the dense path for a dense handle) with the
 * fusions above: y = pool(act(bias + conv(x, W (.) mask) + residual)).  Same argument rules; bf16
 * results are rounded once, after the activation (pooling commutes with that rounding).
 * RT3D_ERR_UNSUPPORTED when a fusion cannot be applied to this call (pooling needs the tensor-core
 * kernels, tile shapes that hold whole windows and output bundles of whole 32-channel pieces); the
 * caller then runs the steps separately.  With p->algo == RT3D_ALGO_AUTO pooling is also declined
 * that way for layers with so few output tiles that the library would split K across SMs (the split
 * plus a separate pool launch is the faster plan); RT3D_ALGO_UMMA fuses regardless. */
rt3d_status rt3d_conv3d_sparse_fused(const rt3d_tensor* x, const rt3d_packed* w, const float* bias,
                                     const rt3d_conv_params* p, const rt3d_fusion* fusion, rt3d_tensor* y,
                                     void* stream);

/*
 * rt3d_conv2plus1d_fused - a factorised (2+1)D convolution in one launch: a spatial 1 x Kh x Kw
 * convolution followed by a temporal Kt x 1 x 1 convolution (the R(2+1)D building block among the
 * paper's models, Section 5.1), both with KGS-pruned (or dense) packed weights:
 *     mid = round_bf16(act_s(bias_s + conv(x, W_s (.) mask_s)))        act_s = ReLU iff p_s->relu
 *     y   = act_t(bias_t + conv(mid, W_t (.) mask_t) + residual)       act_t = ReLU iff p_t->relu
 * i.e. exactly what rt3d_conv3d_sparse on (x, w_s) into a bf16 tensor `mid`, then
 * rt3d_conv3d_sparse_fused on (mid, w_t, residual) compute, but `mid` (usually the widest tensor
 * of the block) stays in shared memory / TMEM and never reaches device memory.
 *   x, y, residual   device NDHWC tensors as elsewhere; residual has y's extents and dtype, or NULL.
 *                    y must not overlap x or residual.
 *   w_s, w_t         packed handles (w_t->N == w_s->M); bias_s [w_s->M], bias_t [w_t->M]: device
 *                    fp32 or NULL.  p_s / p_t: strides, padding, relu of the two convolutions
 *                    (algo ignored).
 * Shape and argument errors are reported as by the separate calls and nothing is launched.
 * RT3D_ERR_UNSUPPORTED (nothing launched; run the two layers separately) unless: bf16; w_s is
 * 1 x Kh x Kw with at most 64 input channels; w_t is 3 x 1 x 1 with temporal padding 1; every stride 1;
 * at most 256 intermediate and 256 output channels with 2*ceil16(mid) + 3*ceil16(out) <= 512; every
 * temporal tap keeps at least one weight group; both packed weight tensors plus one intermediate
 * frame of a 16 x 8 patch fit in shared memory; compute capability 10.x.
 * rt3d_last_plan reports kernel 5.  Same stream, ownership and error conventions as above.
 */
rt3d_status rt3d_conv2plus1d_fused(const rt3d_tensor* x, const rt3d_packed* w_s, const float* bias_s,
                                   const rt3d_conv_params* p_s, const rt3d_packed* w_t, const float* bias_t,
                                   const rt3d_conv_params* p_t, const rt3d_tensor* residual, rt3d_tensor* y,
                                   void* stream);

/*
 * rt3d_conv3d_sparse_noalloc - rt3d_conv3d_sparse for callers that must not allocate.
 * (No counterpart in the paper: this is a deployment variant of the tensor-core kernel.)
 * Some callers cannot call cudaMalloc at the point where they run a layer: code inside a
 * real-time or latency-critical loop, code that runs while another component owns the device's
 * memory budget, or a host thread that must never block on the allocator's device-wide
 * synchronisation.  For them this entry point runs the same tensor-core convolution, including its
 * K-split variant whose fp32 partial tiles need scratch memory, without any allocation: the scratch
 * is a fixed array inside the library (16 MiB of partial tiles plus 4 KiB of counters, resident on
 * every GPU that loads the library until the process exits).
 *   - Same arguments, layouts and alignment rules as rt3d_conv3d_sparse (device x, y, bias); bf16 only.
 *   - Everything that does need an allocation must exist already: call rt3d_packed_prepare(w) on this
 *     device beforehand, else RT3D_ERR_NOT_PREPARED.  Shapes the tensor-core kernel does not take
 *     (fp32, channel pitch not a multiple of 8, p->algo == RT3D_ALGO_SIMT) give RT3D_ERR_UNSUPPORTED.
 *   - K is split S ways, S = min(8, SMs / output tiles, K steps / 8), at least 1, where an output
 *     tile is 128 voxels x up to 256 channels and a K step is one kernel location x 64 input
 *     channels that some kernel group of the tile's channels keeps (the longest such list counts).  If S > 1 and (output tiles x S) partial tiles of 128 x n_tile floats exceed
 *     16 MiB, or there are more than 128 output tiles, the call is rejected with
 *     RT3D_ERR_WORKSPACE and nothing is launched (rt3d_conv3d_sparse has no such limit).
 *   - The device address of the workspace is looked up by rt3d_packed_prepare (once per device, with that
 *     device current; do it before any stream capture begins).  This entry point itself never allocates
 *     or frees device or pinned memory and never triggers that look-up: without a prepared handle on the
 *     device it returns RT3D_ERR_NOT_PREPARED.
 *   - All calls on a device share the one workspace, which keeps the previous call's contents; the
 *     entry point clears the counters it needs on `stream` before the kernel.  Two calls whose
 *     kernels may overlap on the GPU (different streams) race on it: serialise them.
 *   - Results agree with rt3d_conv3d_sparse within the library's tolerance (the split count, and so
 *     the fp32 summation order, may differ); repeated calls give identical bits.
 */
rt3d_status rt3d_conv3d_sparse_noalloc(const rt3d_tensor* x, const rt3d_packed* w, const float* bias,
                                       const rt3d_conv_params* p, rt3d_tensor* y, void* stream);

/*
 * rt3d_conv3d_host - end-to-end variant: x->data and y->data are HOST buffers (pinned
 * memory recommended), bias is HOST [M] or NULL.  Copies x to a library-owned device staging
 * buffer, runs rt3d_conv3d_sparse (or _dense for a dense handle) and copies y back; the work is
 * ordered after what `stream` holds on entry, and the call returns after the stream has been
 * synchronised.  Batches of at least two clips and 8 MiB go through in up to eight chunks of whole
 * clips (clips are independent), with the copies of neighbouring chunks on two internal streams, so
 * that copy-in, convolution and copy-out overlap; each chunk is one rt3d_conv3d_sparse call, so the
 * result agrees with a single call on the whole batch within the library's tolerance (the K split, and
 * with it the fp32 summation order, may differ), not necessarily bit for bit.  Staging buffers, streams
 * and events are cached in the handle (one call at a time per handle).
 */
rt3d_status rt3d_conv3d_host(const rt3d_tensor* x, rt3d_packed* w, const float* bias,
                             const rt3d_conv_params* p, rt3d_tensor* y, void* stream);

/* Layer glue for the C3D- and R(2+1)D-shaped networks (not described by the paper, which
 * only names the models in Section 5). */
/* Max-pool over (t,h,w) windows, padding never wins; x.c == y.c, same dtype. */
rt3d_status rt3d_maxpool3d(const rt3d_tensor* x, int kt, int kh, int kw, int st, int sh, int sw,
                           int pt, int ph, int pw, rt3d_tensor* y, void* stream);
/* y = a + b (optionally ReLU); equal extents and dtype; y may alias a or b. */
rt3d_status rt3d_add_relu(const rt3d_tensor* a, const rt3d_tensor* b, int relu, rt3d_tensor* y, void* stream);

/*
 * Pruning step on the device (Section 4), the stage right before rt3d_pack_kgs.  All pointers DEVICE.
 * rt3d_kgs_group_norms: norms[p][q][k] = group-lasso norm of the weights of kernel group (p,q) at
 *   kernel location k (Fig. 2 caption; Eq. 2), norm = 1 (sum of magnitudes) or 2 (Euclidean);
 *   w is float [M][N][Kt][Kh][Kw], norms float [P][Q][Kt*Kh*Kw]; missing kernels of ragged groups add 0.
 * rt3d_kgs_reweight: one reweighting step on `count` norms (update rule below Eq. 3):
 *   penalty[i] = 1 / (norms[i]^2 + eps), and the pruning decision keep[i] = norms[i] > threshold;
 *   either output may be NULL; eps > 0.
 * rt3d_kgs_expand_mask: group-level decisions [P][Q][Ks] -> per-weight mask [M][N][Ks] (uint8), the
 *   form rt3d_pack_kgs takes once copied to the host.
 * fp32 arithmetic; enqueue on `stream`, no synchronisation.  Errors: INVALID_ARG, CUDA.
 */
rt3d_status rt3d_kgs_group_norms(const float* w, int M, int N, int Kt, int Kh, int Kw, int g_m, int g_n, int norm,
                                 float* norms, void* stream);
rt3d_status rt3d_kgs_reweight(const float* norms, int64_t count, float eps, float threshold, float* penalty,
                              uint8_t* keep, void* stream);
rt3d_status rt3d_kgs_expand_mask(const uint8_t* group_mask, int M, int N, int Kt, int Kh, int Kw, int g_m, int g_n,
                                 uint8_t* mask, void* stream);

/* Work and traffic the method itself requires for one call (Section 3 cost model):
 * kept multiply-accumulates, dense multiply-accumulates, and algorithmic bytes
 * (input once + output once + packed weights and index once + bias). */
rt3d_status rt3d_conv3d_cost(const rt3d_tensor* x, const rt3d_packed* w, const rt3d_conv_params* p,
                             int64_t* kept_macs, int64_t* dense_macs, int64_t* alg_bytes);

/* How the calling thread's most recent successful convolution call was run (for tests and profiling):
 *   kernel       0 CUDA-core kernel, 1 tensor-core single-CTA kernel, 2 tensor-core CTA-pair kernel,
 *                3 tensor-core small-C_in kernel, 4 tensor-core resident-weight (halo) kernel,
 *                5 fused (2+1)D kernel (rt3d_conv2plus1d_fused; n_tile = intermediate width),
 *                6 tensor-core sub-tile kernel (RT3D_ALGO_UMMA_SUB)
 *                7 tensor-core CTA-pair kernel, one deeper input tile per (kh, kw, chunk) shared by all kt
 *   n_tile       output channels per accumulator tile (tensor-core kernels, else 0)
 *   n_splits     K splits per output tile in the single-CTA kernel (1 = none)
 *   tail_workers CTA pairs that share, cut along K, the output tiles which do not fill a last round
 *                of the persistent CTA-pair grid (0 = every tile is computed by one pair)
 *   fused_pool   1 if a max-pool ran in the epilogue
 * RT3D_ERR_INVALID_ARG if info is NULL or the thread has not run a convolution yet. */
typedef struct {
  int32_t kernel, n_tile, n_splits, tail_workers, fused_pool;
} rt3d_plan_info;
rt3d_status rt3d_last_plan(rt3d_plan_info* info);

/* Which kernel family RT3D_ALGO_AUTO would run for this call: writes an rt3d_algo to *algo. */
rt3d_status rt3d_conv3d_query_algo(const rt3d_tensor* x, const rt3d_packed* w, const rt3d_conv_params* p,
                                   const rt3d_tensor* y, int* algo);

/* Synchronises `stream`, then returns RT3D_ERR_TIMEOUT if any kernel of this library
 * recorded a bounded-wait failure on the current device since the last call (and clears
 * the record), RT3D_ERR_CUDA if the stream reports an error, else RT3D_OK. */
rt3d_status rt3d_last_device_status(void* stream);

/* Number of kernels this library has launched in this process (all devices). */
int64_t rt3d_launch_count(void);

/* Number of device allocations (cudaMalloc calls) this library has made in this process. */
int64_t rt3d_alloc_count(void);

/* Planning mode of the calling thread.  Between rt3d_plan_begin and rt3d_plan_end every compute call of this
 * library (convolutions, fused pair, pool, add) validates its arguments, chooses its kernel, builds and uploads
 * the weight layout that kernel needs and sizes the K-split / tail-split workspace of the handle exactly as the
 * real call would, but launches nothing and touches no activation.  Running a network's sequence of calls once in
 * planning mode (same shapes, same parameters) therefore moves every allocation and upload out of the later real
 * calls: afterwards rt3d_alloc_count does not change while those calls run.  rt3d_last_plan reports the planned
 * kernel.  (The paper's counterpart is its compile-time "tuning of the computation configuration", Section 5.2.) */
void rt3d_plan_begin(void);
void rt3d_plan_end(void);

/* Test hooks; no effect on results.  RT3D_DEBUG_WAIT_CYCLES: SM clocks after which a wait inside the single-CTA
 * tensor-core kernel gives up (0 = default, about one second; the environment variable
 * RT3D_DEBUG_TIMEOUT_POLLS sets the initial value).  RT3D_DEBUG_DROP_LAST_LOAD: nonzero makes that kernel's
 * producer skip the loads of each CTA's last pipeline stage, so that the wait on them runs out and the error
 * path (RT3D_ERR_TIMEOUT from rt3d_last_device_status) can be exercised without any fault.
 * RT3D_DEBUG_T_GROUPS: 0 switches off the CTA-pair kernel's variant that stages one deeper input tile per
 * (kh, kw, channel chunk) for all kt (plan kernel 7), so that it can be compared with the step-per-location
 * form (kernel 2) on the same handle; default 1.
 * RT3D_DEBUG_POISON: runs, on the default stream, a kernel that fills the shared memory and the tensor memory of
 * every SM with the 32-bit pattern `value` (e.g. 0x7FC07FC0: two bf16 NaNs) and waits for it: a kernel launched next
 * that reads shared or tensor memory it did not write itself (padding multiplied by zero weights, say) then
 * produces NaNs instead of depending silently on what ran before it.  The partial-tile scratch of every handle's
 * K splits on the device is set to all ones (NaNs) as well.  Device work only; nothing else changes. */
enum { RT3D_DEBUG_WAIT_CYCLES = 1, RT3D_DEBUG_DROP_LAST_LOAD = 2, RT3D_DEBUG_T_GROUPS = 3, RT3D_DEBUG_POISON = 4 };
rt3d_status rt3d_debug_set(int what, long long value);
/* Diagnostics.  RT3D_DEBUG_WAIT_SITE: after a synchronisation of the device, the number of the wait inside a
 * kernel that gave up since the last rt3d_last_device_status (0 = none; the numbers are the last argument of the
 * kernels' bounded waits in the sources); -1 on error.  Does not clear the word. */
enum { RT3D_DEBUG_WAIT_SITE = 1 };
long long rt3d_debug_get(int what);

const char* rt3d_status_string(rt3d_status s);
const char* rt3d_version(void);

#ifdef __cplusplus
}
#endif
#endif /* RT3D_H_ */
