/*
 * ubp.h -- C ABI of the B200 library for unaligned block-wise pruned (UBP) layers.
 *
 * The layer (Section 3.1 of the paper): a weight W[M][C][R] (M output channels,
 * C input channels, R = kh*kw taps) keeps only "blocks": Nb consecutive output
 * channels i..i+Nb-1 at one input channel j, all R taps, starting at ANY row
 * i <= M-Nb, blocks of one input channel never overlapping (Eq. 1, Eq. 2).
 * Inference computes Y = act(Wm * X + bias) with Wm the masked weight.
 *
 * Conventions for every entry point
 *   - returns 0 (UBP_OK) or a negative ubp_status; never throws, aborts, prints
 *     or synchronises the device (exceptions are named below);
 *   - "host" pointers are ordinary CPU memory, "device" pointers are CUDA device
 *     memory of the current device; the caller owns every buffer it passes;
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream); device
 *     work is enqueued on it and the call returns without waiting;
 *   - inputs are assumed finite; input and output buffers must not overlap.
 */
#ifndef UBP_H_
#define UBP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    UBP_OK = 0,
    UBP_E_ARG = -1,       /* null pointer, non-positive size, Nb > M, bad stride ...        */
    UBP_E_RAGGED = -2,    /* a run of ones in a mask column is not a whole number of blocks */
    UBP_E_SPACE = -3,     /* caller buffer too small / host allocation failed               */
    UBP_E_FORMAT = -4,    /* blob or plan is not what it claims to be                       */
    UBP_E_CUDA = -5,      /* a CUDA runtime/driver call failed (see ubp_last_cuda_error)    */
    UBP_E_UNSUPPORTED = -6,
    UBP_E_DEVICE = -7,    /* a kernel reported a bounded wait that ran out                  */
    UBP_E_STATIC_LIMIT = -8 /* layer too large for the fixed scratch of ubp_spmm_static      */
} ubp_status;

const char *ubp_strerror(int status);
/* last cudaError_t seen by this thread inside the library (0 if none) */
int ubp_last_cuda_error(void);

/* ------------------------------------------------------------------ format
 * Canonical packed form of a UBP weight (Section 4.2: "sparse weight format
 * for WROS"): blocks are grouped by the output row they START at --
 *   indptr [M+1]  blocks starting at row i are indptr[i] .. indptr[i+1]-1
 *   indices[m]    input channel j of each block, ascending inside a start row
 *   values [m][Nb][R]  the block's weights, ROTATED: the weight of output row
 *                 rho sits in slot rho mod Nb (so a kernel that keeps Nb
 *                 stationary accumulators never shuffles them); taps in OIHW
 *                 order (tap = 3*r + s for a 3x3 kernel)
 * Blob = 64-byte little-endian header {"UBP1", u32 version=1, i32 M, C, R, Nb, m,
 * u32 flags(bit0 = rotated)} followed by the three arrays, each starting on a
 * 64-byte boundary, padding bytes zero. The blob is a pure function of
 * (W, mask, Nb); weights are copied bit for bit.
 */

/* ubp_pack (host): mask[M][C] of 0/1 + W[M][C][R] -> blob.
 * The mask is decoded by cutting every run of ones in a column into Nb-row
 * blocks from the run's first row (the block-division step, Algorithm 2).
 * blob == NULL: only *blob_len is written (size query).
 * Errors: UBP_E_ARG (null, sizes, Nb > M, mask value > 1), UBP_E_RAGGED,
 * UBP_E_SPACE (blob_cap < needed; *blob_len still holds the needed size). */
int ubp_pack(const float *W, const uint8_t *mask, int M, int C, int R, int Nb,
             void *blob, size_t blob_cap, size_t *blob_len);

/* ubp_unpack (host): blob -> W_out[M][C][R] (zero where pruned) and
 * mask_out[M][C]; either output may be NULL. UBP_E_FORMAT on a bad blob. */
int ubp_unpack(const void *blob, size_t len, float *W_out, uint8_t *mask_out);

typedef struct {
    int32_t M, C, R, Nb, m;
    const int32_t *indptr;   /* point into the blob */
    const int32_t *indices;
    const float *values;
} ubp_view_t;

/* ubp_blob_view (host): validate a blob and expose its arrays (no copy). */
int ubp_blob_view(const void *blob, size_t len, ubp_view_t *view);

/* The other block orientation: B consecutive INPUT channels of ONE output row (runs along K inside a row of W),
 * starting at any input channel <= C-B. It is the same format with the two channel roles exchanged, and R = 1.
 * ubp_pack_kmajor (host): W[M][C], mask[M][C] whose runs of ones along each row are whole multiples of B
 *   -> the canonical blob of the transposed layer (its header reads M' = C, C' = M, Nb = B; indptr runs over the
 *   input channel a block starts at, indices hold the output row). Same size-query and error rules as ubp_pack
 *   (UBP_E_RAGGED for a run that is not a whole number of blocks).
 * ubp_kmajor_to_plan_blob (host): that blob -> a blob ubp_plan_size / ubp_plan_build accept: the same kept weights
 *   in the layer's own orientation as blocks of ONE output channel (any mask is a valid set of such blocks). The
 *   tensor-core kernels work on the densified weight and do not care about the orientation; on the sparse kernel
 *   this form costs one index per kept weight (ubp_plan_build_kmajor below keeps one index per run instead). */
int ubp_pack_kmajor(const float *W, const uint8_t *mask, int M, int C, int B,
                    void *blob, size_t blob_cap, size_t *blob_len);
int ubp_kmajor_to_plan_blob(const void *kblob, size_t klen, void *blob, size_t blob_cap, size_t *blob_len);

/* ------------------------------------------------------------------ plan
 * The kernels do not walk the canonical arrays directly: a plan is the same
 * blocks re-bucketed for the GPU (by row panel, input-channel tile and start
 * offset inside the panel; a block that crosses a panel boundary is listed in
 * both panels, each taking its own rows -- the GPU answer to the "overlapped
 * output tiles" of Section 3.3). The plan lives in a device buffer the CALLER
 * allocates; the library owns only the small host handle.
 *
 * variant: 0 = choose from the layer shape; > 0 = a specific kernel
 * configuration (ubp_variant_count / ubp_variant_describe list them), meant
 * for measuring configurations against each other.
 * Variants 60 and 61 (R == 1, Nb in {1, 2, 4, 8, 16}) are comparison kernels that keep the paper's own dataflow:
 * their plan is the canonical arrays themselves, a thread walks the start rows with row step 1 and keeps Nb
 * stationary accumulators; 60 uses the stored rotation (Section 4.2: the finished row sits in slot i mod Nb, no
 * accumulator ever moves), 61 is the naive form of Section 3.3 (row order, store the first accumulator and move
 * the others down after every start row). With aligned masks they are the aligned kernel, with Nb = 1 the
 * element-wise one (Section 5.4's comparison).
 */
typedef struct ubp_plan ubp_plan_t;

int ubp_variant_count(void);
/* id of the index-th configuration (0 <= index < ubp_variant_count()), or UBP_E_ARG; ids are positive
 * but not contiguous */
int ubp_variant_at(int index);
/* text description of the configuration with this id into buf; UBP_E_ARG if there is none */
int ubp_variant_describe(int variant, char *buf, size_t cap);

/* bytes of device memory a plan of this blob needs (host; no CUDA call) */
int ubp_plan_size(const void *blob, size_t len, int variant, size_t *dev_bytes);

/* ubp_plan_image (host; no CUDA call): write the exact bytes that
 * ubp_plan_build would upload into host_buf (>= ubp_plan_size bytes). Meant for
 * inspection and for checking the plan builder without a GPU. Image layout:
 *   [0,256) header, int32 status word at byte 0;
 *   [256,..) uint32 group_off[nkt*NG + 1] in 16-byte units, groups in (tile, row group) order;
 *   group: uint32 poff[WR+1] (padded to 16), then per panel
 *          uint16 fo[F+1] (F = panel_rows + nbk - 1 start offsets, padded to 16),
 *          uint16 jl[n+4] (input channel inside the tile; 4 trailing zeros so a kernel may read ahead; padded to 16),
 *          float  w[n+2][nbk][R] (weights in row order, i.e. with the rotation undone; 2 trailing zero entries).
 * geom receives {nbk, panel_rows, k_tile, WR, dupw, nkt, NP, NG}. */
int ubp_plan_image(const void *blob, size_t len, int variant, void *host_buf, size_t cap, int32_t geom[8]);

/* Build the plan on the host, copy it into dev_buf (device, >= ubp_plan_size
 * bytes, 256-byte aligned) with one cudaMemcpyAsync on `stream`, return the
 * handle. The handle keeps its host copy until ubp_plan_free, so the copy may
 * still be in flight when this returns. */
int ubp_plan_build(const void *blob, size_t len, int variant, void *dev_buf, size_t dev_bytes,
                   void *stream, ubp_plan_t **plan);
void ubp_plan_free(ubp_plan_t *plan);

/* Plans straight from a K-major blob (the forms of ubp_plan_size / ubp_plan_image / ubp_plan_build for the other
 * orientation; the handle reports the layer's own M and C, and ubp_spmm / ubp_conv1x1 take it like any other).
 * variant 0 chooses: the tensor-core kernel where it pays (at least 3 % of the weights kept -- 0.5 % for layers of a
 * million weights or more --, 128 output and 64 input channels; the weight is densified, the orientation does not matter there), else the K-run sparse kernel
 * (variants 70..73 for B = 2, 4, 8, 16): fp32 FMA, output rows stationary in registers, a plan entry = one run
 * (row, first channel, B weights), i.e. ONE channel index per B weights and B consecutive rows of the staged
 * activation tile per entry; a run that crosses a channel-tile boundary is cut there. Other run lengths fall back
 * to the element-wise configuration (one index per weight). A variant > 0 that is not 70..73 is applied to the
 * re-expressed layer (ubp_kmajor_to_plan_blob). */
int ubp_plan_size_kmajor(const void *kblob, size_t klen, int variant, size_t *dev_bytes);
int ubp_plan_image_kmajor(const void *kblob, size_t klen, int variant, void *host_buf, size_t cap, int32_t geom[8]);
int ubp_plan_build_kmajor(const void *kblob, size_t klen, int variant, void *dev_buf, size_t dev_bytes, void *stream,
                          ubp_plan_t **plan);

typedef struct {
    int32_t M, C, R, Nb, m;      /* layer                                         */
    int32_t variant;             /* configuration actually chosen                 */
    int32_t panel_rows, k_tile;  /* plan geometry                                 */
    int64_t entries;             /* block entries in the plan (incl. duplicates)  */
    int64_t dev_bytes;
} ubp_plan_info_t;
int ubp_plan_info(const ubp_plan_t *plan, ubp_plan_info_t *info);

/* ubp_plan_tile_choice: which kernel a launch of this plan over `Nc` columns uses on the current device when the
 * operands qualify for the fast path (for 3x3: input and output as one [channel][batch, y, x] matrix each), and
 * its output tile. `image_width` is the width of the input planes for a 3x3 plan (Nc = batch * height * width),
 * ignored for 1x1; a negative value asks about a strided 3x3 launch (Nc = batch * Ho * Wo), which the one-CTA kernel
 * serves. *kernel: 0 = sparse FP32 kernel (Section 4.2's output-stationary product on the CUDA cores),
 * 1 = tensor-core kernel with one CTA per tile, 2 = tensor-core kernel with a CTA pair per tile, 3 = the comparison
 * kernels that walk the canonical arrays in the paper's own dataflow (variants 60 and 61; tile_rows is 0).
 * tile_rows is 256 for the CTA-pair kernel, or 512 where a pair stacks two 256-row MMA tiles on one staged activation
 * tile (layers whose rows fill whole 512-row tiles, where the tile estimate prefers that); tile_cols of the CTA-pair
 * kernels is a multiple of 16 (bf16 products) or 64 (TF32 products), at most 256. Host only;
 * enqueues nothing. Not part of the paper's method: it exists so that measurements and tests can name what ran. */
int ubp_plan_tile_choice(const ubp_plan_t *plan, int64_t Nc, int image_width, int *kernel, int *tile_rows,
                         int *tile_cols);

/* ubp_plan_tile_choice_conv: the same question for a 3x3 plan and a batch of B images of H x Wd pixels in the layout
 * the fast paths take (input and output each one [channel][batch, y, x] matrix): *kernel as above, or 4 = the CTA-pair
 * kernel that computes on the zero-padded pixel grid and takes the nine taps as shifts of one staged operand
 * (variants 64..67, stride 1, more than 128 output channels, input channels a multiple of 16); tile_cols then counts
 * padded positions. */
int ubp_plan_tile_choice_conv(const ubp_plan_t *plan, int B, int H, int Wd, int stride, int *kernel, int *tile_rows,
                              int *tile_cols);

/* Read the plan's device status word: blocks until `stream` has finished
 * (cudaStreamSynchronize), then returns UBP_OK or UBP_E_DEVICE if a kernel
 * launched with this plan gave up on a bounded wait (word = 1).
 * The checked build of the library (compiled with -DUBP_DEBUG: libubp_b200_debug.so, same entry points) also
 * compares every index its kernels take from the plan or compute for shared or global memory with the extent
 * it has to stay in; a failing check sets the word (2: shared memory or plan contents, 3: global memory), the
 * access is skipped, the kernel runs to its end and this call reports UBP_E_DEVICE. Nothing traps in either
 * build. */
int ubp_plan_check(const ubp_plan_t *plan, void *stream);

/* ubp_plan_clear_status: reset the plan's device status word to 0 (one 4-byte cudaMemsetAsync on `stream`). */
int ubp_plan_clear_status(const ubp_plan_t *plan, void *stream);

/* ubp_selftest_bounded_wait: enqueue a one-warp kernel that waits on an mbarrier nobody ever completes, with
 * the bounded-wait routine of the tensor-core kernels but a limit of `limit_us` microseconds (1 .. 1 000 000).
 * When the limit runs out the kernel sets the plan's status word and returns, so a following ubp_plan_check
 * reports UBP_E_DEVICE and the context stays usable. Exists so that the "a wait that runs out is reported, not
 * hung" path can be exercised without any fault; not part of the paper's method. */
int ubp_selftest_bounded_wait(const ubp_plan_t *plan, unsigned limit_us, void *stream);

/* ------------------------------------------------------------------ compute
 * ubp_spmm: Y[M][Nc] = act(Wm[M][C] * X[C][Nc] + bias), the 1x1 / fully
 * connected case (R == 1), the weight-rotating output-stationary product of
 * Section 4.2 re-organised for the GPU: accumulators stay in registers for
 * the whole reduction and each output is written once.
 *   X    device, row c at X + c*ldx, Nc contiguous floats (ldx >= Nc)
 *   bias device [M] or NULL;  relu != 0 applies max(.,0)
 *   Y    device, row o at Y + o*ldy (ldy >= Nc)
 * Fast path needs X, Y 16-byte aligned and ldx, ldy multiples of 4; otherwise a
 * slower kernel is used (same arithmetic as the sparse kernel). Nc == 0 is a no-op.
 * Arithmetic, by the kernel the plan's variant selects (ubp_plan_tile_choice names it):
 *   sparse kernel (variants 1..17, 50..57, 70..73, and every fallback) and the comparison kernels 60, 61: fp32 fused
 *     multiply-add, fp32 accumulation: |Y - exact| <= (L + 2) 2^-24 (|Wm||X| + |bias|),
 *     L = kept weights of the output row;
 *   tensor-core kernels, TF32 products (30..33): every fp32 product w x is replaced by
 *     three products of the operands' TF32 heads and remainders, accumulated in fp32 in
 *     tensor memory: error <= 2^-18 |w||x| per product plus the accumulation;
 *   tensor-core kernels, bf16 products (34..37, the choice of variant 0 for layers with
 *     at least 3 % of the weights kept (0.5 % from a million weights on), 128 output and 64 input
 *     channels): three products
 *     of bf16 heads and remainders, fp32 accumulation: error <= 3 * 2^-16 |w||x| per
 *     product in the worst case (about 2 * 10^-6 of |Wm||X| on random data).
 *   tensor-core kernel, three bf16 pieces (84..87): w = w1 + w2 + w3 and x = x1 + x2 + x3 exactly (8 + 8 + 8
 *     significant bits), the six products whose orders add up to at most four, fp32 accumulation: error below
 *     2^-23 |w||x| per product, so that the tensor core's truncating fp32 accumulation is what remains (about
 *     1.5 * 10^-6 of |Wm||X| on random data against 3 * 10^-7 for the fp32 kernel), at twice the tensor-core work
 *     of 34..37.
 * Every kernel sums in a fixed order: results are bitwise reproducible run to run. */
int ubp_spmm(const ubp_plan_t *plan, const float *X, int64_t ldx, int64_t Nc,
             const float *bias, int relu, float *Y, int64_t ldy, void *stream);

/* ubp_conv1x1: 1x1 stride-1 convolution = ubp_spmm over columns n = (b, y, x)
 * (Section 4.2: the pointwise convolution is the sparse matrix product the
 * weight-rotating kernel is written for; Section 3.1 for the block shape).
 * Element strides: in[b][c][y][x] at in + b*in_stride_b + c*in_stride_c + y*Wd + x
 * (NCHW: (C*H*W, H*W); channel-major "CNHW": (H*W, B*H*W)); same for out.
 * If both batch strides equal H*W all images form one product with
 * Nc = B*H*W; otherwise one product per image. */
int ubp_conv1x1(const ubp_plan_t *plan, const float *in, int B, int H, int Wd,
                int64_t in_stride_b, int64_t in_stride_c,
                const float *bias, int relu,
                float *out, int64_t out_stride_b, int64_t out_stride_c, void *stream);

/* ubp_conv3x3_implicit: 3x3, stride 1, zero padding 1, cross-correlation; the
 * plan must come from a blob with R == 9 (a block = Nb output channels x one
 * input channel x all nine taps, Section 3.1). The K = 9*C lowered matrix is
 * never formed in memory. Tensor-core plans (input and output each one
 * [channel][batch, y, x] matrix with 16-byte aligned rows) run an implicit GEMM.
 * Variants 64..67 (the choice of variant 0; more than 128 output channels, input
 * channels a multiple of 16): the outputs are computed on the zero-padded pixel
 * grid, where a tap is a pure shift; per 16 input channels the real pixels a
 * tile touches are copied into shared memory once, split once into the bf16
 * operand pair, and the nine taps read that one operand at nine start offsets.
 * Variants 40..47 (and 64..67 on layers that kernel does not take): reduction
 * index tap * C + channel; per tap and 16-channel chunk the input rows are copied
 * with a halo of columns and a shifted, border-masked operand tile is cut out.
 * Other plans and layouts run a kernel with one lane per output pixel that
 * reads its taps in place. Arithmetic per kernel as for ubp_spmm.
 * Same strides as ubp_conv1x1. */
int ubp_conv3x3_implicit(const ubp_plan_t *plan, const float *in, int B, int H, int Wd,
                         int64_t in_stride_b, int64_t in_stride_c,
                         const float *bias, int relu,
                         float *out, int64_t out_stride_b, int64_t out_stride_c, void *stream);

/* Strided forms (the downsampling layers of ResNet-shaped networks). Output planes are Ho x Wo with
 * Ho = (H-1)/stride + 1, Wo = (W-1)/stride + 1; strides of `out` are in elements of those planes.
 * stride == 1 forwards to the call above.
 * ubp_conv3x3_strided: 3x3, zero padding 1: out[b][o][yo][xo] = act(bias[o] + sum W[o][c][3r+s] *
 *   in[b][c][yo*stride + r - 1][xo*stride + s - 1]). For stride > 1 a tensor-core plan whose output is one
 *   [channel][batch, yo, xo] matrix with 16-byte aligned rows runs the one-CTA implicit-GEMM kernel (its loader warps
 *   gather every tap pixel by pixel, so the stride is only a change of the column -> pixel map); other plans and
 *   layouts are computed by one lane per output pixel that reads its taps in place (correct for any layout, far from
 *   the roofline).
 * ubp_conv1x1_strided: out[b][o][yo][xo] = act(bias[o] + sum W[o][c] * in[b][c][yo*stride][xo*stride]). For
 *   stride > 1 the pixels read are first gathered into `scratch` (device, 16-byte aligned, at least
 *   ubp_conv1x1_strided_scratch(C, B, H, W, stride) bytes, channel-major [C][B][Ho][Wo]) by one extra kernel, then the
 *   stride-1 path runs on them. UBP_E_SPACE if the scratch is too small. Exception: stride 2 under a bf16 tensor-core
 *   plan (variants 34..37), channel-major tensors (both batch strides equal to their plane size), H even, W a multiple
 *   of 4, 16-byte aligned pointers and channel strides that are multiples of 4: the CTA-pair kernel reads the
 *   full-resolution input itself (its copies bring the even rows, its split pass takes every other pixel) and
 *   `scratch` is not touched (it must still be given: which path runs is the library's choice). */
int ubp_conv3x3_strided(const ubp_plan_t *plan, const float *in, int B, int H, int Wd, int stride,
                        int64_t in_stride_b, int64_t in_stride_c, const float *bias, int relu,
                        float *out, int64_t out_stride_b, int64_t out_stride_c, void *stream);
/* ubp_conv3x3_strided_ws: ubp_conv3x3_strided with caller-provided scratch (device, 16-byte aligned, at least
 *   ubp_conv3x3_strided_scratch(C, B, H, W, stride) bytes; that is 0 unless stride == 2). With it, a stride-2 layer
 *   whose plan is a variant 64..67 and whose output is one [channel][batch, yo, xo] matrix runs the padded-grid CTA-pair
 *   kernel: one extra kernel first writes the four phase planes of the input (even/odd rows x even/odd columns,
 *   [4*C][B*Ho*Wo]) into the scratch, on which output (yo, xo) reads tap (dy, dx) at plane (dy != 1, dx != 1), position
 *   (yo - [dy == 0], xo - [dx == 0]): every tap is a shift of 0 or -1 of one plane. scratch == NULL or other cases:
 *   exactly ubp_conv3x3_strided. UBP_E_SPACE if the scratch is too small. (ubp_plan_tile_choice_conv with stride 2
 *   answers for this call.) */
size_t ubp_conv3x3_strided_scratch(int C, int B, int H, int Wd, int stride);
int ubp_conv3x3_strided_ws(const ubp_plan_t *plan, const float *in, int B, int H, int Wd, int stride,
                           int64_t in_stride_b, int64_t in_stride_c, void *scratch, size_t scratch_bytes,
                           const float *bias, int relu, float *out, int64_t out_stride_b, int64_t out_stride_c, void *stream);
size_t ubp_conv1x1_strided_scratch(int C, int B, int H, int Wd, int stride);
int ubp_conv1x1_strided(const ubp_plan_t *plan, const float *in, int B, int H, int Wd, int stride,
                        int64_t in_stride_b, int64_t in_stride_c, void *scratch, size_t scratch_bytes,
                        const float *bias, int relu, float *out, int64_t out_stride_b, int64_t out_stride_c, void *stream);

/* ubp_spmm_static: same result as ubp_spmm, for callers that cannot allocate.
 * (The paper has no counterpart; this is a deployment convenience.)
 *
 * Who needs it: code that has to run a UBP layer but may not obtain device
 * memory at that point -- a plug-in living inside another engine that owns the
 * whole device heap, a service whose memory budget was fixed at start-up, a
 * caller on a path where an allocation (and the implicit synchronisation and
 * possible failure that come with it) is not acceptable. ubp_spmm needs a
 * device buffer for the plan; here the plan goes into a fixed array of
 * ubp_static_plan_capacity() bytes (2 MiB) that is part of the library's
 * device image, so every GPU that loads the library holds those 2 MiB until
 * the process ends, whether or not this function is ever called.
 *
 *   blob/len   host: canonical packed layer (R == 1), as made by ubp_pack
 *   X, bias, Y device, same meaning and alignment rules as ubp_spmm
 * The plan is rebuilt on the host from the blob on EVERY call (host time of the
 * order of a millisecond for a 512x512 layer) and uploaded with one
 * cudaMemcpyAsync from pageable memory -- which may wait for earlier work on
 * `stream` -- then the same kernel as ubp_spmm is launched. The function calls
 * no cudaMalloc / cudaFree and no other device-allocating routine.
 * First call on a device: resolves the array's device address
 * (cudaGetSymbolAddress) with that device current.
 * The call cannot be recorded by a stream capture: the upload's source is a
 * host buffer that lives only for the call, so a replay would read freed
 * memory. A capturing `stream` is refused with UBP_E_UNSUPPORTED before
 * anything is enqueued or the array is touched.
 * All calls on a device share the one array: two calls whose GPU work overlaps
 * (different streams, or threads) race on it -- serialise them. The array
 * keeps the previous call's plan until the next upload overwrites it; the
 * upload rewrites the status word, so nothing has to be cleared by the caller.
 * Errors: as ubp_spmm, plus UBP_E_FORMAT (bad blob) and UBP_E_STATIC_LIMIT when
 * the layer's plan does not fit the array (use ubp_plan_build / ubp_spmm then). */
size_t ubp_static_plan_capacity(void);
int ubp_spmm_static(const void *blob, size_t len, const float *X, int64_t ldx, int64_t Nc,
                    const float *bias, int relu, float *Y, int64_t ldy, void *stream);

/* --------------------------------------------------------- block selection
 * Choosing which blocks to keep (Section 3.1 and Section 4.1): candidate block
 * k = i + M*j starts at output row i of input channel j; its score is the l1
 * norm of W[i..i+Nb-1][j][:] (Eq. 1), -inf when i + Nb > M. Block expansion
 * (Algorithm 1) takes m times the best remaining candidate, re-scores the Nb-1
 * candidates to its left as if the chosen block's kernels were gone (so a block
 * may grow around an earlier choice instead of being excluded by it) and drops
 * the Nb candidates starting inside the chosen block; block division
 * (Algorithm 2) cuts the grown runs every Nb rows. The result is delivered as
 * a mask[M][C] whose runs of ones are whole blocks -- what ubp_pack decodes.
 * The device routines reproduce the sequential procedure bit for bit for this
 * arithmetic: single precision; a kernel's norm = sum of |w| over its R taps in
 * storage order; a block's score = sum of its Nb kernel norms in row order; a
 * re-scored candidate = (S[k-n] + S[k-n+Nb]) - S[k]; ties in an arg max go to
 * the lowest k.
 * Limits: Nb <= M <= 16384, M*C < 2^31 (UBP_E_UNSUPPORTED beyond).
 * All device work is enqueued on `stream`; nothing is synchronised. */

/* bytes of device scratch ubp_block_scores / ubp_bed_select need (256-byte aligned buffer). */
int ubp_bed_workspace_size(int M, int C, int Nb, size_t *dev_bytes);

/* ubp_block_scores: W (device, [M][C][R] row-major) -> S (device, [C][M] floats,
 * S[j*M + i] = score of candidate k = i + M*j). */
int ubp_block_scores(const float *W, int M, int C, int R, int Nb, void *workspace, size_t workspace_bytes,
                     float *S, void *stream);

/* ubp_bed_select: W (device) -> mask (device, [M][C] bytes 0/1) keeping m blocks.
 * n_selected (device, nullable) receives the number of blocks kept: m, or fewer
 * when the columns cannot hold m blocks (each holds floor(M/Nb) at most).
 * Errors: UBP_E_ARG (null, sizes, Nb > M, m < 0, workspace not 256-byte
 * aligned), UBP_E_SPACE (workspace too small), UBP_E_UNSUPPORTED, UBP_E_CUDA. */
int ubp_bed_select(const float *W, int M, int C, int R, int Nb, int64_t m, void *workspace, size_t workspace_bytes,
                   uint8_t *mask, int64_t *n_selected, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* UBP_H_ */
