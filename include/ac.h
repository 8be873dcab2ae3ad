/*
 * ac.h -- C ABI of the compressed-activation backward library (sm_100a).
 *
 * The method (paper: "Less Memory Means smaller GPUs: Backpropagation with
 * Compressed Activations", Section 4 "Compressing Activation Maps" and its
 * figure): a convolution layer computes its forward output from the full
 * input X, but what it keeps for the backward pass is Z, the k x k average
 * pooled copy of X, plus the pooling size and X's shape. In the backward pass
 * the weight gradient is calculated as usual from Z inflated back to X's shape
 * and the uncompressed output gradient dY. Input and bias gradients do not
 * involve X and are not part of this library.
 *
 * Conventions common to every call
 *   - All tensor pointers are DEVICE pointers unless a parameter says "host".
 *     The caller owns every buffer (tensors and workspace). The library never
 *     allocates or frees device memory and never synchronises, except where a
 *     call says so; work is enqueued on `stream` (a cudaStream_t passed as
 *     void*, NULL = the default stream).
 *   - Tensor pointers must be 16-byte aligned (AC_ERR_MISALIGNED otherwise).
 *   - Errors are return codes. No call aborts, throws or traps on the device.
 *     The descriptor is validated before anything is launched.
 *   - Reentrant; no global state except one-time kernel attribute set-up and a small
 *     mutex-protected cache of launch plans keyed by the descriptor.
 *
 * Shapes (logical): X [N, C_in, H, W]; Z [N, C_in, ceil(H/k), ceil(W/k)];
 * dY [N, C_out, H_o, W_o] with H_o = (H + 2 pad_h - R) / stride_h + 1 (floor),
 * likewise W_o; dW [C_out, C_in, R, S]. Dilation 1, one group.
 * Layout AC_NCHW stores X, Z, dY as [N][C][H][W] and dW as [C_out][C_in][R][S];
 * AC_NHWC stores X, Z, dY as [N][H][W][C] and dW as [C_out][R][S][C_in].
 * All buffers are dense (no strides).
 */
#ifndef AC_H_
#define AC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    AC_OK = 0,
    AC_ERR_INVALID_ARG = 1,         /* NULL pointer, non-positive size, bad enum, empty output */
    AC_ERR_UNSUPPORTED = 2,         /* valid problem the library cannot run */
    AC_ERR_MISALIGNED = 3,          /* a tensor or workspace pointer is not 16-byte aligned */
    AC_ERR_WORKSPACE_TOO_SMALL = 4, /* workspace_bytes < ac_workspace_bytes_min(desc) */
    AC_ERR_CUDA = 5,                /* a CUDA runtime call failed (launch, copy, attribute) */
    AC_ERR_TIMEOUT = 6              /* a bounded wait inside a kernel ran out (see ac_workspace_status) */
} ac_status;

typedef enum { AC_F32 = 0, AC_BF16 = 1 } ac_dtype;
typedef enum { AC_NCHW = 0, AC_NHWC = 1 } ac_layout;

/* The problem statement of Section 4: the convolution layer, plus the pooling
 * size k, which together with X's shape is all the metadata the stored Z needs. */
typedef struct {
    int32_t N, C_in, C_out, H, W;   /* X is N x C_in x H x W (logical) */
    int32_t R, S;                   /* filter height, width */
    int32_t stride_h, stride_w, pad_h, pad_w;
    int32_t k;                      /* pooling factor, k >= 1; k = 1 stores X itself */
    int32_t dtype;                  /* ac_dtype of X, Z, dY; dW is always fp32 */
    int32_t layout;                 /* ac_layout of X, Z, dY and dW */
} ac_conv_desc;

/*
 * Bytes of scratch with which ac_conv2d_wgrad_compressed runs this problem on
 * its fastest path: a small status block, the split-K partial sums of dW and,
 * for fp32 and/or NCHW inputs that go to the tensor cores, bf16 NHWC copies of
 * Z and dY, or, for layers with few input channels, the gathered operand matrix
 * (see ac_conv2d_wgrad_compressed). Pure host code. Returns 0 for an invalid
 * descriptor.
 */
size_t ac_workspace_bytes(const ac_conv_desc *desc);

/*
 * The least scratch ac_conv2d_wgrad_compressed accepts for this problem. Equal
 * to ac_workspace_bytes unless the fastest path stages copies of the operands;
 * then this is what the path without copies needs (status block and split-K
 * partial sums only; at most 256 MiB + 256 bytes). A call given at least this
 * much but less than ac_workspace_bytes runs on that slower path. Pure host
 * code. Returns 0 for an invalid descriptor.
 */
size_t ac_workspace_bytes_min(const ac_conv_desc *desc);

/*
 * Compression (Section 4; figure: mu_pq is the mean of the k x k block of X
 * whose first element is X[pk, qk]). Z[n,c,p,q] = mean of X[n,c,h,w] over
 * h in [pk, min(pk+k,H)), w in [qk, min(qk+k,W)): blocks are aligned to X's
 * index 0; a partial last block is averaged over the elements it has. The sum
 * is formed in fp32 and rounded once to the storage dtype.
 *
 *   x      in : [N,C_in,H,W] in desc->layout / desc->dtype. With y_out == NULL
 *               this is the activation X itself.
 *   z      out: [N,C_in,ceil(H/k),ceil(W/k)], same layout and dtype.
 *   y_out  out, optional: if non-NULL the call is the fused form for a layer
 *               whose input is produced by a ReLU: x is the pre-activation A,
 *               y_out = max(A, 0) (same shape as x; may be the same pointer as
 *               x for in-place ReLU) and z = pooling of y_out.
 * Only N, C_in, H, W, k, dtype and layout of the descriptor are used.
 * One kernel launch on `stream`; no scratch memory.
 */
ac_status ac_compress(const ac_conv_desc *desc, const void *x, void *z,
                      void *y_out, void *stream);

/*
 * Fused ReLU + compression that keeps a sign mask instead of the activation
 * (Section 4 replaces the saved conv input by Z; the ReLU in front of it then
 * needs, for its own backward, only where its input was positive). For a
 * caller that does not need Y = max(A, 0) in memory afterwards:
 *
 *   a     in : the pre-activation A, [N,C_in,H,W] in desc->layout / desc->dtype.
 *   z     out: pooling of max(A, 0), exactly as ac_compress with y_out writes.
 *   mask  out: ceil(N*C_in*H*W / 8) bytes on the device; bit (i mod 8) of byte
 *              (i div 8), least significant bit first, is 1 iff element i of A
 *              (i counts in memory order of desc->layout) is greater than zero.
 * The mask is written by the vector kernels only: k must be 1, 2, 4 or 8 and
 * the contiguous axis (C_in for NHWC; W for NCHW, which k must also divide) a
 * multiple of 8, k == 1 needs only N*C_in*H*W to be one. Anything else returns
 * AC_ERR_UNSUPPORTED and launches nothing. All three pointers 16-byte aligned;
 * one kernel launch on `stream`; no scratch memory.
 */
ac_status ac_compress_relu_mask(const ac_conv_desc *desc, const void *a, void *z,
                                void *mask, void *stream);

/*
 * The same pass for a caller that does need Y = max(A, 0) afterwards (as the
 * input of the next convolution's forward pass) but not for the ReLU's
 * backward: writes Y as ac_compress with y_out does, Z, and the mask, reading A
 * once. y_out may alias a (the ReLU in place). Same domain, alignment and
 * errors as ac_compress_relu_mask; y_out must not be NULL.
 */
ac_status ac_compress_relu_mask_y(const ac_conv_desc *desc, const void *a, void *y_out, void *z,
                                  void *mask, void *stream);

/*
 * The backward pass of that ReLU, from the mask alone: dx[i] = dy[i] if bit i of
 * the mask is set, else 0, for the N*C_in*H*W elements of the tensor in memory
 * order (the bit order ac_compress_relu_mask writes; the layout does not matter
 * as long as dy and dx use the one the mask was taken in). This is what lets the
 * ReLU drop its output: Section 4 removes the convolution's claim on X, this
 * call the ReLU's.
 *
 *   mask  in : ceil(N*C_in*H*W / 8) bytes, as written by ac_compress_relu_mask.
 *   dy    in : gradient with respect to the ReLU's output, desc->dtype.
 *   dx    out: gradient with respect to its input, desc->dtype; may alias dy.
 * N*C_in*H*W must be a multiple of 8 (AC_ERR_UNSUPPORTED otherwise; the mask
 * kernels have the same domain). All three pointers 16-byte aligned; one kernel
 * launch on `stream`; no scratch memory. Only N, C_in, H, W and dtype of the
 * descriptor are read.
 */
ac_status ac_relu_mask_backward(const ac_conv_desc *desc, const void *mask, const void *dy,
                                void *dx, void *stream);

/*
 * Weight gradient from the compressed activation (Section 4: Z is expanded to
 * X's shape and the ordinary weight gradient is taken of that; figure:
 * dL/dW ~ Z (*) dL/dY). With Xt[n,c,h,w] = Z[n,c,h/k,w/k] for 0<=h<H, 0<=w<W
 * and 0 elsewhere (the convolution's zero padding, applied after inflation):
 *
 *   dW[co,ci,r,s] = sum_{n,ho,wo} dY[n,co,ho,wo] * Xt[n,ci,ho*stride_h-pad_h+r,
 *                                                          wo*stride_w-pad_w+s]
 *
 * Xt is never written to memory. Products are accumulated in fp32. bf16 inputs
 * are multiplied exactly (tensor cores); fp32 NHWC inputs that the tensor-core
 * kernel takes are each split into three bf16 terms and the six leading partial
 * products are accumulated (terms of relative weight 2^-24 and below are
 * dropped); the split copies of Z and dY live in the workspace, which is why
 * ac_workspace_bytes is then about 3 x (|Z| + |dY|) x 4 bytes larger. NCHW
 * inputs that the tensor-core kernel takes once transposed are copied to NHWC
 * bf16 in the workspace in the same pass. bf16 NHWC layers with fewer than 64
 * input channels (a network's first convolution) have the values every output
 * position reads gathered into a [N*H_o*W_o][taps x C_in] bf16 matrix in the
 * workspace (at most 256 columns, padded to a multiple of 64; taps that read
 * the same element of Z for every position share one column) and run as the
 * equivalent 1x1 problem on the tensor cores; where the strides are multiples
 * of k and k divides H and W (a 7x7 stride-2 stem at k = 2) that matrix is
 * built tile by tile in shared memory instead and needs no workspace. All other problems, and calls
 * whose workspace is smaller than ac_workspace_bytes but at least
 * ac_workspace_bytes_min, use fp32 FMA (or the slower tensor-core kernel) on
 * the operands as they are.
 *
 *   z          in : as produced by ac_compress.
 *   dy         in : [N,C_out,H_o,W_o], desc->layout / desc->dtype.
 *   dw         out: fp32, OVERWRITTEN (not accumulated into); layout per desc->layout.
 *   workspace     : device scratch of at least ac_workspace_bytes_min(desc) bytes,
 *                   16-byte aligned; contents on entry are ignored, contents on
 *                   exit are unspecified except for the status block read by
 *                   ac_workspace_status. Two calls that overlap on the device
 *                   must not share a workspace.
 * Returns AC_ERR_WORKSPACE_TOO_SMALL / AC_ERR_MISALIGNED / AC_ERR_INVALID_ARG
 * before launching anything. Results are deterministic (fixed summation order).
 * Stream semantics are the ordinary ones. Internally the main kernel and the
 * split-K reduction are launched with CUDA's programmatic stream
 * serialization: if the kernel before them in the stream allows it (the
 * library's own compress kernels do), they are brought onto the GPU while
 * that kernel is finishing, but touch global memory only once it has
 * completed and its writes are visible.
 */
ac_status ac_conv2d_wgrad_compressed(const ac_conv_desc *desc, const void *z,
                                     const void *dy, float *dw, void *workspace,
                                     size_t workspace_bytes, void *stream);

/*
 * The same weight gradient added to what dW holds (gradient accumulation over
 * micro-batches): dW <- beta * dW + (the result of ac_conv2d_wgrad_compressed).
 * Section 4 defines dW as a value that is assigned, not added to; accumulation
 * is the usual framework convenience on top. The new gradient is formed
 * in the workspace by exactly the path ac_conv2d_wgrad_compressed would take
 * with `workspace_bytes - 4*|dW|` bytes (rounded down to 256), then one pass
 * combines it with dW, so the result is bitwise beta*dW + that gradient, in
 * fp32. beta may be any finite value; beta == 0 still reads dW (NaNs in it
 * propagate): call the plain entry point to overwrite.
 *   workspace : at least ac_workspace_bytes_min(desc) rounded up to 256, plus
 *               4*|dW| bytes;
 *               ac_accumulate_workspace_bytes(desc) is the size for the
 *               fastest path.
 * Same return codes and status block as ac_conv2d_wgrad_compressed.
 */
size_t ac_accumulate_workspace_bytes(const ac_conv_desc *desc);
ac_status ac_conv2d_wgrad_compressed_accumulate(const ac_conv_desc *desc, const void *z,
                                                const void *dy, float beta, float *dw,
                                                void *workspace, size_t workspace_bytes,
                                                void *stream);

/*
 * Planning hint for callers that run several weight gradients side by side on
 * different streams (independent layers of one backward pass). By default a
 * tensor-core weight gradient launches about one CTA per SM of the GPU (148):
 * kernels of different streams then follow one another, and each pays its fixed
 * costs (set-up, the drain of its partial sums, the split-K reduction) alone.
 * With a budget of `sms` the plans of the calling host thread cut K into about
 * `sms` slices instead, so that 148 / sms kernels are resident together:
 * fewer and smaller partial tensors per layer, and one layer's fixed costs
 * overlap another's main loop. Measured (B200, bf16, k = 2): four ResNet-18-
 * shaped layers at batch 64 on four streams 111 us -> 91 us with a budget of
 * 37; the 53 weight gradients of ResNet-50 at batch 256 on six streams
 * 2540 us -> 2241 us. A single layer on an idle GPU is slower with a budget.
 *
 *   sms : 1 .. 148; 0 or more than 148 restores the default (the whole GPU).
 * The setting is per host thread and affects ac_workspace_bytes*,
 * ac_wgrad_plan_info and every weight-gradient call the thread makes afterwards
 * (size the workspace under the same budget as the call that uses it; a
 * workspace that is too small for the plan is refused, never overrun).
 * Results do not depend on the budget beyond the order of the fp32 sums.
 * Returns AC_ERR_INVALID_ARG for a negative value.
 */
ac_status ac_set_sm_budget(int32_t sms);
int32_t ac_get_sm_budget(void);

/*
 * Profiling aid (not part of the paper's method). While a pair of CUDA events
 * (cudaEvent_t, created with timing enabled) is set for the calling host thread,
 * every weight-gradient call made from that thread records `before` and
 * `after` on its stream immediately around the main weight-gradient kernel
 * alone: not the staging passes, not the split-K reduction (with two main
 * launches in one call the events end up around the last). Under stream
 * capture the records become external event-record nodes of the graph.
 * Passing NULL for either clears the pair. The events stay the caller's.
 */
ac_status ac_set_kernel_timing_events(void *before, void *after);

/*
 * Reads back the status block a previous ac_conv2d_wgrad_compressed call left
 * in `workspace`: synchronises `stream`, then returns AC_OK, or AC_ERR_TIMEOUT
 * if a bounded wait inside a kernel gave up (dW is then not valid), or
 * AC_ERR_CUDA if the stream reports an error. `detail`, if non-NULL, receives
 * a kernel-specific code saying which wait ran out (0 when AC_OK).
 */
ac_status ac_workspace_status(const void *workspace, void *stream, uint32_t *detail);

/*
 * One backward step of a compressed layer on HOST buffers (Section 4, whole
 * path): copies X and dY to the device, compresses X to Z, computes dW from Z
 * and dY, copies dW back. For callers that hold their tensors in host memory
 * and for end-to-end timing.
 *
 *   x_host, dy_host in : host memory (pinned for asynchronous copies),
 *                        desc->layout / desc->dtype.
 *   dw_host        out : host memory, fp32.
 *   z_host    optional : if non-NULL also receives Z (desc->dtype).
 *   arena              : DEVICE scratch of at least ac_host_step_arena_bytes(desc)
 *                        bytes, 256-byte aligned; holds X, Z, dY, dW and the
 *                        wgrad workspace for the duration of the call.
 * Enqueues the copies and kernels on `stream` and returns without waiting;
 * the caller synchronises the stream before reading dw_host.
 */
size_t ac_host_step_arena_bytes(const ac_conv_desc *desc);
ac_status ac_backward_step_host(const ac_conv_desc *desc, const void *x_host,
                                const void *dy_host, float *dw_host, void *z_host,
                                void *arena, size_t arena_bytes, void *stream);

/*
 * The weight gradient without a workspace argument, for callers that cannot
 * allocate device memory. (The paper has no counterpart to this call; it
 * exists for the library's users, not for the method.)
 *
 * Some callers have no way to get scratch memory: they run inside a framework
 * whose memory pool already holds the whole device, so a raw cudaMalloc fails
 * or stalls every stream; or in a loop that must never wait on the allocator;
 * or as a plug-in that receives tensors but no allocator. For them the scratch
 * is a fixed array of AC_STATIC_SCRATCH_BYTES bytes of device memory that
 * belongs to the library image: every GPU that loads the library holds it
 * until the process ends. The call allocates and frees nothing.
 *
 * Computes the same dW as ac_conv2d_wgrad_compressed (same arguments z, dy,
 * dw, same layouts, dW overwritten), always on the fp32-ALU kernel.
 *   - The sum over the N*H_o*W_o positions is cut into as many slices as the
 *     array holds partial dW tensors for (256 bytes of it are the status
 *     block), each slice one fp32 running sum per output. A slice may be up to
 *     16384 positions long (the ordinary call stops at 2048, so this call's
 *     fp32 rounding error can be a few times larger); a problem that would
 *     need longer slices, because |dW| x 4 bytes x slices does not fit
 *     AC_STATIC_SCRATCH_BYTES, is refused with AC_ERR_WORKSPACE_TOO_SMALL
 *     before anything is launched. Problems of at most 16384 positions are
 *     never refused (one slice goes straight to dW).
 *   - The first call on each device looks up the array's device address (the
 *     device must be current). Make that first call outside any stream capture.
 *   - All calls on a device share the one array, which still holds the last
 *     call's partial sums: two calls that overlap on the GPU (different streams,
 *     or different host threads without ordering) race. Issue them on one stream
 *     or order them yourself.
 */
#define AC_STATIC_SCRATCH_BYTES (32u << 20)
ac_status ac_conv2d_wgrad_compressed_static(const ac_conv_desc *desc, const void *z,
                                            const void *dy, float *dw, void *stream);

/*
 * Non-uniform pooling blocks: k_h rows by k_w columns instead of k x k. The
 * paper (Section 6) lists such shapes as future work; Section 4's definitions
 * carry over unchanged with Z[n,c,p,q] = mean of X over h in [p k_h,
 * min((p+1) k_h, H)), w in [q k_w, min((q+1) k_w, W)), Z of size ceil(H/k_h) x
 * ceil(W/k_w), and Xt[n,c,h,w] = Z[n,c,h/k_h,w/k_w]. The three calls below are
 * ac_workspace_bytes, ac_compress and ac_conv2d_wgrad_compressed with the block
 * given beside the descriptor (k_h, k_w >= 1; desc->k is ignored); every other
 * argument, the layouts, the return codes and the status block are theirs.
 * k_h == k_w gives bit for bit what the square calls give. With k_h != k_w:
 * compression runs on the NHWC vector kernel (C_in a multiple of the 16-byte
 * vector) or the generic kernel; the weight gradient runs on the TMA-fed
 * tensor-core kernel when stride_h divides k_h and stride_w divides k_w
 * (bf16 NHWC directly, fp32 / NCHW staged through the workspace), else on the
 * fp32-ALU kernel. Passing k_h = k_w = 0 means desc->k.
 */
size_t ac_workspace_bytes_rect(const ac_conv_desc *desc, int32_t k_h, int32_t k_w);
ac_status ac_compress_rect(const ac_conv_desc *desc, int32_t k_h, int32_t k_w,
                           const void *x, void *z, void *y_out, void *stream);
ac_status ac_conv2d_wgrad_compressed_rect(const ac_conv_desc *desc, int32_t k_h, int32_t k_w,
                                          const void *z, const void *dy, float *dw,
                                          void *workspace, size_t workspace_bytes,
                                          void *stream);

/*
 * How ac_conv2d_wgrad_compressed will run this problem (pure host code; for
 * reports and tests). Returns AC_ERR_INVALID_ARG for an invalid descriptor.
 */
typedef struct {
    int32_t tensor_core;     /* 7: bf16 NHWC problems with partial pooling blocks next to the padding (an
                                odd map, padded taps) on which kernel 2 is expected to be slower reading
                                Z than reading the inflated map (3x3 on 7x7 at k = 2: four differently
                                zeroed copies of a 5x5-cell tile per image and class), or cannot keep its
                                tile copies in shared memory at all: the inflated map Xt is written to the
                                workspace (|X| bytes) and kernel 2 runs on it with k = 1 (described by
                                the other fields); with a workspace of ac_workspace_bytes_min() bytes
                                the kernel reads Z itself where it can. For square blocks of 4 and more
                                the same route is taken with Z re-blocked to a smaller block k' that
                                divides k, Z'[p][q] = Z[p*k'/k][q*k'/k] (|X| / k'^2 elements; the same
                                inflated map), where the plan for k' is expected to be faster (fewer
                                output classes; 64-channel layers pair their taps at k' = 2); `phases`
                                then counts the classes of that plan,
                                6: as 5 when taps share columns (both strides multiples of k, k divides H
                                and W, at most 128 columns, rows of Z a multiple of 16 bytes long): the matrix
                                is never written to memory; sixteen warps of the kernel build each K-tile
                                of it in shared memory from a strip of Z rows fetched by TMA, beside the
                                warp that issues the MMAs (band_rows = whole output rows per K-tile); a pooling block
                                that is a multiple k = f * s of the stride s is first re-blocked to k' = s
                                in the workspace, Z'[p][q] = Z[p/f][q/f] (|X| / s^2 elements: the same
                                inflated map), and runs as that,
                                5: bf16 NHWC with fewer than 64 input channels (a 3-channel stem): the
                                inflated, zero-padded values every output position reads are gathered
                                into a [positions][taps x C_in] matrix in the workspace (one column
                                per distinct shift of Z instead of per tap when both strides are
                                multiples of k and k divides H and W), then as 2 on the equivalent
                                1x1 problem over the output map (described by the other fields),
                                4: as 3, but as two launches whose results are added: the five small
                                partial products (five times the images; described by the other
                                fields), then the leading one, 3: fp32 and/or NCHW inputs staged
                                as bf16 NHWC terms in the workspace (fp32: six partial products =
                                six times the images), then as 2, 2: TMA-fed tcgen05
                                kernel, 1: tcgen05 kernel with inflating producer warps,
                                0: fp32-ALU kernel */
    int32_t splits;          /* K-slices summed by the split-K reduction */
    int32_t ctas;            /* CTAs of the main kernel */
    int32_t groups;          /* tensor-core path: CTAs that share one K-slice */
    int32_t band_rows;       /* tensor-core path: output rows of one image per K-tile */
    int32_t k_tile;          /* tensor-core path: positions per K-tile (kernel 2: per class; may span
                                several whole images of a small map) incl. zero fill */
    int32_t row_pitch;       /* tensor-core path: flat row pitch Wq of the tiles */
    int32_t stages;          /* tensor-core path: shared-memory pipeline depth */
    int32_t smem_bytes;      /* dynamic shared memory per CTA */
    int32_t tmem_columns;    /* tensor-memory columns allocated per CTA */
    int32_t units_per_cta;   /* tensor-core path: accumulator tiles (128 x block_n) per CTA; with 64
                                input channels a tile may hold two filter taps */
    int32_t block_n;         /* tensor-core path: output channels per accumulator tile */
    int32_t a_cells;         /* tensor-core path: cells per 64-channel chunk (kernel 2) or per 8-channel
                                plane (kernel 1) of the input tile in shared memory */
    int32_t phases;          /* tensor-core path: stride phases (kernel 1) or output classes
                                (kernel 2) per K-tile */
} ac_plan_info;
ac_status ac_wgrad_plan_info(const ac_conv_desc *desc, ac_plan_info *info);

/*
 * The same weight gradient with the repeated products taken out (Section 4 notes that a fused
 * operator on the compressed form could also cut memory traffic; this goes one step further and
 * cuts arithmetic. Section 4 defines only the result, which is unchanged). Inflation makes neighbouring taps read the same
 * pooled value: for the outputs of one class (ho mod k/s_h, wo mod k/s_w) every filter tap reads Z
 * at one of a few distinct shifts, and taps with the same shift form identical products. This call
 * accumulates one tile per (class, distinct shift) and adds each tile to all taps that map to it:
 * for a 3x3 filter at k = 2 that is 16 tiles instead of 36, at k = 4 36 instead of 144.
 * dW equals ac_conv2d_wgrad_compressed's up to fp32 summation order.
 *
 * When to call it (measured on B200, bf16 NHWC): it pays on large maps with many positions per
 * output class -- 3x3, 128 channels and more, maps of 64 x 64, k = 2 or 4: 1.4-1.6 times faster than
 * the dense call. It loses, by 10-25 %, on layers of 64 channels (the dense call computes two taps
 * per MMA there, this one cannot), on maps of 28 x 28 and smaller (each tile's fixed cost is paid
 * for fewer MMAs), at stride 2 with k = 2 (4 tiles instead of 9, but short ones) and at k = 8 (64
 * classes of 8 x 8 positions): call ac_conv2d_wgrad_compressed for those.
 *
 * ac_collapsed_workspace_bytes returns the scratch size, or 0 if the problem is not taken in this
 * form (not bf16/NHWC, channels not multiples of 64, strides not dividing k, k not dividing H and
 * W, or nothing to collapse such as k = 1 or a 1x1 filter at stride 1); it also reports the number of
 * accumulated tiles per block of 128 x C_out-block outputs in the collapsed and in the dense
 * form (their ratio is the saving in tensor-core work). ac_conv2d_wgrad_compressed_collapsed then
 * returns AC_ERR_UNSUPPORTED for such problems; arguments and conventions are those of
 * ac_conv2d_wgrad_compressed.
 */
size_t ac_collapsed_workspace_bytes(const ac_conv_desc *desc, int32_t *tiles_collapsed,
                                    int32_t *tiles_dense);
ac_status ac_conv2d_wgrad_compressed_collapsed(const ac_conv_desc *desc, const void *z,
                                               const void *dy, float *dw, void *workspace,
                                               size_t workspace_bytes, void *stream);

/*
 * Self-test of the kernels' failure reporting. Every wait inside the tensor-core kernels is
 * bounded: when it runs out, the kernel records it in the workspace status block and returns
 * instead of hanging. This call launches one small kernel that waits, with that same bounded
 * wait and a limit of `limit_cycles` SM clock cycles (1 .. 2^32), on a barrier nothing will
 * ever complete. Afterwards ac_workspace_status(workspace) must report AC_ERR_TIMEOUT with
 * detail 0x7E57. `workspace`: at least 256 bytes of device memory, 16-byte aligned.
 */
ac_status ac_selftest_bounded_wait(void *workspace, uint64_t limit_cycles, void *stream);

/* Static, human-readable name of a status code. */
const char *ac_status_string(ac_status status);

#ifdef __cplusplus
}
#endif
#endif /* AC_H_ */
