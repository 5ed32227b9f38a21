/*
 * libfsoftmax -- last-dimension softmax for NVIDIA B200 (sm_100a), C ABI, with the operators that
 * share its row skeleton (causal softmax, router softmax + top-k, layer_norm, group_norm).
 *
 * The operation is the `softmax` operator the paper reports its largest gains on (abstract and
 * Sec. IV-C: Gemma 4 E2B and Qwen 3.5 35B-A3B eager-attention softmax); its semantics are the
 * eager framework's on the same inputs (Sec. III-C, "Kernel Validator"):
 *
 *     y[i][j] = exp(z[i][j] - max_k z[i][k]) / sum_k exp(z[i][k] - max_k z[i][k]),   z = scale * x
 *
 * over the last dimension of a contiguous row-major [rows, cols] tensor. Arithmetic is fp32 inside
 * (fp32 accumulation of the row sum), the result is rounded once, to nearest even, to the tensor's
 * dtype. IEEE special values follow the formula literally: a -inf entry beside finite ones gives
 * exactly +0; a NaN or +inf entry (after scaling), or a row holding only -inf, makes that whole row
 * NaN. `scale` may be zero or negative.
 *
 * General conventions
 *   - Pointers named `x`/`y` are DEVICE pointers unless the entry point says "host".
 *   - The caller owns every buffer and the stream. Device entry points only enqueue work on
 *     `stream` (a cudaStream_t passed as void*, NULL = default stream): they never synchronise
 *     and keep no reference to the buffers after the enqueued work has run.
 *   - All entry points return an fs_status as int and enqueue nothing when they return an error.
 *   - The library works on the calling thread's current CUDA device. One GPU; no host fallback:
 *     without a usable CUDA device every compute entry point returns FS_ERR_CUDA.
 *   - Thread-safe. Per-device attributes are cached on first use.
 *   - Device memory: no entry point allocates per call. On first use per device the library
 *     allocates a 4-byte status word; the two-kernel path of very long rows (fs_softmax,
 *     fs_layer_norm, fs_group_norm on rows beyond FS_STATIC_MAX_ROW_BYTES) keeps one scratch buffer
 *     per device, allocated when first needed, grown when a call needs more, and fs_softmax_host
 *     keeps its staging buffers; fs_release frees the last two. fs_softmax_static allocates nothing.
 *   - Environment switches (each read once per process): FS_LOG=1 prints one line per call with the
 *     dispatcher's decision and launch geometry on stderr; FS_FORCE_KERNEL=warp|block|block_tma|
 *     cluster|generic replaces the choice of fs_softmax's dispatcher (a shape that kernel cannot run
 *     returns FS_ERR_UNSUPPORTED); FS_CHECK=1 validates every tensor pointer with
 *     cudaPointerGetAttributes (memory the current device cannot address is FS_ERR_INVALID_ARG);
 *     FS_SIM_NO_CLUSTER=1 and FS_SIM_SMEM_OPTIN=<bytes> make the library behave as on a device
 *     without cluster launch / with less shared memory, so that its downgrade paths can be tested.
 *   - Stream order is all a caller has to respect. Kernels are launched with programmatic dependent
 *     launch: they may become resident while the previous kernel of the stream drains, and read their
 *     inputs only after it has completed. Before that point the first wave of the long-row kernels
 *     asks the L2 cache for its own input (a prefetch, never a read: whatever the previous kernel
 *     still writes there is what the later read returns). FS_PDL=0 / FS_EARLY_PF=0 turn the two off.
 */
#ifndef FSOFTMAX_H_
#define FSOFTMAX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { FS_DTYPE_FP32 = 0, FS_DTYPE_BF16 = 1, FS_DTYPE_FP16 = 2 } fs_dtype;

/* Longest row (bytes) the split-row kernel holds in the shared memory of a 16-block cluster. */
#define FS_STATIC_MAX_ROW_BYTES (16 * 192 * 1024)
/* fs_softmax_static: size of the fixed device array every GPU holds, and the number of per-segment
 * (max, sum) pairs of its long-row path that fit behind the array's 256-byte header. */
#define FS_STATIC_SCRATCH_BYTES 65536
#define FS_STATIC_MAX_PAIRS ((FS_STATIC_SCRATCH_BYTES - 256) / 8)

typedef enum {
    FS_OK = 0,
    FS_ERR_INVALID_ARG = 1,    /* null pointer, negative size, unknown dtype/kernel, non-finite scale, partial overlap */
    FS_ERR_UNSUPPORTED = 2,    /* a forced kernel cannot handle this shape/alignment/launch geometry */
    FS_ERR_CUDA = 3,           /* a CUDA call failed; see fs_last_cuda_error() */
    FS_ERR_DEVICE_TIMEOUT = 4, /* a bounded device-side wait expired (reported by fs_device_status) */
    FS_ERR_DEVICE_BOUNDS = 5   /* checked build only: a kernel tried to touch memory outside its call's tensors */
} fs_status;

/* The kernels behind the size-based dispatcher (the "variants" of the operator in the sense of
 * the paper's Sec. III-A: same operator, different shape/dtype/layout -> different kernel). */
typedef enum {
    FS_KERNEL_AUTO = 0,
    FS_KERNEL_WARP = 1,       /* (sub-)warp per row, row held in registers */
    FS_KERNEL_BLOCK = 2,      /* block per row, 128-bit global loads, row held in registers */
    FS_KERNEL_BLOCK_TMA = 3,  /* rows staged in shared memory by bulk async copies: a block per row; the dispatcher's own choice for
                                 16-bit rows of 4.5-14 KiB is four rows per block, a warp per row */
    FS_KERNEL_CLUSTER = 4,    /* row split over a thread-block cluster of 1..16 blocks, slices resident in shared memory,
                                 (max,sum) pairs exchanged through distributed shared memory */
    FS_KERNEL_GENERIC = 5     /* any cols, any alignment. Element-wise accesses, the row read twice -- except rows whose byte length
                                 is not a multiple of 16 in 16-byte aligned tensors, which (up to what a cluster's shared memory holds)
                                 are read and written as the aligned 16-byte vectors that cover them, unless a block size is forced */
} fs_kernel;

/*
 * fs_softmax -- y = softmax(scale * x) over the last dimension; the dispatcher picks the kernel.
 *   x, y   device pointers to rows*cols elements of `dtype`, row-major, row pitch = cols elements.
 *          x == y (exact aliasing) is allowed; any other overlap returns FS_ERR_INVALID_ARG.
 *          Any alignment is accepted; the fast kernels need 16-byte aligned x and y and a row size
 *          that is a multiple of 16 bytes, other cases run the generic kernel.
 *   rows, cols  >= 0. rows == 0 or cols == 0 returns FS_OK without a launch.
 *   dtype  an fs_dtype; x and y share it.
 *   scale  finite float, multiplies x before the max is taken (scale <= 0 is legal).
 *   stream cudaStream_t as void*.
 */
int fs_softmax(const void* x, void* y, int64_t rows, int64_t cols, int dtype, float scale, void* stream);

/*
 * fs_softmax_ex -- as fs_softmax, with the kernel and its launch geometry forced (tests, tuning).
 *   kernel   an fs_kernel; FS_KERNEL_AUTO behaves like fs_softmax.
 *   threads  threads per block, 0 = the kernel's own choice. Must be a multiple of 32.
 *   cluster  blocks per cluster for FS_KERNEL_CLUSTER (1 .. 16), 0 = the kernel's choice;
 *            ignored by the other kernels.
 * Returns FS_ERR_UNSUPPORTED when the forced kernel cannot run this shape, alignment or geometry.
 */
int fs_softmax_ex(const void* x, void* y, int64_t rows, int64_t cols, int dtype, float scale,
                  void* stream, int kernel, int threads, int cluster);

/*
 * fs_softmax_causal -- softmax with the causal mask of eager attention applied inside the kernel
 * (the operator fusion the paper lists among its levers, Sec. II-B; the workloads are the
 * eager-attention softmax calls of its Table I). Row i keeps columns j <= i + q_offset:
 *
 *     y[i][j] = softmax over the kept columns of scale * x[i][.]   for j <= i + q_offset
 *     y[i][j] = +0                                                   for j >  i + q_offset
 *
 * i.e. what fs_softmax returns when every masked x[i][j] holds -inf (for scale > 0), except that
 * masked inputs are never read, so they may hold anything, and only the kept part of x crosses the
 * memory bus. q_offset = 0 is the square case (row i sees columns 0..i), q_offset = cols - rows
 * aligns the last row with the last column (decoding with a key/value cache); q_offset >= cols - 1
 * masks nothing. A row with no kept column (i + q_offset < 0) is all NaN, like an all -inf row,
 * and a row made NaN by a kept NaN or +inf is NaN in its masked part too.
 *   x, y, rows, cols, dtype, scale, stream   as for fs_softmax (x == y allowed).
 * Vector-aligned tensors with rows up to FS_STATIC_MAX_ROW_BYTES run the split-row kernel, one
 * cluster per row; everything else the generic kernel.
 */
int fs_softmax_causal(const void* x, void* y, int64_t rows, int64_t cols, int64_t q_offset, int dtype, float scale,
                      void* stream);

/*
 * fs_router_topk -- the router step of a mixture-of-experts layer: softmax over the expert logits
 * of each token, then the k most probable experts (the softmax of the paper's Qwen 3.5 35B-A3B
 * workload, Table I, fused with the selection that follows it in such a router; operator fusion
 * is the lever of Sec. II-B).
 *
 *     p = softmax(scale * x[i][.]);   idx[i][0..k) = the k columns with the largest p, largest
 *     first, equal values in column order;   w[i][j] = p[idx[i][j]], or, with `renormalize`,
 *     p[idx[i][j]] / sum_j p[idx[i][j]].
 *
 *   x     device pointer, rows*cols elements of `dtype`, 16-byte aligned, row size a multiple of
 *         16 bytes and cols <= 1024 (rows live in the registers of a warp); other shapes return
 *         FS_ERR_UNSUPPORTED.
 *   w     device pointer to rows*k floats (fp32 whatever `dtype` is); idx: rows*k int32.
 *   k     1 <= k <= min(cols, FS_ROUTER_MAX_K).
 * The selection is made on the inputs (the order of p is the order of scale*x), so it is exact: a
 * negative scale selects the smallest x, a zero scale the first k columns. NaN inputs count as the
 * smallest value for the selection; a row with a NaN or +inf (after scaling), or with only -inf,
 * has NaN weights. Weights meet the fp32 bound of fs_softmax (|error| <= 1e-6).
 */
#define FS_ROUTER_MAX_K 64
int fs_router_topk(const void* x, float* w, int32_t* idx, int64_t rows, int64_t cols, int k, int dtype, float scale,
                   int renormalize, void* stream);

/*
 * fs_log_softmax -- the logarithm of the same operator, formed directly (the variant of the softmax
 * family that language-model heads consume; operator variants are the paper's Sec. III-A):
 *
 *     y[i][j] = z[i][j] - max_k z[i][k] - ln sum_k exp(z[i][k] - max_k z[i][k]),   z = scale * x
 *
 *   x, y, rows, cols, dtype, scale, stream   as for fs_softmax (x == y allowed; scale may be zero
 *   or negative). A -inf entry beside finite ones gives -inf; a NaN or +inf entry (after scaling),
 *   or a row holding only -inf, makes the whole row NaN.
 * fp32 output is within 1e-6 * max(1, |y|) of the fp64 value, 16-bit output within one unit in the
 * last place of the correctly rounded fp64 value. Rows up to 9 KiB stay in the registers of a
 * (sub-)warp, longer rows are split over a cluster with the slices resident in shared memory (one
 * read and one write of HBM per element), ragged or misaligned rows take a three-pass kernel.
 */
int fs_log_softmax(const void* x, void* y, int64_t rows, int64_t cols, int dtype, float scale, void* stream);

/*
 * fs_softmax_f32out -- softmax of a bf16/fp16 tensor written as binary32: what eager attention asks
 * for with softmax(scores, dim=-1, dtype=float32) before it casts back (the mixed-dtype variant of
 * the operator; variants are the paper's Sec. III-A).
 *   x      device pointer, rows*cols elements of `dtype` (FS_DTYPE_BF16 or FS_DTYPE_FP16 only).
 *   y      device pointer, rows*cols floats; must not overlap x.
 * Same formula, special values and scale rules as fs_softmax; every output is within 1e-6 of the
 * fp64 value. Traffic is 6 bytes per element (2 in, 4 out).
 */
int fs_softmax_f32out(const void* x, float* y, int64_t rows, int64_t cols, int dtype, float scale, void* stream);

/*
 * fs_softmax_masked -- softmax with an additive mask applied inside the kernel, the other half of the
 * `scores + mask -> softmax` pair of eager attention (operator fusion, the paper's Sec. II-B; the
 * workloads are the eager-attention softmax calls of its Table I):
 *
 *     y[i][j] = softmax over j of ( scale * x[i][j] + mask[mrow(i)][j] )
 *
 * The rows of x are ordered (batch, head, query); the mask has one row per (batch, query) and is
 * shared by the heads: mrow(i) = (i / (heads * q_rows)) * q_rows + i % q_rows. The mask is added
 * unscaled; -inf entries mask a column (a fully masked row is NaN, like an all -inf row), finite
 * entries act as a bias.
 *   x, y    as for fs_softmax (x == y allowed); rows must be a multiple of heads * q_rows.
 *   mask    device pointer, (rows / heads) * cols elements of `dtype`, dense, never written.
 * Parity: the exponent scale * x + mask is formed in binary32 before the row maximum is taken off,
 * so fp32 output is within 1e-6 + 2.5e-7 * Z * y of the fp64 value, Z the largest finite |scale * x
 * + mask| of the row (1e-6 for |z| up to a few units); 16-bit output within one unit in the last
 * place of the correctly rounded value.
 */
int fs_softmax_masked(const void* x, const void* mask, void* y, int64_t rows, int64_t cols, int64_t q_rows, int64_t heads,
                      int dtype, float scale, void* stream);

/*
 * fs_softmax_backward -- the gradient of y = softmax(scale * x) with respect to x (what a training
 * step asks of the same operator):
 *
 *     dx[i][j] = scale * y[i][j] * (dy[i][j] - sum_k dy[i][k] * y[i][k])
 *
 *   dy, y  device pointers, rows*cols elements of `dtype`: the upstream gradient and the forward output.
 *   dx     device pointer, rows*cols elements; may be the same buffer as dy or as y (partial overlap
 *          is FS_ERR_INVALID_ARG).
 *   scale  the forward call's scale (finite).
 * Binary32 arithmetic and accumulation; the result is rounded once. Rows up to 4 KiB stay in
 * registers, longer rows are split over a cluster with both slices resident in shared memory (two
 * reads and one write of HBM per element), ragged or misaligned rows take a two-pass kernel.
 */
int fs_softmax_backward(const void* dy, const void* y, void* dx, int64_t rows, int64_t cols, int dtype, float scale,
                        void* stream);

/*
 * fs_layer_norm -- layer normalisation over the last dimension, one of the two normalisation
 * operators the paper reports generated kernels for (Sec. IV-C, Stable Diffusion 3.5 Medium):
 *
 *     mu_i = mean_j x[i][j],   var_i = mean_j (x[i][j] - mu_i)^2   (biased),
 *     y[i][j] = (x[i][j] - mu_i) / sqrt(var_i + eps) * gamma[j] + beta[j]
 *
 *   x, y    device pointers, rows*cols elements of `dtype`, row-major, dense; x == y allowed,
 *           partial overlap is FS_ERR_INVALID_ARG.
 *   gamma, beta   device pointers to cols elements of `dtype`, or NULL (1 and 0), independently.
 *   eps     finite, >= 0. Statistics and arithmetic are binary32; the output is rounded once.
 *   stream  cudaStream_t as void*.
 * Rows up to 4 KiB stay in the registers of a (sub-)warp, 16-bit rows up to 9 KiB too (packed, and
 * widened where they are used); longer rows are split over
 * a cluster of 1..16 blocks with the slices resident in shared memory (one read and one write of
 * HBM per element, as for fs_softmax); rows beyond a cluster's shared memory (about 3 MiB) are
 * cut into segments over two kernels, whose partial statistics pass through the library's
 * per-device scratch buffer (16 bytes per segment; see "Device memory" above: a call allocates
 * only when the buffer has to grow, which it cannot do inside a stream capture); ragged or
 * misaligned rows take a three-pass kernel.
 * A NaN or infinity in a row makes the whole row NaN. rows == 0 or cols == 0 launches nothing.
 */
int fs_layer_norm(const void* x, const void* gamma, const void* beta, void* y, int64_t rows, int64_t cols, int dtype,
                  float eps, void* stream);

/*
 * fs_group_norm -- group normalisation (the paper's largest normalisation result, Sec. IV-C) of a
 * dense [n, channels, spatial] tensor (NCHW with the spatial dimensions flattened): each
 * (sample, group) block of channels/groups * spatial contiguous elements is normalised like one
 * row of fs_layer_norm; gamma and beta (channels elements each, or NULL) are indexed by channel.
 *   groups  >= 1 and a divisor of channels.
 * The same kernels as fs_layer_norm run on rows of channels/groups * spatial elements; the fast
 * path needs spatial * element size to be a multiple of 16 bytes.
 */
int fs_group_norm(const void* x, const void* gamma, const void* beta, void* y, int64_t n, int64_t channels, int64_t spatial,
                  int64_t groups, int dtype, float eps, void* stream);

/*
 * fs_split_geometry -- the launch geometry the dispatcher gives the split-row kernels (softmax,
 * log_softmax, masked, backward, normalisations) for rows of `cols` elements: blocks per cluster
 * (1..16), threads per block and the bytes of a row each block holds in shared memory. Pure host
 * arithmetic, no CUDA call. FS_ERR_UNSUPPORTED when the row size is not a multiple of 16 bytes or
 * exceeds what a 16-block cluster holds.
 */
int fs_split_geometry(int64_t cols, int dtype, int* cluster, int* threads, int64_t* slice_bytes);

/*
 * fs_select_kernel -- the dispatcher's decision, without a launch (no CUDA call is made when the
 * device attributes are already cached or `x_align`/`y_align` rule the fast paths out).
 *   x_align, y_align  the largest power of two (<= 16 is enough) dividing each base address.
 * Returns an fs_kernel (>= 1), or a negative fs_status on invalid arguments. FS_KERNEL_GENERIC
 * covers two forms: vector-aligned rows of 1 MiB or more that no cluster holds are cut into
 * segments over two kernels (partial (max, sum) pairs, 8 bytes per segment, through the library's
 * per-device scratch buffer; calls that use it are ordered on the device by an event, whatever
 * their streams; inside a stream capture the buffer cannot grow, so the first such call should
 * come before the capture); everything else runs one block per row.
 * On a device without cluster launch, or with too little shared memory for the split-row kernel,
 * fs_softmax runs FS_KERNEL_CLUSTER's one-block form where the row fits one block and the generic
 * forms otherwise; fs_softmax_ex with a forced kernel returns FS_ERR_UNSUPPORTED instead.
 */
int fs_select_kernel(int64_t rows, int64_t cols, int dtype, int x_align, int y_align);

/*
 * fs_softmax_host -- the same operation on HOST buffers, end to end.
 *   x_host, y_host  host pointers (pinned memory gives full copy bandwidth; pageable works).
 * Splits the rows into chunks of about 8 MiB and pipelines host->device copy, kernel and
 * device->host copy on three internal streams through four pairs of device staging buffers the
 * library allocates on first use and keeps (grown on demand, released by fs_release). Blocks until
 * y_host is complete. Calls on one device are serialised.
 */
int fs_softmax_host(const void* x_host, void* y_host, int64_t rows, int64_t cols, int dtype, float scale);

/*
 * fs_copy -- speed-of-light calibration: copies `bytes` bytes from x to y (device pointers, both
 * 16-byte aligned, bytes a multiple of 16) with the same 128-bit streaming accesses and grid
 * sizing as the softmax kernels. Same traffic as a softmax over the same buffers, no arithmetic.
 */
int fs_copy(const void* x, void* y, int64_t bytes, void* stream);

/*
 * fs_device_status -- reads and clears the device-side status word of the current device
 * (synchronises the device). FS_OK, or FS_ERR_DEVICE_TIMEOUT if a bounded wait on an async copy
 * expired inside a kernel since the last call (the outputs of that launch are then undefined).
 */
int fs_device_status(void);

/*
 * fs_softmax_static -- fs_softmax for callers that must not allocate device memory.
 * (The paper has no counterpart: this entry point exists for the library's users only.)
 *
 * Every other compute entry point calls cudaMalloc on its first use per device (the status buffer
 * its kernels write when a bounded wait expires), the long-row path of fs_softmax again whenever
 * its scratch buffer must grow, fs_softmax_host for its staging buffers. Some callers cannot afford
 * such a call: a process that has handed all device memory to its own pool and must not touch the
 * driver's allocator again, a service that has to prove it cannot run out of memory after start-up,
 * or a latency-critical loop in which the implicit device synchronisation of an allocation is
 * unacceptable. This entry point makes no cudaMalloc, cudaFree or other allocating call, ever.
 * What the other paths keep in allocated memory lives in one array of FS_STATIC_SCRATCH_BYTES that
 * is part of the library's device code: every GPU that loads the library holds those bytes until the
 * process exits. The array carries the status buffer and the scratch of the long-row path:
 *   - rows up to FS_STATIC_MAX_ROW_BYTES run the split-row kernel (FS_KERNEL_CLUSTER's
 *     shared-memory-resident form), which needs the status buffer only;
 *   - longer rows are cut into segments over two kernels, as in fs_softmax; the first writes one
 *     (max, sum) pair per row and segment into the array, the second reads them back. rows times
 *     segments per row (about 8 * SM count / rows, at least 1, at most 1024) must not exceed
 *     FS_STATIC_MAX_PAIRS: FS_ERR_UNSUPPORTED otherwise.
 *
 *   x, y, rows, cols, dtype, scale, stream   as for fs_softmax; x and y are DEVICE pointers.
 *   Limits: x and y 16-byte aligned, row size a multiple of 16 bytes, rows * blocks-per-row
 *           below 2^31; scale == 0 only for rows that split into whole chunks (powers of two do)
 *           or that take the long-row path. Anything else returns FS_ERR_UNSUPPORTED and enqueues
 *           nothing; there is no silent switch to a path that allocates.
 *   First call on a device: looks up the array's device address (cudaGetSymbolAddress, with that
 *           device current) and raises the kernel's shared-memory limit: queries and attribute
 *           calls, no allocation. Make that first call before starting any stream capture.
 *   Sharing: all calls on a device share the one array, and it keeps what the last call left
 *           there. Nothing in it has to start at zero except the status word, which is cleared when
 *           fs_static_status reads it: the pairs are all written by a call's first kernel before
 *           its second kernel reads them. Two long-row calls whose work overlaps on the GPU
 *           (different streams, no event between them) race on the pairs and produce wrong
 *           results: keep such calls on one stream or order them yourself. Calls on the split-row
 *           kernel only OR bits into the status word and may overlap freely.
 */
int fs_softmax_static(const void* x, void* y, int64_t rows, int64_t cols, int dtype, float scale, void* stream);

/*
 * fs_static_status -- fs_device_status for fs_softmax_static: synchronises the device, reads the
 * status word of the fixed array and clears it if set. Allocates nothing (a copy from the address
 * cudaGetSymbolAddress gave). FS_OK, or FS_ERR_DEVICE_TIMEOUT if a bounded wait expired inside a
 * kernel launched by fs_softmax_static since the last call.
 * (The paper has no counterpart.)
 */
int fs_static_status(void);

/*
 * Self-tests of the bounded device-side waits (the paper's validator watches for launches that do not
 * come back, Sec. III-C; these calls let a test see the library's own guard work without any fault).
 * Every wait on an async copy polls at most N times (2^23, about two seconds); a wait that runs out
 * sets a status bit, the kernel carries on without waiting again and returns, and fs_device_status
 * reports FS_ERR_DEVICE_TIMEOUT once.
 *   fs_debug_set_wait_polls(polls)  sets N for the two calls below and for FS_KERNEL_CLUSTER launches
 *           of fs_softmax / fs_softmax_ex on the current device (polls <= 0 restores 2^23); the
 *           other kernels keep 2^23.
 *   fs_debug_wait_probe(stream)     launches one block that arms a barrier for 16 bytes nobody
 *           copies and waits for it: the wait must run out. Touches no tensor.
 *   fs_debug_softmax_expire(...)    fs_softmax_ex(..., FS_KERNEL_CLUSTER, threads, cluster) with every
 *           chunk barrier armed for 16 bytes more than are copied: the copies complete, the waits
 *           run out, every warp gives up once and finishes the row. Call it with a small poll cap
 *           (a few thousand: long enough for the copies to land) and restore the default after.
 *           y receives the normal result when the cap was long enough for the data to arrive.
 */
/*
 * The checked build (libfsoftmax_debug.so: the same sources compiled with -DFS_DEBUG_BOUNDS; the paper's
 * validator lists illegal memory accesses among the failures it must catch, Sec. III-C). In it every
 * global load, store and bulk copy of every kernel is checked against the address ranges of the
 * tensors its entry point was given; an access outside them, or a store into an input, is skipped and
 * recorded instead of performed: fs_device_status then returns FS_ERR_DEVICE_BOUNDS (once) and
 * fs_debug_bad_address the first offending address. Several times slower; one stream at a time (the
 * ranges are one table per device); fs_softmax_static and fs_softmax_host go unchecked.
 *   fs_debug_checked_build()        1 in the checked build, 0 in the normal one.
 *   fs_debug_bad_address(&a)        reads and clears the first refused address (0 if none); synchronises.
 *                                   FS_ERR_UNSUPPORTED in the normal build.
 *   fs_debug_shrink_writable(n)     self-test: until called again with 0, the output ranges this thread
 *                                   registers end n bytes early, so a correct kernel "overruns" them by
 *                                   n bytes without touching anything it should not; the checker must
 *                                   refuse exactly those stores. FS_ERR_UNSUPPORTED in the normal build.
 */
int fs_debug_checked_build(void);
int fs_debug_bad_address(uint64_t* address);
int fs_debug_shrink_writable(int64_t bytes);

int fs_debug_set_wait_polls(int polls);
int fs_debug_wait_probe(void* stream);
int fs_debug_softmax_expire(const void* x, void* y, int64_t rows, int64_t cols, int dtype, float scale, void* stream,
                            int threads, int cluster);

/* fs_release -- frees the staging buffers and streams fs_softmax_host created on the current device and the
 * scratch buffer of the two-kernel long-row paths (synchronises the device if there is one to free). */
int fs_release(void);

/* The cudaError_t behind the last FS_ERR_CUDA returned on this thread (0 if none). */
int fs_last_cuda_error(void);

/* Static strings. */
const char* fs_strerror(int status);
const char* fs_kernel_name(int kernel);
const char* fs_version(void);

#ifdef __cplusplus
}
#endif
#endif /* FSOFTMAX_H_ */
