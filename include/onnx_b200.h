/*
 * onnx_b200.h - C ABI of the ONNX Conv / Gemm library for NVIDIA B200 (sm_100a).
 *
 * The library computes the two operators at the centre of the inference code an
 * ONNX compiler emits for MNIST- and ResNet-50-class models (the paper's Sec. 4.1
 * names convolution and Gemm as supported operators; Sec. 4.2 runs both models):
 * ONNX Conv (2-D, NCHW) and ONNX Gemm, each with a fused bias and an optional
 * fused Relu (the producer/consumer fusion idea of Sec. 3.4.3).  Operator
 * semantics follow the ONNX standard the paper builds on (Sec. 2.1); shapes are
 * inferred from input shapes and attributes as in the shape-inference pass of
 * Sec. 3.4.2, restricted to static shapes.
 *
 * General conventions
 *   - All tensors are dense, row-major, 32-bit float.  Conv tensors are NCHW.
 *   - Pointers named X, W, B, A, C, Y and `workspace` are DEVICE pointers owned
 *     by the caller.  Attribute structs, dims arrays and out-parameters are HOST
 *     memory.  `cuda_stream` is a cudaStream_t passed as void* (NULL = the
 *     default stream).
 *   - Run calls enqueue work on the given stream and return without
 *     synchronising.  They never allocate or free device memory.
 *   - Inputs are read-only; Y must not overlap any input or the workspace.
 *   - Every device pointer must be 16-byte aligned.
 *   - No C++ exception crosses this boundary; every failure is a status code and
 *     leaves Y untouched (errors are detected before anything is launched).
 *   - Tensors with more than 2^31-1 elements are rejected (ONNXB_ERR_UNSUPPORTED).
 *   - Arithmetic: fp32 inputs and outputs.  Kernels of the tensor-core family
 *     multiply in TF32 (10-bit mantissa operands) and accumulate in fp32; kernels
 *     of the SIMT family use fp32 FMA.  Operands are rounded to TF32 to nearest
 *     (2^-11 per operand) before they reach the tensor core, which gives
 *         |Y - exact| <= 1e-3 * sum|x*w| + 1e-5       per output element
 *     for finite inputs of moderate magnitude.  One exception: a 1x1, stride-1
 *     convolution whose image planes TMA can address (ONNXB_KERNEL_MMA_GEMM) feeds
 *     X to the tensor core as stored, and the hardware drops the low 13 mantissa
 *     bits (truncation: up to 2^-10, 3.4e-4 on average, always towards zero); W is
 *     still rounded.  There the bound is 1.5e-3 * sum|x*w| + 1e-5 in the worst case
 *     (every activation just below a TF32 grid point and every term of one sign); it
 *     stays below 1e-3 * sum|x*w| + 1e-5 whenever the weights are exact in TF32, and
 *     measured 0.53 of that on uniform non-negative operands.
 */
#ifndef ONNX_B200_H_
#define ONNX_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ONNXB_OK = 0,
    ONNXB_ERR_NULL = 1,            /* a required pointer is NULL (or B given/omitted against has_bias) */
    ONNXB_ERR_ATTR = 2,            /* an attribute value ONNX does not admit */
    ONNXB_ERR_SHAPE = 3,           /* shapes inconsistent with each other or with the attributes */
    ONNXB_ERR_UNSUPPORTED = 4,     /* valid ONNX, outside this library's range (size, alignment, negative pads) */
    ONNXB_ERR_WORKSPACE = 5,       /* workspace missing or smaller than the descriptor asks for */
    ONNXB_ERR_CUDA = 6,            /* a CUDA runtime/driver call failed (launch configuration, no device) */
    ONNXB_ERR_DEVICE_TIMEOUT = 7   /* a bounded device-side wait ran out (see onnxb_last_device_status) */
} onnxb_status;

typedef enum {
    ONNXB_NOTSET = 0,              /* use `pads` */
    ONNXB_SAME_UPPER = 1,          /* out = ceil(in/stride); odd padding unit at the end */
    ONNXB_SAME_LOWER = 2,          /* out = ceil(in/stride); odd padding unit at the beginning */
    ONNXB_VALID = 3                /* no padding */
} onnxb_auto_pad;

/* Kernel family a descriptor resolved to (reported by onnx_conv2d_desc_query_kernel). */
typedef enum {
    ONNXB_KERNEL_SIMT_DIRECT = 0,  /* fp32 FMA direct convolution (thin contractions, any attributes) */
    ONNXB_KERNEL_SIMT_DEPTHWISE = 1, /* fp32 FMA, one input channel per output channel, smem row tiles */
    ONNXB_KERNEL_MMA_GEMM = 2,     /* 1x1 stride-1: batched tcgen05 TF32 GEMM straight from NCHW via TMA */
    ONNXB_KERNEL_MMA_IMPLICIT = 3, /* general implicit GEMM: TMA staging + in-smem im2col + tcgen05 TF32 */
    ONNXB_KERNEL_MMA_GATHER_GEMM = 4 /* other 1x1 (strided, or H*W not a multiple of 4): the pixels read are
                                        gathered (and rounded) into the workspace, then the same batched TF32 GEMM */
} onnxb_kernel_family;

/*
 * Attribute set of ONNX Conv, one field per ONNX attribute (the paper's onnx
 * dialect mirrors ONNX attributes one for one, Sec. 3.2), plus the two fusion
 * switches.  Zero-initialise the struct to get every ONNX default.
 */
typedef struct {
    int64_t x_dims[4];        /* N, C, H, W */
    int64_t w_dims[4];        /* M, C/group, kH, kW */
    int64_t kernel_shape[2];  /* {0,0}: infer from w_dims; otherwise must equal w_dims[2..3] */
    int64_t pads[4];          /* ONNX order: h_begin, w_begin, h_end, w_end; >= 0 */
    int64_t strides[2];       /* along H, along W; {0,0} = default {1,1} */
    int64_t dilations[2];     /* along H, along W; {0,0} = default {1,1} */
    int64_t group;            /* 0 = default 1 */
    int32_t auto_pad;         /* onnxb_auto_pad; anything but NOTSET excludes non-zero pads */
    int32_t has_bias;         /* non-zero: B[M] is added */
    int32_t fuse_relu;        /* non-zero: max(.,0) applied to the result */
    int32_t reserved;         /* must be 0 */
} onnxb_conv2d_attrs;

typedef struct onnxb_conv2d_desc_s *onnxb_conv2d_desc_t;

/*
 * onnx_conv2d_desc - validate attributes, resolve auto_pad, infer the output
 * shape (Sec. 3.4.2) and choose a kernel (host only, no CUDA call).
 *
 *   P = floor((H + h_begin + h_end - ((kH-1)*dh + 1)) / sh) + 1, likewise Q.
 *   SAME_*: P = ceil(H/sh), total = max((P-1)*sh + (kH-1)*dh + 1 - H, 0),
 *           UPPER: begin = total/2, end = total - begin; LOWER the other way.
 *
 * attrs (host, read) ; out (host, written on success; destroy with
 * onnx_conv2d_desc_destroy).  Descriptors are immutable and may be shared by
 * threads.  Errors: NULL arguments -> ERR_NULL; non-positive stride/dilation,
 * unknown auto_pad, auto_pad with non-zero pads, kernel_shape != W dims,
 * reserved != 0 -> ERR_ATTR; non-positive dims, C % group, M % group,
 * w_dims[1] != C/group, kernel larger than the padded input -> ERR_SHAPE;
 * negative pads or a tensor above 2^31-1 elements -> ERR_UNSUPPORTED.
 */
onnxb_status onnx_conv2d_desc(const onnxb_conv2d_attrs *attrs, onnxb_conv2d_desc_t *out);

/*
 * onnx_conv2d_desc_query - read back what the descriptor resolved.  Any of the
 * out-pointers (host) may be NULL.  y_dims = {N, M, P, Q}; resolved_pads in ONNX
 * order; workspace_bytes = device scratch onnx_conv2d_run needs (may be 0).
 */
onnxb_status onnx_conv2d_desc_query(onnxb_conv2d_desc_t desc, int64_t y_dims[4],
                                    int64_t resolved_pads[4], size_t *workspace_bytes);

/* Kernel family the descriptor will launch (the dispatch step: a contraction of
 * C/group*kH*kW terms that is too thin for the tensor cores, or a depthwise
 * convolution, goes to a SIMT kernel).  Returns -1 for a NULL descriptor. */
int onnx_conv2d_desc_query_kernel(onnxb_conv2d_desc_t desc);

/*
 * onnx_conv2d_run - Y = relu?( conv(X, W) + B ), ONNX Conv (Sec. 4.1), i.e.
 *
 *   Y[n,m,p,q] = B[m] + sum_{c<C/g, r<kH, s<kW}
 *       Xpad[n, (m div (M/g))*(C/g)+c, p*sh + r*dh - h_begin, q*sw + s*dw - w_begin] * W[m,c,r,s]
 *
 * with Xpad = X inside the image and 0 outside; the kernel is not flipped.
 *
 * X [N,C,H,W], W [M,C/g,kH,kW], B [M] (NULL exactly when has_bias == 0),
 * Y [N,M,P,Q]: device, fp32, dense.  workspace: device scratch of at least the
 * queried size (NULL allowed when that size is 0); its contents are undefined on
 * return and two runs that share a workspace must not overlap in time.
 * Errors: ERR_NULL, ERR_WORKSPACE, ERR_UNSUPPORTED (misaligned pointer),
 * ERR_CUDA (launch failure).
 */
onnxb_status onnx_conv2d_run(onnxb_conv2d_desc_t desc, const float *X, const float *W,
                             const float *B, float *Y, void *workspace, size_t workspace_bytes,
                             void *cuda_stream);

/*
 * onnx_conv2d_add_run - Conv, then Add of a second tensor, then the descriptor's Relu, in one
 * pass: Y = relu?( Conv(X, W) + B + R ).  This is a residual connection written the way the
 * compiler's fusion of a single-use producer into its consumer leaves it (Sec. 3.4.3; elementwise
 * Add is the paper's running example, Sec. 3.2): the convolution's output is never written and
 * read back.  R: device, same shape and layout as Y ([N, M, P, Q], dense, 16-byte aligned), read
 * only, must not overlap Y; every other argument and error exactly as for onnx_conv2d_run
 * (ERR_NULL when R is NULL).  The addition is one fp32 add per element before the Relu.
 */
onnxb_status onnx_conv2d_add_run(onnxb_conv2d_desc_t desc, const float *X, const float *W, const float *B,
                                 const float *R, float *Y, void *workspace, size_t workspace_bytes,
                                 void *cuda_stream);

/*
 * onnx_conv2d_prepack / onnx_conv2d_run_prepacked - for weights that are constants of the graph
 * (the usual case in inference; the compiler propagates constants ahead of time, Sec. 3.4.4):
 * the weight re-layout that onnx_conv2d_run performs at every call is done once.
 *
 * onnx_conv2d_prepack writes the derived copy of W that the descriptor's kernel reads (packed and
 * rounded to TF32 for ONNXB_KERNEL_MMA_IMPLICIT, rounded to TF32 for ONNXB_KERNEL_MMA_GEMM and
 * ONNXB_KERNEL_MMA_GATHER_GEMM) into `packed` (device, caller-owned, at least the workspace_bytes
 * of onnx_conv2d_desc_query, 16-byte aligned).  Descriptors of the SIMT kernels read W directly:
 * the call then does nothing and returns OK.
 * onnx_conv2d_run_prepacked computes what onnx_conv2d_run (R == NULL) or onnx_conv2d_add_run
 * (R != NULL) computes, from that copy, bit for bit.  W must still be passed (the kernels that use
 * no copy read it) and must be the tensor that was packed; `packed` is read only.  workspace /
 * workspace_bytes: as for onnx_conv2d_run for the SIMT kernels and for
 * ONNXB_KERNEL_MMA_GATHER_GEMM (whose gathered input still needs scratch: the queried
 * workspace_bytes always suffice), ignored (may be NULL / 0) otherwise.  Errors: as the calls they
 * stand for; ERR_WORKSPACE when `packed` is too small, ERR_NULL when it is missing where needed.
 */
onnxb_status onnx_conv2d_prepack(onnxb_conv2d_desc_t desc, const float *W, void *packed, size_t packed_bytes,
                                 void *cuda_stream);
onnxb_status onnx_conv2d_run_prepacked(onnxb_conv2d_desc_t desc, const float *X, const float *W, const void *packed,
                                       const float *B, const float *R, float *Y, void *workspace,
                                       size_t workspace_bytes, void *cuda_stream);

void onnx_conv2d_desc_destroy(onnxb_conv2d_desc_t desc);

/*
 * onnx_conv2d_run_static - the same computation as onnx_conv2d_run, for callers that
 * cannot allocate device memory and therefore have no workspace to pass: a control loop
 * whose memory budget was frozen at start-up, a plugin inside a host application that owns
 * the allocator, a process whose device memory is already fully committed.  (This entry
 * point is a convenience of this library; the paper has no counterpart.)
 *
 * The scratch comes from a fixed array of onnx_conv2d_static_scratch_bytes() bytes
 * (10 MiB) that is part of the library image: every GPU the library is loaded on holds it
 * until the process exits.  The call allocates and frees nothing.  A descriptor whose
 * queried workspace_bytes exceeds that size is rejected with ONNXB_ERR_WORKSPACE and
 * nothing is launched; use onnx_conv2d_run with your own workspace for such layers.
 *
 * X, W, B, Y, cuda_stream: exactly as for onnx_conv2d_run (device pointers, caller-owned).
 * The first call on each device looks up the array's device address (a host-side query,
 * not an allocation); make that first call outside any stream capture.
 * All calls on a device share the one array, and it keeps whatever the previous call left
 * there.  Each call overwrites all of the scratch it later reads, so stale contents are
 * harmless, but two calls whose kernels may overlap on the GPU (different streams, or
 * several host threads) race on it: serialise them, e.g. by using one stream.
 * Errors: as onnx_conv2d_run, plus ONNXB_ERR_WORKSPACE as described above.
 */
onnxb_status onnx_conv2d_run_static(onnxb_conv2d_desc_t desc, const float *X, const float *W,
                                    const float *B, float *Y, void *cuda_stream);

/* Size in bytes of the built-in scratch array used by onnx_conv2d_run_static. */
size_t onnx_conv2d_static_scratch_bytes(void);

/*
 * onnx_gemm_workspace_bytes - device scratch onnx_gemm_run needs for this
 * problem (0 when none).  Host only.  The tensor-core path keeps TF32-rounded
 * copies of A and B there (4 * (M*K + K*N) bytes; its split-K form for small M
 * rounds in shared memory and leaves the workspace untouched, but the size is
 * asked for all the same); the SIMT path needs none.
 */
size_t onnx_gemm_workspace_bytes(int transA, int transB, int64_t M, int64_t N, int64_t K);

/*
 * onnx_gemm_run - ONNX Gemm (Sec. 3.4.3: Gemm(m1,m2,m3) = Add(MatMul(m1,m2),m3)):
 *
 *   Y[i,j] = relu?( alpha * sum_k A'[i,k] * B'[k,j] + beta * Cb[i,j] )
 *
 * A' = transA ? A^T : A is M x K (A stored [M,K], or [K,M] when transA != 0);
 * B' = transB ? B^T : B is K x N (B stored [K,N], or [N,K] when transB != 0);
 * Cb is C broadcast one-directionally to [M,N].  C == NULL omits the term;
 * otherwise c_rank in {0,1,2} and c_dims (host) hold its shape: (), (1), (N),
 * (1,N), (M,1), (1,1) or (M,N); a 1-D C is per column.  Y [M,N].
 * Errors: ERR_NULL; ERR_SHAPE (M,N,K < 1, C shape not broadcastable);
 * ERR_UNSUPPORTED (size, alignment); ERR_WORKSPACE; ERR_CUDA.
 */
onnxb_status onnx_gemm_run(int transA, int transB, float alpha, float beta,
                           int64_t M, int64_t N, int64_t K,
                           const float *A, const float *B,
                           const float *C, int c_rank, const int64_t *c_dims,
                           int fuse_relu, float *Y, void *workspace, size_t workspace_bytes,
                           void *cuda_stream);

/*
 * onnx_matmul_add_run - the pair MatMul(A, B) followed by Add(., C) that the compiler's
 * graph rewriting fuses into one Gemm (Sec. 3.4.3, the MulAddToGemm pattern):
 *
 *   Y[i,j] = relu?( sum_k A[i,k] * B[k,j] + Cb[i,j] )
 *
 * A [M,K], B [K,N], C broadcast as in onnx_gemm_run (C == NULL: plain MatMul), Y [M,N];
 * exactly onnx_gemm_run with transA = transB = 0 and alpha = beta = 1, same pointers,
 * workspace and errors.
 */
onnxb_status onnx_matmul_add_run(int64_t M, int64_t N, int64_t K, const float *A, const float *B,
                                 const float *C, int c_rank, const int64_t *c_dims, int fuse_relu,
                                 float *Y, void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * onnx_maxpool2d_shape / onnx_maxpool2d_run - ONNX MaxPool, 2-D, NCHW, dilation 1, ceil_mode 0
 * (pooling is among the operators the paper lowers, Sec. 4.1; both of its models use it, Sec. 4.2):
 *
 *   Y[n,c,p,q] = max over r < kH, s < kW of X[n,c, p*sh + r - pt, q*sw + s - pl]
 *
 * where positions outside the image do not take part (the padding value is minus infinity),
 * P = floor((H + pt + pb - kH) / sh) + 1 and Q likewise.  x_dims = {N,C,H,W}; kernel_shape = {kH,kW};
 * pads = {h_begin, w_begin, h_end, w_end} or NULL for none; strides = {sh, sw}, NULL or 0 = 1.
 * All four arrays are host memory.  X [N,C,H,W] and Y [N,C,P,Q] are caller-owned device memory, dense;
 * the kernel is enqueued on cuda_stream, nothing is allocated or synchronised.  The result is exact.
 * Errors: ERR_NULL; ERR_SHAPE (non-positive sizes, negative pads, a pad as large as the kernel,
 * kernel larger than the padded input); ERR_UNSUPPORTED (more than 2^31-1 elements); ERR_CUDA.
 * onnx_maxpool2d_shape only computes y_dims (host).
 */
onnxb_status onnx_maxpool2d_shape(const int64_t x_dims[4], const int64_t kernel_shape[2], const int64_t pads[4],
                                  const int64_t strides[2], int64_t y_dims[4]);
onnxb_status onnx_maxpool2d_run(const int64_t x_dims[4], const int64_t kernel_shape[2], const int64_t pads[4],
                                const int64_t strides[2], const float *X, float *Y, void *cuda_stream);

/*
 * onnx_global_average_pool_run - ONNX GlobalAveragePool (ResNet50's last pooling, Sec. 4.2):
 * Y[n,c,0,0] = mean over h, w of X[n,c,h,w].  x_dims = {N,C,H,W} (host); X device [N,C,H,W],
 * Y device [N,C,1,1]; fp32 accumulation (32 partial sums per plane, then a tree).  Enqueued on
 * cuda_stream; allocates and synchronises nothing.  Errors: ERR_NULL, ERR_SHAPE, ERR_UNSUPPORTED, ERR_CUDA.
 */
onnxb_status onnx_global_average_pool_run(const int64_t x_dims[4], const float *X, float *Y, void *cuda_stream);

/* Human-readable name of a status code (static storage, never NULL). */
const char *onnxb_status_string(onnxb_status status);

/*
 * onnxb_last_device_status - every device-side wait in the tensor-core kernels
 * is bounded; a wait that runs out sets an error word in device memory and the
 * kernel drains and returns.  This call synchronises `cuda_stream`, reads and
 * clears that word and returns ONNXB_ERR_DEVICE_TIMEOUT if it was set,
 * ONNXB_ERR_CUDA if the stream reports an error, else ONNXB_OK.
 */
onnxb_status onnxb_last_device_status(void *cuda_stream);

/*
 * onnxb_set_kernel_override - force a kernel family for descriptors created
 * afterwards (A/B measurements and tests): -1 = automatic choice (default),
 * otherwise an onnxb_kernel_family value.  A forced family that cannot compute a
 * given problem makes onnx_conv2d_desc return ERR_UNSUPPORTED.  Also settable
 * through the environment variable ONNXB_FORCE = simt | mma | auto, read once.
 */
void onnxb_set_kernel_override(int family);

/* Number of kernels this library has launched since it was loaded (all streams). */
uint64_t onnxb_launch_count(void);

/*
 * Measurement aid (no operator of the paper behind it; Sec. 4.2 reports whole-model times only):
 * the issue-rate ceiling of the TF32 tensor-core instruction the Conv and Gemm kernels are built
 * from.  Every SM issues `instructions` tcgen05.mma kind::tf32 instructions of shape 128 x n x 8
 * back to back on operands already in shared memory; *cycles_per_instruction receives the SM
 * cycles per instruction of the slowest SM (ideal: n / 2).  n: multiple of 16 in [16, 256];
 * instructions in [16, 2^20].  Unlike the run calls this one allocates a small device buffer,
 * launches on `cuda_stream` and synchronises it before returning.  Host pointer out; ERR_ATTR for
 * arguments out of range, ERR_CUDA if the device refuses.
 */
onnxb_status onnxb_probe_tf32_mma_rate(int n, int instructions, double *cycles_per_instruction,
                                       void *cuda_stream);

/*
 * Test aid for the failure-detection path (no operator of the paper behind it): launches one CTA
 * that waits, with the bounded wait the tensor-core kernels use, on a barrier nothing will ever
 * signal.  After limit_cycles SM cycles (1 .. 1e8, i.e. at most ~50 ms) the wait gives up, sets the
 * device error word and the kernel returns normally; the next onnxb_last_device_status on that
 * stream therefore reports ONNXB_ERR_DEVICE_TIMEOUT once, and ONNXB_OK afterwards.  Nothing faults,
 * traps or hangs, and the context stays usable.  Enqueues on cuda_stream without synchronising.
 * Errors: ERR_ATTR (limit out of range), ERR_CUDA.
 */
onnxb_status onnxb_probe_wait_timeout(long long limit_cycles, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* ONNX_B200_H_ */
