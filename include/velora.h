/*
 * velora.h -- C-ABI of the B200 (sm_100a) VeLoRA linear-layer library.
 *
 * VeLoRA (arxiv 2405.17991) replaces the input X[N, D] that a linear layer
 * saves for its backward pass by one scalar per sub-token: every token is cut
 * into M = ceil(D / Dsub) contiguous sub-tokens of length Dsub and each is
 * projected onto one fixed unit vector v[Dsub] (Section 3.1).  The backward
 * pass rebuilds a coarse input Xhat = Z (x) v for the weight gradient
 * (Algorithm 1).
 *
 * Naming.  The paper calls the sub-token LENGTH "M"; this header calls it
 * Dsub and uses M for the NUMBER of sub-tokens per token.
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers owned by the caller; the library
 *     never allocates or frees device memory.  Scratch is a caller-provided
 *     device workspace sized by velora_workspace_bytes().  State kept between
 *     calls: a per-process cache of immutable launch attributes (safe to fill
 *     from several host threads), and ONE sticky error word per device that
 *     the entry points without a workspace raise when a bounded wait expires
 *     (see velora_device_error: shared by all streams and callers of the device).
 *   - Matrices are row-major with an explicit leading dimension counted in
 *     ELEMENTS.  W is [O, D] (nn.Linear convention): Y = X W^T, dX = dY W,
 *     dW = dY^T Xhat.  The listing in Algorithm 1 is only consistent with
 *     this layout.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Work is enqueued asynchronously; only velora_init_v, velora_normalize_v and the
 *     two status readers synchronise.  The asynchronous entry points use nothing but
 *     kernel launches (and, for the host-buffer step, asynchronous copies) on `stream`,
 *     so after one ordinary call per shape (which sets the kernels' shared-memory
 *     limits on that device) a sequence of them can be captured into a CUDA graph:
 *     the forward + backward of a layer replayed from a graph gives the same bits.
 *   - Return value: a velora_status.  Arguments are validated on the host
 *     before anything is launched; on a non-zero status no output is written
 *     (VELORA_ERR_CUDA and VELORA_ERR_TIMEOUT excepted, which report a failure
 *     of an already enqueued launch).  Nothing throws, aborts or prints.
 *   - When Dsub does not divide D the last sub-token is the remaining
 *     D - (M-1)*Dsub entries followed by zeros (the paper's group() is a
 *     reshape and is silent on this case); outputs of width D are written on
 *     their first D columns only.
 *   - N == 0 (data pointers may then be NULL): velora_compress, velora_reconstruct, velora_linear_forward
 *     and the dX half of velora_linear_backward write nothing and succeed; velora_init_v returns
 *     VELORA_ERR_DEGENERATE_V (an empty batch has no mean); the weight gradient of an empty batch is the
 *     empty sum, dW = beta * dW: beta = 0 fills dW with zeros, beta = 1 leaves it.
 *   - Vector (128-bit) kernels are used when base pointers are 16-byte aligned,
 *     leading dimensions are multiples of 16 bytes and Dsub is a multiple of 8
 *     (fastest for 8 * 2^k) or one of 1, 2, 4; otherwise the element-wise kernels
 *     run (same results, lower speed).  The
 *     tensor-core GEMMs need 16-byte aligned bf16 rows; other cases run on the
 *     CUDA-core GEMM.
 */
#ifndef VELORA_H
#define VELORA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    VELORA_OK = 0,
    VELORA_ERR_INVALID_ARG = 1,   /* null pointer, negative size, ld < width, Dsub out of range */
    VELORA_ERR_UNSUPPORTED = 2,   /* dtype combination or size outside what the kernels cover  */
    VELORA_ERR_ALIGNMENT = 3,     /* pointer not aligned to its element size                   */
    VELORA_ERR_WORKSPACE = 4,     /* workspace missing or smaller than velora_workspace_bytes  */
    VELORA_ERR_DEGENERATE_V = 5,  /* the sub-token sum has zero or non-finite length           */
    VELORA_ERR_TIMEOUT = 6,       /* a bounded device-side wait expired (reported by status)   */
    VELORA_ERR_CUDA = 7           /* a CUDA runtime call or launch failed                      */
} velora_status;

/* VELORA_FP8_E4M3 is a storage type for Z only (see "8-bit storage of Z" below). */
typedef enum { VELORA_F32 = 0, VELORA_BF16 = 1, VELORA_FP8_E4M3 = 2 } velora_dtype;

/* How velora_weight_grad forms dW. */
typedef enum {
    VELORA_WG_FACTORED = 0,  /* P = dY^T Z on tensor cores, dW = P (x) v in the epilogue; Xhat never exists */
    VELORA_WG_EXPLICIT = 1   /* Xhat = reconstruct(Z, v) into the workspace, then the dense GEMM dY^T Xhat    */
} velora_wg_mode;

typedef enum {
    VELORA_OP_INIT_V = 0,
    VELORA_OP_WEIGHT_GRAD_FACTORED = 1,
    VELORA_OP_WEIGHT_GRAD_EXPLICIT = 2,
    VELORA_OP_LINEAR_FORWARD = 3,
    VELORA_OP_LINEAR_BACKWARD_FACTORED = 4,
    VELORA_OP_LINEAR_BACKWARD_EXPLICIT = 5,
    VELORA_OP_UPDATE_V = 6,
    VELORA_OP_Z8_CALIBRATE = 7
} velora_op;

#define VELORA_MAX_DSUB 1024

/* Library version, major*10000 + minor*100 + patch. */
int velora_version(void);

/* Number of kernels this library has launched in the calling process so far (all devices). */
unsigned long long velora_launch_count(void);

/* Static, human-readable name of a status code. */
const char* velora_status_string(int status);

/*
 * Bytes of device workspace the given entry point needs for these sizes
 * (0 if it needs none).  Independent of pointer values; deterministic.
 */
size_t velora_workspace_bytes(int op, int64_t N, int64_t D, int64_t O, int Dsub);

/*
 * Workspace header.  The first 256 bytes of every workspace are a status area; word 0 is a sticky
 * device error flag that a kernel raises when one of its bounded waits (on a shared-memory barrier
 * fed by a tile copy or by the tensor cores) gives up after one second instead of spinning for ever.
 * velora_workspace_init zeroes the header (asynchronously, on `stream`): call it once after
 * allocating a workspace.  velora_workspace_status synchronises `stream`, reads the flag and returns
 * VELORA_OK or VELORA_ERR_TIMEOUT; outputs of a call that raised the flag are undefined.  (The one other
 * value is VELORA_ERR_DEGENERATE_V, which velora_update_v leaves there instead of synchronising.)
 * The paper has no counterpart: this is run-time hygiene of the implementation.
 */
int velora_workspace_init(void* ws, size_t ws_bytes, void* stream);
int velora_workspace_status(const void* ws, void* stream);

/*
 * The entry points that take no workspace (velora_compress, and velora_init_v's first pass) record an
 * expired bounded wait in a word inside the library instead.  velora_device_error synchronises
 * `stream`, returns VELORA_OK or VELORA_ERR_TIMEOUT for the current device and clears the word.
 * There is one such word per device, whichever stream raised it: the call sees (and clears) what kernels
 * already completed on ANY stream have recorded, but synchronises only `stream`, so a caller that runs
 * several streams should drain them before it asks, and only one party per device should do the asking.
 */
int velora_device_error(void* stream);

/*
 * Self-test of the bounded waits (the paper has no counterpart; a test hook of the implementation).
 * Launches ONE small CTA that holds no tile copy and no tensor memory.  Its first warp waits, through the
 * very routine all pipelines of this library wait with, on a shared-memory barrier that nothing ever
 * signals, and gives up after limit_ns; its second warp waits on another such barrier with the ordinary
 * one-second limit and is released early by the abort flag the first warp raises on giving up.  The kernel
 * then returns normally, having set the workspace's status word and the per-device error word, so
 * velora_workspace_status(ws) and velora_device_error() both report VELORA_ERR_TIMEOUT (until
 * velora_workspace_init / the read that clears the word).  Asynchronous.
 *   limit_ns: 1000 .. 100000000 (1 us .. 100 ms), else VELORA_ERR_INVALID_ARG.
 *   observed: DEVICE int[4], written by the kernel: [0] first wait gave up (1), [1] microseconds it waited,
 *             [2] second wait gave up (1), [3] microseconds it waited.
 *   ws: any initialised workspace (>= 256 bytes).
 */
int velora_selftest_wait_timeout(void* ws, size_t ws_bytes, unsigned long long limit_ns, int* observed, void* stream);

/*
 * Initialise the projection vector from a batch (Section 3.2, "Cheap
 * initialisation strategies": the average of the first batch's sub-tokens;
 * Section 3.1: v has unit length):
 *     s[j] = sum_n sum_m X[n, m*Dsub + j],   v = s / ||s||_2      (fp32, v[Dsub])
 * X: [N, D], x_dtype bf16 or f32, leading dimension ldx.  The sum over tokens
 * uses a fixed order, so results are run-to-run identical.
 * ws: device workspace of velora_workspace_bytes(VELORA_OP_INIT_V, ...) bytes.
 * Synchronises `stream` once to read back whether the sum is degenerate;
 * returns VELORA_ERR_DEGENERATE_V and leaves v untouched if ||s|| is zero or
 * not finite.
 */
int velora_init_v(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub,
                  float* v, void* ws, size_t ws_bytes, void* stream);

/*
 * velora_init_v for callers that have no device memory to lend.  The paper has no counterpart: it is
 * the same operation and the same kernels as velora_init_v, but the partial sums go to a fixed array
 * inside the library instead of a caller-provided workspace.  It exists for code that runs where
 * allocating is not an option: a plugin handed only its input and output buffers by a host framework
 * that owns the allocator, a real-time loop that must not touch the driver's allocator once started,
 * or start-up code that runs before the application's memory pool exists.  The call itself allocates
 * and frees nothing, on the host or on the device.
 *   - Limit: Dsub <= VELORA_INIT_V_STATIC_MAX_DSUB, else VELORA_ERR_UNSUPPORTED (use velora_init_v).
 *   - Cost: the array (about 1.2 MB) is part of the library image, so every GPU on which the library
 *     is used keeps it until the process ends.
 *   - The first call on each device looks up the array's device address (once, cached); make that
 *     first call outside any stream capture.
 *   - All calls on a device share the one array.  Each call overwrites what it reads, so calls need
 *     no clearing between them, but two calls whose work overlaps on the GPU (different streams or
 *     threads) race on it: serialise them.  Like velora_init_v it synchronises `stream` once.
 * Arguments, results and errors otherwise as velora_init_v.
 */
#define VELORA_INIT_V_STATIC_MAX_DSUB 256
int velora_init_v_static(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub,
                         float* v, void* stream);

/*
 * compress (Section 3.1, Eq. 1):  Z[n, m] = sum_j X[n, m*Dsub + j] * v[j].
 * X: [N, D] bf16 or f32.  v: fp32 [Dsub].  Z: [N, M] f32, bf16 or E4M3, ldz >= M.
 * Products and sums are formed in fp32.
 */
int velora_compress(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub,
                    const float* v, void* Z, int z_dtype, int64_t ldz, void* stream);

/*
 * reconstruct + ungroup (Section 3.1, Eq. 2):  Xhat[n, m*Dsub + j] = Z[n, m] * v[j].
 * Z: [N, M] f32, bf16 or E4M3.  Xhat: [N, D] bf16 or f32 (rounded to nearest even).
 */
int velora_reconstruct(const void* Z, int z_dtype, int64_t ldz, int64_t N, int64_t D, int Dsub,
                       const float* v, void* Xhat, int x_dtype, int64_t ldxhat, void* stream);

/*
 * Weight gradient of Algorithm 1's backward with the reconstructed input:
 *     dW[o, d] = beta * dW[o, d] + sum_n dY[n, o] * Xhat[n, d],  Xhat = Z (x) v
 * dY: [N, O] bf16 or f32.  Z: [N, M] f32, bf16 or E4M3.  dW: [O, D] bf16 or f32.
 * beta is 0 (overwrite) or 1 (accumulate into dW).
 * mode VELORA_WG_FACTORED uses dW[o, m*Dsub+j] = (dY^T Z)[o, m] * v[j]
 * (the Dsub = D case is the paper's g v v^T, Section 3.2); VELORA_WG_EXPLICIT
 * materialises Xhat in the workspace and multiplies -- kept as a cross-check.
 * ws: velora_workspace_bytes(VELORA_OP_WEIGHT_GRAD_{FACTORED,EXPLICIT}, N, D, O, Dsub).
 */
int velora_weight_grad(const void* dY, int dy_dtype, int64_t N, int64_t O, int64_t lddy,
                       const void* Z, int z_dtype, int64_t ldz, const float* v, int64_t D, int Dsub,
                       void* dW, int dw_dtype, int64_t lddw, int beta, int mode,
                       void* ws, size_t ws_bytes, void* stream);

/*
 * Forward of the VeLoRA linear (Algorithm 1, forward):
 *     Y[N, O] = X W^T      and      Z = compress(X, v)
 * `dtype` is the storage type of X, W and Y (bf16: tensor cores with fp32
 * accumulation; f32: CUDA cores).  Z as in velora_compress.  X itself need not
 * be kept by the caller afterwards: (Z, W, v) is all the backward needs.
 * With bf16 data, 16-byte aligned rows and Dsub a power of two in 8 .. 1024, X is read
 * from HBM once for both results: inside the tensor-core product for wide layers
 * (O > 768), in a single streaming pass for adapter-shaped ones (O <= 64, Section 4:
 * down projections of adapters); other shapes run the product and then velora_compress.
 * ws: velora_workspace_bytes(VELORA_OP_LINEAR_FORWARD, ...) bytes.
 */
int velora_linear_forward(const void* X, int64_t ldx, const void* W, int64_t ldw, const float* v,
                          void* Y, int64_t ldy, void* Z, int z_dtype, int64_t ldz,
                          int dtype, int64_t N, int64_t D, int64_t O, int Dsub,
                          void* ws, size_t ws_bytes, void* stream);

/*
 * Backward of the VeLoRA linear (Algorithm 1, backward):
 *     dX[N, D] = dY W                  (exact; skipped when dX == NULL)
 *     dW[O, D] as velora_weight_grad   (skipped when dW == NULL)
 * `dtype` is the storage type of dY, W and dX.
 * ws: velora_workspace_bytes(VELORA_OP_LINEAR_BACKWARD_{FACTORED,EXPLICIT}, ...) bytes, always required.
 */
int velora_linear_backward(const void* dY, int64_t lddy, const void* W, int64_t ldw,
                           const void* Z, int z_dtype, int64_t ldz, const float* v,
                           void* dX, int64_t lddx, void* dW, int dw_dtype, int64_t lddw, int beta, int mode,
                           int dtype, int64_t N, int64_t D, int64_t O, int Dsub,
                           void* ws, size_t ws_bytes, void* stream);

/*
 * 8-bit storage of Z (an extension of Section 3.1: what the forward pass keeps for the backward pass is the
 * array of scalars Z, and the paper's memory tables (Table 5(b), Table 6) count exactly those bytes; it
 * stores them in the training precision, this stores them in one byte each).
 *
 * Every entry point that writes or reads Z accepts z_dtype = VELORA_FP8_E4M3: Z is then [N, M] bytes (ldz in
 * bytes) in the E4M3 format (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities, largest
 * value 448).  A writer stores round_to_nearest_even(<sub-token, v>), saturating at +-448; a reader uses the
 * decoded value as Z.  The scale that brings Z into E4M3's range travels in the VECTOR argument, since
 * compress is linear in v and the backward pass is linear in v as well:
 *     writers (velora_compress, velora_linear_forward):                      pass v_store = v / zscale
 *     readers (velora_reconstruct, velora_weight_grad, velora_linear_backward,
 *              velora_expand_p after velora_weight_grad_p):                   pass v_load  = v * zscale
 * so that Xhat = decode(Z8) (x) v_load approximates Z (x) v and no kernel needs a scale argument.  The
 * weight gradient feeds the decoded values to the tensor cores as they are (every E4M3 value is a bf16
 * value), so an 8-bit Z adds no rounding beyond the store's own: relative error at most 2^-4 per scalar
 * for |Z| >= zscale * 2^-6, absolute error at most zscale * 2^-10 below that.
 *
 * velora_z8_calibrate chooses the scale from a batch (like v itself it is meant to be fixed on the first
 * batch and kept):  zscale = headroom * max_{n,m} |<x_nm, v>| / 448   (1 if that maximum is zero or not
 * finite), v_store = v / zscale, v_load = v * zscale.  headroom in [1, 1024] leaves room for later batches
 * (2 puts the calibration batch's largest scalar at 224); scalars beyond the range saturate.
 * zscale[1], v_store[Dsub], v_load[Dsub]: device fp32.  Asynchronous.
 * ws: velora_workspace_bytes(VELORA_OP_Z8_CALIBRATE, N, D, 0, Dsub) bytes (holds Z of the batch in fp32).
 */
int velora_z8_calibrate(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub, const float* v,
                        float headroom, float* zscale, float* v_store, float* v_load,
                        void* ws, size_t ws_bytes, void* stream);

/*
 * The dense products of Algorithm 1 on their own, i.e. the layer WITHOUT the method: Y = X W^T (forward),
 * dX = dY W and dW = dY^T X (backward, with the input X kept instead of Z).  They are the same tensor-core
 * kernels the VeLoRA entry points use, exported so that the cost of an uncompressed layer can be measured
 * beside the compressed one (Section 5, the speed comparison with full fine-tuning).
 *     C[Mdim, Ndim] = beta * C + op(A) op(B),  fp32 accumulation, beta in {0, 1}
 *   VELORA_PRODUCT_A_BT:  A[Mdim, Kdim], B[Ndim, Kdim]    (C = A B^T)
 *   VELORA_PRODUCT_A_B:   A[Mdim, Kdim], B[Kdim, Ndim]    (C = A B)
 *   VELORA_PRODUCT_AT_B:  A[Kdim, Mdim], B[Kdim, Ndim]    (C = A^T B)
 * `dtype`: storage type of A and B (bf16: tensor cores when rows are 16-byte aligned; otherwise and for
 * f32 the CUDA-core product).  C: c_dtype, bf16 or f32.  ws: at least 256 bytes, initialised (status header).
 */
typedef enum { VELORA_PRODUCT_A_BT = 0, VELORA_PRODUCT_A_B = 1, VELORA_PRODUCT_AT_B = 2 } velora_product;
int velora_dense_product(int kind, const void* A, int64_t lda, const void* B, int64_t ldb,
                         void* C, int c_dtype, int64_t ldc, int beta,
                         int64_t Mdim, int64_t Ndim, int64_t Kdim, int dtype,
                         void* ws, size_t ws_bytes, void* stream);

/*
 * The two halves of velora_init_v, for a batch that is sharded over several processes (Section 3.2:
 * the average runs over ALL sub-tokens of the first batch, so every rank must end up with the same v).
 *   velora_subtoken_sum:  s[j] = sum_n sum_m X[n, m*Dsub + j]   (fp32, s[Dsub]; asynchronous; N == 0 gives 0)
 *   velora_normalize_v:   v = s / ||s||_2; synchronises `stream`; VELORA_ERR_DEGENERATE_V as velora_init_v
 * Between the two the caller adds the s of all ranks (an all-reduce of Dsub floats).
 * ws: velora_workspace_bytes(VELORA_OP_INIT_V, ...) bytes for the sum, at least 256 bytes for the normalisation.
 */
int velora_subtoken_sum(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub,
                        float* s, void* ws, size_t ws_bytes, void* stream);
int velora_normalize_v(const float* s, int Dsub, float* v, void* ws, size_t ws_bytes, void* stream);

/*
 * Running-average variant of the initialisation (Section 5, ablation on the initialisation strategy,
 * row "Running average").  The paper names the variant without a formula; the reading implemented is an
 * exponential average of the per-batch sub-token means, re-normalised:
 *   a[j] <- (1 - rho) * a[j] + rho * s[j] / (N * M),  s as in velora_subtoken_sum;   v <- a / ||a||_2
 * rho in [0, 1].  rho = 1 makes v follow each incoming batch (a is not read, so it needs no initial value);
 * rho = 1/t at the t-th call of equal-size batches keeps a at the mean of everything seen, i.e. v at the
 * fixed average of velora_init_v over the concatenated batches.
 * a[Dsub], v[Dsub]: device fp32, the caller's running state and the vector to use from now on.
 * Asynchronous (no synchronisation).  If ||a|| comes out zero or not finite, a and v are left as they
 * were and the workspace's status word is set: velora_workspace_status then returns
 * VELORA_ERR_DEGENERATE_V until velora_workspace_init.  N == 0 changes nothing.
 * ws: velora_workspace_bytes(VELORA_OP_UPDATE_V, ...) bytes, initialised once with velora_workspace_init.
 */
int velora_update_v(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub, float rho,
                    float* a, float* v, void* ws, size_t ws_bytes, void* stream);

/*
 * The factored weight gradient kept in factored form (the rank-1 structure of Section 3.2, per sub-token):
 *   velora_weight_grad_p:  P[O, M] = beta * P + dY^T Z      (fp32, ldp >= M)
 *   velora_expand_p:       dW[o, m*Dsub + j] = beta * dW + P[o, m] * v[j]
 * Since v is frozen, P can be accumulated over micro-batches (beta = 1) and summed over data-parallel
 * ranks (an all-reduce of O*M floats instead of O*D gradients) before it is expanded ONCE; the two calls in
 * sequence give the same dW as velora_weight_grad in VELORA_WG_FACTORED mode.
 * Because the expansion is linear in v, a plain gradient step needs no dW at all: velora_expand_p with
 * beta = 1, the weight matrix as `dW` and a copy of v scaled by -lr gives W <- W - lr * (P (x) v).
 * ws of velora_weight_grad_p: velora_workspace_bytes(VELORA_OP_WEIGHT_GRAD_FACTORED, N, D, O, Dsub).
 */
int velora_weight_grad_p(const void* dY, int dy_dtype, int64_t N, int64_t O, int64_t lddy,
                         const void* Z, int z_dtype, int64_t ldz, int64_t D, int Dsub,
                         float* P, int64_t ldp, int beta, void* ws, size_t ws_bytes, void* stream);
int velora_expand_p(const float* P, int64_t ldp, const float* v, int64_t O, int64_t D, int Dsub,
                    void* dW, int dw_dtype, int64_t lddw, int beta, void* stream);

/*
 * One forward + backward of a VeLoRA linear (Algorithm 1, both functions) on data
 * that lives in HOST memory (bf16, dense rows: ld = width).  On `stream`, in order:
 * copies X[N, D] and dY[N, O] from the host into the device staging area, runs
 * velora_linear_forward and velora_linear_backward (factored weight gradient,
 * beta = 0, fp32 Z), and copies Y[N, O], dX[N, D] and dW[O, D] back to the host
 * (each host output may be NULL to skip its copy).  Nothing is synchronised: the
 * host buffers must stay valid until the stream has drained, and should be
 * page-locked for the copies to be asynchronous.
 * hX, hdY, hY, hdX, hdW: HOST pointers.  W[O, D] (ld = D) and v[Dsub]: DEVICE.
 * staging: DEVICE memory of velora_host_step_staging_bytes(N, D, O, Dsub) bytes,
 * 256-byte aligned.  ws: velora_workspace_bytes(VELORA_OP_LINEAR_BACKWARD_FACTORED, ...).
 */
size_t velora_host_step_staging_bytes(int64_t N, int64_t D, int64_t O, int Dsub);
int velora_linear_step_host(const void* hX, const void* hdY, void* hY, void* hdX, void* hdW,
                            const void* W, const float* v, void* staging, size_t staging_bytes,
                            int64_t N, int64_t D, int64_t O, int Dsub,
                            void* ws, size_t ws_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* VELORA_H */
