/*
 * libab: the per-GPU hot path of AB-Training on NVIDIA B200 (sm_100a).
 *
 * Notation (the paper's Eq. 3, with its k written r): a layer weight W (m x n,
 * out-features x in-features) is held as W = A B with A (m x r) and B (r x n).
 * Activations x are N x n, outputs y and upstream gradients dY are N x m,
 * T = x B^T and dT = dY A are N x r.  Every matrix is row-major.
 *
 * Conventions for every call
 *  - Pointers are DEVICE pointers owned by the caller unless a parameter says "host".
 *    The library allocates no device memory; scratch space is passed in as `ws` (size from
 *    ab_workspace_bytes, 256-byte aligned).  No result depends on an earlier call.  What the
 *    library does keep per process: a count of its kernel launches (ab_launch_count), cached
 *    device properties, the address of the built-in array of ab_layer_forward_static, and one
 *    low-priority helper stream per device that ab_group_sync creates on first use (see there).
 *  - Calls are asynchronous on `cuda_stream` (a cudaStream_t passed as void*; NULL = the
 *    default stream).  Buffers must stay valid until the stream has run the call.
 *  - Arguments that can be checked on the host (NULL, non-positive sizes, r > min(m,n),
 *    a short workspace, a misaligned pointer) are rejected with a negative status and
 *    nothing is launched.  Conditions only the device can see (an iteration that did not
 *    converge, a bounded wait that ran out) are written to a device status word and never
 *    trap; the context stays usable.
 *  - There is no CPU fallback: without a CUDA device every compute call returns AB_ERR_CUDA.
 *  - bf16 storage always means fp32 accumulation.  dA, dB, sigma are always fp32.
 */
#ifndef AB_H_
#define AB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  AB_OK = 0,
  AB_ERR_INVALID_ARG = -1,   /* NULL pointer, non-positive size, r > min(m,n), bad leading dimension */
  AB_ERR_UNSUPPORTED = -2,   /* a size beyond what the kernels handle (stated per call) */
  AB_ERR_WORKSPACE = -3,     /* ws NULL, misaligned or smaller than ab_workspace_bytes says */
  AB_ERR_NOT_CONVERGED = -4, /* device status: Jacobi sweep cap reached */
  AB_ERR_TIMEOUT = -5,       /* device status: a bounded on-chip wait expired */
  AB_ERR_CUDA = -6,          /* a CUDA runtime call failed (no device, launch error) */
  AB_ERR_ACCURACY = -7       /* device status: the split kept singular values below the accuracy domain of
                                the route that computed them (stated at ab_svd_split / ab_group_sync); the
                                outputs are written, those values are not accurate to 1e-4 */
} ab_status;

typedef enum { AB_F32 = 0, AB_BF16 = 1 } ab_dtype;

typedef enum {
  AB_OP_LAYER_FORWARD = 0,
  AB_OP_LAYER_BACKWARD = 1,
  AB_OP_GROUP_AVERAGE = 2,
  AB_OP_RECOMBINE = 3,
  AB_OP_SVD_SPLIT = 4,
  AB_OP_DENSE_FORWARD = 5,
  AB_OP_DENSE_BACKWARD = 6
} ab_op;

/* Human-readable name of a status code (static storage, never NULL). */
const char* ab_status_string(int status);

/* Library version, "major.minor". */
const char* ab_version(void);

/* Number of kernels this library has launched in this process since it was loaded. */
long long ab_launch_count(void);

/*
 * Self-test of the failure path (no counterpart in the paper).  Every on-chip wait of the fused kernels
 * is bounded: when it runs out the kernel writes AB_ERR_TIMEOUT to its status word and exits normally.
 * This call launches one small kernel whose only thread waits, with the same wait routine, on a barrier
 * that nothing ever signals, for limit_us microseconds (1 .. 1,000,000); dev_status (device int) then
 * holds AB_ERR_TIMEOUT.  Nothing hangs, traps or faults; the context stays usable.
 */
int ab_selftest_bounded_wait(int* dev_status, unsigned limit_us, void* cuda_stream);

/*
 * The same for the whole failure path of the fused chain kernel (no counterpart in the paper): the kernel
 * is launched on scratch operands inside ws with its loader switched off, so the waits of its other roles
 * run out after limit_us microseconds; each role gives up, the kernel unwinds through its common exit,
 * releases its tensor memory and leaves AB_ERR_TIMEOUT in the first int of ws.  ws: device memory of
 * ab_selftest_chain_stall_workspace_bytes() bytes, 256-byte aligned.  Nothing hangs, traps or faults.
 */
int ab_selftest_chain_stall(void* ws, size_t ws_bytes, unsigned limit_us, void* cuda_stream);
size_t ab_selftest_chain_stall_workspace_bytes(void);

/*
 * Scratch bytes a call needs (0 if none).  Arguments a given op does not use are ignored
 * (pass 0).  For AB_OP_SVD_SPLIT, r is r_max.  Returns 0 for unknown ops or bad sizes.
 */
size_t ab_workspace_bytes(int op, int64_t N, int m, int n, int r, int K, int dt);

/*
 * Forward of the factorised layer (Eq. 3 used as a linear map): y = (x B^T) A^T.
 *   x [N,n], A [m,r] (row stride ldA >= r), B [r,n] (row stride ldB >= n), y [N,m], all of
 *   storage type dt.  T_save: NULL, or [N,r] of type dt that receives T = x B^T for the
 *   backward call.  The rank-r intermediate stays on chip when dt = AB_BF16, r is a
 *   multiple of 8 with 8 <= r <= 256 and m, n are multiples of 8; other shapes take a
 *   slower general kernel (same results to rounding).  N = 0 is a no-op.
 *   Device status: the first int of ws receives AB_OK, or AB_ERR_TIMEOUT if a bounded
 *   on-chip wait of the fused kernel expired (outputs are then undefined).  The same holds
 *   for ab_layer_backward.
 */
int ab_layer_forward(const void* x, const void* A, const void* B, void* y, void* T_save,
                     int64_t N, int m, int n, int r, int ldA, int ldB, int dt,
                     void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * ab_layer_forward for callers that cannot allocate.  (The paper has no counterpart; this is
 * a packaging variant of the call above.)  Some callers have no way to give the library a
 * workspace: they run where device allocation is forbidden or impossible -- inside a host
 * application that has reserved all device memory for its own pool, in a plug-in without
 * access to that pool, in a latency-critical loop that must not hit cudaMalloc's implicit
 * synchronisation.  For them the rank-r intermediate T = x B^T is kept in a fixed 4 MiB
 * array built into the library (each GPU that loads the library holds it until the process
 * ends), so the call needs only its inputs and its output and never calls cudaMalloc,
 * cudaFree or any allocating routine.
 *   Same arguments and results as ab_layer_forward without T_save and ws; always runs the
 *   general kernels.  Limit: N * r <= ab_static_scratch_elems() (1,048,576); larger calls
 *   return AB_ERR_UNSUPPORTED and launch nothing.
 *   The first call on each device looks up the array's device address (with that device
 *   current); make that first call outside of any stream capture.
 *   All calls on a device share the one array, which keeps whatever the previous call left
 *   in it (this call overwrites all it reads, so nothing has to be cleared).  Two calls
 *   that may run on the GPU at the same time -- different streams, or different host
 *   threads -- race on it: serialise them on one stream.
 */
int ab_layer_forward_static(const void* x, const void* A, const void* B, void* y,
                            int64_t N, int m, int n, int r, int ldA, int ldB, int dt,
                            void* cuda_stream);
size_t ab_static_scratch_elems(void);

/*
 * Backward of the factorised layer (chain rule through T):
 *   dT = dY A, dX = dT B, dA = dY^T T, dB = dT^T x.
 *   dX [N,n] of type dt; dA [m,r] and dB [r,n] are fp32 and dense (row strides r and n).
 *   Any of dX, dA, dB may be NULL (not wanted: groups that train only A or only B).
 *   T_saved: the T written by ab_layer_forward, or NULL to recompute it from x.
 *   Sums over N are taken in a fixed order: two runs give identical bits.
 *   No output may overlap an input or another output (the kernels of one call run partly side
 *   by side: dA is accumulated from dY and T while dX is still being written).
 */
int ab_layer_backward(const void* x, const void* dY, const void* A, const void* B,
                      const void* T_saved, void* dX, float* dA, float* dB,
                      int64_t N, int m, int n, int r, int ldA, int ldB, int dt,
                      void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Factorised 3 x 3 convolution (stride 1, zero padding 1) on NHWC activations, without materialised im2col
 * rows.  The paper flattens the trailing dimensions of a convolution weight into a matrix before Eq. 3
 * (Section "Methodology", after Eq. 3); here the flattened weight is W [m, 9 C] = A B with column
 * (ky * 3 + kx) * C + c for tap (ky, kx) and input channel c, and
 *   forward : y [B,H,W,m] = (rows(x) B^T) A^T, where rows(x) are the 9 C-wide im2col rows of x [B,H,W,C]; they
 *             are never formed: every tap's shifted view of x is loaded straight from the activation (what
 *             falls outside an image is zero), so x is read from device memory once instead of nine times.
 *             T_save: NULL, or [B H W, r] that receives T for the backward call.
 *   backward: dT = dY A;  dX [B,H,W,C] = the col2im sum of dT B over the nine taps (folded into the
 *             reduction: no 9 C-wide gradient rows are formed);  dA [m,r] = dY^T T;  dB [r,9C] = dT^T rows(x).
 *             Any of dX, dA, dB may be NULL; T_saved NULL recomputes T.  dA, dB fp32, fixed summation order.
 *   Supported: dt = AB_BF16, C, m, r multiples of 8, 8 <= r <= 256, W <= 64, H <= 256; anything else returns
 *   AB_ERR_UNSUPPORTED (materialise the rows and call ab_layer_forward / ab_layer_backward instead).
 *   Workspace: ab_conv3x3_workspace_bytes; its first int is the device status word as for ab_layer_forward.
 */
int ab_conv3x3_forward(const void* x, const void* A, const void* B, void* y, void* T_save,
                       int batch, int H, int W, int C, int m, int r, int ldA, int ldB, int dt,
                       void* ws, size_t ws_bytes, void* cuda_stream);
int ab_conv3x3_backward(const void* x, const void* dY, const void* A, const void* B, const void* T_saved,
                        void* dX, float* dA, float* dB, int batch, int H, int W, int C, int m, int r,
                        int ldA, int ldB, int dt, void* ws, size_t ws_bytes, void* cuda_stream);
size_t ab_conv3x3_workspace_bytes(int batch, int H, int W, int C, int m, int r);

/*
 * Dense layer of the full-rank phases of a training cycle (Algorithm 1: the warm-up steps before the
 * first decomposition and the full-rank rebound steps after W <- A B; Section "Methodology", full-rank
 * rebound): the same linear map with W held dense.
 *   forward : y [N,m] = x [N,n] W^T, W [m,n] dense (row stride n); all of storage type dt.
 *   backward: dX [N,n] = dY [N,m] W (type dt), dW [m,n] = dY^T x (fp32, sums over N in a fixed order).
 *   Either of dX, dW may be NULL.  bf16 storage with m, n multiples of 8 runs on the tensor cores
 *   (fp32 accumulation); other shapes and fp32 storage take the general kernel.  N = 0 is a no-op
 *   (dW is zeroed).  Workspace: ab_workspace_bytes(AB_OP_DENSE_FORWARD / AB_OP_DENSE_BACKWARD, N, m, n,
 *   0, 0, dt); its first int receives AB_OK or AB_ERR_TIMEOUT as for ab_layer_forward.
 */
int ab_dense_forward(const void* x, const void* W, void* y, int64_t N, int m, int n, int dt,
                     void* ws, size_t ws_bytes, void* cuda_stream);
int ab_dense_backward(const void* x, const void* dY, const void* W, void* dX, float* dW,
                      int64_t N, int m, int n, int dt, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * One AdamW update of a factor from the gradient ab_layer_backward left (the paper trains with
 * AdamW, Section "Experiments"; decoupled weight decay):
 *   p <- p (1 - lr wd);  m <- b1 m + (1-b1) g;  v <- b2 v + (1-b2) g^2;
 *   p <- p - lr (m / (1-b1^step)) / (sqrt(v / (1-b2^step)) + eps).
 * param, m, v: fp32 [count], updated in place; grad: fp32 [count]; param_bf16: NULL, or bf16
 * [count] that receives the updated values rounded to nearest even (the copy the tensor-core
 * chain reads).  step >= 1.  lr is the rate of this step: multiply ab_lr_rebound_factor in
 * while a rebound is running.  All pointers device memory; one launch on the stream.
 */
int ab_adamw_step(float* param, const float* grad, float* m, float* v, void* param_bf16, int64_t count,
                  float lr, float beta1, float beta2, float eps, float weight_decay, int step,
                  void* cuda_stream);

/*
 * Learning-rate rebound (Section "Methodology", "learning rate rebound"): whenever the parameters
 * change shape the rate drops to near zero and climbs back to its scheduled value over
 * rebound_steps steps.  The paper does not give the shape of the climb; this is the linear
 * one: floor + (1 - floor) * min(1, steps_since_change / rebound_steps).  Host function.
 */
float ab_lr_rebound_factor(int steps_since_change, int rebound_steps, float floor);

/*
 * Mean of K group copies (Algorithm 1: A <- allReduce(A / worldSize), likewise B), the K
 * workers being K arenas in one device's memory: copy k starts at base + k*stride_elems
 * (elements of in_dt).  In fp32 and in a fixed order:
 *   out[i] = fl( (((c0[i] + c1[i]) + c2[i]) + ...) * fl(1/K) ),   i < count.
 * For K a power of two this equals the paper's divide-then-sum bit for bit.
 * out has type out_dt (fp32 -> bf16 rounds to nearest even).  1 <= K <= 64.
 */
int ab_group_average(const void* base, int64_t stride_elems, int K, int64_t count,
                     int in_dt, int out_dt, void* out, void* cuda_stream);

/*
 * Recombination (Algorithm 1: W <- A B): W [m,n] fp32 (dense) = Abar [m,r] Bbar [r,n],
 * factors of type dt, product accurate to fp32 rounding.  With a workspace of
 * ab_workspace_bytes(AB_OP_RECOMBINE, 0, m, n, r, 0, dt) bytes and n a multiple of 4 it runs on the tensor
 * cores: bf16 factors multiply exactly in fp32; fp32 factors are cut into three bf16 pieces each (24 bits)
 * and multiplied as six bf16 products accumulated in fp32.  With ws = NULL (or too small) the same product
 * runs on the fp32 pipes.
 */
int ab_recombine(const void* Abar, const void* Bbar, float* W, int m, int n, int r,
                 int ldA, int ldB, int dt, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * The two all-reduces and the recombination of Algorithm 1 in ONE kernel: W = mean_k(A_k) mean_k(B_k), the mean
 * taken in the product's operand loader (fp32, copies added in ascending k, times fl(1/K): the bits of
 * ab_group_average); Abar [m,r] and Bbar [r,n], when not NULL, receive the averaged factors (written by the
 * CTAs of the first tile column / row).  fp32 factors only (AB_ERR_UNSUPPORTED otherwise); product on the fp32
 * pipes.  Every output tile re-reads the K copies of its operand panels, so for K > 1 this is slower than
 * ab_group_average + ab_recombine on all but small matrices (measured: the bench line's fused_mean_recombine);
 * it is here for callers who want one launch and no intermediate.
 */
int ab_recombine_mean(const void* A_copies, int64_t strideA, const void* B_copies, int64_t strideB, int K,
                      float* W, float* Abar, float* Bbar, int m, int n, int r, int dt, void* cuda_stream);

/*
 * Truncated SVD and split (Eq. 3 with the rank rule of the AB-decomposition phase):
 *   W = U S V^T;  r' = #{ i < r_cap : s_i >= sigma_cutoff * s_0 }, at least 1, where
 *   r_cap = min(r_max, m, n);  A = U_r' S_r'^(1/2),  B = S_r'^(1/2) V_r'^T.
 *   W [m,n] dense of type w_dt.  A [m,r_max] (row stride r_max) and B [r_max,n] of type
 *   out_dt; columns of A and rows of B with index >= r' are zero.  sigma [r_cap] fp32,
 *   descending up to rounding; r_out: device int that receives r'; dev_status: device
 *   int that receives AB_OK, AB_ERR_NOT_CONVERGED or AB_ERR_ACCURACY.  sigma_cutoff = 0 keeps r_cap.
 *   Accuracy domain: the decomposition works on the Gram matrix of the shorter side in fp32, so
 *   singular values below 2% of the largest lose relative accuracy (they keep absolute accuracy
 *   1e-6 * s_0).  If a value between 1e-5 and 2e-2 of the largest is among the kept ones,
 *   dev_status says AB_ERR_ACCURACY (outputs are still written); with sigma_cutoff >= 0.02 every
 *   kept value is inside the domain.  Values below 1e-5 * s_0 count as zero (a W of lower rank
 *   than r_max).  min(m,n) <= 3072.
 */
int ab_svd_split(const void* W, int m, int n, int r_max, float sigma_cutoff,
                 void* A, void* B, float* sigma, int* r_out, int* dev_status,
                 int w_dt, int out_dt, void* ws, size_t ws_bytes, void* cuda_stream);

/* One matrix of a batched group synchronisation.  All pointers are device pointers. */
typedef struct {
  const void* A_copies;   /* K copies of A [m,r], copy k at A_copies + k*strideA elements */
  const void* B_copies;   /* K copies of B [r,n] */
  int64_t strideA, strideB;
  int m, n, r;            /* r = rank of the incoming factors = r_max of the outgoing ones */
  void* A_out;            /* [m,r] */
  void* B_out;            /* [r,n] */
  float* sigma;           /* [min(r,m,n)] */
  int* r_out;             /* device int */
  float* W_out;           /* NULL, or [m,n] fp32 that receives the recombination W = Abar Bbar */
} ab_sync_desc;

typedef enum {
  AB_SYNC_AUTO = 0,      /* factored when it applies, else dense */
  AB_SYNC_DENSE = 1,     /* form W, then the dense split of ab_svd_split */
  AB_SYNC_FACTORED = 2   /* never form W: r x r Cholesky/SVD problems only (rank(W) <= r makes this exact) */
} ab_sync_path;

/*
 * Group synchronisation of a whole model (Algorithm 1 from the two all-reduces to the next
 * decomposition): for each of the L matrices, mean of the K copies of A and of B, W = Abar
 * Bbar, then the split of W as in ab_svd_split.  descs: HOST array of L descriptors (read
 * before the call returns).  Factor storage dt on both sides.  dev_status: device int[L].
 * path: an ab_sync_path.  The factored path uses that W = Abar Bbar has rank <= r: the
 * decomposition reduces to Cholesky factors of Abar^T Abar and Bbar Bbar^T and the SVD of an
 * r x r core, each solved inside shared memory (one CTA, or a cluster of CTAs, per matrix); W
 * itself is only written if W_out asks for it.  It needs r <= 236 (shared-memory capacity);
 * AB_SYNC_FACTORED returns AB_ERR_UNSUPPORTED when r is too large, AB_SYNC_AUTO falls back to the
 * dense path.  Accuracy domain of the factored path: singular values down to 1e-2 of the largest
 * come out to 1e-4 relative.  dev_status[i] says AB_ERR_ACCURACY (outputs still written) when a
 * kept value lies between 1e-6 and 1e-2 of the largest, or when a Cholesky pivot of a Gram matrix
 * fell under 1e-6 of its largest diagonal entry without being exactly zero (exactly zero pivots
 * are the columns of A / rows of B that an earlier rank rule removed: dropping them is exact).
 * A caller that gets this status can rerun that matrix with AB_SYNC_DENSE, whose domain is
 * stated at ab_svd_split; with sigma_cutoff >= 0.02 neither path keeps a value outside its domain.
 * Workspace: ab_sync_workspace_bytes (covers either path).  When a W_out is given, the factored
 * path runs that product on a helper stream of the library (one per device, lowest priority,
 * created on first use) beside its Jacobi kernel and joins it before the call's last kernel, so
 * the caller's stream order still covers everything the call writes.
 */
int ab_group_sync(const ab_sync_desc* descs, int L, int K, float sigma_cutoff, int dt,
                  int* dev_status, void* ws, size_t ws_bytes, void* cuda_stream, int path);
size_t ab_sync_workspace_bytes(const ab_sync_desc* descs, int L, int K, int dt);

#ifdef __cplusplus
}
#endif
#endif /* AB_H_ */
