/*
 * tarflow.h -- C ABI of the B200 selective-Jacobi TarFlow sampling library (libtarflow.so).
 *
 * The library implements, as hand-written CUDA kernels for sm_100a, the inference hot path of a
 * TarFlow-style block-autoregressive normalizing flow:
 *   - the autoregressive affine block and its inverse            (paper Eq. 4 and Eq. 5),
 *   - Jacobi decoding of a block's inverse                        (paper Algorithm 1, Eq. 8),
 *   - the selective policy: per block, sequential decoding with a
 *     key/value cache or Jacobi iteration                         (paper Sec. 3.5),
 *   - token-order reversal between blocks                         (remark after Eq. 4).
 * Notation: mu = g_k, alpha = -s_k, so a block's inverse is  u_l = v_l * exp(alpha_l) + mu_l  and
 * log|det d z / d x| = -sum(alpha).  Blocks are indexed in GENERATION order: block 0 is the first
 * inverse applied to the noise (the paper's "first (K-th) layer").
 *
 * Conventions for every call
 *   - Pointers named *_dev are device pointers on the current CUDA device, *_host are host
 *     pointers.  The caller owns every buffer it passes; the library neither frees nor keeps them
 *     after the call returns.  Images are fp32 [B, C, H, W], contiguous.
 *   - `cuda_stream` is a cudaStream_t cast to void* (NULL = the legacy default stream).  Work is
 *     enqueued on it; calls that fill host outputs synchronise that stream before returning.
 *   - Return value: 0 = TF_OK; TF_MAXITER (1) = a Jacobi block hit max_iters before every sample
 *     passed the stopping test (x holds the last iterate; not an error); negative = error, with a
 *     message available from tf_last_error().  Nothing aborts, throws or traps.
 *   - A tf_model is not thread-safe: it owns one workspace; use it from one thread/stream at a time.
 *   - Device-side waits (mbarrier waits inside the tensor-core kernels) are bounded by wall time (2 s).  A wait
 *     that runs out records a code in the model's error word; kernels that see the word set return without
 *     work.  The next synchronising call (tf_forward, tf_inverse_*) returns TF_ETIMEOUT ONCE and clears the
 *     word: the outputs of that call are undefined, the model is usable again for the next call.
 *   - Class labels are read from caller memory, so they are validated on the device before any kernel uses
 *     them: an id outside [0, n_classes) makes the call return TF_EINVAL (no table is ever indexed with it).
 *   - Tuning aids read from the environment (bf16 engine, sequential decoding only; results are unchanged
 *     up to summation order): TARFLOW_SEQ_MMA=1 selects the mma.sync step GEMM instead of the tcgen05 one,
 *     TARFLOW_SEQ_KBN=1|2|4 the 64-wide k slabs per CTA of the tcgen05 step GEMM, TARFLOW_SEQ_NC=8|16|32|64
 *     the column-slice width of the mma.sync step GEMM, TARFLOW_SEQ_FUSE_GELU=1 lets the MLP-up step GEMM
 *     apply bias + GELU itself when its reduction fits one CTA (K <= 512), TARFLOW_SEQ_FUSE_TAIL=0|1 switches the one-kernel
 *     step tail (final LayerNorm, head, update, embedding, next LayerNorm) off or on whatever the head's size.  Sweeps: TARFLOW_PAIR_GEMM=0 runs the projections with
 *     one CTA per 128x256 tile instead of 2-CTA pairs; TARFLOW_ATTN_TC=0 runs attention on the mma.sync kernel
 *     instead of the tcgen05 one, TARFLOW_ATTN_TC_SPLIT=0 does so for two-term operands only.  TARFLOW_SEQ_CHAINS=1|2|4
 *     sets how many sample chains decode a sequential block side by side (default: 2 from 32 samples up),
 *     TARFLOW_SEQ_ATTN_THREADS=128|256 the CTA size of the decoding step's attention (default: 128 when there are
 *     more (sample, head) pairs than three 256-thread CTAs per SM hold at once);
 *     TARFLOW_SEQ_FIN=1 lets the last K slice of a step projection finish its tile (residual add or bias + GELU) and
 *     the next projection normalise its own operand slice, five kernels per layer instead of eight (measured slower
 *     than the default chain), TARFLOW_SEQ_KBN8=0 keeps such launches at four k slabs per CTA;
 *     TARFLOW_SWEEP_GRAPH_ROWS=n replays Jacobi sweeps of at most n rows (slots x tokens, default 4096) from CUDA
 *     graphs, 0 launches every kernel directly; TARFLOW_GRAPHS=0 replays nothing from graphs, the decoding steps of a
 *     sequential block included (same kernels in the same order, for tools that list launches).  TARFLOW_SMALL_M_ROWS=n (default 1024): sweeps of at most n rows run
 *     their projections on 128 x 128 single-CTA tiles; TARFLOW_SPLIT_M_ROWS=n (default 4096): up to n rows the two
 *     projections into the residual stream are cut into K slices whose partial products the next LayerNorm adds in
 *     slice order (TARFLOW_SMALL_M_SPLIT=0: never); 0 for both keeps one tile shape for every sweep.  These paths
 *     hold a [8192, width] fp32 buffer per model.
 */
#ifndef TARFLOW_H_
#define TARFLOW_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TF_OK 0
#define TF_MAXITER 1
#define TF_EINVAL (-1)     /* bad argument or configuration                       */
#define TF_ESIZE (-2)      /* weight blob size / header mismatch                  */
#define TF_ENOMEM (-3)     /* host or device allocation failed                    */
#define TF_ECUDA (-4)      /* a CUDA runtime/driver call failed                   */
#define TF_ETIMEOUT (-5)   /* a bounded device-side wait expired                  */
#define TF_ENONFINITE (-6) /* NaN/Inf reached the convergence reduction           */

typedef struct tf_model tf_model; /* opaque: device weights, KV cache, workspace */

typedef struct {
  int32_t C, H, W, patch; /* L = (H/patch)*(W/patch) tokens of D = C*patch*patch values         */
  int32_t n_blocks;       /* K flow blocks                                                      */
  int32_t n_layers;       /* transformer layers per block                                       */
  int32_t width;          /* transformer width d (multiple of n_heads; bf16 engine: of 64)      */
  int32_t n_heads;        /* head_dim = width / n_heads; bf16 engine needs head_dim == 64       */
  int32_t mlp_ratio;      /* MLP hidden = mlp_ratio * width                                     */
  int32_t n_classes;      /* 0 = unconditional, else rows of the per-block class embedding      */
  int32_t dtype;          /* 0 = fp32 SIMT engine, 1 = bf16 tensor-core engine (fp32 accumulate)*/
  int32_t max_batch;      /* largest B any later call may use (sizes workspace and KV cache)    */
} tf_config;

/*
 * tf_load -- build a model from seeded weights (paper Sec. 3.1: the functions s_k, g_k of Eq. 4).
 *   weights_host: flat little-endian blob: 16 int32 header {magic 0x31574654, version 1, C, H, W,
 *     patch, n_blocks, n_layers, width, n_heads, mlp_ratio, n_classes, dtype, seed, 0, 0} followed
 *     by fp32 tensors, block by block (generation order), each block in this order:
 *       w_in [d,D], b_in [d], pos [L,d], cls [n_classes,d] (only if n_classes>0),
 *       per layer: ln1_g[d] ln1_b[d] w_qkv[3d,d] b_qkv[3d] w_o[d,d] b_o[d]
 *                  ln2_g[d] ln2_b[d] w_1[hid,d] b_1[hid] w_2[d,hid] b_2[d],
 *       lnf_g[d] lnf_b[d] w_out[2D,d] b_out[2D].
 *     Linear layers are [out_features, in_features] (y = x W^T + b); w_qkv rows are q | k | v;
 *     w_out rows are mu~ (first D) | alpha~ (last D).  The blob is copied, not retained.
 *     For dtype 1 the matrices are converted to bf16 (round to nearest even).
 *   nbytes: size of the blob; must equal the size implied by cfg (else TF_ESIZE); the header
 *     fields must equal cfg's (else TF_ESIZE).
 *   out: receives the model.  Allocates all device memory the other calls use.
 */
int tf_load(const tf_config* cfg, const void* weights_host, size_t nbytes, tf_model** out);

/* tf_free -- release a model and everything it owns.  tf_free(NULL) is a no-op. */
void tf_free(tf_model* m);

/*
 * tf_forward -- data to latent, x -> z, and logdet = -sum(alpha) (paper Eq. 4 applied through
 * blocks K-1 .. 0, Eq. 1 for the log-determinant).  One causal pass per block, no iteration.
 *   x_dev [B,C,H,W] in, labels_dev [B] int32 class ids or NULL, z_dev [B,C,H,W] out,
 *   logdet_dev [B] fp32 out (may be NULL).  1 <= B <= max_batch.  Synchronises the stream before returning
 *   (that is where a device-side timeout is reported).
 */
int tf_forward(tf_model* m, const float* x_dev, const int32_t* labels_dev, int32_t B, float* z_dev,
               float* logdet_dev, void* cuda_stream);

/*
 * tf_inverse_sequential -- latent to data, z -> x, every block decoded token by token with a
 * key/value cache (paper Eq. 5; the sequential baseline of Sec. 3.5).  L-1 steps per block.
 */
int tf_inverse_sequential(tf_model* m, const float* z_dev, const int32_t* labels_dev, int32_t B,
                          float* x_dev, void* cuda_stream);

/*
 * tf_inverse_jacobi -- latent to data under a per-block policy (paper Algorithm 1 and Sec. 3.5).
 *   policy_host [n_blocks], generation order: 0 = sequential with KV cache, 1 = Jacobi.
 *     The paper's selective policy is {0,1,1,...}; uniform Jacobi is all ones.
 *   tau >= 0: a sample leaves a Jacobi block after the first sweep whose
 *     max over all its L*D entries of |u^t - u^{t-1}| <= tau (per-sample test; converged samples
 *     are dropped from later sweeps).  tau < 0: fixed-iteration mode, exactly max_iters sweeps.
 *   max_iters >= 1: sweep cap per Jacobi block (L sweeps reproduce sequential decoding exactly,
 *     Prop. 3.2; passing the test on an exact iterate can need sweep L+1).
 *   init_mode: 0 = u^0 = 0 (Algorithm 1);  1 = u^0 = v (the block's input);  other values EINVAL.
 *   x_dev [B,C,H,W] out.
 *   iters_block_host [n_blocks] out (may be NULL): sweeps executed by a Jacobi block (max over
 *     samples, counting the passing sweep); L-1 for a sequential block.
 *   iters_sample_dev [n_blocks, B] int32 out (may be NULL): the same per sample.
 *   Synchronises the stream before returning.
 */
int tf_inverse_jacobi(tf_model* m, const float* z_dev, const int32_t* labels_dev, int32_t B,
                      const uint8_t* policy_host, float tau, int32_t max_iters, int32_t init_mode,
                      float* x_dev, int32_t* iters_block_host, int32_t* iters_sample_dev,
                      void* cuda_stream);

/*
 * tf_inverse_jacobi_ex -- tf_inverse_jacobi with the variants the paper discusses around Algorithm 1 and the
 * selective policy (Sec. 3.5, Sec. 4.4; Fig. "Convergence dynamics", the initialisation ablation, the table of
 * Jacobi iterations per block whose second CIFAR-10 block needs 54 sweeps).  opts == NULL behaves like
 * tf_inverse_jacobi with init_mode 0.  Fields of tf_jacobi_opts:
 *   struct_bytes      sizeof(tf_jacobi_opts) as the caller compiled it (checked).
 *   init_mode         0: u^0 = 0 (Algorithm 1);  1: u^0 = the block's input v;  2: u^0 = u0_dev (for instance the
 *                     caller's N(0, I) draws: the library draws no random numbers itself).
 *   u0_dev            init_mode 2: [n_blocks, B, C, H, W] fp32 on the device, image-shaped like z; Jacobi block g
 *                     starts from slice g (slices of sequential blocks are not read).
 *   tau_block_host    NULL, or [n_blocks] host floats: block g uses tau_block_host[g] instead of tau (negative:
 *                     that block runs max_iters sweeps without the test).
 *   fallback_sweeps   0: off.  n > 0: a Jacobi block that still has unconverged samples after n sweeps decodes
 *                     exactly those samples sequentially (Eq. 5) from the block's input, so a slowly converging
 *                     block costs at most n sweeps plus one sequential pass over the stragglers; such a sample
 *                     reports n + L - 1 iterations, the block reports the maximum.  Ignored when tau < 0 or
 *                     n >= max_iters.
 *   states_dev        NULL, or out [n_blocks, B, C, H, W] fp32: the sequence after each block, image-shaped
 *                     (slice n_blocks - 1 equals x).
 *   ref_states_dev    NULL, or in [n_blocks, B, C, H, W]: reference states, e.g. states_dev of an all-sequential
 *                     call.  With the trace enabled every sweep of Jacobi block g also records, per sample,
 *                     || u^t - ref_g ||_2 (the quantity the paper's convergence figure plots); read it with
 *                     tf_trace_read_l2.
 */
typedef struct {
  int32_t struct_bytes;
  int32_t init_mode;
  const float* u0_dev;
  const float* tau_block_host;
  int32_t fallback_sweeps;
  int32_t reserved;
  float* states_dev;
  const float* ref_states_dev;
} tf_jacobi_opts;

int tf_inverse_jacobi_ex(tf_model* m, const float* z_dev, const int32_t* labels_dev, int32_t B,
                         const uint8_t* policy_host, float tau, int32_t max_iters, const tf_jacobi_opts* opts,
                         float* x_dev, int32_t* iters_block_host, int32_t* iters_sample_dev, void* cuda_stream);

/*
 * tf_block_times -- device time of every block of the last tf_inverse_jacobi* call on this model, from CUDA
 * events the call records on its stream around each block (the per-block breakdown of the paper's runtime table).
 * Fills ms_host[0 .. min(cap, n_blocks)) and returns n_blocks; returns 0 when no call has completed yet.
 */
int tf_block_times(tf_model* m, float* ms_host, int32_t cap);

/*
 * tf_inverse_jacobi_host -- the same operation for callers that hold host memory: copies z (and
 * labels) to the device, runs tf_inverse_jacobi, copies x back.  z_host/x_host [B,C,H,W] fp32,
 * labels_host [B] or NULL; pinned host memory makes the copies asynchronous.  iters_sample_host
 * [n_blocks,B] may be NULL.  Synchronises before returning.
 */
int tf_inverse_jacobi_host(tf_model* m, const float* z_host, const int32_t* labels_host, int32_t B,
                           const uint8_t* policy_host, float tau, int32_t max_iters,
                           int32_t init_mode, float* x_host, int32_t* iters_block_host,
                           int32_t* iters_sample_host, void* cuda_stream);

/*
 * Second workload: Jacobi decoding of an MLP-based masked autoregressive flow (paper App. E.3: Algorithm 1 on every
 * layer of a flow whose networks have no key/value cache).  Each layer is the affine autoregressive block of Eq. 4 /
 * Eq. 5 over the D scalar dimensions of a sample, x_i = z_i * exp(alpha_i(x_<i)) + mu_i(x_<i), with (mu, alpha) from a
 * MADE network (two hidden layers of `hidden` ReLU units; input i and output i have degree i, hidden unit j degree
 * 1 + (j mod (D - 1)); a hidden unit sees degrees <= its own, an output degrees < its own), and the order of the
 * dimensions is reversed between layers.  Samples are fp32 [B, D].
 *   tf_maf_load: blob = 16 int32 header {magic 0x3146414D, version 1, D, hidden, n_blocks, dtype, seed, 0...} then per
 *     layer the dense fp32 tensors w1 [hidden, D], b1 [hidden], w2 [hidden, hidden], b2 [hidden], w3 [2D, hidden]
 *     (rows mu | alpha), b3 [2D]; the masks are applied by the library.  bf16 engine: D % 8 == 0, hidden % 64 == 0.
 *     The model is released with tf_free; tf_set_precision, tf_trace_*, tf_profile_*, tf_block_times,
 *     tf_launch_count and tf_device_bytes apply to it, the TarFlow calls refuse it (TF_EINVAL) and vice versa.
 *   tf_maf_forward: x -> z and logdet = -sum(alpha) (Eq. 4 through layers K-1 .. 0).  Synchronises.
 *   tf_maf_inverse_sequential: Eq. 5, D whole passes of the network per layer (dimension i is final after pass i).
 *   tf_maf_inverse_jacobi: Algorithm 1 on every layer with the per-sample stopping test (tau, max_iters, init_mode
 *     0 | 1, outputs as for tf_inverse_jacobi; D sweeps reproduce sequential decoding, Prop. 3.2).  Synchronises.
 */
typedef struct {
  int32_t D, hidden, n_blocks;
  int32_t dtype;      /* 0 = fp32 SIMT engine, 1 = bf16 tensor-core engine */
  int32_t max_batch;
} tf_maf_config;
int tf_maf_load(const tf_maf_config* cfg, const void* weights_host, size_t nbytes, tf_model** out);
int tf_maf_forward(tf_model* m, const float* x_dev, int32_t B, float* z_dev, float* logdet_dev, void* cuda_stream);
int tf_maf_inverse_sequential(tf_model* m, const float* z_dev, int32_t B, float* x_dev, void* cuda_stream);
int tf_maf_inverse_jacobi(tf_model* m, const float* z_dev, int32_t B, float tau, int32_t max_iters, int32_t init_mode,
                          float* x_dev, int32_t* iters_block_host, int32_t* iters_sample_dev, void* cuda_stream);

/*
 * tf_jacobi_update -- the fused step of Algorithm 1 on its own: given the un-shifted head output
 * o_dev [B, L, 2D] = (mu~ | alpha~) of one causal pass, the block input v_dev [B,L,D] and the
 * previous iterate u_dev [B,L,D] (updated in place), set u_1 = v_1, u_l = v_l * exp(alpha~_{l-1})
 * + mu~_{l-1}, and write maxdiff_dev[b] = max |u^t - u^{t-1}| over sample b.  `reversed` != 0
 * applies the block permutation (core position l is raster position L-1-l).  Asynchronous.
 */
int tf_jacobi_update(const float* o_dev, const float* v_dev, float* u_dev, float* maxdiff_dev,
                     int32_t B, int32_t L, int32_t D, int32_t reversed, void* cuda_stream);

/*
 * tf_gemm_bf16 -- the tensor-core GEMM used by every projection of a sweep, exposed for tests and
 * profiling:  C[M,N] (fp32, row-major) = A[M,K] (bf16 row-major) * W[N,K]^T (bf16 row-major) +
 * bias[N] (fp32, may be NULL).  K % 64 == 0, N % 8 == 0, pointers 16-byte aligned.  Asynchronous:
 * a device-side wait that expired is reported by tf_gemm_status.
 */
int tf_gemm_bf16(const void* a_dev, const void* w_dev, const float* bias_dev, float* c_dev,
                 int32_t M, int32_t N, int32_t K, void* cuda_stream);

/*
 * tf_skinny_gemm_noalloc -- C[M,N] (fp32) = A[M,K] (bf16) * W[N,K]^T (bf16) + bias[N] (fp32, may be NULL),
 * the same product as tf_gemm_bf16, computed by the split-K kernel of the sequential decoding path, for
 * callers that must not allocate device memory.  (The paper has no counterpart; this is a property of
 * the library, not of the method.)
 *   Who needs it: a caller that has handed all device memory to its own pool or arena, a caller inside a
 *   latency-critical loop where cudaMalloc's implicit device-wide synchronisation is not acceptable, or
 *   one that runs where the allocator may not be entered at all (for instance from a callback).  Every
 *   other entry point of this library takes its working memory from cudaMalloc (tf_load for a model,
 *   tf_gemm_bf16 for its error word on first use); this one calls neither cudaMalloc nor cudaFree nor any
 *   routine that does.
 *   How: the fp32 partial tiles of the K slices ((K/256) * M * N * 4 bytes) and one control word live in a
 *   static device array of TF_NOALLOC_SCRATCH_BYTES that every GPU which loads the library holds until
 *   the process exits.  A problem whose tiles do not fit is refused with TF_EINVAL and a message that
 *   names both sizes.  Requirements: M >= 1, N % 8 == 0, K % 256 == 0, a_dev and w_dev 16-byte aligned, c_dev and
 *   bias_dev 4-byte aligned (checked: TF_EINVAL, nothing is launched).
 *   First call on a device: looks up the array's device address (cudaGetSymbolAddress) and raises the
 *   kernel's shared-memory limit, with that device current; make this first call outside any stream capture.
 *   Sharing: all calls on a device use the one array, which keeps the contents of the previous call; the
 *   call re-zeroes what has to start at zero.  Two calls whose work overlaps on the GPU (different streams
 *   without ordering between them) race on it and give wrong results: order them.
 *   Asynchronous on `cuda_stream`; the caller owns every buffer.
 */
#define TF_NOALLOC_SCRATCH_BYTES (8u << 20)
int tf_skinny_gemm_noalloc(const void* a_dev, const void* w_dev, const float* bias_dev, float* c_dev,
                           int32_t M, int32_t N, int32_t K, void* cuda_stream);

/* tf_gemm_status -- synchronise `cuda_stream` and report whether any tf_gemm_bf16 launch on the current device
 * since the last report gave up on a bounded device-side wait (TF_ETIMEOUT, reported once) or all completed (TF_OK). */
int tf_gemm_status(void* cuda_stream);

/*
 * Profiling aid: when enabled, calls on this model bracket every kernel class with CUDA events on
 * the caller's stream and accumulate elapsed milliseconds and launch counts.
 *   tf_profile_enable(m, on): switch on (1), off (0) and reset the counters.  on == 2: the kernels of Jacobi sweeps
 *     are bracketed one by one as with 1, while a sequentially decoded block runs exactly as it does unprofiled
 *     (replayed graphs, sample chains) and is timed as ONE unit of the class "seq_block" (rows = B * (L - 1)).
 *   tf_profile_read(m, names, ms, launches, rows, cap): fills up to cap entries, returns how many
 *     classes exist; names[i] points to a static string; rows[i] is the number of activation
 *     rows (tokens of a sweep, samples of a sequential step) the class's launches processed.
 *   tf_launch_count(m): kernels launched by the library on this model since load (always counted).
 */
int tf_profile_enable(tf_model* m, int32_t on);
int tf_profile_read(tf_model* m, const char** names, double* ms, int64_t* launches, double* rows,
                    int32_t cap);
int64_t tf_launch_count(tf_model* m);

/*
 * tf_set_precision -- operand precision of Jacobi sweeps on the bf16 engine (no effect on fp32).
 * With single bf16 operands the rounding of activations puts a floor of a few 1e-3 under
 * max|u^t - u^{t-1}|, so the stopping test of Algorithm 1 cannot pass for a smaller tau.  In the
 * two-term mode every activation operand is a bf16 pair (hi + lo, about 16 significant bits) and
 * every product keeps the leading cross terms; the tensor-core work of such a sweep roughly doubles.
 *   mode 0 (default): per sample, sweeps use single operands until that sample's max|du| drops to
 *     switch_threshold, two-term operands afterwards; used only when 0 <= tau < single_ok_tau.
 *   mode 1: single operands always.   mode 2: two-term operands for every Jacobi sweep.
 *   switch_threshold / single_ok_tau <= 0 select the defaults 2^-5 and 2^-6.
 * Fixed-iteration mode (tau < 0) uses single operands unless mode is 2.
 */
int tf_set_precision(tf_model* m, int32_t mode, float switch_threshold, float single_ok_tau);

/*
 * Convergence trace (paper Fig. "Convergence dynamics of Jacobi decoding", and the stopping test of
 * Algorithm 1): when enabled, every Jacobi sweep of later tf_inverse_jacobi calls records
 * (block, sweep number, samples active in that sweep, max over those samples of
 * max|u^t - u^{t-1}|).  Enabling it makes every sweep synchronise, also in fixed-iteration mode.
 *   tf_trace_read fills up to cap records of the last call and returns how many exist.
 *   Enabling the trace for the first time allocates the buffer of tf_trace_read_l2 (device memory).
 */
int tf_trace_enable(tf_model* m, int32_t on);
int tf_trace_read(tf_model* m, int32_t* block, int32_t* sweep, int32_t* active, float* maxdiff,
                  int32_t cap);
/* tf_trace_read_l2 -- the distances || u^t - ref ||_2 recorded for Jacobi block `block` of the last
 * tf_inverse_jacobi_ex call that supplied ref_states_dev: l2_host[t * B + b] for sweep t + 1 and sample b (samples
 * that have converged keep their final iterate).  Returns the number of sweeps recorded (0 if none). */
int tf_trace_read_l2(tf_model* m, int32_t block, int32_t B, float* l2_host, int32_t cap_sweeps);

/*
 * tf_selftest_wait_timeout -- exercises the bounded-wait path without any fault: launches one CTA whose thread
 * waits, for at most limit_us microseconds (1 .. 1 000 000), on an mbarrier that nothing arrives on.  The wait runs
 * out, the kernel records its code in the model's error word and returns; the call then synchronises and returns
 * what any synchronising call would: TF_ETIMEOUT, once, with the word cleared.  The model remains usable.
 */
int tf_selftest_wait_timeout(tf_model* m, int32_t limit_us, void* cuda_stream);

/*
 * tf_debug_check_guards -- every device buffer of a model lies between two 256-byte guard regions filled with a
 * fixed pattern when the model is loaded.  This call counts, on the device, the guard words that no longer hold the
 * pattern and returns that number (0 = no kernel has written outside its buffer since the model was loaded;
 * negative = error).  It synchronises the stream.  A substitute for a memory checker where none can be run.
 */
int64_t tf_debug_check_guards(tf_model* m, void* cuda_stream);

/* tf_device_bytes -- device memory owned by the model (weights + workspace + KV cache), bytes. */
int64_t tf_device_bytes(tf_model* m);

/* tf_last_error -- message of the last failing call on this thread ("" if none). */
const char* tf_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* TARFLOW_H_ */
