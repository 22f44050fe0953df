/*
 * pestats -- per-example gradient statistics for linear layers on NVIDIA B200 (sm_100a).
 *
 * C ABI.  Every pointer is a DEVICE pointer unless its name starts with "h_" or the comment says
 * "host".  The caller owns every buffer and the stream; the library allocates nothing and enqueues
 * its work asynchronously on `stream` (0 = the legacy default stream).  State kept between calls: the
 * process-wide path override and wait limit below, and a per-device cache of device properties and
 * kernel attributes that the first call on a device fills in (guarded by a mutex, so first calls
 * from several host threads are safe).  Functions return a pe_status_t and
 * never throw.  Errors detected on the host (bad arguments, unsupported shape, CUDA launch
 * failure) are returned immediately and nothing is enqueued.  Errors detected on the device (a
 * bounded wait inside a kernel that ran out) are latched in a device status word that
 * pe_get_async_status() reads back.
 *
 * Layout conventions (row-major, contiguous):
 *   X   [B, T, d_in]   activations entering the layer            (the paper's H, "BLD")
 *   dY  [B, T, d_out]  cotangents of the layer's output          (the paper's Lambda, "BLF")
 *   per-example gradient  G_b = dY_b^T X_b  is [d_out, d_in]     (transpose of the paper's D x F)
 *   every statistic is [d_out, d_in] fp32.
 * There is no CPU fallback: on a machine without an sm_100 GPU the compute calls return
 * PE_ERR_ARCH or PE_ERR_CUDA.
 */
#ifndef PESTATS_H_
#define PESTATS_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  PE_OK = 0,
  PE_ERR_NULL = 1,              /* a required pointer is NULL */
  PE_ERR_DIM = 2,               /* a size is zero/negative/too large, or step < 1, or B < 1 */
  PE_ERR_ALIGN = 3,             /* a pointer is not aligned as documented */
  PE_ERR_UNSUPPORTED_SHAPE = 4, /* the forced path cannot run this shape */
  PE_ERR_PHI = 5,               /* phi is not one of pe_phi_t */
  PE_ERR_ARCH = 6,              /* current device is not compute capability 10.x */
  PE_ERR_CUDA = 7,              /* a CUDA runtime/driver call failed */
  PE_ERR_TIMEOUT = 8,           /* a bounded device-side wait ran out (see pe_get_async_status) */
  PE_ERR_WORKSPACE = 9          /* workspace missing or smaller than *_workspace_bytes() */
} pe_status_t;

/* The elementwise function applied to each per-example gradient before the sum over examples
 * (Eq. (2): the nonlinear statistic (1/B) sum_i phi(grad f(theta; x_i)); square gives Eq. (3)'s
 * nu_micro, sign gives the MicroSignSGD statistic of Section 3.1).  sign(+0) = sign(-0) = 0; every other fp32 value of
 * G_b, denormals included, counts with its sign. */
typedef enum { PE_PHI_IDENTITY = 0, PE_PHI_SQUARE = 1, PE_PHI_SIGN = 2 } pe_phi_t;

/* Which kernel family a call may use.  AUTO picks the tensor-core kernel whenever the shape allows
 * it (bf16 inputs, d_in % 8 == 0, d_out % 8 == 0) and the SIMT kernel otherwise.  When both outputs
 * are wanted AUTO and TENSOR keep both running sums in registers: on a 256 x 192 tile for T >= 64 when
 * d_in rounded up to a multiple of 192 is at most 13 % above d_in rounded up to a multiple of 128, else
 * on a 256 x 128 tile, except that from T = 4096 on those remaining shapes keep sum_b G_b in tensor
 * memory beside a 256 x 256 tile.  TENSOR_NARROW is TENSOR with the 256 x 128 tile and TENSOR_WIDE is
 * TENSOR with the 256 x 192 tile, both at any T; they exist so that tests can reach those kernels on
 * every shape. */
typedef enum { PE_PATH_AUTO = 0, PE_PATH_SIMT = 1, PE_PATH_TENSOR = 2, PE_PATH_TENSOR_NARROW = 3, PE_PATH_TENSOR_WIDE = 4 } pe_path_t;

typedef struct CUstream_st* pe_stream_t; /* a cudaStream_t */

/*
 * Sequence-level per-example statistics of a linear layer (Section 2.3, "Dense layers in
 * sequence-level architectures"; Eq. (2)).  For every example b the gradient
 *     G_b[o,i] = sum_{t<T} dY[b,t,o] * X[b,t,i]
 * is formed on chip (it is never written to global memory), and
 *     out_mean[o,i] = sum_b G_b[o,i]            (the ordinary batch weight gradient, NOT divided by B)
 *     out_stat[o,i] = sum_b phi(G_b[o,i])
 * X, dY: bf16, 16-byte aligned.  out_mean, out_stat: fp32 [d_out, d_in], 16-byte aligned, OVERWRITTEN;
 * either may be NULL to skip it (not both).  Products are exact in fp32 and accumulated in fp32.
 * B, T >= 0 (B == 0 or T == 0 writes zeros, and X, dY may then be NULL); d_in, d_out >= 1; B*T*max(d_in,d_out) < 2^40.
 * When the batch is split across thread blocks the outputs are zeroed first and every block adds its
 * partial tile with fp32 reduce-add bulk stores (the SIMT kernel: fp32 atomic adds), so the low bits
 * of out_mean / the square statistic may differ between runs; the sign statistic is always
 * exact-integer valued.
 */
pe_status_t pe_linear_stats(const void* X, const void* dY, int B, int T, int d_in, int d_out,
                            pe_phi_t phi, float* out_mean, float* out_stat, pe_stream_t stream);

/* Same for fp32 inputs (4-byte aligned suffices); always the SIMT kernel, fp32 FMA accumulation. */
pe_status_t pe_linear_stats_f32(const float* X, const float* dY, int B, int T, int d_in, int d_out,
                                pe_phi_t phi, float* out_mean, float* out_stat, pe_stream_t stream);

/*
 * Per-example squared gradient norms (Section 2.3: N_b = ||grad_W f(theta; x_b)||_2^2, the quantity
 * behind per-example clipping, one of the transformations phi of Section 2.1):
 *     out_norms[b] = sum_{o,i} G_b[o,i]^2,     G_b = dY_b^T X_b.
 * bf16 inputs as for pe_linear_stats; out_norms: fp32 [B], 4-byte aligned, overwritten (may be NULL
 * only if B = 0).  Each G_b tile is formed on chip, squared and reduced there; every tile adds its
 * share to out_norms[b] with an fp32 atomic, so the result is reproducible only to rounding.  A
 * clipped batch gradient is then sum_b c_b G_b with c_b = min(1, C / sqrt(N_b)): pe_linear_clipped_sum.
 */
pe_status_t pe_example_sqnorms(const void* X, const void* dY, int B, int T, int d_in, int d_out,
                               float* out_norms, pe_stream_t stream);

/*
 * pe_linear_stats for a PACKED batch of sequences of different lengths (Section 2.3: the per-example
 * gradient of a sequence-level dense layer is the contraction over THAT sequence's tokens; Eq. (2)).
 * X is [total_rows, d_in] and dY [total_rows, d_out] (bf16, 16-byte aligned); example b owns the token
 * rows seq_offsets[b] .. seq_offsets[b+1]-1, so
 *     G_b[o,i] = sum_{r in example b} dY[r,o] * X[r,i],   out_mean = sum_b G_b,   out_stat = sum_b phi(G_b).
 * seq_offsets: DEVICE array of B+1 int32, 4-byte aligned, non-decreasing, 0 <= seq_offsets[0],
 * seq_offsets[B] <= total_rows < 2^31 (it is read by the kernels only, so a producer on the same stream
 * may still be writing it when this call returns).  An empty sequence contributes nothing.  Offsets
 * that break these rules give unspecified statistics but never an access outside the tensors.
 * workspace: device memory, 256-byte aligned, at least pe_linear_stats_ragged_workspace_bytes(B, d_in,
 * d_out) bytes (32 * B * (d_in + d_out) bytes plus padding), contents undefined afterwards: the tensor-core
 * kernel contracts 16 tokens per instruction, and a pre-pass copies every sequence's last len % 16
 * tokens there, zero-padded to 16.  The SIMT path (widths not multiples of 8, or forced) ignores it.
 * Outputs and phi as for pe_linear_stats; B == 0 or total_rows == 0 writes zeros.
 */
pe_status_t pe_linear_stats_ragged(const void* X, const void* dY, const int* seq_offsets, int B,
                                   long long total_rows, int d_in, int d_out, pe_phi_t phi, float* out_mean,
                                   float* out_stat, void* workspace, size_t workspace_bytes, pe_stream_t stream);
/* Bytes of workspace the packed-batch calls need under the current path setting (0 on the SIMT path). */
size_t pe_linear_stats_ragged_workspace_bytes(int B, int d_in, int d_out);
/* pe_example_sqnorms for a packed batch (same layout, offsets and workspace as pe_linear_stats_ragged):
 * out_norms[b] = ||G_b||_F^2 (Section 2.3). */
pe_status_t pe_example_sqnorms_ragged(const void* X, const void* dY, const int* seq_offsets, int B,
                                      long long total_rows, int d_in, int d_out, float* out_norms,
                                      void* workspace, size_t workspace_bytes, pe_stream_t stream);

/*
 * Sum of norm-clipped per-example gradients (Section 2.1 lists clipping among the statistics
 * E[phi(grad f)] of Eq. (2); Section 2.3 names the per-example squared norms N_b it needs).  The paper
 * does not spell the function out; per-example L2 clipping is taken:
 *     c_b = min(1, clip_norm / sqrt(N_b)),     out_sum[o,i] = sum_b c_b * G_b[o,i],     G_b = dY_b^T X_b
 * (not divided by B).  sq_norms: fp32 [B], 4-byte aligned.  norms_given == 0: the call first computes
 * this layer's N_b = ||G_b||_F^2 into sq_norms (pe_example_sqnorms) and clips by them; norms_given != 0:
 * sq_norms is an input, e.g. the squared norms summed over all layers of a model for a model-wide clip.
 * N_b = 0 gives c_b = 1.  Two passes over the inputs (norms, then the contraction with every G_b scaled
 * on chip as it is added); G_b never reaches global memory.  X, dY, shapes as for pe_linear_stats;
 * out_sum fp32 [d_out, d_in], 16-byte aligned, overwritten; clip_norm >= 0.
 */
pe_status_t pe_linear_clipped_sum(const void* X, const void* dY, int B, int T, int d_in, int d_out,
                                  float clip_norm, float* sq_norms, int norms_given, float* out_sum,
                                  pe_stream_t stream);

/*
 * pe_linear_stats for gradient accumulation over micro-batches: the statistics of this call's B
 * examples are ADDED to what out_mean / out_stat already hold (both sums of Eq. (2) are additive over
 * examples, so running this over the micro-batches of a batch, after zeroing the outputs once, gives
 * the statistics of the whole batch; the caller divides by the total number of examples).  Same
 * arguments and rules otherwise; an empty micro-batch leaves the outputs untouched.  Partial results
 * are added with fp32 reduce operations, so the summation order over micro-batches is the call order
 * but within a call it is unspecified.
 */
pe_status_t pe_linear_stats_accumulate(const void* X, const void* dY, int B, int T, int d_in, int d_out,
                                       pe_phi_t phi, float* out_mean, float* out_stat, pe_stream_t stream);

/*
 * The three statistics of pe_linear_stats in one pass over the examples (Eq. (2) with phi = identity,
 * square and sign at once; Sections 2.1 and 3.1):
 *     out_mean = sum_b G_b,   out_square = sum_b G_b^2,   out_sign = sum_b sign(G_b),   G_b = dY_b^T X_b.
 * bf16 inputs as for pe_linear_stats; all three outputs [d_out, d_in] fp32, 16-byte aligned, non-NULL,
 * overwritten.  Each G_b tile is formed once and feeds all three running sums (the sign sum is kept
 * as a per-column count), so the call costs about one pe_linear_stats(square) instead of that plus a
 * pe_linear_stats(sign).  Shapes the one-pass kernel does not take (widths that are not multiples of 8,
 * the SIMT path forced) are served by those two calls.
 */
pe_status_t pe_linear_stats_all(const void* X, const void* dY, int B, int T, int d_in, int d_out,
                                float* out_mean, float* out_square, float* out_sign, pe_stream_t stream);

/*
 * Per-token second moment (Section 2.3, the "per-token" alternative):
 *     out_stat[o,i] = sum_{b,t} dY[b,t,o]^2 * X[b,t,i]^2  =  ((dY o dY)^T (X o X))[o,i].
 * B and T only enter through the row count B*T.  bf16 inputs, 16-byte aligned; out_stat fp32
 * [d_out, d_in], 16-byte aligned, overwritten.  On the tensor-core path (taken when the shape allows
 * it and B*T >= 256) one kernel squares the operands on chip (exact in fp32), rounds each square to
 * tf32 (11 significant bits, so every entry is within about 1e-3 relative of the exact sum) and
 * contracts them; nothing is staged in global memory.  Otherwise the SIMT kernel squares in fp32.
 */
pe_status_t pe_token_sqstats(const void* X, const void* dY, int B, int T, int d_in, int d_out,
                             float* out_stat, pe_stream_t stream);
pe_status_t pe_token_sqstats_f32(const float* X, const float* dY, int B, int T, int d_in, int d_out,
                                 float* out_stat, pe_stream_t stream);

/*
 * The same statistic in two passes (Section 2.3), for callers that can lend a workspace as large as
 * the inputs.  Streaming kernels find the largest magnitude of every column of X and of dY and write
 * the squares, each multiplied by a power of two chosen from its column's maximum so that it fits
 * IEEE half, into `workspace` (device memory, 256-byte aligned, at least
 * pe_token_sqstats_staged_workspace_bytes() bytes, contents undefined afterwards); the plain
 * tensor-core contraction then runs on the half operands at the full 16-bit rate (the one-kernel
 * pe_token_sqstats contracts tf32 at half that rate), and a last kernel undoes the scales.  Half keeps
 * the same 11 significant bits as tf32, rounded to nearest even; within a column, entries more than
 * 2^14 below the column's largest magnitude lose bits gradually and vanish 2^20 below it.  Faster
 * than pe_token_sqstats once B*T*(d_in + d_out) reaches about 10^8 elements, slower below (several
 * launches instead of one).  Also the kernel sequence behind pe_token_sqstats_static.  The SIMT path
 * ignores the workspace (it may then be NULL).
 */
pe_status_t pe_token_sqstats_staged(const void* X, const void* dY, int B, int T, int d_in, int d_out,
                                    float* out_stat, void* workspace, size_t workspace_bytes,
                                    pe_stream_t stream);
/* Bytes of workspace pe_token_sqstats_staged needs for this shape under the current path setting
 * (0 when the SIMT kernel will be used). */
size_t pe_token_sqstats_staged_workspace_bytes(int B, int T, int d_in, int d_out);

/*
 * The two-pass per-token statistic (Section 2.3) with fp8 operands: as pe_token_sqstats_staged, but the
 * scaled squares are staged as e4m3 (one byte each: half the workspace and half the staged traffic) and
 * contracted by the 8-bit tensor-core path at twice the 16-bit rate.  Two error sources, both measured:
 * (1) e4m3 keeps 4 significant bits, so a staged square carries up to 2^-4 relative rounding error (0.027
 * rms, to nearest even, unbiased) and a term of the sum about 0.0375 rms, independent from row to row:
 * with w_r = dY[r,o]^2 X[r,i]^2 >= 0 an entry's random relative error is about
 * 0.0375 * sqrt(sum_r w_r^2) / sum_r w_r, i.e. 0.11 / sqrt(B*T) for Gaussian inputs (9e-4 at B*T = 16384),
 * more when a few rows carry the sum; (2) the 8-bit tensor-core path aligns the products of one instruction
 * to their largest exponent and drops what falls below its internal width, which for these all-positive
 * sums is a systematic deficit of about 2.4e-3, whatever the number of rows.  Together: 2.6e-3 to 3.1e-3
 * relative Frobenius error on 16384-row layers, ABOVE the 2e-3 the other routes are held to (they reach
 * 1e-5).  An approximation to opt into where that is acceptable; pe_token_sqstats and pe_token_sqstats_staged keep
 * 11 significant bits.  Needs d_in % 16 == 0 and d_out % 16 == 0; other tensor-core shapes are served by
 * the half route (same workspace call, which then reports the larger size), tiny or odd ones by the SIMT
 * kernel.  workspace: 256-byte aligned, pe_token_sqstats_fp8_workspace_bytes() bytes.
 */
pe_status_t pe_token_sqstats_fp8(const void* X, const void* dY, int B, int T, int d_in, int d_out,
                                 float* out_stat, void* workspace, size_t workspace_bytes,
                                 pe_stream_t stream);
size_t pe_token_sqstats_fp8_workspace_bytes(int B, int T, int d_in, int d_out);

/*
 * pe_token_sqstats_staged for callers that have no device memory to give as workspace and no way to
 * get some.  (The paper has no counterpart; this is a convenience of this library.)  Typical cases: a
 * plug-in that is handed input and output pointers but no allocator; a process whose framework
 * reserved all of the GPU's memory in its own pool at start-up, so that cudaMalloc would fail; a
 * latency-critical loop that must not pay cudaMalloc / cudaFree's device-wide synchronisation.
 *
 * Same arguments, result and path selection as pe_token_sqstats_staged, minus the workspace: the
 * staging of the squared operands lives in an array of PE_STATIC_SCRATCH_BYTES bytes that is part
 * of the library's device image, so every GPU on which the library is used holds that much memory
 * from module load until the process exits.  The call allocates and frees nothing, on the device or
 * through any library.
 *
 * Limit: shapes whose staging (pe_token_sqstats_staged_workspace_bytes) exceeds
 * PE_STATIC_SCRATCH_BYTES are refused with PE_ERR_WORKSPACE and nothing is enqueued; use
 * pe_token_sqstats (which needs no workspace at all) or pe_token_sqstats_staged with your own
 * workspace for those.
 * First call on a device: looks up the array's device address (a host-side query, done once per
 * device with that device current) before enqueuing; make that first call outside any stream
 * capture.  The array belongs to the one device module that holds all of this library's kernels, and
 * CUDA loads a module when its first kernel or symbol is used: a process that is going to hand the
 * whole GPU to a memory pool must make its first call into this library on each device (any entry
 * point) BEFORE doing so, or the module load itself fails for want of 32 MiB and every pestats call
 * on that device returns PE_ERR_CUDA.
 * Speed: every shape that fits the array is small enough that the one-kernel pe_token_sqstats, which
 * needs no workspace either, is the faster route; this entry point is for callers that want the two-pass
 * route's arithmetic (IEEE-half squares at the full 16-bit tensor rate) without owning memory.
 * Sharing: all calls on a device use the same array and it keeps whatever the previous call left
 * there.  Each call overwrites the part it reads before reading it, so stale contents never reach
 * a result; but two calls whose kernels can overlap on the GPU (different streams, no dependency
 * between them) race on the array and both results are then undefined.  Calls on one stream are
 * ordered and safe.
 */
#define PE_STATIC_SCRATCH_BYTES (32u * 1024u * 1024u)
pe_status_t pe_token_sqstats_static(const void* X, const void* dY, int B, int T, int d_in, int d_out,
                                    float* out_stat, pe_stream_t stream);

/*
 * One MicroAdam step over n parameters (Algorithm 1, MicroAdam branch; Eq. (3)):
 *     mu = s*sum_g/B;  nu = s^2*sum_g2/B;   m = beta1*m + (1-beta1)*mu;   v = beta2*v + (1-beta2)*nu
 *     mh = m/(1-beta1^step);  vh = v/(1-beta2^step)
 *     u  = mh/(sqrt(vh)+eps)            if eps_inside_sqrt == 0  (the form of Section 3.2.3)
 *     u  = mh/sqrt(eps+vh)              otherwise                (Algorithm 1 as printed)
 *     theta = theta - lr*u - weight_decay*theta                  (decay not scaled by lr, Appendix E)
 * theta, m, v: fp32 [n], updated in place.  sum_g, sum_g2: fp32 [n], the out_mean / out_stat(square)
 * of pe_linear_stats.  s = grad_scale converts the passed sums to sums of per-example gradients
 * (1 if dY came from sum_b f_b, B if it came from the mean loss).  theta_lp: optional bf16 [n] copy
 * of the new theta (NULL to skip).  step is 1-based.  All pointers 16-byte aligned.
 */
pe_status_t microadam_step(float* theta, void* theta_lp, float* m, float* v, const float* sum_g,
                           const float* sum_g2, long long n, int B, float grad_scale, float lr,
                           float beta1, float beta2, float eps, int eps_inside_sqrt,
                           float weight_decay, int step, pe_stream_t stream);

/*
 * One step of a member of the extended Adam family (Section 3.2.3, "A new family of Adam methods";
 * Algorithm 1).  As microadam_step, except for what feeds the second-moment EMA:
 *     nu_adam = mu^2,   nu_micro = s^2*sum_g2/B
 *     PE_ADAM_ORIGINAL   nu = nu_adam                                   (Adam on the average gradient)
 *     PE_ADAM_MICRO      nu = nu_micro                                  (microadam_step)
 *     PE_ADAM_MICRO_VAR  nu = (nu_micro - nu_adam)   / (1 - 1/B)        (Eq. (6): unbiased variance)
 *     PE_ADAM_MICRO_MSQ  nu = (nu_adam - nu_micro/B) / (1 - 1/B)        (Eq. (6): unbiased squared mean)
 * Algorithm 1 prints the factor of the last two as B/(1-B); Eq. (6), which Section 3.2.3 says they
 * implement, is followed.  PE_ADAM_MICRO_MSQ clamps vh at zero where it enters u (v itself keeps its
 * sign, so the estimator stays unbiased); the paper runs it with eps = 1e-6.  The last two need
 * B >= 2 (PE_ERR_DIM otherwise); an unknown variant is PE_ERR_PHI.
 */
typedef enum { PE_ADAM_ORIGINAL = 0, PE_ADAM_MICRO = 1, PE_ADAM_MICRO_VAR = 2, PE_ADAM_MICRO_MSQ = 3 } pe_adam_variant_t;
pe_status_t microadam_family_step(float* theta, void* theta_lp, float* m, float* v, const float* sum_g,
                                  const float* sum_g2, long long n, int B, pe_adam_variant_t variant,
                                  float grad_scale, float lr, float beta1, float beta2, float eps,
                                  int eps_inside_sqrt, float weight_decay, int step, pe_stream_t stream);

/*
 * One MicroSignSGD step (Section 3.1: EMA o avg o sign):
 *     sbar = sum_sign/B;   m = beta*m + (1-beta)*sbar;   theta = theta - lr*m - weight_decay*theta
 * sum_sign: fp32 [n], the out_stat(sign) of pe_linear_stats.  No bias correction.
 */
pe_status_t microsignsgd_step(float* theta, void* theta_lp, float* m, const float* sum_sign,
                              long long n, int B, float lr, float beta, float weight_decay,
                              pe_stream_t stream);

/*
 * Statistics and parameter update in ONE launch (Algorithm 1 applied to the statistics of Eq. (2) where
 * they are formed: the thread block that holds, or completes, a tile's sums over the whole batch applies
 * the update to that tile of the parameters, so the sums need not be written out and read back and the
 * update needs no launch of its own).  The result is that of pe_linear_stats(phi = square) followed by
 * microadam_family_step on its two outputs:
 *     theta, m, v [d_out, d_in] fp32 updated in place, theta_lp the optional bf16 copy of the new theta.
 * out_mean / out_stat (sum_b G_b, sum_b G_b^2): written when not NULL.  workspace: device memory, 256-byte
 * aligned, pe_linear_fused_workspace_bytes(d_in, d_out) bytes (tile counters; contents undefined
 * afterwards); needed, together with both outputs, when the schedule splits the batch across thread
 * blocks: every block then adds its partial sums to the outputs and the one that adds the last part
 * of a tile applies the update.  If the workspace or an output is missing the batch is not split (one
 * block per tile walks all examples: correct, slower on layers with few tiles).  B >= 1, T >= 1; other
 * arguments as for pe_linear_stats and microadam_family_step.  The _f32 form takes fp32 inputs (SIMT
 * kernel, never splits the batch).  After PE_ERR_TIMEOUT the parameters of unfinished tiles are left as
 * they were (the two-kernel sequence skips its update kernel while the device status word is set, i.e.
 * until pe_get_async_status has read and cleared it).
 * What the fusion buys is MEMORY, not time: with out_mean = out_stat = NULL no [d_out, d_in] statistic
 * buffer exists anywhere (2 x 4 bytes per parameter saved).  In time there is little to gain (the update
 * moves 34 bytes per parameter whoever performs it; fusing saves the 8 bytes of re-reading the sums) and
 * something to lose: the blocks of a wave finish their tiles together, so the update's traffic reaches
 * memory in bursts during which the tensor cores idle (about 25 us per wave, measured), while a separate
 * update kernel streams at the HBM rate after the statistics kernel.  By default
 * (PE_FUSED_AUTO) the call therefore fuses only when it was given no statistic buffers and otherwise
 * runs the statistics kernel and the update kernel back to back on `stream`; pe_set_fused_update
 * overrides that choice.
 */
pe_status_t pe_linear_microadam_step(const void* X, const void* dY, int B, int T, int d_in, int d_out,
                                     float* theta, void* theta_lp, float* m, float* v, float* out_mean,
                                     float* out_stat, pe_adam_variant_t variant, float grad_scale, float lr,
                                     float beta1, float beta2, float eps, int eps_inside_sqrt,
                                     float weight_decay, int step, void* workspace, size_t workspace_bytes,
                                     pe_stream_t stream);
pe_status_t pe_linear_microadam_step_f32(const float* X, const float* dY, int B, int T, int d_in, int d_out,
                                         float* theta, void* theta_lp, float* m, float* v, float* out_mean,
                                         float* out_stat, pe_adam_variant_t variant, float grad_scale,
                                         float lr, float beta1, float beta2, float eps, int eps_inside_sqrt,
                                         float weight_decay, int step, pe_stream_t stream);
/*
 * The same for MicroSignSGD (Section 3.1: EMA o avg o sign): pe_linear_stats(phi = sign, statistic only)
 * followed by microsignsgd_step, in one launch.  out_sign (sum_b sign(G_b)) is written when not NULL and,
 * like the workspace, is needed for a split batch.
 */
pe_status_t pe_linear_microsignsgd_step(const void* X, const void* dY, int B, int T, int d_in, int d_out,
                                        float* theta, void* theta_lp, float* m, float* out_sign, float lr,
                                        float beta, float weight_decay, void* workspace,
                                        size_t workspace_bytes, pe_stream_t stream);
/* Bytes of workspace the two calls above can use (one 32-bit counter per thread block of the widest grid). */
size_t pe_linear_fused_workspace_bytes(int d_in, int d_out);
/* How pe_linear_microadam_step / pe_linear_microsignsgd_step run on the tensor-core path (process-wide;
 * returns the previous mode, -1 for an unknown one): AUTO = one fused launch when no statistic buffers
 * were given, the two-kernel sequence otherwise; ALWAYS = the fused launch whenever possible; NEVER =
 * the two-kernel sequence (the statistic buffers are then required: PE_ERR_NULL without them). */
typedef enum { PE_FUSED_AUTO = 0, PE_FUSED_ALWAYS = 1, PE_FUSED_NEVER = 2 } pe_fused_mode_t;
int pe_set_fused_update(int mode /* pe_fused_mode_t */);

/* Human-readable name of a status code (static storage). */
const char* pe_status_string(pe_status_t status);

/* Synchronises `stream`, then reads and clears the device status word.  Returns PE_OK, PE_ERR_TIMEOUT
 * (a kernel gave up on a bounded wait; its outputs are invalid), or PE_ERR_CUDA.  If `detail` is not
 * NULL it receives a host int identifying the wait that expired (0 if none). */
pe_status_t pe_get_async_status(pe_stream_t stream, int* detail);

/* Cycle budget of every wait inside the tensor-core kernels on the CURRENT device (each wait of a thread
 * on an on-chip barrier is bounded; a wait that exhausts the budget makes its kernel give up cleanly,
 * skip its outputs and latch PE_ERR_TIMEOUT for pe_get_async_status).  The default, restored by
 * cycles <= 0, is 2^32 cycles (about two seconds), far beyond any wait of a healthy launch; tests lower it
 * to a few cycles to drive the give-up path, which makes ordinary launches time out.  Synchronous (a
 * small host-to-device copy); set it while no library kernel is running on the device. */
pe_status_t pe_set_wait_limit_cycles(long long cycles);

/* Process-wide override of the kernel family (for tests and benchmarks). Returns the previous value. */
int pe_set_path(int path /* pe_path_t */);
/* The family the most recent pe_linear_stats / pe_token_sqstats call on this thread's process used
 * (PE_PATH_SIMT or PE_PATH_TENSOR; PE_PATH_AUTO if none yet). */
int pe_last_path(void);
/* The tile order a tensor-core launch would use, as a host-side query (no GPU is touched): the number of 256-row pair
 * rows of d_out that consecutive thread-block pairs walk before they move to the next column tile of d_in.  tile_cols is
 * the tile's width in d_in (128, 192 or 256), batch_slices the number of slices the batch is split into (>= 1),
 * sm_count the device's SM count (two SMs hold one pair).  The library picks, per launch, the band that minimises the
 * operand columns its waves of sm_count / 2 pairs stream from memory, sum over waves of (pair rows x 256 + column tiles x
 * tile_cols); the paper has no counterpart (it leaves scheduling to XLA).  Returns 0 for arguments out of range. */
int pe_tile_order_band(int d_in, int d_out, int tile_cols, int batch_slices, int sm_count);
/* Number of kernels the library has launched since load (or since the last reset to 0 via
 * pe_reset_launch_count). */
long long pe_launch_count(void);
void pe_reset_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* PESTATS_H_ */
