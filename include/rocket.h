/*
 * rocket.h - C ABI of the B200 ROCKET transform library.
 *
 * The library computes the random-convolution transform of ROCKET (Section 3 of "Making the
 * exceptionally fast ROCKET model faster"): K random dilated, optionally "same"-padded,
 * multichannel 1-D convolution kernels are applied to a batch of series X[N][C][L] and each
 * kernel's output is reduced on the fly to two pooled features, so the N*K*L_out convolution
 * outputs never leave the chip.
 *
 *   z[n,k,i] = b_k + sum_{q<m_k} sum_{j<len_k} W_k[q][j] * xpad[n, S_k[q], i - p_k + j*d_k]
 *              for 0 <= i < L_out,k = L + 2 p_k - (len_k - 1) d_k, xpad = 0 outside [0, L)
 *   PPV      = (1/L_out) #{ i : z_i > 0 }                               (Eq. 1-2)
 *   MAX      = max_i z_i                                                (Section 3, step (2))
 *   softPPV  = (1/L_out) sum_i 1 / (1 + exp(-(lambda z_i + shift)))     (Eq. 3-4)
 *
 * Conventions common to every call
 *   - Pointers named *_dev are device pointers; pointers named *_host and all other pointers
 *     are host pointers.  A handle binds to the device that is current at its first device
 *     call (its parameters are uploaded then, once) and every later call with that handle
 *     runs on that device.  Creating, inspecting and destroying a handle needs no device.
 *   - X is dense row-major [N][C][L] fp32.  Features are fp32 [N][2K], interleaved:
 *     feat[n][2k] = PPV_k (or softPPV_k), feat[n][2k+1] = MAX_k.
 *   - Kernel parameters are ragged: kernel k owns num_channels[k] consecutive entries of
 *     channel_idx and num_channels[k]*length[k] consecutive weights, row-major [q][j].
 *   - Device calls enqueue work on the caller's stream (a cudaStream_t passed as void*, NULL =
 *     the legacy default stream).  Outputs are fully overwritten.  The caller owns every buffer
 *     it passes; the library owns the handle and the workspace inside it.  Two calls that use
 *     the same handle must be ordered on the device (same stream, or an event between them):
 *     they share the handle's workspace.
 *   - Workspace.  The handle's workspace (parameter upload, zero-margined staging copies and
 *     their tensor maps, per-pair and per-weight accumulators) is allocated either up front by
 *     rocket_params_reserve, or lazily: the first device call, the first call of a kind (soft,
 *     backward, 8-bit input) and any call with more examples than every call before it may
 *     allocate, free, clear and upload, which synchronises the device.  Once the workspace
 *     covers a call - after rocket_params_reserve for its size and passes, or after an earlier
 *     call at least as large - the device calls only enqueue kernels and return without
 *     allocating or synchronising.  rocket_device_alloc_count lets a caller verify that.
 *   - Every function returns a rocket_status_t (0 = success).  Argument errors are detected
 *     on the host before anything is launched and leave the outputs untouched.  Nothing
 *     aborts and nothing throws across this boundary.  There is no CPU fallback: without a
 *     CUDA device the device calls fail with ROCKET_ECUDA.
 */
#ifndef ROCKET_B200_H
#define ROCKET_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct rocket_params rocket_params_t; /* opaque: host arrays, device copies, launch plan */

typedef enum {
    ROCKET_OK = 0,
    ROCKET_EINVAL = -1,       /* null pointer, negative size, parameter out of range            */
    ROCKET_ESHAPE = -2,       /* C or L of the call differ from the handle's                    */
    ROCKET_EUNSUPPORTED = -3, /* valid request outside what the kernels implement               */
    ROCKET_ENOMEM = -4,       /* host or device allocation failed                               */
    ROCKET_ECUDA = -5         /* a CUDA call failed (no device, launch error, copy error)       */
} rocket_status_t;

/* Largest kernel length and channel count per kernel the kernels are built for (Section 3.1
 * draws lengths from {7, 9, 11} and at most min(C, len) channels). */
#define ROCKET_MAX_LENGTH 11
#define ROCKET_MAX_CHANNELS_PER_KERNEL 11

/* Human-readable text for a status code.  Never NULL; static storage. */
const char* rocket_strerror(int status);

/*
 * Random kernel initialisation (Section 3.1), on the host, from one seed.  Kernel k is a pure
 * function of (seed, k, C, L): length uniform over {7,9,11}; weights N(0,1), each chosen
 * channel's row mean-centred; bias U(-1,1); dilation floor(2^x), x ~ U(0, log2((L-1)/(len-1)));
 * padding (len-1)d/2 with probability 1/2, else 0; floor(2^U(0, log2(min(C,len)+1))) channels
 * drawn without replacement.  Draws are made in fp64 by a counter-based generator (splitmix64
 * finaliser) and rounded once to fp32.  Needs K >= 1, C >= 1, L >= 11.  On success *out owns
 * the host arrays and the launch plan; release with rocket_params_destroy.
 */
int rocket_params_generate(uint64_t seed, int K, int C, int L, rocket_params_t** out);

/*
 * Adopt caller-supplied kernels (the arrays are copied; the caller keeps ownership of its own).
 * Requirements, else ROCKET_EINVAL: 1 <= length[k] <= 11; dilation[k] >= 1; padding[k] >= 0;
 * L_out,k >= 1; 1 <= num_channels[k] <= min(C, 11); channel indices of one kernel distinct and
 * in [0, C).  Any such kernel is accepted, up to L_out,k <= 2^30 (ROCKET_EUNSUPPORTED beyond);
 * kernels of length 7, 9 or 11 are served by the fused kernels (for C <= 20 channels and L >= 16),
 * every other kernel of the same handle by the generic ones, in every pass.
 */
int rocket_params_from_arrays(int K, int C, int L, const int32_t* length, const int32_t* dilation,
                              const int32_t* padding, const int32_t* num_channels,
                              const int32_t* channel_idx, const float* weights, const float* bias,
                              rocket_params_t** out);

/* Sizes of the handle's arrays.  Any output pointer may be NULL. */
int rocket_params_counts(const rocket_params_t* p, int* K, int* C, int* L, int64_t* n_channel_idx,
                         int64_t* n_weights);

/*
 * Read-only views of the handle's host arrays (valid until rocket_params_destroy), so that a
 * checker can consume exactly the numbers the device uses.  Any output pointer may be NULL.
 */
int rocket_params_host_view(const rocket_params_t* p, const int32_t** length, const int32_t** dilation,
                            const int32_t** padding, const int32_t** num_channels,
                            const int32_t** channel_idx, const float** weights, const float** bias);

/* Convolution work of one example under the explicit count 2*len*channels*L_out summed over
 * kernels (flop), and the number of conv outputs sum_k L_out,k.  Outputs may be NULL. */
int rocket_params_work(const rocket_params_t* p, double* conv_flops_per_example,
                       double* conv_outputs_per_example);

/*
 * Bind the handle to the current CUDA device now (upload its parameters) instead of at its
 * first device call.  Allocates device memory; a no-op returning ROCKET_OK when already bound.
 */
int rocket_params_bind_device(const rocket_params_t* p);

/*
 * Allocate, now, everything the device calls with this handle will need for up to max_N examples
 * per call, on the current device (binding the handle to it if it is not bound yet), so that the
 * calls themselves never allocate, free or synchronise.  passes is a bit set of the calls to
 * prepare for: ROCKET_PASS_HARD (rocket_transform), ROCKET_PASS_SOFT (rocket_transform_soft),
 * ROCKET_PASS_BACKWARD (rocket_transform_soft_backward) and ROCKET_PASS_U8_INPUT (the *_u8 forms of
 * the passes named).  May be called again with a larger max_N or more passes; never shrinks.  The
 * host-buffer forms (*_host) stage through buffers of their own and synchronise by design; they
 * are not covered.  ROCKET_EINVAL for max_N < 1 or an empty / unknown set of passes, ROCKET_ENOMEM
 * when the device memory does not suffice (what was allocated before stays usable).
 */
#define ROCKET_PASS_HARD 1
#define ROCKET_PASS_SOFT 2
#define ROCKET_PASS_BACKWARD 4
#define ROCKET_PASS_U8_INPUT 8
int rocket_params_reserve(rocket_params_t* p, int max_N, int passes);

/* Number of device allocations (cudaMalloc) the library has made in this process so far.  A
 * caller that must not allocate in its steady state reads it before and after a call. */
int64_t rocket_device_alloc_count(void);

/* Free the handle, its device copies and its workspace.  NULL is allowed.  The caller must
 * have synchronised any stream that still runs work enqueued with this handle. */
void rocket_params_destroy(rocket_params_t* p);

/*
 * Hard transform: PPV (Eq. 1-2, strict z > 0) and max for every (example, kernel).
 *   X_dev    [N][C][L] fp32, device (a 16-byte aligned base with L a multiple of 4 lets the staging copy
 *            move 16 bytes at a time; any other base or length works, one float at a time);  C and L must
 *            equal the handle's
 *   feat_dev [N][2K] fp32, device, written
 * N = 0 is a successful no-op.
 */
int rocket_transform(const rocket_params_t* p, const float* X_dev, int N, int C, int L, float* feat_dev,
                     void* cuda_stream);

/*
 * Hard transform in half precision (Section 5 of the paper names FP16 compute as a further speed-up).  Same
 * arguments and layout as rocket_transform.  What it computes: samples, weights and biases rounded to binary16
 * (nearest, ties to even); every conv output starts at the bias and takes one fused multiply-add per tap -
 * channels in the order of the kernel's channel list, taps 0 .. len - 1 - each rounded once to binary16; PPV
 * (strict) and max of those outputs, the max returned exactly, PPV as count / L_out in fp32.  Errors against the
 * FP32 transform are of the order of 1e-3 (PPV) and 1e-3 of the max; on this hardware the gain in speed is small
 * (packed half-precision and packed FP32 multiply-adds issue at the same rate).  Served by the fused kernels
 * only: ROCKET_EUNSUPPORTED when the handle has a kernel they do not take (a length other than 7, 9, 11, more
 * than 20 channels); ROCKET_EINVAL for a base that is not 4-byte aligned; samples beyond +-65504 overflow.
 */
int rocket_transform_f16(const rocket_params_t* p, const float* X_dev, int N, int C, int L, float* feat_dev,
                         void* cuda_stream);

/*
 * Soft transform: softPPV (Eq. 3-4) with softness lambda and shift (Eq. 3 as printed: shift =
 * +3; the accompanying prose describes shift = -3; both are valid arguments), and max.
 *   argmax_dev [N][K] int32, device, written when not NULL: the lowest output index attaining
 *              the max, the sub-gradient choice the backward pass uses.
 */
int rocket_transform_soft(const rocket_params_t* p, const float* X_dev, int N, int C, int L, float lambda,
                          float shift, float* feat_dev, int32_t* argmax_dev, void* cuda_stream);

/*
 * Backward of the soft transform for kernel weights and biases (the paper states that softPPV
 * lets gradients flow; this is the chain rule through Eq. 3-4 and the convolution):
 *   gz[n,k,i] = dfeat[n][2k] * (lambda / L_out) * h_i (1 - h_i) + dfeat[n][2k+1] * [i == argmax[n][k]]
 *   db[k]       = sum_n sum_i gz[n,k,i]
 *   dW_k[q][j]  = sum_n sum_i gz[n,k,i] * xpad[n, S_k[q], i - p_k + j d_k]
 *   dfeat_dev  [N][2K] fp32, device      argmax_dev [N][K] int32, device (from the soft forward)
 *   dW_dev     fp32, device, ragged exactly like the weights, assigned (not accumulated)
 *   db_dev     [K] fp32, device, assigned
 * No gradient with respect to X is produced.  N = 0 writes zeros.
 */
int rocket_transform_soft_backward(const rocket_params_t* p, const float* X_dev, int N, int C, int L,
                                   float lambda, float shift, const float* dfeat_dev,
                                   const int32_t* argmax_dev, float* dW_dev, float* db_dev,
                                   void* cuda_stream);

/*
 * Host-buffer convenience forms of the three passes: inputs and outputs are HOST pointers
 * (pinned memory makes the copies asynchronous, pageable memory works too).  The call copies the inputs to
 * device buffers kept inside the handle (grown on demand, ROCKET_ENOMEM if that fails), runs
 * the pass, copies the results back and returns after they have arrived (the forward forms upload
 * the batch in chunks on a second stream of the handle and start on a chunk as soon as it is there).  argmax_host may be
 * NULL in the forward; it is required in the backward.  These calls mutate the handle's
 * staging buffers: one such call per handle at a time.
 */
int rocket_transform_host(rocket_params_t* p, const float* X_host, int N, int C, int L, float* feat_host);
int rocket_transform_soft_host(rocket_params_t* p, const float* X_host, int N, int C, int L, float lambda,
                               float shift, float* feat_host, int32_t* argmax_host);
int rocket_transform_soft_backward_host(rocket_params_t* p, const float* X_host, int N, int C, int L,
                                        float lambda, float shift, const float* dfeat_host,
                                        const int32_t* argmax_host, float* dW_host, float* db_host);

/*
 * The transform of raw 8-bit sensor intensities (Section 4.1: integer light intensities 0..255)
 * under per-channel feature scaling (Section 4.3: every sensor channel is normalised on its own):
 *     x[n][c][i] = ((float)X_u8[n][c][i] - mean[c]) * inv_std[c]      (two fp32 operations)
 * followed by rocket_transform / rocket_transform_soft on x.  X_u8_dev is [N][C][L] bytes on the
 * device; mean and inv_std are HOST arrays of C floats (statistics of the training set, not of the
 * batch) and are read before the call returns; outputs, stream, ownership and errors as in the fp32
 * forms, plus ROCKET_EINVAL for a NULL or NaN statistic.  When every kernel of the handle is served
 * by the fused kernels (lengths 7/9/11, C <= 20), L is a multiple of 4 and X_u8_dev is 4-byte aligned, the
 * scaling happens while the kernels' staging copy of the batch is written and no fp32 copy of the
 * batch exists; otherwise the call first writes a scaled fp32 copy into a buffer of the handle
 * (grown with cudaMalloc on demand, ROCKET_ENOMEM if that fails) and takes the fp32 route.
 * The host form copies the bytes to the device inside the call (a quarter of the fp32 form's traffic).
 */
int rocket_transform_u8(const rocket_params_t* p, const uint8_t* X_u8_dev, int N, int C, int L, const float* mean,
                        const float* inv_std, float* feat_dev, void* cuda_stream);
int rocket_transform_soft_u8(const rocket_params_t* p, const uint8_t* X_u8_dev, int N, int C, int L, const float* mean,
                             const float* inv_std, float lambda, float shift, float* feat_dev, int32_t* argmax_dev,
                             void* cuda_stream);
int rocket_transform_u8_host(rocket_params_t* p, const uint8_t* X_u8_host, int N, int C, int L, const float* mean,
                             const float* inv_std, float* feat_host);

/*
 * The linear regressor on the pooled features (Section 3 step (3), Section 3.3: a ridge regressor on
 * the 2K features of every example), fitted and applied on the device so that the features of the
 * transform never leave it.
 *
 * rocket_ridge_fit: feat_dev [N][P] fp32 (row-major, P = 2K for the transform's output), y_dev [N]
 * fp32 targets, alpha >= 0 the penalty on the weights.  The intercept is fitted and not penalised:
 * with Fc, yc the column-centred features and targets, w minimises |Fc w - yc|^2 + alpha |w|^2 and
 * b = mean(y) - mean(F) . w.  Solved in its dual form (an N x N system, N <= ROCKET_RIDGE_MAX_EXAMPLES)
 * in double precision; w_dev [P] and b_dev [1] receive the result as fp32.  The call allocates its
 * workspace ((P + N*N + N) doubles) with cudaMalloc, frees it, and returns after the work on
 * cuda_stream has finished.  Errors: ROCKET_EINVAL for NULL pointers, N < 1, P < 1, a negative or
 * non-finite alpha, or a system that is not positive definite (alpha = 0 with dependent rows);
 * ROCKET_EUNSUPPORTED beyond the size limit; ROCKET_ENOMEM / ROCKET_ECUDA from the runtime.
 *
 * rocket_ridge_predict: yhat_dev[n] = b + sum_p feat_dev[n][p] w_dev[p] for n < N (products summed in
 * double), enqueued on cuda_stream, no allocation.  All pointers are device pointers on the current device.
 */
#define ROCKET_RIDGE_MAX_EXAMPLES 4096
int rocket_ridge_fit(const float* feat_dev, int N, int P, const float* y_dev, float alpha, float* w_dev, float* b_dev,
                     void* cuda_stream);
int rocket_ridge_predict(const float* feat_dev, int N, int P, const float* w_dev, const float* b_dev, float* yhat_dev,
                         void* cuda_stream);

/*
 * Replaces the weights and biases of the handle's kernels (host arrays laid out as
 * rocket_params_host_view returns them: n_weights ragged weights, K biases); lengths, dilations,
 * paddings and channels stay.  This is the step that makes the kernels trainable (the paper's
 * stated use of the soft PPV, Sections 1 and 6): rocket_transform_soft and
 * rocket_transform_soft_backward give the loss gradient for the current values, the caller's
 * optimiser produces new ones, this call installs them on the host and, if the handle is bound, on
 * its device (it waits for the device first).  ROCKET_EINVAL for NULL or non-finite values (nothing
 * is changed then).  Not to be called while another thread uses the handle.
 */
int rocket_params_set_weights(rocket_params_t* p, const float* weights, const float* bias);

/*
 * Which kernels serve the handle: 0 = automatic (fast path where it applies), 1 = force the
 * generic kernels.  For tests and measurements; returns ROCKET_EINVAL for other values.
 */
int rocket_params_set_path(rocket_params_t* p, int path);

/*
 * Device-side health of the handle.  Every wait inside the kernels (on a bulk-copy barrier) is
 * bounded; a wait that gives up sets a flag instead of hanging the GPU, and the results of that
 * call are then invalid.  This call synchronises the device, reads the flag into *wait_timeouts
 * (0 = healthy) and returns ROCKET_OK unless the read itself failed.
 */
int rocket_params_device_status(const rocket_params_t* p, int* wait_timeouts);

/*
 * Per-kernel timing of the hard transform, for benchmarks.  With profiling enabled, every
 * rocket_transform call through the fast path records CUDA events on the caller's stream around
 * its two fused kernels: the one that serves the small dilations (tiles shared by all kernels of
 * one dilation) and the one that serves the large dilations (one kernel per tile).
 * The batch goes through both kernels in chunks of a few examples; rocket_params_last_profile waits
 * for the last such call and returns the two durations, summed over the chunks, in milliseconds
 * (0 when nothing was recorded), and the convolution work of one example in either
 * kernel under the count 2*len*channels*L_out (flop).  Any output pointer may be NULL.
 */
int rocket_params_set_profiling(rocket_params_t* p, int enable);
int rocket_params_last_profile(const rocket_params_t* p, double* ms_small_dilations, double* ms_large_dilations,
                               double* flops_small_dilations, double* flops_large_dilations);

/* Number of device kernels this library has launched in this process so far. */
int64_t rocket_kernel_launch_count(void);

/*
 * Allocation-free form of rocket_transform_soft_backward.  (The paper has no counterpart; this
 * entry point exists for callers that are not allowed to allocate device memory.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a real-time control loop
 * that must not take the allocator's locks or its implicit device synchronisation, inside a
 * host process whose memory pool is fixed at start-up, or on a stream that another component is
 * recording.  rocket_transform_soft_backward keeps its per-example partial sums in a workspace
 * that it grows with cudaMalloc on demand; this form keeps them in a fixed array that is part
 * of the library image instead, so the call itself never allocates or frees anything.
 *
 * Same arguments, same results and same error rules as rocket_transform_soft_backward, plus:
 *   - The scratch array holds ROCKET_NOALLOC_MAX_SCRATCH_FLOATS floats (16 MiB).  Every GPU
 *     that loads the library carries it until the process exits.  The call needs
 *     N * (n_weights + K) floats of it and returns ROCKET_EUNSUPPORTED, launching nothing,
 *     when that is more than the array holds.
 *   - The handle must already be bound to its device (rocket_params_bind_device, or any
 *     earlier device call with it); binding allocates, so do it during set-up.  An unbound
 *     handle gives ROCKET_EINVAL.
 *   - The first call on each device looks up the array's device address.  With the runtime's
 *     lazy module loading that query, and the first launch of the kernels behind this call, may
 *     load the library's device code onto the GPU, which allocates and synchronises inside the
 *     driver.  So make one small call during set-up (N = 1 on any example will do: it runs the
 *     look-up and both kernels), before any stream capture and before the phase that must not
 *     allocate.
 *   - All calls on one device share the one array, and it keeps the previous call's contents.
 *     Nothing in it needs clearing: each call writes every element it later reads.  Two calls
 *     that overlap on the GPU (different streams, no event between them) race on it and give
 *     wrong gradients; order them on the device.
 */
#define ROCKET_NOALLOC_MAX_SCRATCH_FLOATS (4 * 1024 * 1024)
int rocket_transform_soft_backward_noalloc(const rocket_params_t* p, const float* X_dev, int N, int C, int L,
                                           float lambda, float shift, const float* dfeat_dev,
                                           const int32_t* argmax_dev, float* dW_dev, float* db_dev,
                                           void* cuda_stream);

/*
 * MINIROCKET (Section 2: the model that followed ROCKET - two-valued kernels from a fixed set, so that the
 * convolution needs additions only, biases sampled from the input data, PPV as the only pooled feature;
 * Section 6 names it as the extension of the GPU implementation).
 *
 * What the paper leaves open is fixed as follows.  Kernels: the 84 ways to give three of nine taps the weight
 * 2 and the other six -1.  num_features is rounded down to a multiple of 84 (10,000 -> 9,996); every kernel
 * owns the same number of features, spread over the distinct values of floor(2^x), x equally spaced on
 * [0, log2((L - 1) / 8)] (at most 32 of them; computed as floor(exp2(x) * (1 + 2^-40)) in double precision, so
 * that a power that is an integer - the largest is (L - 1) / 8 itself - is not lost to a rounding error).  Combination c = dilation_index * 84 + kernel_index owns the
 * features feature_offset[c] .. feature_offset[c + 1] - 1, has padding 4 d (outputs 0 .. L - 1) when
 * dilation_index + kernel_index is even and none otherwise (outputs 4 d .. L - 4 d - 1), and a random subset of
 * floor(2^U(0, log2(min(C, 9) + 1))) channels whose samples are summed before the convolution (the same
 * weights apply to every channel).  Feature f is
 *     #{ i : z_i > bias_f } / number of outputs,   z_i = sum_{c in S} sum_{j<9} w_j xpad[c][i + (j - 4) d]
 * and bias_f is the quantile frac((f + 1) / golden ratio) - linear interpolation between order statistics -
 * of the outputs of training example floor(example_draw[c] * N).
 *
 * rocket_mini_create   host only; *out owns the parameters (release with rocket_mini_destroy).  Needs C >= 1,
 *                      L >= 9, num_features >= 84 (ROCKET_EINVAL otherwise); C * L < 2^31
 *                      (ROCKET_EUNSUPPORTED beyond: positions within an example are 32-bit).
 * rocket_mini_fit      X_host [N][C][L] fp32 on the HOST; computes every bias (a one-off over one example per
 *                      combination, on the host's cores); returns when done.
 * rocket_mini_set_biases  installs biases computed elsewhere ([n_features] floats, host).
 * rocket_mini_transform   X_dev [N][C][L] fp32 and feat_dev [N][n_features] fp32 on the device; one fused kernel
 *                      on the caller's stream (convolution outputs never reach memory; any L, any 4-byte
 *                      aligned X_dev); the first call binds the handle to the current device, uploads its
 *                      parameters (one allocation) and opts the kernel into 64 KB of shared memory.  ROCKET_EINVAL before
 *                      a fit or set_biases; ROCKET_ESHAPE when C or L differ from the handle's.
 * rocket_mini_host_view   read-only views of the host arrays (taps [84][3], per combination: dilation,
 *                      kernel_index, padded, num_channels, ragged channel_idx, feature_offset [n + 1],
 *                      example_draw; per feature: quantile, bias); any output pointer may be NULL.
 */
typedef struct rocket_mini rocket_mini_t;
int rocket_mini_create(uint64_t seed, int C, int L, int num_features, rocket_mini_t** out);
int rocket_mini_counts(const rocket_mini_t* p, int* C, int* L, int* n_features, int* n_combinations,
                       int64_t* n_channel_idx);
int rocket_mini_host_view(const rocket_mini_t* p, const int32_t** taps, const int32_t** dilation,
                          const int32_t** kernel_index, const int32_t** padded, const int32_t** num_channels,
                          const int32_t** channel_idx, const int32_t** feature_offset, const double** example_draw,
                          const double** quantile, const float** bias);
int rocket_mini_fit(rocket_mini_t* p, const float* X_host, int N);
int rocket_mini_set_biases(rocket_mini_t* p, const float* bias);
int rocket_mini_transform(const rocket_mini_t* p, const float* X_dev, int N, int C, int L, float* feat_dev,
                          void* cuda_stream);
void rocket_mini_destroy(rocket_mini_t* p);

#ifdef __cplusplus
}
#endif
#endif /* ROCKET_B200_H */
