/*
 * jacobi_sample.h - C ABI of the parallel autoregressive sampler for NVIDIA B200.
 *
 * The library draws samples x_1..x_T from a masked autoregressive network by
 * solving the triangular system  x_t = h_t(u, x_{1:t-1}),  t = 1..T  (Eq. 1 and
 * Eq. 5 of arXiv 2002.03629) with the random numbers u drawn beforehand by the
 * caller (Appendix A.3).  Solvers: nonlinear Jacobi (Algorithm 1), Gauss-Seidel
 * (Eq. 4; one sweep is the ordinary feedforward pass, Section 3.2) and the two
 * block hybrids Jacobi-GS (Algorithm 2) and GS-Jacobi (Algorithm 3).  Every
 * solver returns exactly the feedforward sample (Propositions 1 and 2).
 *
 * Conventions
 *   - Pointers named *_dev are DEVICE pointers owned by the caller; pointers in
 *     the model descriptors are HOST pointers, read during the create call only.
 *   - Calls enqueue their work on `cuda_stream` (a cudaStream_t passed as
 *     void*, NULL = default stream) and synchronise that stream before they
 *     return, so outputs are complete and the return value is final.
 *   - Return value: 0 = done and converged; JS_NOT_CONVERGED (1) = max_iters
 *     reached while some sample still changed, outputs hold the last iterate;
 *     negative = error, outputs unspecified.  No exceptions, no exit().
 *   - One call at a time per model (the model owns the activation scratch).
 *   - Positions are 0-based here (the paper counts from 1).  Symbols are bytes:
 *     0/1 for binary positions, 0..C-1 for C-way positions.
 *   - There is no CPU fallback: without a CUDA device every call fails with
 *     JS_ERR_CUDA.
 */
#ifndef JACOBI_SAMPLE_H
#define JACOBI_SAMPLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct js_model js_model;   /* opaque; library-owned device memory */

/* solver selection; the block hybrid with blocks in order and Jacobi inside (Algorithm 3) is
 * JS_GS_JACOBI, the one with all blocks in parallel and a sweep inside (Algorithm 2) JS_JACOBI_GS */
typedef enum { JS_JACOBI = 0, JS_GAUSS_SEIDEL = 1, JS_GS_JACOBI = 2, JS_JACOBI_GS = 3 } js_mode;

/* how u_t turns the conditional's logits z_t into x_t (Appendix A.3):
 *   UNIFORM_ICDF  x = [u < sigmoid(z)]      noise [batch][T]      in (0,1)
 *   LOGISTIC      x = [z + eps > 0]         noise [batch][T]      logistic
 *   GUMBEL        x = argmax_c (z_c + g_c)  noise [batch][T][C]   Gumbel(0,1), lowest index wins ties
 *   UNIFORM_CAT   x = first class c with u < F_c, F_c = sum_{i<=c} softmax(z)_i (inverse CDF of a C-way
 *                 position)                 noise [batch][T]      in (0,1); one number per position, so
 *                 1/C of the noise bytes of GUMBEL */
typedef enum { JS_NOISE_UNIFORM_ICDF = 0, JS_NOISE_LOGISTIC = 1, JS_NOISE_GUMBEL = 2, JS_NOISE_UNIFORM_CAT = 3 } js_noise_kind;
typedef enum { JS_ACT_RELU = 0, JS_ACT_GELU_TANH = 1 } js_act;
/* JS_F32: fp32 weights and activations.  JS_BF16: weights rounded to bf16 after
 * masking, hidden activations rounded to bf16 after bias and nonlinearity,
 * fp32 accumulation, fp32 logits. */
typedef enum { JS_F32 = 0, JS_BF16 = 1 } js_prec;

enum {
    JS_OK = 0,
    JS_NOT_CONVERGED = 1,
    JS_ERR_ARG = -1,          /* null pointer, bad enum, batch > max_batch, ... */
    JS_ERR_UNSUPPORTED = -2,  /* shape or mode the kernels do not cover */
    JS_ERR_CUDA = -3,         /* a CUDA runtime call failed (js_last_cuda_error) */
    JS_ERR_TIMEOUT = -4       /* a bounded device-side wait gave up; model stays usable */
};

/* Masked MLP (MADE).  Widths n = (T, H[0..L-1], T*C).  Input position d has
 * degree d+1, output (d, c) has degree d+1, hidden unit j of a layer of width H
 * has degree 1 + floor(j*(T-1)/H) unless hidden_deg gives it.  Hidden units read
 * units of the layer below with degree <= their own, outputs read hidden units
 * of strictly smaller degree, so position d depends on positions < d only.
 * The library applies the masks and the rounding itself. */
typedef struct {
    int T;                         /* positions */
    int C;                         /* logits per position: 1 = binary, else classes (<= 256) */
    int L;                         /* hidden layers, 1..8 */
    const int *H;                  /* [L] hidden widths */
    int act;                       /* js_act */
    int prec;                      /* js_prec */
    const float *const *W;         /* [L+1] host pointers, W[l] unmasked [n[l+1]][n[l]] row-major */
    const float *const *b;         /* [L+1] host pointers, b[l] [n[l+1]] */
    const float *lut;              /* [n_lut] network input for symbol value v */
    int n_lut;                     /* 2 for binary, C otherwise */
    const int *const *hidden_deg;  /* NULL, or [L] host arrays of degrees (1..T-1) */
    int max_batch;                 /* scratch is sized for this many samples */
} js_made_desc;

/* Masked-convolution stack (PixelCNN style): n_conv masked 3x3 convolutions
 * with ReLU and zero padding, then a 1x1 head.  Image [height][width][in_ch],
 * position t = (y*width + x)*in_ch + c.  Hidden channel k is in colour group
 * floor(in_ch*k/ch).  Kernels keep the row above and the left neighbour; at the
 * centre tap layer 0 keeps input groups < output group (type A), later layers
 * groups <= (type B); the head gives sub-pixel c its C logits from groups <= c.
 * W[0] [ch][3][3][in_ch], W[1..n_conv-1] [ch][3][3][ch], W[n_conv] [in_ch*C][ch]. */
typedef struct {
    int height, width, in_ch, ch, n_conv, C;
    int prec;                      /* js_prec */
    const float *const *W;         /* [n_conv+1] host pointers */
    const float *const *b;         /* [n_conv+1] host pointers */
    const float *lut;              /* [C] */
    int n_lut;
    int max_batch;
} js_conv_desc;

int js_made_create(const js_made_desc *desc, js_model **out);
int js_conv_create(const js_conv_desc *desc, js_model **out);
void js_model_destroy(js_model *m);

/*
 * Solve for all positions at once (Algorithms 1-3).
 *   noise_dev        fp32, layout by `nk` above; the same values serve every iteration
 *   init_dev         uint8 [batch][T] start iterate s^0, NULL = zeros; may alias out_samples_dev
 *   mode, block      block = B, the number of consecutive positions per block, for the hybrids
 *   max_iters        <= 0: the algorithm's own cap (T for Jacobi, |B_i| per block for
 *                    GS-Jacobi, number of blocks for Jacobi-GS); otherwise that cap lowered
 *   out_samples_dev  uint8 [batch][T]
 *   out_iters_dev    int32 [batch] (may be NULL): iteration at which the sample's forward
 *                    difference vanished, the confirming iteration included, or the cap;
 *                    GS-Jacobi: summed over blocks; Jacobi-GS: outer iterations; Gauss-Seidel: 1
 * A sample whose iterate did not change in an iteration is at its fixed point and stops
 * counting; the call ends when every sample has stopped or the cap is reached.
 */
int jacobi_sample(const js_model *m, int batch, const float *noise_dev, int nk,
                  const uint8_t *init_dev, int mode, int block, int max_iters,
                  uint8_t *out_samples_dev, int32_t *out_iters_dev, void *cuda_stream);

/*
 * The same solve (Algorithms 1-3) for callers whose noise and samples live in HOST memory.
 *   noise_host        fp32, same layout as noise_dev above; pinned memory makes the upload
 *                     asynchronous, pageable memory works too
 *   init_host         uint8 [batch][T] or NULL (zeros)
 *   out_samples_host  uint8 [batch][T]; out_iters_host int32 [batch] or NULL
 * The library owns the device-side staging buffers (allocated on the first call of a model,
 * sized for its max_batch) and a copy stream.  The upload of the noise runs beside the first
 * hidden layers: noise is not needed before the first sampling step (Appendix A.3: it only
 * turns the conditional of a position into a symbol), and the tensor-core kernel waits
 * (bounded) for it there; the other kernels start after the upload.  The call returns when
 * the samples are in out_samples_host.  Return codes as jacobi_sample; the caller's buffers
 * are only read (noise, init) or written (samples, iters) during the call.
 */
int jacobi_sample_host(const js_model *m, int batch, const float *noise_host, int nk,
                       const uint8_t *init_host, int mode, int block, int max_iters,
                       uint8_t *out_samples_host, int32_t *out_iters_host, void *cuda_stream);

/* Strict feedforward order (Eq. 1): T steps, each a forward pass of the same kernels of
 * which one position is kept. */
int sequential_sample(const js_model *m, int batch, const float *noise_dev, int nk,
                      uint8_t *out_samples_dev, void *cuda_stream);

/* Logits of every position for given symbols x (teacher forcing): logits_dev fp32
 * [batch][T][C].  For parity checks of the network itself. */
int js_forward_logits(const js_model *m, int batch, const uint8_t *x_dev, float *logits_dev,
                      void *cuda_stream);

/*
 * Continuous states with logistic conditionals (the paper's MADE: Section 5.3.1, Appendix C.3).  The model is
 * a masked MLP created with C = 2 (n_lut = 2, the table is not used): the states x_t are real numbers, the
 * network reads the states themselves (rounded to bf16 in a JS_BF16 model, like any activation) and gives
 * position t a location m_t (logit 2t) and a log-scale l_t (logit 2t+1) from x_{<t};
 *     x_t = m_t + exp(l_t) * noise_t,    noise_t = logit(u_t)   (inverse CDF of the logistic law, Appendix A.3)
 *   noise_dev        fp32 [batch][T], logistic numbers (as for JS_NOISE_LOGISTIC)
 *   init_dev         fp32 [batch][T] start iterate s^0, or NULL (zeros)
 *   eps              >= 0: a sample stops at the first iteration whose largest change max_t |x^k_t - x^{k-1}_t|
 *                    is <= eps (forward-difference rule of Section 2.2.1 in the maximum norm) or at the
 *                    algorithm's cap; eps = 0 gives the exact feedforward result (Proposition 1), eps > 0
 *                    trades error for iterations
 *   out_states_dev   fp32 [batch][T];  out_iters_dev as in jacobi_sample
 * Modes JS_JACOBI, JS_GAUSS_SEIDEL and JS_GS_JACOBI (JS_JACOBI_GS: JS_ERR_UNSUPPORTED).  CUDA-core kernels.
 * js_forward_logits_real gives the [batch][T][2] outputs of the network for given states.
 */
int jacobi_sample_real(const js_model *m, int batch, const float *noise_dev, const float *init_dev, int mode,
                       int block, int max_iters, float eps, float *out_states_dev, int32_t *out_iters_dev,
                       void *cuda_stream);
int sequential_sample_real(const js_model *m, int batch, const float *noise_dev, float *out_states_dev,
                           void *cuda_stream);
int js_forward_logits_real(const js_model *m, int batch, const float *x_dev, float *logits_dev, void *cuda_stream);

typedef enum {
    JS_OPT_FRONTIER_SKIP = 0,  /* 1 (default): skip positions and hidden units already final (proof of Prop. 1) */
    JS_OPT_SEQ_SKIP = 1,       /* how sequential_sample and JS_GAUSS_SEIDEL walk the strict order.  0: a full forward pass per
                                  position; 1: per position only the tiles of the band that changed; 2 (default): the cached
                                  sweep, every hidden unit evaluated once (Section 4.2; binary bf16 masked MLPs with sorted
                                  degrees - other models take 0) */
    JS_OPT_SPIN_LIMIT = 2,     /* polls before a device-side wait gives up (default 1<<22) */
    JS_OPT_PATH = 3,           /* 0 (default): tensor-core kernels where the model allows; 1: CUDA-core kernels only */
    JS_OPT_COMPACT = 4,        /* 1 (default): move finished samples out of the working batch */
    JS_OPT_TRACE = 5           /* 0 (default); 1: record device timestamps of the next calls (js_get_trace) for the
                                  first and the last CTA; n >= 2: for the first CTA and CTA n - 2 */
} js_option;
int js_set_option(js_model *m, int option, int value);

/* counters of the most recent sampling call on this model */
typedef struct {
    int iterations;            /* forward passes executed; outer iterations for Jacobi-GS on the tensor cores (micro-steps
                                  on the CUDA-core kernels); 1 for the cached sweep */
    int batch_iters_max;       /* largest per-sample iteration count */
    int final_frontier;        /* leading positions known final when the loop ended */
    long long tiles_issued;    /* output tiles computed */
    long long tiles_skipped;   /* output tiles skipped as final, finished or masked */
    int path;                  /* 0 tensor-core kernels, 1 CUDA-core kernels */
    int status;                /* the call's return value */
    int compactions;           /* times finished samples were moved out of the working batch */
    long long mma_flops;       /* tensor-core kernels: flops of the MMA instructions issued (tile padding included) */
    long long weight_bytes;    /* tensor-core kernels: weight bytes the call had to stream (each weight tile counted once per pass) */
} js_stats;
int js_get_stats(const js_model *m, js_stats *out);

/* Device-side timeline of the most recent call made with JS_OPT_TRACE on (tensor-core kernels):
 * globaltimer nanoseconds, layout [2][256][12] = [first CTA, last (or chosen) CTA][phase][slot]; a phase is one
 * layer of one forward pass; slots: 0 phase start, 1 first operands landed, 2 last MMA issued,
 * 3 accumulator complete, 4 epilogue stored, 5 left the grid barrier, 6-11 points inside the
 * epilogue; 0 = not recorded.
 * Copies at most `capacity` values to the HOST array `out`, returns how many. */
int js_get_trace(const js_model *m, unsigned long long *out, int capacity);

const char *js_strerror(int code);
const char *js_last_cuda_error(void);   /* text of the last failed CUDA call on this thread */

/*
 * jacobi_sample_noalloc - JS_JACOBI sampling of a small fp32 masked MLP without any
 * device-memory allocation.  The paper has no counterpart for this entry point; it exists
 * for callers that are not allowed to call cudaMalloc when they sample (a real-time loop
 * that must not block on the allocator, a process whose device memory belongs to another
 * framework's pool), and who therefore cannot use js_made_create.
 *
 * The caller owns and passes everything: the UNMASKED fp32 weights W_dev[l] [n[l+1]][n[l]],
 * biases b_dev[l] and the input table lut_dev as DEVICE pointers (masks of the default
 * degree rule are applied on the fly; there are no custom degrees), the noise, the optional
 * start iterate and the outputs, with the layouts of jacobi_sample.  All other memory the
 * kernel needs is one fixed device array inside the library, js_noalloc_scratch_limit()
 * bytes (4 MiB), which every GPU that loads the library holds until the process exits.
 * A shape whose scratch (js_noalloc_scratch_needed) exceeds it is rejected with JS_ERR_ARG
 * and a message in js_noalloc_last_error().  The call itself makes no cudaMalloc/cudaFree
 * and calls no allocating library routine.
 *
 * All calls share the one array and find the previous call's contents in it; the kernel
 * clears what must start at zero.  Calls that overlap on the GPU race on it: serialise them.
 * The first call on each device looks up the array's device address (with that device
 * current); it is also the call on which the driver loads this library's device code and
 * the array onto that GPU, which may take the driver's allocator once.  So make one warm-up
 * call per device at start-up, before the phase that must not allocate and before any
 * stream capture begins.  The array of the CURRENT device serves the call: cuda_stream must
 * belong to that device.  Every call copies a status word back and synchronises cuda_stream
 * before it returns.  Runs on one CTA: meant for small models.  Results equal
 * jacobi_sample(..., JS_JACOBI, ...) on the same fp32 model: same samples, same out_iters,
 * same return codes (0, JS_NOT_CONVERGED, negative on error).  A position whose scores are
 * all NaN or -inf gets class 0.
 */
typedef struct {
    int T, C, L;
    int H[8];
    int act;                    /* js_act */
    const float *W_dev[9];      /* device pointers, l = 0..L */
    const float *b_dev[9];
    const float *lut_dev;       /* device pointer, 2 entries (binary) or C entries */
} js_noalloc_made;

int jacobi_sample_noalloc(const js_noalloc_made *net, int batch, const float *noise_dev, int nk,
                          const uint8_t *init_dev, int max_iters, uint8_t *out_samples_dev,
                          int32_t *out_iters_dev, void *cuda_stream);
size_t js_noalloc_scratch_limit(void);
size_t js_noalloc_scratch_needed(const js_noalloc_made *net, int batch);
const char *js_noalloc_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* JACOBI_SAMPLE_H */
