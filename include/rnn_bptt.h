/*
 * rnn_bptt.h - C ABI of the recurrent-network workload of arXiv 2002.03629 (Section 5.1 "Backpropagation
 * of RNNs"; appendix "Backpropagation" for the reduction to feedforward computation; appendix "Extra
 * Experimental Details: RNN" for the model): back-propagation through time as a triangular system,
 * solved by back-substitution or by n Jacobi iterations ("Jacobi_n", Algorithm 1 truncated).
 *
 * Model (one hidden layer, SoftPlus), per sequence, t = 1..T, h_0 = 0:
 *     a_t = W_h h_{t-1} + W_x x_t + b,   h_t = softplus(a_t),   y_t = W_o h_t + b_o,
 *     loss = 1/2 sum_t |y_t - r_t|^2                         (the loss touches every step)
 * Backward states s_t = d loss / d h_t with l_t = W_o^T (y_t - r_t) and d_t = sigmoid(a_t):
 *     s_T = l_T,   s_t = l_t + W_h^T (d_{t+1} * s_{t+1})     (Eq. 1 with the states taken from T downwards)
 * A Jacobi iteration evaluates the right-hand side for every t at once from the previous iterate; after n
 * iterations the last n states are exact (Proposition 1), all of them after T.
 *
 * Conventions.  Every pointer is a DEVICE pointer to fp32, row-major, owned by the caller; the calls are
 * asynchronous on `stream` (a cudaStream_t; NULL = the default stream) and allocate nothing.  Sequences of
 * a batch are independent (one thread block each).  Limits: 1 <= T <= 128, 1 <= H <= 128 with H a multiple
 * of 4, 1 <= d_in, d_out <= 16, B >= 1.  Return value: 0, RNN_ERR_INVALID (-1) for a null pointer or a size
 * outside the limits (nothing is launched), RNN_ERR_CUDA (-2) if the launch failed (rnn_last_error() names
 * the CUDA error).  Arithmetic: fp32 fused multiply-adds in a fixed order (results are reproducible run to
 * run); exp/log from the fast-math intrinsics are not used.
 */
#ifndef RNN_BPTT_H
#define RNN_BPTT_H

#ifdef __cplusplus
extern "C" {
#endif

#define RNN_OK 0
#define RNN_ERR_INVALID (-1)
#define RNN_ERR_CUDA (-2)
#define RNN_MAX_T 128
#define RNN_MAX_H 128
#define RNN_MAX_IO 16

/* Forward pass and everything the backward pass needs.
 *   Wh [H][H], Wx [H][d_in], b [H], Wo [d_out][H], bo [d_out]: parameters
 *   x [B][T][d_in] inputs, r [B][T][d_out] targets
 *   out: h [B][T][H] hidden states, d [B][T][H] activation derivatives sigmoid(a_t),
 *        l [B][T][H] direct gradients W_o^T (y_t - r_t), loss [B] */
int rnn_forward(const float *Wh, const float *Wx, const float *b, const float *Wo, const float *bo, const float *x,
                const float *r, int B, int T, int H, int d_in, int d_out, float *h, float *d, float *l, float *loss,
                void *stream);

/* Exact backward pass by back-substitution, last step first.  l, d [B][T][H] in, s [B][T][H] out. */
int rnn_bptt_sequential(const float *Wh, const float *l, const float *d, int B, int T, int H, float *s, void *stream);

/* Jacobi_n: n_iters >= 0 Jacobi iterations from the iterate s0 [B][T][H] (NULL: zeros).  n_iters >= T gives
 * the exact states whatever s0 is. */
int rnn_bptt_jacobi(const float *Wh, const float *l, const float *d, int B, int T, int H, int n_iters, const float *s0,
                    float *s, void *stream);

/* Parameter gradients of each sequence from its state gradients: with g_t = d_t * s_t,
 *   dWh [B][H][H] = sum_{t>=2} g_t h_{t-1}^T,  dWx [B][H][d_in] = sum_t g_t x_t^T,  db [B][H] = sum_t g_t. */
int rnn_param_grads(const float *s, const float *d, const float *h, const float *x, int B, int T, int H, int d_in,
                    float *dWh, float *dWx, float *db, void *stream);

/* Text of the last CUDA error seen by these calls in this process ("" if none). */
const char *rnn_last_error(void);

#ifdef __cplusplus
}
#endif
#endif
