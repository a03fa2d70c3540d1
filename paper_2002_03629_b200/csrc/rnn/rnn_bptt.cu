// Back-propagation through time of a one-layer recurrent network as a triangular system (arXiv 2002.03629,
// Section 5.1; appendix "Backpropagation"): forward pass, exact back-substitution, truncated Jacobi
// iterations (Algorithm 1) and the parameter gradients.  One thread block per sequence; fp32 fused
// multiply-adds in a fixed order.
//
// The Jacobi iteration is the only step with parallel slack: all T states at once, a [T x H] x [H x H]
// product per iteration, here a register-tiled product out of shared memory (the iterate, premultiplied by
// the activation derivative and shifted by one step, stays in shared memory between iterations, and so do
// the weights).  Back-substitution is a chain of T matrix-vector products with a column of W_h per thread
// in registers.
#include <cuda_runtime.h>

#include <cstdio>

#include "../../../include/rnn_bptt.h"

namespace {

constexpr int MT = RNN_MAX_T, MH = RNN_MAX_H, MIO = RNN_MAX_IO;

char g_err[256] = "";

int launch_status()
{
    const cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) return RNN_OK;
    snprintf(g_err, sizeof g_err, "%s", cudaGetErrorString(e));
    return RNN_ERR_CUDA;
}

__device__ __forceinline__ float softplus_f(float a) { return fmaxf(a, 0.0f) + log1pf(expf(-fabsf(a))); }
__device__ __forceinline__ float sigmoid_f(float a) { return 1.0f / (1.0f + expf(-a)); }

// ------------------------------------------------------------------ forward
// thread j owns hidden unit j: row j of W_h in registers, the previous state in shared memory
__global__ void __launch_bounds__(MH, 1)
rnn_forward_kernel(const float *__restrict__ Wh, const float *__restrict__ Wx, const float *__restrict__ b,
                   const float *__restrict__ Wo, const float *__restrict__ bo, const float *__restrict__ x,
                   const float *__restrict__ r, int T, int H, int d_in, int d_out, float *__restrict__ h,
                   float *__restrict__ d, float *__restrict__ l, float *__restrict__ loss)
{
    extern __shared__ float hs[];                       // [T][MH]: the hidden states, zero beyond H
    __shared__ float es[MT * MIO];                      // y_t - r_t
    __shared__ float red[MH];
    const int j = threadIdx.x, seq = blockIdx.x;
    const bool on = j < H;
    float w[MH], wx[MIO];
#pragma unroll
    for (int i = 0; i < MH; ++i) w[i] = (on && i < H) ? Wh[(size_t)j * H + i] : 0.0f;
#pragma unroll
    for (int c = 0; c < MIO; ++c) wx[c] = (on && c < d_in) ? Wx[(size_t)j * d_in + c] : 0.0f;
    const float bj = on ? b[j] : 0.0f;
    const float *xs = x + (size_t)seq * T * d_in;
    for (int t = 0; t < T; ++t) {
        float a = bj;
        for (int c = 0; c < d_in; ++c) a = fmaf(wx[c], xs[(size_t)t * d_in + c], a);
        if (t > 0) {
            const float4 *hp = reinterpret_cast<const float4 *>(hs + (size_t)(t - 1) * MH);
#pragma unroll
            for (int i = 0; i < MH / 4; ++i) {
                const float4 v = hp[i];
                a = fmaf(w[4 * i], v.x, a);
                a = fmaf(w[4 * i + 1], v.y, a);
                a = fmaf(w[4 * i + 2], v.z, a);
                a = fmaf(w[4 * i + 3], v.w, a);
            }
        }
        const float hv = on ? softplus_f(a) : 0.0f;
        hs[(size_t)t * MH + j] = hv;
        if (on) {
            const size_t o = ((size_t)seq * T + t) * H + j;
            h[o] = hv;
            d[o] = sigmoid_f(a);
        }
        __syncthreads();
    }
    // outputs, residuals and the loss
    float part = 0.0f;
    for (int p = j; p < T * d_out; p += MH) {
        const int t = p / d_out, o = p % d_out;
        float y = bo[o];
        for (int i = 0; i < H; ++i) y = fmaf(Wo[(size_t)o * H + i], hs[(size_t)t * MH + i], y);
        const float e = y - r[((size_t)seq * T + t) * d_out + o];
        es[t * MIO + o] = e;
        part = fmaf(0.5f * e, e, part);
    }
    red[j] = part;
    __syncthreads();
    for (int w2 = MH / 2; w2 > 0; w2 >>= 1) {
        if (j < w2) red[j] += red[j + w2];
        __syncthreads();
    }
    if (j == 0) loss[seq] = red[0];
    // direct gradients l_t = W_o^T (y_t - r_t)
    if (on) {
        float wo[MIO];
#pragma unroll
        for (int o = 0; o < MIO; ++o) wo[o] = o < d_out ? Wo[(size_t)o * H + j] : 0.0f;
        for (int t = 0; t < T; ++t) {
            float v = 0.0f;
#pragma unroll
            for (int o = 0; o < MIO; ++o)
                if (o < d_out) v = fmaf(wo[o], es[t * MIO + o], v);
            l[((size_t)seq * T + t) * H + j] = v;
        }
    }
}

// ------------------------------------------------------------------ exact back-substitution
// thread i owns component i of the states: column i of W_h in registers
__global__ void __launch_bounds__(MH, 1)
rnn_bptt_sequential_kernel(const float *__restrict__ Wh, const float *__restrict__ l, const float *__restrict__ d,
                           int T, int H, float *__restrict__ s)
{
    __shared__ __align__(16) float u[2][MH];            // d_{t+1} * s_{t+1}
    const int i = threadIdx.x, seq = blockIdx.x;
    const bool on = i < H;
    float wc[MH];
#pragma unroll
    for (int j = 0; j < MH; ++j) wc[j] = (on && j < H) ? Wh[(size_t)j * H + i] : 0.0f;
    const size_t base = (size_t)seq * T * H;
    u[0][i] = 0.0f;
    u[1][i] = 0.0f;
    float ln = on ? l[base + (size_t)(T - 1) * H + i] : 0.0f, dn = on ? d[base + (size_t)(T - 1) * H + i] : 0.0f;
    __syncthreads();
    for (int t = T - 1; t >= 0; --t) {
        const float lt = ln, dt = dn;
        if (t > 0 && on) {                               // the next step's operands while this one computes
            ln = l[base + (size_t)(t - 1) * H + i];
            dn = d[base + (size_t)(t - 1) * H + i];
        }
        float acc = lt;
        if (t < T - 1) {
            const float4 *up = reinterpret_cast<const float4 *>(u[(t + 1) & 1]);
#pragma unroll
            for (int j = 0; j < MH / 4; ++j) {
                const float4 v = up[j];
                acc = fmaf(wc[4 * j], v.x, acc);
                acc = fmaf(wc[4 * j + 1], v.y, acc);
                acc = fmaf(wc[4 * j + 2], v.z, acc);
                acc = fmaf(wc[4 * j + 3], v.w, acc);
            }
        }
        if (on) {
            s[base + (size_t)t * H + i] = acc;
            u[t & 1][i] = dt * acc;
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------ Jacobi iterations
// 512 threads; thread (lane = tid % 32, wy = tid / 32) owns the states t = 4 lane .. 4 lane + 3, components
// i = 8 wy .. 8 wy + 7.  VT[buf][k][t] = d_{t+1}[k] * s_{t+1}[k] of the current iterate (zero where t + 1 >= T
// or k >= H), so that  s_new[t][i] = l[t][i] + sum_k VT[k][t] * W_h[k][i].
constexpr int JT = 512;
constexpr int VS = MT;                                   // row stride of VT
constexpr size_t JACOBI_SMEM = (size_t)(2 * MH * VS + MH * MH) * sizeof(float);

__global__ void __launch_bounds__(JT, 1)
rnn_bptt_jacobi_kernel(const float *__restrict__ Wh, const float *__restrict__ l, const float *__restrict__ d,
                       int T, int H, int n_iters, const float *__restrict__ s0, float *__restrict__ s)
{
    extern __shared__ __align__(16) float sm[];
    float *VT = sm;                                      // [2][MH][VS]
    float *W = sm + 2 * MH * VS;                         // [MH][MH], W[k][i] = W_h[k][i], zero beyond H
    const int tid = threadIdx.x, lane = tid & 31, wy = tid >> 5, seq = blockIdx.x;
    const size_t base = (size_t)seq * T * H;
    for (int p = tid; p < 2 * MH * VS; p += JT) VT[p] = 0.0f;
    for (int p = tid; p < MH * MH; p += JT) {
        const int k = p / MH, i = p % MH;
        W[p] = (k < H && i < H) ? Wh[(size_t)k * H + i] : 0.0f;
    }
    __syncthreads();
    if (s0 != nullptr)
        for (int p = tid; p < (T - 1) * H; p += JT) {
            const int t = p / H, k = p % H;              // column t holds step t + 1
            VT[k * VS + t] = d[base + (size_t)(t + 1) * H + k] * s0[base + (size_t)(t + 1) * H + k];
        }
    if (n_iters <= 0) {
        for (int p = tid; p < T * H; p += JT) s[base + p] = s0 != nullptr ? s0[base + p] : 0.0f;
        return;
    }
    float cl[4][8], dd[4][8];
#pragma unroll
    for (int rr = 0; rr < 4; ++rr)
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const int t = 4 * lane + rr, i = 8 * wy + c;
            const bool in = t < T && i < H;
            cl[rr][c] = in ? l[base + (size_t)t * H + i] : 0.0f;
            dd[rr][c] = in ? d[base + (size_t)t * H + i] : 0.0f;
        }
    __syncthreads();
    for (int it = 0; it < n_iters; ++it) {
        const float *cur = VT + (size_t)(it & 1) * MH * VS;
        float *nxt = VT + (size_t)((it + 1) & 1) * MH * VS;
        float acc[4][8];
#pragma unroll
        for (int rr = 0; rr < 4; ++rr)
#pragma unroll
            for (int c = 0; c < 8; ++c) acc[rr][c] = cl[rr][c];
#pragma unroll 4
        for (int k = 0; k < H; ++k) {
            const float4 a = *reinterpret_cast<const float4 *>(cur + (size_t)k * VS + 4 * lane);
            const float4 w0 = *reinterpret_cast<const float4 *>(W + (size_t)k * MH + 8 * wy);
            const float4 w1 = *reinterpret_cast<const float4 *>(W + (size_t)k * MH + 8 * wy + 4);
            const float av[4] = {a.x, a.y, a.z, a.w};
            const float wv[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
            for (int rr = 0; rr < 4; ++rr)
#pragma unroll
                for (int c = 0; c < 8; ++c) acc[rr][c] = fmaf(av[rr], wv[c], acc[rr][c]);
        }
        const bool last = it + 1 == n_iters;
#pragma unroll
        for (int rr = 0; rr < 4; ++rr)
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const int t = 4 * lane + rr, i = 8 * wy + c;
                if (t < T && i < H) {
                    if (last) s[base + (size_t)t * H + i] = acc[rr][c];
                    else if (t >= 1) nxt[(size_t)i * VS + t - 1] = dd[rr][c] * acc[rr][c];
                }
            }
        __syncthreads();
    }
}

// ------------------------------------------------------------------ parameter gradients
// 256 threads; thread (tx = tid % 16, ty = tid / 16) owns dWh[8 ty .. +7][8 tx .. +7]
__global__ void __launch_bounds__(256, 1)
rnn_param_grads_kernel(const float *__restrict__ s, const float *__restrict__ d, const float *__restrict__ h,
                       const float *__restrict__ x, int T, int H, int d_in, float *__restrict__ dWh,
                       float *__restrict__ dWx, float *__restrict__ db)
{
    extern __shared__ __align__(16) float sm[];
    float *g = sm;                                       // [T][MH]  d_t * s_t
    float *hh = sm + (size_t)MT * MH;                    // [T][MH]
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4, seq = blockIdx.x;
    const size_t base = (size_t)seq * T * H;
    for (int p = tid; p < T * MH; p += 256) {
        const int t = p / MH, i = p % MH;
        const bool in = i < H;
        g[p] = in ? d[base + (size_t)t * H + i] * s[base + (size_t)t * H + i] : 0.0f;
        hh[p] = in ? h[base + (size_t)t * H + i] : 0.0f;
    }
    __syncthreads();
    float acc[8][8];
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[a][c] = 0.0f;
    for (int t = 1; t < T; ++t) {
        const float4 g0 = *reinterpret_cast<const float4 *>(g + (size_t)t * MH + 8 * ty);
        const float4 g1 = *reinterpret_cast<const float4 *>(g + (size_t)t * MH + 8 * ty + 4);
        const float4 h0 = *reinterpret_cast<const float4 *>(hh + (size_t)(t - 1) * MH + 8 * tx);
        const float4 h1 = *reinterpret_cast<const float4 *>(hh + (size_t)(t - 1) * MH + 8 * tx + 4);
        const float gv[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
        const float hv[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
#pragma unroll
        for (int a = 0; a < 8; ++a)
#pragma unroll
            for (int c = 0; c < 8; ++c) acc[a][c] = fmaf(gv[a], hv[c], acc[a][c]);
    }
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const int j = 8 * ty + a, i = 8 * tx + c;
            if (j < H && i < H) dWh[((size_t)seq * H + j) * H + i] = acc[a][c];
        }
    if (tid < H) {
        float sb = 0.0f;
        for (int t = 0; t < T; ++t) sb += g[(size_t)t * MH + tid];
        db[(size_t)seq * H + tid] = sb;
        for (int c = 0; c < d_in; ++c) {
            float sx = 0.0f;
            for (int t = 0; t < T; ++t) sx = fmaf(g[(size_t)t * MH + tid], x[((size_t)seq * T + t) * d_in + c], sx);
            dWx[((size_t)seq * H + tid) * d_in + c] = sx;
        }
    }
}

bool sizes_ok(int B, int T, int H) { return B >= 1 && T >= 1 && T <= MT && H >= 1 && H <= MH && H % 4 == 0; }

template <typename K>
bool allow_smem(K kernel, size_t bytes)
{
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) {
        launch_status();
        return false;
    }
    return true;
}

}  // namespace

extern "C" {

int rnn_forward(const float *Wh, const float *Wx, const float *b, const float *Wo, const float *bo, const float *x,
                const float *r, int B, int T, int H, int d_in, int d_out, float *h, float *d, float *l, float *loss,
                void *stream)
{
    if (!Wh || !Wx || !b || !Wo || !bo || !x || !r || !h || !d || !l || !loss) return RNN_ERR_INVALID;
    if (!sizes_ok(B, T, H) || d_in < 1 || d_in > MIO || d_out < 1 || d_out > MIO) return RNN_ERR_INVALID;
    const size_t smem = (size_t)T * MH * sizeof(float);
    if (!allow_smem(rnn_forward_kernel, smem)) return RNN_ERR_CUDA;
    rnn_forward_kernel<<<B, MH, smem, (cudaStream_t)stream>>>(Wh, Wx, b, Wo, bo, x, r, T, H, d_in, d_out, h, d, l, loss);
    return launch_status();
}

int rnn_bptt_sequential(const float *Wh, const float *l, const float *d, int B, int T, int H, float *s, void *stream)
{
    if (!Wh || !l || !d || !s || !sizes_ok(B, T, H)) return RNN_ERR_INVALID;
    rnn_bptt_sequential_kernel<<<B, MH, 0, (cudaStream_t)stream>>>(Wh, l, d, T, H, s);
    return launch_status();
}

int rnn_bptt_jacobi(const float *Wh, const float *l, const float *d, int B, int T, int H, int n_iters, const float *s0,
                    float *s, void *stream)
{
    if (!Wh || !l || !d || !s || !sizes_ok(B, T, H) || n_iters < 0) return RNN_ERR_INVALID;
    if (!allow_smem(rnn_bptt_jacobi_kernel, JACOBI_SMEM)) return RNN_ERR_CUDA;
    rnn_bptt_jacobi_kernel<<<B, JT, JACOBI_SMEM, (cudaStream_t)stream>>>(Wh, l, d, T, H, n_iters, s0, s);
    return launch_status();
}

int rnn_param_grads(const float *s, const float *d, const float *h, const float *x, int B, int T, int H, int d_in,
                    float *dWh, float *dWx, float *db, void *stream)
{
    if (!s || !d || !h || !x || !dWh || !dWx || !db || !sizes_ok(B, T, H) || d_in < 1 || d_in > MIO) return RNN_ERR_INVALID;
    const size_t smem = (size_t)2 * MT * MH * sizeof(float);
    if (!allow_smem(rnn_param_grads_kernel, smem)) return RNN_ERR_CUDA;
    rnn_param_grads_kernel<<<B, 256, smem, (cudaStream_t)stream>>>(s, d, h, x, T, H, d_in, dWh, dWx, db);
    return launch_status();
}

const char *rnn_last_error(void) { return g_err; }

}  // extern "C"
