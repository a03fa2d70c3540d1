// CUDA-core path of the masked-MLP sampler: one persistent cooperative kernel
// that runs the whole solver (Algorithms 1-3 of arXiv 2002.03629, or the strict
// feedforward order of Eq. 1) on the device.  It serves fp32 models, shapes the
// tensor-core path does not cover, and the fine-grained sweeps of Jacobi-GS.
//
// Every CTA executes the same driver loop; decisions are taken from values all
// CTAs read identically after a grid barrier, so control flow never diverges
// between CTAs.  Each output value is accumulated in a fixed order over k that
// does not depend on what else is skipped, so h_t is the same function in every
// iteration (the convergence proofs need that).
#include <limits.h>

#include "js_common.cuh"
#include "made_driver.cuh"

namespace {

constexpr int GT = JS_GT;      // 64x64 output tile
constexpr int KC = 32;         // k chunk staged in shared memory
constexpr int NTHREADS = 256;

struct Smem {
    alignas(16) float As[KC][GT + 4];       // read as float4: rows of GT + 4 floats keep every group of four on 16 bytes
    alignas(16) float Bs[KC][GT + 4];
    int list[4096];            // Jacobi-GS: units to evaluate in this micro-step
    int list_n;
    int wcnt[NTHREADS / 32];
};

// One 64x64 tile of  out = A[batch][K] * W[N][K]^T  over k in [0, kend).
template <typename T>
__device__ void gemm_tile(Smem &s, const T *A, int lda, const T *__restrict__ W, int ldw,
                          int M, int N, int kend, int m0, int n0, float (&acc)[4][4])
{
    const int tid = threadIdx.x;
    const int ty = tid >> 4, tx = tid & 15;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;
    // the operands of the next K step are fetched into registers while the current one is multiplied
    // (the sums themselves are taken in the same order as without the prefetch)
    constexpr int PER = (GT * KC) / NTHREADS;
    float av[PER], bv[PER];
    auto fetch = [&](int k0) {
#pragma unroll
        for (int it = 0; it < PER; ++it) {
            const int idx = tid + it * NTHREADS;
            const int kk = idx % KC, row = idx / KC;
            const int k = k0 + kk;
            av[it] = 0.0f;
            bv[it] = 0.0f;
            if (k < kend) {
                if (m0 + row < M) av[it] = to_f32<T>(A[(size_t)(m0 + row) * lda + k]);
                if (n0 + row < N) bv[it] = to_f32<T>(W[(size_t)(n0 + row) * ldw + k]);
            }
        }
    };
    if (kend > 0) fetch(0);
    for (int k0 = 0; k0 < kend; k0 += KC) {
#pragma unroll
        for (int it = 0; it < PER; ++it) {
            const int idx = tid + it * NTHREADS;
            const int kk = idx % KC, row = idx / KC;
            s.As[kk][row] = av[it];
            s.Bs[kk][row] = bv[it];
        }
        __syncthreads();
        if (k0 + KC < kend) fetch(k0 + KC);
#pragma unroll 8
        for (int kk = 0; kk < KC; ++kk) {
            // (rows of As / Bs are GT + 4 floats: every row and every group of four starts on 16 bytes)
            const float4 a4 = *reinterpret_cast<const float4 *>(&s.As[kk][ty * 4]);
            const float4 b4 = *reinterpret_cast<const float4 *>(&s.Bs[kk][tx * 4]);
            const float a[4] = {a4.x, a4.y, a4.z, a4.w}, b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
}

// Layer l over the window: hidden layers store act(pre) into `out`; the output
// layer (l == L) stores fp32 logits into `zout` [batch][T*C].
template <typename T>
__device__ void gemm_phase(Smem &s, const MadeDev &m, int l, const T *Asrc, T *out, float *zout, int batch,
                           const Win &w, unsigned long long &issued, unsigned long long &skipped)
{
    const int N = m.n[l + 1], K = m.n[l];
    const int mt = (batch + GT - 1) / GT, nt = (N + GT - 1) / GT;
    const bool is_out = (l == m.L);
    const T *Wl = (const T *)m.W[l];
    for (int tile = blockIdx.x; tile < mt * nt; tile += gridDim.x) {
        const int tn = tile / mt, tm = tile % mt;
        const int dmin = m.t_dmin[l][tn], dmax = m.t_dmax[l][tn];
        bool live;
        if (is_out) live = (dmax - 1 >= w.olo) && (dmin - 1 < w.ohi);
        else live = (dmax > w.hdeg_lo) && (dmin <= w.hdeg_hi);
        if (!live) { if (threadIdx.x == 0) skipped++; continue; }
        if (threadIdx.x == 0) issued++;
        float acc[4][4];
        const int m0 = tm * GT, n0 = tn * GT;
        gemm_tile<T>(s, Asrc, K, Wl, K, batch, N, m.t_kend[l][tn], m0, n0, acc);
        const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = m0 + ty * 4 + i;
            if (row >= batch) continue;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int col = n0 + tx * 4 + j;
                if (col >= N) continue;
                const float pre = acc[i][j] + m.bias[l][col];
                if (is_out) zout[(size_t)row * N + col] = pre;
                else out[(size_t)row * N + col] = from_f32<T>(js_act_fn(m.act, pre));
            }
        }
    }
}

// x = init (or zeros), a[0] = lut[x]; also clears the per-sample bookkeeping.
template <typename T>
__device__ void init_phase(const MadeDev &m, const RunArgs &r, const uint8_t *src)
{
    const size_t n = (size_t)r.batch * m.T;
    T *a0 = (T *)m.a[0];
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const uint8_t v = src ? src[i] : (uint8_t)0;
        if (r.x) r.x[i] = v;
        a0[i] = from_f32<T>(m.lut[v]);
    }
    if (blockIdx.x == 0) {
        for (int i = threadIdx.x; i < 2 * r.batch; i += blockDim.x) {
            r.smp_changed[i] = 0;
            r.smp_state[i] = 0;
        }
        if (threadIdx.x == 0) {
            r.ctl->agg_any[0] = r.ctl->agg_any[1] = 0;
            r.ctl->agg_minfirst[0] = r.ctl->agg_minfirst[1] = INT_MAX;
        }
    }
}

// Sample positions [plo, phi) of every sample from the logits scratch, compare
// with the current iterate, store the new symbol and its encoding.
template <typename T>
__device__ void sample_phase(const MadeDev &m, const RunArgs &r, const float *z, int plo, int phi, bool flag,
                             int parity)
{
    const int T_ = m.T, C = m.C, np = phi - plo;
    T *a0 = (T *)m.a[0];
    if (C == 1) {
        const size_t n = (size_t)r.batch * np;
        for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
            const int b = (int)(i / np), d = plo + (int)(i % np);
            const size_t at = (size_t)b * T_ + d;
            const int xn = js_sample_binary(r.nk, z[at], r.noise[at]);
            if (xn != r.x[at]) {
                r.x[at] = (uint8_t)xn;
                a0[at] = from_f32<T>(m.lut[xn]);
                if (flag) note_change(r, parity, b, d);
            }
        }
        return;
    }
    const int lane = threadIdx.x & 31;
    const size_t warps = ((size_t)gridDim.x * blockDim.x) >> 5;
    const size_t n = (size_t)r.batch * np;
    for (size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; i < n; i += warps) {
        const int b = (int)(i / np), d = plo + (int)(i % np);
        const size_t at = (size_t)b * T_ + d;
        const int bi = js_warp_sample_cat(r.nk, z + at * C, r.noise + (r.nk == JS_NOISE_GUMBEL ? at * C : at), C, lane);
        if (lane == 0 && bi != r.x[at]) {
            r.x[at] = (uint8_t)bi;
            a0[at] = from_f32<T>(m.lut[bi]);
            if (flag) note_change(r, parity, b, d);
        }
    }
}

// Continuous states: x = start values (or zeros), a[0] = x (rounded like any activation in a bf16 model).
template <typename T>
__device__ void init_phase_real(const MadeDev &m, const RunArgs &r, const float *src)
{
    const size_t n = (size_t)r.batch * m.T;
    T *a0 = (T *)m.a[0];
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const float v = src ? src[i] : 0.0f;
        if (r.xr) r.xr[i] = v;
        a0[i] = from_f32<T>(v);
    }
    if (blockIdx.x == 0) {
        for (int i = threadIdx.x; i < 2 * r.batch; i += blockDim.x) {
            r.smp_changed[i] = 0;
            r.smp_state[i] = 0;
        }
        if (threadIdx.x == 0) {
            r.ctl->agg_any[0] = r.ctl->agg_any[1] = 0;
            r.ctl->agg_minfirst[0] = r.ctl->agg_minfirst[1] = INT_MAX;
        }
    }
}

// Continuous states with logistic conditionals (Section 5.3.1, Appendix C.3 of arXiv 2002.03629): logit 2t
// is the location m_t, logit 2t+1 the log-scale l_t, and the position's reserved noise e_t = logit(u_t) gives
// x_t = m_t + exp(l_t) e_t (inverse CDF of the logistic law).  A position counts as changed when it moved by
// more than eps, so "no position changed" is the stopping rule  max_t |x^k_t - x^{k-1}_t| <= eps  of
// Section 2.2.1 in the maximum norm.
template <typename T>
__device__ void sample_real_phase(const MadeDev &m, const RunArgs &r, const float *z, int plo, int phi, bool flag,
                                  int parity)
{
    const int T_ = m.T, np = phi - plo;
    T *a0 = (T *)m.a[0];
    const size_t n = (size_t)r.batch * np;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const int b = (int)(i / np), d = plo + (int)(i % np);
        // a sample whose stopping test has fired keeps the iterate it stopped at (with eps > 0 a further
        // update would still move it)
        if (flag && r.smp_state[b] != 0) continue;
        const size_t at = (size_t)b * T_ + d;
        const float xn = fmaf(expf(z[2 * at + 1]), r.noise[at], z[2 * at]);
        const float xo = r.xr[at];
        r.xr[at] = xn;
        a0[at] = from_f32<T>(xn);
        if (flag && !(fabsf(xn - xo) <= r.eps)) note_change(r, parity, b, d);     // a NaN difference is a change
    }
}

template <typename T>
__device__ bool forward_pass(Smem &s, const MadeDev &m, const RunArgs &r, T *const *acts, float *zout, const Win &w,
                             unsigned &epoch, unsigned long long &issued, unsigned long long &skipped)
{
    for (int l = 0; l <= m.L; ++l) {
        gemm_phase<T>(s, m, l, (const T *)acts[l], l < m.L ? acts[l + 1] : (T *)nullptr, zout, r.batch, w, issued,
                      skipped);
        if (!grid_barrier(r.ctl, epoch, r.spin_limit)) return false;
    }
    return true;
}

// ---- Jacobi-GS micro-steps (Algorithm 2): warp-per-dot-product evaluation of
// the units that become computable at step j of every block's sequential sweep.
// A unit of block i reads, from the layer below, units of earlier blocks at the
// previous outer iterate (`old`) and units of its own block at the current one.
template <typename T>
__device__ float mixed_dot(const MadeDev &m, int l, int unit, int blk, int B, const T *old_row, const T *new_row,
                           int kend)
{
    const int lane = threadIdx.x & 31;
    const T *w = (const T *)m.W[l] + (size_t)unit * m.n[l];
    const int *dg = m.deg[l];
    float acc = 0.0f;
    for (int k = lane; k < kend; k += 32) {
        const bool use_old = ((dg[k] - 1) / B) < blk;
        acc = fmaf(to_f32<T>(w[k]), to_f32<T>(use_old ? old_row[k] : new_row[k]), acc);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    return acc;
}

template <typename T>
__device__ void jgs_hidden_phase(Smem &s, const MadeDev &m, const RunArgs &r, int l, int j, int B, int blk_lo)
{
    // units of layer l+1 whose degree g satisfies g % B == j, in blocks >= blk_lo.
    // The list is built in index order so that every CTA holds the same list.
    const int N = m.n[l + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const size_t warps = ((size_t)gridDim.x * blockDim.x) >> 5;
    for (int ubase = 0; ubase < N; ubase += 4096) {
        const int uend = min(N, ubase + 4096);
        if (threadIdx.x == 0) s.list_n = 0;
        __syncthreads();
        for (int base = ubase; base < uend; base += NTHREADS) {
            const int i = base + threadIdx.x;
            bool pred = false;
            if (i < uend) {
                const int g = m.deg[l + 1][i];
                pred = (g % B == j) && ((g - 1) / B >= blk_lo);
            }
            const unsigned bal = __ballot_sync(0xffffffffu, pred);
            if (lane == 0) s.wcnt[warp] = __popc(bal);
            __syncthreads();
            int off = s.list_n;
            for (int w2 = 0; w2 < warp; ++w2) off += s.wcnt[w2];
            if (pred) s.list[off + __popc(bal & ((1u << lane) - 1u))] = i;
            __syncthreads();
            if (threadIdx.x == 0) {
                int tot = 0;
                for (int w2 = 0; w2 < NTHREADS / 32; ++w2) tot += s.wcnt[w2];
                s.list_n += tot;
            }
            __syncthreads();
        }
        const int cnt = s.list_n;
        const size_t items = (size_t)cnt * r.batch;
        for (size_t it = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; it < items; it += warps) {
            const int unit = s.list[it / r.batch], b = (int)(it % r.batch);
            const int g = m.deg[l + 1][unit];
            const float pre = mixed_dot<T>(m, l, unit, (g - 1) / B, B, (const T *)m.a_old[l] + (size_t)b * m.n[l],
                                           (const T *)m.a[l] + (size_t)b * m.n[l], m.t_kend[l][unit / GT]) +
                              m.bias[l][unit];
            if (lane == 0) ((T *)m.a[l + 1])[(size_t)b * N + unit] = from_f32<T>(js_act_fn(m.act, pre));
        }
        __syncthreads();
    }
}

template <typename T>
__device__ void jgs_output_phase(const MadeDev &m, const RunArgs &r, int j, int B, int blk_lo)
{
    const int L = m.L, C = m.C, nblk = (m.T + B - 1) / B;
    const size_t warps = ((size_t)gridDim.x * blockDim.x) >> 5;
    const size_t items = (size_t)(nblk - blk_lo) * C * r.batch;
    const int lane = threadIdx.x & 31;
    for (size_t it = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; it < items; it += warps) {
        const int b = (int)(it % r.batch);
        const int c = (int)((it / r.batch) % C);
        const int blk = blk_lo + (int)(it / ((size_t)r.batch * C));
        const int t = blk * B + j;
        if (t >= m.T) continue;
        const int unit = t * C + c;
        const float z = mixed_dot<T>(m, L, unit, blk, B, (const T *)m.a_old[L] + (size_t)b * m.n[L],
                                     (const T *)m.a[L] + (size_t)b * m.n[L], m.t_kend[L][unit / GT]) +
                        m.bias[L][unit];
        if (C == 1) {
            if (lane == 0) {
                const size_t at = (size_t)b * m.T + t;
                const int xn = js_sample_binary(r.nk, z, r.noise[at]);
                r.x[at] = (uint8_t)xn;
                ((T *)m.a[0])[at] = from_f32<T>(m.lut[xn]);
            }
        } else if (lane == 0) {
            m.logits[(size_t)b * m.n[L + 1] + unit] = z;
        }
    }
}

// categorical commit of position blk*B + j for every block (no change flags here)
template <typename T>
__device__ void jgs_commit_phase(const MadeDev &m, const RunArgs &r, int j, int B, int blk_lo)
{
    const int C = m.C, nblk = (m.T + B - 1) / B;
    const size_t warps = ((size_t)gridDim.x * blockDim.x) >> 5;
    const size_t items = (size_t)(nblk - blk_lo) * r.batch;
    const int lane = threadIdx.x & 31;
    for (size_t it = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; it < items; it += warps) {
        const int b = (int)(it % r.batch);
        const int t = (blk_lo + (int)(it / r.batch)) * B + j;
        if (t >= m.T) continue;
        const size_t at = (size_t)b * m.T + t;
        const int bi = js_warp_sample_cat(r.nk, m.logits + at * C, r.noise + (r.nk == JS_NOISE_GUMBEL ? at * C : at), C, lane);
        if (lane == 0) {
            r.x[at] = (uint8_t)bi;
            ((T *)m.a[0])[at] = from_f32<T>(m.lut[bi]);
        }
    }
}

// x_old = x and a_old[0] = a[0] (start of an outer iteration); or compare x with
// x_old and raise change flags (end of an outer iteration).
template <typename T>
__device__ void jgs_copy_or_compare(const MadeDev &m, const RunArgs &r, bool compare, int parity)
{
    const size_t n = (size_t)r.batch * m.T;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        if (compare) {
            if (r.x[i] != r.x_old[i]) note_change(r, parity, (int)(i / m.T), (int)(i % m.T));
        } else {
            r.x_old[i] = r.x[i];
            ((T *)m.a_old[0])[i] = ((const T *)m.a[0])[i];
        }
    }
}

// ------------------------------------------------------------------ engine
template <typename T>
struct GenericEngine {
    static constexpr bool has_jgs = true;
    Smem &s;
    const MadeDev &m;
    const RunArgs &r;
    unsigned epoch = 0;
    unsigned long long issued = 0, skipped = 0;
    T *acts[JS_MAXL + 1], *acts_old[JS_MAXL + 1];

    __device__ GenericEngine(Smem &s_, const MadeDev &m_, const RunArgs &r_) : s(s_), m(m_), r(r_)
    {
        for (int l = 0; l <= m.L; ++l) { acts[l] = (T *)m.a[l]; acts_old[l] = (T *)m.a_old[l]; }
    }
    __device__ bool barrier() { return grid_barrier(r.ctl, epoch, r.spin_limit); }
    __device__ void init(const uint8_t *src)
    {
        if (r.real)
            init_phase_real<T>(m, r, r.kmode == KM_FORWARD ? r.xin_r : r.kmode == KM_SEQ ? (const float *)nullptr : r.init_r);
        else
            init_phase<T>(m, r, src);
    }
    __device__ int compact(int) { return 0; }      // the CUDA-core path keeps the batch as it is
    // one forward pass over the window; then either the logits go to zout (teacher forcing) or
    // positions [w.plo, w.phi) are sampled and committed
    __device__ bool step(const Win &w, bool flag, int parity, float *zout)
    {
        if (zout) return forward_pass<T>(s, m, r, acts, zout, w, epoch, issued, skipped);
        if (!forward_pass<T>(s, m, r, acts, m.logits, w, epoch, issued, skipped)) return false;
        if (r.real) sample_real_phase<T>(m, r, m.logits, w.plo, w.phi, flag, parity);
        else sample_phase<T>(m, r, m.logits, w.plo, w.phi, flag, parity);
        return barrier();
    }
    // one outer iteration of Algorithm 2
    __device__ bool jgs_outer(int parity, int fin_h, int blk_lo, int &iterations)
    {
        const int B = r.block, T_ = m.T;
        jgs_copy_or_compare<T>(m, r, false, parity);
        if (!barrier()) return false;
        // hidden activations of the previous outer iterate
        const Win w = make_win(fin_h, T_, T_, T_);
        for (int l = 0; l < m.L; ++l) {
            gemm_phase<T>(s, m, l, acts_old[l], acts_old[l + 1], nullptr, r.batch, w, issued, skipped);
            if (!barrier()) return false;
        }
        const int jmax = min(B, T_);
        for (int j = 0; j < jmax; ++j) {
            if (j >= 1)
                for (int l = 0; l < m.L; ++l) {
                    jgs_hidden_phase<T>(s, m, r, l, j, B, blk_lo);
                    if (!barrier()) return false;
                }
            jgs_output_phase<T>(m, r, j, B, blk_lo);
            if (!barrier()) return false;
            if (m.C > 1) {
                jgs_commit_phase<T>(m, r, j, B, blk_lo);
                if (!barrier()) return false;
            }
            iterations++;
        }
        jgs_copy_or_compare<T>(m, r, true, parity);
        return barrier();
    }
};

template <typename T>
__global__ void __launch_bounds__(NTHREADS) made_generic_kernel(const __grid_constant__ MadeDev m, const __grid_constant__ RunArgs r)
{
    __shared__ Smem s;
    GenericEngine<T> e(s, m, r);
    const DriverResult res = made_driver(e, m.T, r);
    driver_finish(r, res, e.issued, e.skipped);
}

}  // namespace

int js_made_generic_max_grid(int prec)
{
    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return -1;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
    cudaError_t e = prec == JS_BF16
        ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, made_generic_kernel<__nv_bfloat16>, NTHREADS, 0)
        : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, made_generic_kernel<float>, NTHREADS, 0);
    if (e != cudaSuccess || per_sm < 1) return -1;
    return sms * per_sm;
}

int js_launch_made_generic(const MadeDev &m, const RunArgs &r, int grid, cudaStream_t stream)
{
    void *args[2] = {(void *)&m, (void *)&r};
    const void *fn = m.prec == JS_BF16 ? (const void *)made_generic_kernel<__nv_bfloat16>
                                       : (const void *)made_generic_kernel<float>;
    cudaError_t e = cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(NTHREADS), args, 0, stream);
    return e == cudaSuccess ? 0 : (int)e;
}
