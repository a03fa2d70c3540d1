// C ABI of the sampler library: model construction (masking, rounding, tile
// metadata), argument checks, kernel selection and launch, status read-back.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "js_common.cuh"
#include "js_model.h"

static thread_local char g_cuda_err[256] = "";

#define CU_TRY(call)                                                                         \
    do {                                                                                     \
        cudaError_t e__ = (call);                                                            \
        if (e__ != cudaSuccess) {                                                            \
            snprintf(g_cuda_err, sizeof g_cuda_err, "%s: %s", #call, cudaGetErrorString(e__)); \
            return JS_ERR_CUDA;                                                              \
        }                                                                                    \
    } while (0)

namespace {

// masked, rounded copy of one weight matrix:  Wm[i][j] = keep(i, j) ? W[i][j] : 0
template <typename T>
__global__ void pack_made_weights(const float *__restrict__ W, const int *__restrict__ deg_out,
                                  const int *__restrict__ deg_in, int n_out, int n_in, int strict, T *__restrict__ out)
{
    const size_t n = (size_t)n_out * n_in;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const int r = (int)(i / n_in), c = (int)(i % n_in);
        const bool keep = strict ? (deg_out[r] > deg_in[c]) : (deg_out[r] >= deg_in[c]);
        out[i] = from_f32<T>(keep ? W[i] : 0.0f);
    }
}

template <typename T>
int dev_alloc(js_model *m, T **p, size_t count, bool zero)
{
    void *q = nullptr;
    const size_t bytes = std::max<size_t>(count * sizeof(T), 16);
    CU_TRY(cudaMalloc(&q, bytes));
    m->allocs.push_back(q);
    if (zero) CU_TRY(cudaMemset(q, 0, bytes));
    *p = (T *)q;
    return JS_OK;
}

template <typename T>
int dev_upload(js_model *m, const T **p, const T *host, size_t count)
{
    T *q = nullptr;
    int rc = dev_alloc(m, &q, count, false);
    if (rc != JS_OK) return rc;
    CU_TRY(cudaMemcpy(q, host, count * sizeof(T), cudaMemcpyHostToDevice));
    *p = q;
    return JS_OK;
}

int made_build(js_model *m, const js_made_desc *d)
{
    MadeDev &v = m->made;
    v.T = d->T; v.C = d->C; v.L = d->L; v.act = d->act; v.prec = d->prec;
    v.n[0] = d->T;
    for (int l = 0; l < d->L; ++l) v.n[l + 1] = d->H[l];
    v.n[d->L + 1] = d->T * d->C;
    const int L = d->L;
    const size_t esz = d->prec == JS_BF16 ? 2 : 4;

    // degrees
    std::vector<std::vector<int>> deg(L + 2);
    for (int l = 0; l <= L + 1; ++l) deg[l].resize(v.n[l]);
    for (int i = 0; i < d->T; ++i) deg[0][i] = i + 1;
    for (int l = 1; l <= L; ++l)
        for (int j = 0; j < v.n[l]; ++j) {
            int g = (d->hidden_deg && d->hidden_deg[l - 1]) ? d->hidden_deg[l - 1][j]
                                                            : 1 + (int)(((long long)j * (d->T - 1)) / v.n[l]);
            if (g < 1 || g > d->T) return JS_ERR_ARG;
            deg[l][j] = g;
        }
    for (int i = 0; i < d->T * d->C; ++i) deg[L + 1][i] = i / d->C + 1;
    for (int l = 0; l <= L + 1; ++l) {
        int rc = dev_upload<int>(m, &v.deg[l], deg[l].data(), deg[l].size());
        if (rc != JS_OK) return rc;
    }

    // per-tile metadata for the 64-wide output tiles of every layer
    for (int l = 0; l <= L; ++l) {
        const int N = v.n[l + 1], K = v.n[l], nt = (N + JS_GT - 1) / JS_GT;
        std::vector<int> kend(nt), dmin(nt), dmax(nt);
        for (int t = 0; t < nt; ++t) {
            int lo = INT32_MAX, hi = 0;
            for (int i = t * JS_GT; i < std::min(N, (t + 1) * JS_GT); ++i) {
                lo = std::min(lo, deg[l + 1][i]);
                hi = std::max(hi, deg[l + 1][i]);
            }
            int ke = K;
            while (ke > 0 && !(l == L ? deg[l][ke - 1] < hi : deg[l][ke - 1] <= hi)) --ke;
            kend[t] = ke; dmin[t] = lo; dmax[t] = hi;
        }
        int rc;
        if ((rc = dev_upload<int>(m, &v.t_kend[l], kend.data(), nt)) != JS_OK) return rc;
        if ((rc = dev_upload<int>(m, &v.t_dmin[l], dmin.data(), nt)) != JS_OK) return rc;
        if ((rc = dev_upload<int>(m, &v.t_dmax[l], dmax.data(), nt)) != JS_OK) return rc;
        m->host_deg = deg;
    }

    // weights: upload unmasked fp32, mask and round on the device
    int sms = 1;
    {
        int dev = 0;
        CU_TRY(cudaGetDevice(&dev));
        CU_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    }
    for (int l = 0; l <= L; ++l) {
        const size_t cnt = (size_t)v.n[l + 1] * v.n[l];
        float *tmp = nullptr;
        CU_TRY(cudaMalloc((void **)&tmp, cnt * sizeof(float)));
        cudaError_t e = cudaMemcpy(tmp, d->W[l], cnt * sizeof(float), cudaMemcpyHostToDevice);
        void *wm = nullptr;
        if (e == cudaSuccess) e = cudaMalloc(&wm, cnt * esz);
        if (e == cudaSuccess) {
            m->allocs.push_back(wm);
            const int grid = (int)std::min<size_t>((cnt + 255) / 256, (size_t)sms * 16);
            if (d->prec == JS_BF16)
                pack_made_weights<__nv_bfloat16><<<grid, 256>>>(tmp, v.deg[l + 1], v.deg[l], v.n[l + 1], v.n[l],
                                                                 l == L, (__nv_bfloat16 *)wm);
            else
                pack_made_weights<float><<<grid, 256>>>(tmp, v.deg[l + 1], v.deg[l], v.n[l + 1], v.n[l], l == L,
                                                         (float *)wm);
            e = cudaGetLastError();
            if (e == cudaSuccess) e = cudaDeviceSynchronize();
        }
        cudaFree(tmp);
        CU_TRY(e);
        v.W[l] = wm;
        int rc = dev_upload<float>(m, &v.bias[l], d->b[l], v.n[l + 1]);
        if (rc != JS_OK) return rc;
    }

    // input table, rounded like an activation
    {
        std::vector<float> lut(d->lut, d->lut + d->n_lut);
        if (d->prec == JS_BF16)
            for (auto &f : lut) f = __bfloat162float(__float2bfloat16_rn(f));
        int rc = dev_upload<float>(m, &v.lut, lut.data(), lut.size());
        if (rc != JS_OK) return rc;
    }

    // activations and scratch
    m->rows = (m->max_batch + 127) / 128 * 128;
    for (int l = 0; l <= L; ++l) {
        char *p = nullptr, *q = nullptr;
        int rc;
        if ((rc = dev_alloc<char>(m, &p, (size_t)m->rows * v.n[l] * esz, true)) != JS_OK) return rc;
        if ((rc = dev_alloc<char>(m, &q, (size_t)m->rows * v.n[l] * esz, true)) != JS_OK) return rc;
        v.a[l] = p; v.a_old[l] = q;
    }
    int rc;
    if ((rc = dev_alloc<float>(m, &v.logits, (size_t)m->rows * v.n[L + 1], true)) != JS_OK) return rc;
    return JS_OK;
}

int common_scratch(js_model *m, int T)
{
    int rc;
    if ((rc = dev_alloc<JsCtl>(m, &m->ctl, 1, true)) != JS_OK) return rc;
    CU_TRY(cudaHostAlloc((void **)&m->h_result, sizeof(JsCtl), cudaHostAllocMapped));
    CU_TRY(cudaHostGetDevicePointer((void **)&m->d_result, m->h_result, 0));
    if ((rc = dev_alloc<int>(m, &m->smp_changed, 2 * (size_t)m->rows, true)) != JS_OK) return rc;
    if ((rc = dev_alloc<int>(m, &m->smp_state, 2 * (size_t)m->rows, true)) != JS_OK) return rc;
    if ((rc = dev_alloc<int>(m, &m->perm, 2 * (size_t)m->rows, true)) != JS_OK) return rc;
    if ((rc = dev_alloc<uint8_t>(m, &m->x_old, (size_t)m->rows * T, true)) != JS_OK) return rc;
    if ((rc = dev_alloc<uint8_t>(m, &m->x_tmp, (size_t)m->rows * T, true)) != JS_OK) return rc;
    if ((rc = dev_alloc<unsigned long long>(m, &m->trace, 2 * JS_TRACE_PHASES * JS_TRACE_SLOTS, true)) != JS_OK) return rc;
    return JS_OK;
}

bool noise_kind_ok(const js_model *m, int nk)
{
    const int C = m->kind == 0 ? m->made.C : m->conv_C;
    if (nk == JS_NOISE_GUMBEL || nk == JS_NOISE_UNIFORM_CAT) return C > 1;
    if (nk == JS_NOISE_UNIFORM_ICDF || nk == JS_NOISE_LOGISTIC) return C == 1;
    return false;
}

const int NOT_REPORTED = -1000000;

// model-owned fields of the launch arguments; the control block is cleared if the last call left it dirty
int prep_args(js_model *m, RunArgs &r, cudaStream_t st)
{
    r.ctl = m->ctl;
    r.smp_changed = m->smp_changed;
    r.smp_state = m->smp_state;
    r.x_old = m->x_old;
    // with a tolerance eps > 0 an unchanged position is not a final one: no skipping on continuous states
    r.frontier_skip = r.real ? 0 : m->opt_frontier_skip;
    r.seq_skip = (!r.real && m->opt_seq_skip == 1) ? 1 : 0;
    r.compact = m->opt_compact;
    r.perm = m->perm;
    r.perm_stride = m->rows;
    r.spin_limit = (unsigned)m->opt_spin_limit;
    r.trace = m->opt_trace ? m->trace : nullptr;
    r.trace_cta = m->opt_trace >= 2 ? m->opt_trace - 2 : -1;
    if (r.trace) CU_TRY(cudaMemsetAsync(m->trace, 0, sizeof(unsigned long long) * 2 * JS_TRACE_PHASES * JS_TRACE_SLOTS, st));
    // a call that ended normally left the control block zeroed
    if (!m->ctl_clean) CU_TRY(cudaMemsetAsync(m->ctl, 0, sizeof(JsCtl), st));
    m->ctl_clean = false;
    r.result = m->d_result;
    m->h_result->status = NOT_REPORTED;
    return JS_OK;
}

// waits for the launch and reads what the kernel reported through mapped host memory
int wait_result(js_model *m, cudaStream_t st, JsCtl &h)
{
    CU_TRY(cudaStreamSynchronize(st));
    h = *m->h_result;
    if (h.status == NOT_REPORTED) {
        snprintf(g_cuda_err, sizeof g_cuda_err, "the kernel ended without reporting");
        return JS_ERR_CUDA;
    }
    m->ctl_clean = h.status >= 0;
    return JS_OK;
}

int launch_failed(int rc_launch)
{
    snprintf(g_cuda_err, sizeof g_cuda_err, "kernel launch: %s", cudaGetErrorString((cudaError_t)rc_launch));
    return JS_ERR_CUDA;
}

void fill_stats(js_model *m, const JsCtl &h, int used_path)
{
    m->stats.iterations = h.iterations;
    m->stats.final_frontier = h.frontier;
    m->stats.tiles_issued = (long long)h.tiles_issued;
    m->stats.tiles_skipped = (long long)h.tiles_skipped;
    m->stats.batch_iters_max = h.iters_max;
    m->stats.mma_flops = (long long)h.mma_flops;
    m->stats.weight_bytes = (long long)h.weight_bytes;
    m->stats.path = used_path;
    m->stats.compactions = h.compactions;
    m->stats.status = h.status;
}

// can the cached sweeps (made_sweep.cu) serve this call?
bool sweeps_usable(js_model *m, const RunArgs &r)
{
    if (m->kind != 0 || !m->tc_ok || m->opt_path != 0 || m->made.C != 1) return false;
    if ((((uintptr_t)r.noise | (uintptr_t)r.x) & 15u) != 0) return false;
    return js_sweep_prepare(m) == 1;
}

// The feedforward pass with every hidden unit evaluated once: one sweep over all positions.
int run_sweep_sequential(js_model *m, RunArgs &r, cudaStream_t st)
{
    int rc = prep_args(m, r, st);
    if (rc != JS_OK) return rc;
    r.block = m->made.T;
    r.blk_lo = 0;
    r.smp_changed = m->sw_flags;
    const int rl = js_launch_made_sweep(m, r, st);
    if (rl != 0) return launch_failed(rl);
    JsCtl h;
    if ((rc = wait_result(m, st, h)) != JS_OK) return rc;
    fill_stats(m, h, 0);
    m->stats.iterations = 1;
    m->stats.final_frontier = m->made.T;
    if (h.status == JS_OK && r.out_iters) {
        std::vector<int32_t> ones(r.batch, 1);
        CU_TRY(cudaMemcpyAsync(r.out_iters, ones.data(), sizeof(int32_t) * r.batch, cudaMemcpyHostToDevice, st));
        CU_TRY(cudaStreamSynchronize(st));
    }
    return h.status;
}

// Algorithm 2 on the tensor cores.  Outer iteration k: the hidden layers on x^{k-1} (tensor-core
// kernel, hidden layers only), then every block swept from that prefix (sweep kernel), then the
// per-sample bookkeeping; the host looks at one word per outer iteration.  After k outer iterations
// the first k blocks are final (proof of Proposition 2): they are not swept again, and the hidden
// units that depend on them alone are not recomputed.
int run_jacobi_gs_tc(js_model *m, RunArgs &r, cudaStream_t st)
{
    const MadeDev &v = m->made;
    const int T = v.T, B = r.block, M = (T + B - 1) / B;
    const int cap = (r.max_iters > 0 && r.max_iters < M) ? r.max_iters : M;
    if (r.init != r.x) {
        if (r.init) CU_TRY(cudaMemcpyAsync(r.x, r.init, (size_t)r.batch * T, cudaMemcpyDeviceToDevice, st));
        else CU_TRY(cudaMemsetAsync(r.x, 0, (size_t)r.batch * T, st));
    }
    CU_TRY(cudaMemsetAsync(m->sw_flags, 0, 2 * (size_t)m->rows * sizeof(int), st));
    long long flops = 0;
    int status = JS_OK, k = 0;
    for (k = 1;; ++k) {
        const int fin_blocks = m->opt_frontier_skip ? k - 1 : 0;          // blocks known final before this iteration
        RunArgs f = r;
        int rc = prep_args(m, f, st);
        if (rc != JS_OK) return rc;
        f.kmode = KM_HIDDEN;
        f.x_in = r.x;
        f.x = nullptr;
        f.out_iters = nullptr;
        f.hid_lo = m->opt_frontier_skip ? std::max(0, (k - 2) * B) : 0;   // final since the previous forward pass
        int rl = js_launch_made_tc(m, f, st);
        if (rl != 0) return launch_failed(rl);
        JsCtl h;
        if ((rc = wait_result(m, st, h)) != JS_OK) return rc;
        if (h.status < 0) { fill_stats(m, h, 0); return h.status; }
        flops += (long long)h.mma_flops;
        RunArgs s2 = r;
        if ((rc = prep_args(m, s2, st)) != JS_OK) return rc;
        s2.blk_lo = std::min(fin_blocks, M - 1);
        s2.smp_changed = m->sw_flags;
        rl = js_launch_made_sweep(m, s2, st);
        if (rl != 0) return launch_failed(rl);
        *m->h_any = -1;
        rl = js_launch_jgs_book(m, r.batch, k, k == cap, r.out_iters, st);
        if (rl != 0) return launch_failed(rl);
        if ((rc = wait_result(m, st, h)) != JS_OK) return rc;
        flops += (long long)h.mma_flops;
        if (h.status < 0) { fill_stats(m, h, 0); return h.status; }
        const int any = *m->h_any;
        if (any < 0) {
            snprintf(g_cuda_err, sizeof g_cuda_err, "the bookkeeping kernel did not report");
            return JS_ERR_CUDA;
        }
        fill_stats(m, h, 0);
        if (!any || k == cap) {
            if (any && cap < M) status = JS_NOT_CONVERGED;
            break;
        }
    }
    m->stats.iterations = k;
    m->stats.mma_flops = flops;
    m->stats.final_frontier = status == JS_OK ? T : std::min(T, k * B);
    m->stats.status = status;
    return status;
}

int run_made(js_model *m, RunArgs &r, cudaStream_t st)
{
    const MadeDev &v = m->made;
    // Algorithm 2 on the masked-conv stack: blocks of one image row (the paper's choice, Section 5.3.2)
    if (m->kind == 1 && r.kmode == KM_JACOBI_GS && r.block != m->conv.width * m->conv.in_ch) return JS_ERR_UNSUPPORTED;
    // the sweeps: the strict order with cached hidden units, and Algorithm 2
    if (r.kmode == KM_SEQ && m->opt_seq_skip == 2 && sweeps_usable(m, r)) return run_sweep_sequential(m, r, st);
    if (r.kmode == KM_JACOBI_GS && sweeps_usable(m, r)) return run_jacobi_gs_tc(m, r, st);
    int rc = prep_args(m, r, st);
    if (rc != JS_OK) return rc;

    int used_path = 1;
    int rc_launch;
    // the tensor-core epilogues use 16-byte vector accesses on the caller's buffers
    const bool aligned = (((uintptr_t)r.noise | (uintptr_t)r.x | (uintptr_t)r.logits_out) & 15u) == 0;
    if (m->kind == 1) {
        if (!aligned) return JS_ERR_ARG;
        used_path = 0;
        rc_launch = js_launch_conv_tc(m, r, st);
    } else if (m->tc_ok && m->opt_path == 0 && r.kmode != KM_JACOBI_GS && aligned) {
        used_path = 0;
        rc_launch = js_launch_made_tc(m, r, st);
    } else {
        if (m->max_grid_generic <= 0) m->max_grid_generic = js_made_generic_max_grid(v.prec);
        if (m->max_grid_generic <= 0) {
            snprintf(g_cuda_err, sizeof g_cuda_err, "occupancy query failed");
            return JS_ERR_CUDA;
        }
        long long tiles = 1;
        for (int l = 0; l <= v.L; ++l)
            tiles = std::max<long long>(tiles, (long long)((r.batch + JS_GT - 1) / JS_GT) * ((v.n[l + 1] + JS_GT - 1) / JS_GT));
        const long long elems = ((long long)r.batch * v.T * (v.C > 1 ? 32 : 1) + 255) / 256;
        const int grid = (int)std::min<long long>(m->max_grid_generic, std::max(tiles, elems));
        rc_launch = js_launch_made_generic(v, r, std::max(grid, 1), st);
    }
    if (rc_launch != 0) return launch_failed(rc_launch);
    JsCtl h;
    if ((rc = wait_result(m, st, h)) != JS_OK) return rc;
    fill_stats(m, h, used_path);
    return h.status;
}

}  // namespace

extern "C" {

int js_made_create(const js_made_desc *d, js_model **out)
{
    if (!d || !out) return JS_ERR_ARG;
    *out = nullptr;
    if (d->T < 1 || d->C < 1 || d->C > 256 || d->L < 1 || d->L > JS_MAXL || !d->H || !d->W || !d->b || !d->lut ||
        d->max_batch < 1)
        return JS_ERR_ARG;
    if (d->act != JS_ACT_RELU && d->act != JS_ACT_GELU_TANH) return JS_ERR_ARG;
    if (d->prec != JS_F32 && d->prec != JS_BF16) return JS_ERR_ARG;
    if (d->n_lut != (d->C == 1 ? 2 : d->C)) return JS_ERR_ARG;
    for (int l = 0; l < d->L; ++l)
        if (d->H[l] < 1) return JS_ERR_ARG;
    for (int l = 0; l <= d->L; ++l)
        if (!d->W[l] || !d->b[l]) return JS_ERR_ARG;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) {
        snprintf(g_cuda_err, sizeof g_cuda_err, "no CUDA device");
        return JS_ERR_CUDA;
    }
    js_model *m = new (std::nothrow) js_model();
    if (!m) return JS_ERR_ARG;
    m->kind = 0;
    m->max_batch = d->max_batch;
    int rc = made_build(m, d);
    if (rc == JS_OK) rc = common_scratch(m, d->T);
    if (rc == JS_OK && js_tc_prepare(m) < 0) rc = JS_ERR_CUDA;
    if (rc != JS_OK) { js_model_destroy(m); return rc; }
    *out = m;
    return JS_OK;
}

int js_conv_create(const js_conv_desc *d, js_model **out)
{
    if (!d || !out) return JS_ERR_ARG;
    *out = nullptr;
    if (!d->W || !d->b || !d->lut || d->max_batch < 1 || d->n_conv < 1 || d->n_conv > JS_MAXL) return JS_ERR_ARG;
    for (int l = 0; l <= d->n_conv; ++l)
        if (!d->W[l] || !d->b[l]) return JS_ERR_ARG;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) {
        snprintf(g_cuda_err, sizeof g_cuda_err, "no CUDA device");
        return JS_ERR_CUDA;
    }
    js_model *m = new (std::nothrow) js_model();
    if (!m) return JS_ERR_ARG;
    m->kind = 1;
    m->max_batch = d->max_batch;
    m->rows = d->max_batch;
    int rc = js_conv_build(m, d);
    if (rc == JS_ERR_CUDA) snprintf(g_cuda_err, sizeof g_cuda_err, "conv model: %s", cudaGetErrorString(cudaGetLastError()));
    if (rc == JS_OK) rc = common_scratch(m, m->conv.T);
    if (rc != JS_OK) { js_model_destroy(m); return rc; }
    *out = m;
    return JS_OK;
}

void js_model_destroy(js_model *m)
{
    if (!m) return;
    for (void *p : m->allocs) cudaFree(p);
    if (m->h_result) cudaFreeHost(m->h_result);
    if (m->h_nflag) cudaFreeHost(m->h_nflag);
    if (m->h_any) cudaFreeHost(m->h_any);
    if (m->ev_main) cudaEventDestroy(m->ev_main);
    if (m->ev_copy) cudaEventDestroy(m->ev_copy);
    if (m->copy_stream) cudaStreamDestroy(m->copy_stream);
    delete m;
}

int jacobi_sample(const js_model *cm, int batch, const float *noise_dev, int nk, const uint8_t *init_dev, int mode,
                  int block, int max_iters, uint8_t *out_samples_dev, int32_t *out_iters_dev, void *cuda_stream)
{
    js_model *m = const_cast<js_model *>(cm);
    if (!m || !noise_dev || !out_samples_dev) return JS_ERR_ARG;
    if (batch < 1 || batch > m->max_batch) return JS_ERR_ARG;
    if (mode < JS_JACOBI || mode > JS_JACOBI_GS) return JS_ERR_ARG;
    if (!noise_kind_ok(m, nk)) return JS_ERR_ARG;
    const int T = m->kind == 0 ? m->made.T : m->conv_T;
    if ((mode == JS_GS_JACOBI || mode == JS_JACOBI_GS) && (block < 1 || block > T)) return JS_ERR_ARG;
    RunArgs r;
    memset(&r, 0, sizeof r);
    r.batch = batch; r.noise = noise_dev; r.nk = nk; r.init = init_dev;
    r.kmode = mode == JS_JACOBI ? KM_JACOBI : mode == JS_GAUSS_SEIDEL ? KM_SEQ : mode == JS_GS_JACOBI ? KM_GS_JACOBI
                                                                                                        : KM_JACOBI_GS;
    r.block = block; r.max_iters = max_iters;
    r.x = out_samples_dev; r.out_iters = out_iters_dev;
    int rc = run_made(m, r, (cudaStream_t)cuda_stream);
    return rc;
}

// device staging, copy stream and events of the host-buffer entry point, on first use
static int ensure_host_staging(js_model *m)
{
    if (m->copy_stream) return JS_OK;
    const int T = m->kind == 0 ? m->made.T : m->conv_T;
    const int C = m->kind == 0 ? m->made.C : m->conv_C;
    int rc;
    if ((rc = dev_alloc<float>(m, &m->st_noise, (size_t)m->max_batch * T * C, false)) != JS_OK) return rc;
    if ((rc = dev_alloc<uint8_t>(m, &m->st_x, (size_t)m->max_batch * T, false)) != JS_OK) return rc;
    if ((rc = dev_alloc<uint8_t>(m, &m->st_init, (size_t)m->max_batch * T, false)) != JS_OK) return rc;
    if ((rc = dev_alloc<int32_t>(m, &m->st_iters, (size_t)m->max_batch, false)) != JS_OK) return rc;
    if ((rc = dev_alloc<unsigned>(m, &m->d_nflag, 4, true)) != JS_OK) return rc;
    CU_TRY(cudaHostAlloc((void **)&m->h_nflag, sizeof(unsigned), cudaHostAllocDefault));
    CU_TRY(cudaEventCreateWithFlags(&m->ev_main, cudaEventDisableTiming));
    CU_TRY(cudaEventCreateWithFlags(&m->ev_copy, cudaEventDisableTiming));
    CU_TRY(cudaStreamCreateWithFlags(&m->copy_stream, cudaStreamNonBlocking));
    return JS_OK;
}

int jacobi_sample_host(const js_model *cm, int batch, const float *noise_host, int nk, const uint8_t *init_host,
                       int mode, int block, int max_iters, uint8_t *out_samples_host, int32_t *out_iters_host,
                       void *cuda_stream)
{
    js_model *m = const_cast<js_model *>(cm);
    if (!m || !noise_host || !out_samples_host) return JS_ERR_ARG;
    if (batch < 1 || batch > m->max_batch) return JS_ERR_ARG;
    if (mode < JS_JACOBI || mode > JS_JACOBI_GS) return JS_ERR_ARG;
    if (!noise_kind_ok(m, nk)) return JS_ERR_ARG;
    const int T = m->kind == 0 ? m->made.T : m->conv_T;
    const int C = m->kind == 0 ? m->made.C : m->conv_C;
    if ((mode == JS_GS_JACOBI || mode == JS_JACOBI_GS) && (block < 1 || block > T)) return JS_ERR_ARG;
    int rc = ensure_host_staging(m);
    if (rc != JS_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream, cs = m->copy_stream;
    // From the first enqueue on, every way out drains both streams first: the caller's buffers and
    // the arrival word may only be touched during the call.
    auto leave = [&](int code) {
        cudaStreamSynchronize(cs);
        cudaStreamSynchronize(st);
        return code;
    };
#define HOST_TRY(call)                                                                       \
    do {                                                                                     \
        cudaError_t e__ = (call);                                                            \
        if (e__ != cudaSuccess) {                                                            \
            snprintf(g_cuda_err, sizeof g_cuda_err, "%s: %s", #call, cudaGetErrorString(e__)); \
            return leave(JS_ERR_CUDA);                                                       \
        }                                                                                    \
    } while (0)
    // the uploads start once the work the caller queued on `st` before this call is done
    HOST_TRY(cudaEventRecord(m->ev_main, st));
    HOST_TRY(cudaStreamWaitEvent(cs, m->ev_main, 0));
    if (init_host) {
        HOST_TRY(cudaMemcpyAsync(m->st_init, init_host, (size_t)batch * T, cudaMemcpyHostToDevice, cs));
        HOST_TRY(cudaEventRecord(m->ev_copy, cs));
        HOST_TRY(cudaStreamWaitEvent(st, m->ev_copy, 0));       // the start iterate is needed at once
    }
    HOST_TRY(cudaMemcpyAsync(m->st_noise, noise_host, (size_t)batch * T * (nk == JS_NOISE_GUMBEL ? C : 1) * sizeof(float),
                             cudaMemcpyHostToDevice, cs));
    // copies of one stream run in order: this word changes after the noise has arrived
    *m->h_nflag = ++m->n_uploads;
    HOST_TRY(cudaMemcpyAsync(m->d_nflag, m->h_nflag, sizeof(unsigned), cudaMemcpyHostToDevice, cs));
    RunArgs r;
    memset(&r, 0, sizeof r);
    r.batch = batch; r.noise = m->st_noise; r.nk = nk; r.init = init_host ? m->st_init : nullptr;
    r.kmode = mode == JS_JACOBI ? KM_JACOBI : mode == JS_GAUSS_SEIDEL ? KM_SEQ : mode == JS_GS_JACOBI ? KM_GS_JACOBI
                                                                                                        : KM_JACOBI_GS;
    r.block = block; r.max_iters = max_iters;
    r.x = m->st_x; r.out_iters = m->st_iters;
    // only the tensor-core kernel of the masked MLPs waits for the noise by itself
    const bool overlap = m->kind == 0 && m->tc_ok && m->opt_path == 0 && (r.kmode == KM_JACOBI || r.kmode == KM_GS_JACOBI);
    if (overlap) {
        r.noise_ready = m->d_nflag;
        r.noise_stamp = m->n_uploads;
    } else {
        HOST_TRY(cudaEventRecord(m->ev_copy, cs));
        HOST_TRY(cudaStreamWaitEvent(st, m->ev_copy, 0));
    }
    rc = run_made(m, r, st);
    if (rc < 0) return leave(rc);
    HOST_TRY(cudaStreamSynchronize(cs));
    HOST_TRY(cudaMemcpyAsync(out_samples_host, m->st_x, (size_t)batch * T, cudaMemcpyDeviceToHost, st));
    if (out_iters_host)
        HOST_TRY(cudaMemcpyAsync(out_iters_host, m->st_iters, (size_t)batch * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    HOST_TRY(cudaStreamSynchronize(st));
#undef HOST_TRY
    return rc;
}

// ---- continuous states (logistic conditionals): masked MLPs with C == 2, CUDA-core kernels
static bool real_model_ok(const js_model *m) { return m && m->kind == 0 && m->made.C == 2; }

int jacobi_sample_real(const js_model *cm, int batch, const float *noise_dev, const float *init_dev, int mode, int block,
                       int max_iters, float eps, float *out_states_dev, int32_t *out_iters_dev, void *cuda_stream)
{
    js_model *m = const_cast<js_model *>(cm);
    if (!m || !noise_dev || !out_states_dev) return JS_ERR_ARG;
    if (!real_model_ok(m)) return JS_ERR_UNSUPPORTED;
    if (batch < 1 || batch > m->max_batch || !(eps >= 0.0f)) return JS_ERR_ARG;
    if (mode < JS_JACOBI || mode > JS_JACOBI_GS) return JS_ERR_ARG;
    if (mode == JS_JACOBI_GS) return JS_ERR_UNSUPPORTED;
    if (mode == JS_GS_JACOBI && (block < 1 || block > m->made.T)) return JS_ERR_ARG;
    RunArgs r;
    memset(&r, 0, sizeof r);
    r.batch = batch; r.noise = noise_dev; r.nk = JS_NOISE_LOGISTIC;
    r.kmode = mode == JS_JACOBI ? KM_JACOBI : mode == JS_GAUSS_SEIDEL ? KM_SEQ : KM_GS_JACOBI;
    r.block = block; r.max_iters = max_iters;
    r.real = 1; r.eps = eps; r.xr = out_states_dev; r.init_r = init_dev; r.out_iters = out_iters_dev;
    return run_made(m, r, (cudaStream_t)cuda_stream);
}

int sequential_sample_real(const js_model *cm, int batch, const float *noise_dev, float *out_states_dev, void *cuda_stream)
{
    js_model *m = const_cast<js_model *>(cm);
    if (!m || !noise_dev || !out_states_dev) return JS_ERR_ARG;
    if (!real_model_ok(m)) return JS_ERR_UNSUPPORTED;
    if (batch < 1 || batch > m->max_batch) return JS_ERR_ARG;
    RunArgs r;
    memset(&r, 0, sizeof r);
    r.batch = batch; r.noise = noise_dev; r.nk = JS_NOISE_LOGISTIC; r.kmode = KM_SEQ;
    r.real = 1; r.xr = out_states_dev;
    return run_made(m, r, (cudaStream_t)cuda_stream);
}

int js_forward_logits_real(const js_model *cm, int batch, const float *x_dev, float *logits_dev, void *cuda_stream)
{
    js_model *m = const_cast<js_model *>(cm);
    if (!m || !x_dev || !logits_dev) return JS_ERR_ARG;
    if (!real_model_ok(m)) return JS_ERR_UNSUPPORTED;
    if (batch < 1 || batch > m->max_batch) return JS_ERR_ARG;
    RunArgs r;
    memset(&r, 0, sizeof r);
    r.batch = batch; r.kmode = KM_FORWARD; r.real = 1; r.xin_r = x_dev; r.logits_out = logits_dev;
    return run_made(m, r, (cudaStream_t)cuda_stream);
}

int sequential_sample(const js_model *cm, int batch, const float *noise_dev, int nk, uint8_t *out_samples_dev,
                      void *cuda_stream)
{
    js_model *m = const_cast<js_model *>(cm);
    if (!m || !noise_dev || !out_samples_dev) return JS_ERR_ARG;
    if (batch < 1 || batch > m->max_batch) return JS_ERR_ARG;
    if (!noise_kind_ok(m, nk)) return JS_ERR_ARG;
    RunArgs r;
    memset(&r, 0, sizeof r);
    r.batch = batch; r.noise = noise_dev; r.nk = nk; r.kmode = KM_SEQ;
    r.x = out_samples_dev;
    return run_made(m, r, (cudaStream_t)cuda_stream);
}

int js_forward_logits(const js_model *cm, int batch, const uint8_t *x_dev, float *logits_dev, void *cuda_stream)
{
    js_model *m = const_cast<js_model *>(cm);
    if (!m || !x_dev || !logits_dev) return JS_ERR_ARG;
    if (batch < 1 || batch > m->max_batch) return JS_ERR_ARG;
    RunArgs r;
    memset(&r, 0, sizeof r);
    r.batch = batch; r.kmode = KM_FORWARD; r.x_in = x_dev; r.logits_out = logits_dev;
    r.x = m->x_tmp;
    return run_made(m, r, (cudaStream_t)cuda_stream);
}

int js_set_option(js_model *m, int option, int value)
{
    if (!m) return JS_ERR_ARG;
    switch (option) {
    case JS_OPT_FRONTIER_SKIP: m->opt_frontier_skip = value ? 1 : 0; return JS_OK;
    case JS_OPT_SEQ_SKIP: if (value < 0 || value > 2) return JS_ERR_ARG; m->opt_seq_skip = value; return JS_OK;
    case JS_OPT_SPIN_LIMIT: if (value < 0) return JS_ERR_ARG; m->opt_spin_limit = value; return JS_OK;
    case JS_OPT_PATH: if (value != 0 && value != 1) return JS_ERR_ARG; m->opt_path = value; return JS_OK;
    case JS_OPT_COMPACT: m->opt_compact = value ? 1 : 0; return JS_OK;
    case JS_OPT_TRACE: m->opt_trace = value > 0 ? value : 0; return JS_OK;
    default: return JS_ERR_ARG;
    }
}

int js_get_trace(const js_model *m, unsigned long long *out, int capacity)
{
    if (!m || !out || capacity < 0) return JS_ERR_ARG;
    const int n = 2 * JS_TRACE_PHASES * JS_TRACE_SLOTS;
    const int k = capacity < n ? capacity : n;
    if (cudaMemcpy(out, m->trace, sizeof(unsigned long long) * k, cudaMemcpyDeviceToHost) != cudaSuccess) return JS_ERR_CUDA;
    return k;
}

int js_get_stats(const js_model *m, js_stats *out)
{
    if (!m || !out) return JS_ERR_ARG;
    *out = m->stats;
    return JS_OK;
}

const char *js_strerror(int code)
{
    switch (code) {
    case JS_OK: return "ok";
    case JS_NOT_CONVERGED: return "iteration cap reached before every sample stopped changing";
    case JS_ERR_ARG: return "invalid argument";
    case JS_ERR_UNSUPPORTED: return "unsupported model shape or mode";
    case JS_ERR_CUDA: return "CUDA runtime error";
    case JS_ERR_TIMEOUT: return "a bounded device-side wait gave up";
    default: return "unknown code";
    }
}

const char *js_last_cuda_error(void) { return g_cuda_err; }

}  // extern "C"
