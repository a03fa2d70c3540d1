// jacobi_sample_noalloc: Jacobi sampling of a small fp32 masked MLP for callers
// that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the time they sample: a
// real-time loop that may not block on the allocator, a process whose device
// memory is entirely owned by another framework's pool, code running between
// two phases that forbid allocation.  js_made_create allocates (packed weights,
// activations, control words), so those callers cannot use it.  This entry
// point allocates nothing: the caller passes every input and output as device
// pointers (unmasked fp32 weights included; the masks of the default degree
// rule are applied on the fly), and everything the kernel needs besides -
// activations, logits, per-sample flags, the status word - lives in one
// file-scope device array of fixed size, below.
//
// Consequences the caller has to know:
//   * the array costs JS_NOALLOC_SCRATCH_BYTES on every GPU that loads the
//     library, until the process exits;
//   * a problem that needs more scratch than that is rejected with JS_ERR_ARG
//     (js_noalloc_scratch_needed tells how much a shape needs);
//   * every call uses the same array and finds the previous call's contents in
//     it; the kernel clears what has to start at zero.  Two calls that overlap
//     on the GPU (different streams or threads) race on it: serialise them;
//   * the first call on a device looks up the array's device address
//     (cudaGetSymbolAddress, with that device current) and is the call that makes
//     the driver load this library's device code and the array itself onto that
//     GPU, so it may take the driver's allocator once: make one warm-up call per
//     device at start-up, before the phase that must not allocate and before any
//     stream capture begins.  The array that serves a call is the one of the
//     CURRENT device; cuda_stream must belong to that device;
//   * every call copies a status word back and synchronises cuda_stream before it
//     returns.
// The kernel is a single-CTA restatement of the CUDA-core sampler (same
// accumulation order, same sampling rule), so its samples and iteration counts
// equal jacobi_sample's in JS_JACOBI mode on the same fp32 model.
#include <cstdio>
#include <cstring>

#include "js_common.cuh"

#define JS_NOALLOC_SCRATCH_BYTES (4u << 20)
#define JS_NOALLOC_THREADS 512
#define JS_NOALLOC_MAX_DEVICES 64

static __device__ __align__(256) unsigned char g_noalloc_scratch[JS_NOALLOC_SCRATCH_BYTES];

namespace {

struct NoallocNet {
    int T, C, L, act;
    int n[JS_MAXL + 2];
    const float *W[JS_MAXL + 1];
    const float *b[JS_MAXL + 1];
    const float *lut;
};

struct NoallocHeader {      // first 256 bytes of the scratch
    int status;
    int iterations;
    int any;
    int pad[61];
};

__host__ __device__ inline size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

// degree of unit i of layer l (0 = inputs, 1..L hidden, L+1 outputs) under the default rule
__device__ __forceinline__ int unit_degree(const NoallocNet &net, int l, int i)
{
    if (l == 0) return i + 1;
    if (l == net.L + 1) return i / net.C + 1;
    return 1 + (int)(((long long)i * (net.T - 1)) / net.n[l]);
}

__global__ void __launch_bounds__(JS_NOALLOC_THREADS)
noalloc_jacobi_kernel(const NoallocNet net, unsigned char *scratch, int batch, const float *noise, int nk,
                      const uint8_t *init, int max_iters, uint8_t *x, int32_t *out_iters)
{
    // carve the scratch; the host checked that it fits
    NoallocHeader *hdr = reinterpret_cast<NoallocHeader *>(scratch);
    size_t off = sizeof(NoallocHeader);
    int *changed = reinterpret_cast<int *>(scratch + off); off = align256(off + sizeof(int) * batch);
    int *done = reinterpret_cast<int *>(scratch + off); off = align256(off + sizeof(int) * batch);
    float *a[JS_MAXL + 1];
    for (int l = 0; l <= net.L; ++l) {
        a[l] = reinterpret_cast<float *>(scratch + off);
        off = align256(off + sizeof(float) * (size_t)batch * net.n[l]);
    }
    float *z = reinterpret_cast<float *>(scratch + off);

    const int tid = threadIdx.x, nth = blockDim.x;
    const int T = net.T, C = net.C, L = net.L;

    // the array keeps the last call's contents: clear what must start at zero
    if (tid == 0) { hdr->status = JS_OK; hdr->iterations = 0; hdr->any = 0; }
    for (int b = tid; b < batch; b += nth) { changed[b] = 0; done[b] = 0; }
    for (int i = tid; i < batch * T; i += nth) {
        const uint8_t v = init ? init[i] : (uint8_t)0;
        x[i] = v;
        a[0][i] = net.lut[v];
    }
    __syncthreads();

    const int cap = (max_iters > 0 && max_iters < T) ? max_iters : T;
    int status = JS_OK, k = 0;
    for (k = 1;; ++k) {
        // masked forward pass on the current iterate
        for (int l = 0; l <= L; ++l) {
            const int nin = net.n[l], nout = net.n[l + 1];
            const bool is_out = (l == L);
            for (int idx = tid; idx < batch * nout; idx += nth) {
                const int b = idx / nout, i = idx % nout;
                const int gi = unit_degree(net, l + 1, i);
                const float *w = net.W[l] + (size_t)i * nin;
                const float *in = a[l] + (size_t)b * nin;
                float acc = 0.0f;
                for (int j = 0; j < nin; ++j) {
                    const int gj = unit_degree(net, l, j);
                    const bool keep = is_out ? (gi > gj) : (gi >= gj);
                    acc = fmaf(in[j], keep ? w[j] : 0.0f, acc);
                }
                const float pre = acc + net.b[l][i];
                if (is_out) z[(size_t)b * nout + i] = pre;
                else a[l + 1][(size_t)b * nout + i] = js_act_fn(net.act, pre);
            }
            __syncthreads();
        }
        // sampling against the fixed noise, compare with the previous iterate
        if (C == 1) {
            for (int i = tid; i < batch * T; i += nth) {
                const int xn = js_sample_binary(nk, z[i], noise[i]);
                if (xn != x[i]) {
                    x[i] = (uint8_t)xn;
                    a[0][i] = net.lut[xn];
                    changed[i / T] = 1;
                    hdr->any = 1;
                }
            }
        } else {
            const int lane = tid & 31;
            for (int i = tid >> 5; i < batch * T; i += nth >> 5) {
                const float *zz = z + (size_t)i * C, *gg = noise + (size_t)i * C;
                float best = -INFINITY;
                int bi = INT_MAX;
                for (int c = lane; c < C; c += 32) {
                    const float v = zz[c] + gg[c];
                    if (v > best) { best = v; bi = c; }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    const float ov = __shfl_xor_sync(0xffffffffu, best, o);
                    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                    if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
                }
                if ((unsigned)bi >= (unsigned)C) bi = 0;      // no finite score in the row (NaN or -inf everywhere): class 0
                if (lane == 0 && bi != x[i]) {
                    x[i] = (uint8_t)bi;
                    a[0][i] = net.lut[bi];
                    changed[i / T] = 1;
                    hdr->any = 1;
                }
            }
        }
        __syncthreads();
        const int any = hdr->any;
        for (int b = tid; b < batch; b += nth) {
            if (!done[b] && (changed[b] == 0 || k == cap)) {
                done[b] = 1;
                if (out_iters) out_iters[b] = k;
            }
            changed[b] = 0;
        }
        __syncthreads();
        if (tid == 0) hdr->any = 0;
        __syncthreads();
        if (!any || k == cap) {
            if (any && cap < T) status = JS_NOT_CONVERGED;
            break;
        }
    }
    if (tid == 0) { hdr->status = status; hdr->iterations = k; }
}

size_t scratch_needed(const js_noalloc_made *net, int batch)
{
    size_t off = sizeof(NoallocHeader);
    off = align256(off + sizeof(int) * (size_t)batch);
    off = align256(off + sizeof(int) * (size_t)batch);
    off = align256(off + sizeof(float) * (size_t)batch * net->T);
    for (int l = 0; l < net->L; ++l) off = align256(off + sizeof(float) * (size_t)batch * net->H[l]);
    off += sizeof(float) * (size_t)batch * net->T * net->C;
    return off;
}

thread_local char g_noalloc_err[200] = "";
unsigned char *g_scratch_ptr[JS_NOALLOC_MAX_DEVICES];   // device address of the array, per device

}  // namespace

extern "C" {

size_t js_noalloc_scratch_limit(void) { return JS_NOALLOC_SCRATCH_BYTES; }

size_t js_noalloc_scratch_needed(const js_noalloc_made *net, int batch)
{
    if (!net || batch < 1 || net->L < 1 || net->L > JS_MAXL) return 0;
    return scratch_needed(net, batch);
}

const char *js_noalloc_last_error(void) { return g_noalloc_err; }

int jacobi_sample_noalloc(const js_noalloc_made *net, int batch, const float *noise_dev, int nk,
                          const uint8_t *init_dev, int max_iters, uint8_t *out_samples_dev, int32_t *out_iters_dev,
                          void *cuda_stream)
{
    g_noalloc_err[0] = 0;
    if (!net || !noise_dev || !out_samples_dev || batch < 1) return JS_ERR_ARG;
    if (net->T < 1 || net->C < 1 || net->C > 256 || net->L < 1 || net->L > JS_MAXL || !net->lut_dev) return JS_ERR_ARG;
    if (net->act != JS_ACT_RELU && net->act != JS_ACT_GELU_TANH) return JS_ERR_ARG;
    for (int l = 0; l < net->L; ++l)
        if (net->H[l] < 1) return JS_ERR_ARG;
    for (int l = 0; l <= net->L; ++l)
        if (!net->W_dev[l] || !net->b_dev[l]) return JS_ERR_ARG;
    if (nk == JS_NOISE_GUMBEL ? net->C == 1 : (net->C != 1 || (nk != JS_NOISE_UNIFORM_ICDF && nk != JS_NOISE_LOGISTIC)))
        return JS_ERR_ARG;
    const size_t need = scratch_needed(net, batch);
    if (need > JS_NOALLOC_SCRATCH_BYTES) {
        snprintf(g_noalloc_err, sizeof g_noalloc_err,
                 "jacobi_sample_noalloc: this shape needs %zu bytes of scratch, the built-in array holds %u",
                 need, JS_NOALLOC_SCRATCH_BYTES);
        return JS_ERR_ARG;
    }
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= JS_NOALLOC_MAX_DEVICES) {
        snprintf(g_noalloc_err, sizeof g_noalloc_err, "jacobi_sample_noalloc: no usable current CUDA device");
        return JS_ERR_CUDA;
    }
    // set-up, once per device, with that device current: in host code the array's name is only a
    // stand-in, the kernel needs the address the runtime reports for it
    if (!g_scratch_ptr[dev]) {
        unsigned char *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress((void **)&p, g_noalloc_scratch);
        if (e != cudaSuccess || !p) {
            snprintf(g_noalloc_err, sizeof g_noalloc_err, "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
            return JS_ERR_CUDA;
        }
        g_scratch_ptr[dev] = p;
    }
    unsigned char *scratch = g_scratch_ptr[dev];

    NoallocNet k;
    memset(&k, 0, sizeof k);
    k.T = net->T; k.C = net->C; k.L = net->L; k.act = net->act;
    k.n[0] = net->T;
    for (int l = 0; l < net->L; ++l) k.n[l + 1] = net->H[l];
    k.n[net->L + 1] = net->T * net->C;
    for (int l = 0; l <= net->L; ++l) { k.W[l] = net->W_dev[l]; k.b[l] = net->b_dev[l]; }
    k.lut = net->lut_dev;

    cudaStream_t st = (cudaStream_t)cuda_stream;
    noalloc_jacobi_kernel<<<1, JS_NOALLOC_THREADS, 0, st>>>(k, scratch, batch, noise_dev, nk, init_dev, max_iters,
                                                             out_samples_dev, out_iters_dev);
    cudaError_t e = cudaGetLastError();
    NoallocHeader h;
    if (e == cudaSuccess) e = cudaMemcpyAsync(&h, scratch, sizeof h, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) {
        snprintf(g_noalloc_err, sizeof g_noalloc_err, "jacobi_sample_noalloc: %s", cudaGetErrorString(e));
        return JS_ERR_CUDA;
    }
    return h.status;
}

}  // extern "C"
