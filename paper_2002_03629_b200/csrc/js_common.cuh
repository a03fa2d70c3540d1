// Shared declarations of the sampler library: device-side model views, the
// control block of the persistent kernels and the bounded grid barrier.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <limits.h>
#include <stdint.h>

#include "../../include/jacobi_sample.h"

#define JS_MAXL 8
#define JS_TRACE_PHASES 256
#define JS_TRACE_SLOTS 12
#define JS_GT 64          // output-tile edge of the CUDA-core GEMM phases

enum { KM_JACOBI = 0, KM_SEQ = 1, KM_GS_JACOBI = 2, KM_JACOBI_GS = 3, KM_FORWARD = 4,
       KM_HIDDEN = 5 };      // KM_HIDDEN: hidden layers only, on the symbols x_in (activations for the sweeps)

// Control block in device memory, zeroed by the host before every launch.
struct JsCtl {
    unsigned bar_count;     // grid barrier: monotonically increasing arrival counter
    int abort;              // set when a bounded wait gave up; every CTA then leaves
    int status;             // JS_OK / JS_NOT_CONVERGED / JS_ERR_TIMEOUT
    int agg_any[2];         // per iteration parity: did any sample change
    int agg_minfirst[2];    // per iteration parity: smallest changed position
    int iterations;         // forward passes executed
    int frontier;           // leading positions known final at exit
    int iters_max;
    int live;               // samples still iterating (tensor-core path)
    int compactions;        // times the working batch was compacted
    unsigned long long tiles_issued, tiles_skipped;
    unsigned long long mma_flops;       // flops of the tcgen05.mma instructions issued (tile padding included)
    unsigned long long weight_bytes;    // bytes of weight tiles loaded for the first row tile of every unit (unique weight bytes a pass streams)
    unsigned exit_count;    // CTAs that have left; the last one reports and clears the block
};

// Device view of a masked MLP.  Layer l maps a[l] (width n[l]) to a[l+1].
struct MadeDev {
    int T, C, L, act, prec;
    int n[JS_MAXL + 2];
    const void *W[JS_MAXL + 1];       // masked weights [n[l+1]][n[l]], float or bf16
    const float *bias[JS_MAXL + 1];
    void *a[JS_MAXL + 1];             // activations [rows][n[l]], float or bf16 (a[0] = encoded iterate)
    void *a_old[JS_MAXL + 1];         // Jacobi-GS: activations of the previous outer iterate
    const int *deg[JS_MAXL + 2];      // degree of every unit
    const int *t_kend[JS_MAXL + 1];   // per JS_GT-wide output tile: inputs beyond this index are masked
    const int *t_dmin[JS_MAXL + 1];   // per tile: smallest / largest degree inside
    const int *t_dmax[JS_MAXL + 1];
    const float *lut;
    float *logits;                    // scratch [rows][T*C]
};

struct RunArgs {
    int batch;
    const float *noise;
    int nk;
    const uint8_t *init;
    int kmode;
    int block;
    int max_iters;
    uint8_t *x;               // working iterate = output samples [batch][T]
    uint8_t *x_old;           // scratch [batch][T] (Jacobi-GS)
    int32_t *out_iters;       // may be NULL
    int *smp_changed;         // [2][batch] per-sample change flags by iteration parity
    int *smp_state;           // [2][batch] per-sample bookkeeping (done flag, running count)
    const uint8_t *x_in;      // KM_FORWARD: symbols
    float *logits_out;        // KM_FORWARD: destination
    int *perm;                // [2][perm_stride]: working row -> sample index, by compaction parity
    int perm_stride;
    int frontier_skip, seq_skip, compact;
    // continuous states (C == 2: location and log-scale per position): real != 0, states are floats
    int real;
    float eps;                // stop when the largest change of a sample's states is <= eps
    float *xr;                // working iterate = output states [batch][T]
    const float *init_r;      // start iterate or NULL (zeros)
    const float *xin_r;       // KM_FORWARD: states to evaluate the network on
    int blk_lo;               // sweeps: first block that is swept (earlier ones are final)
    int hid_lo;               // KM_HIDDEN: hidden units of degree <= hid_lo are final already
    unsigned spin_limit;
    JsCtl *ctl;
    const unsigned *noise_ready;   // NULL, or a word that takes the value noise_stamp once `noise` has arrived
    unsigned noise_stamp;
    JsCtl *result;            // host memory mapped into the device: the last CTA to leave copies ctl here
    unsigned long long *trace;   // [2 CTAs][JS_TRACE_PHASES][JS_TRACE_SLOTS] globaltimer stamps, or NULL
    int trace_cta;               // the second traced CTA (the first is CTA 0); < 0: the last CTA of the grid
};

// which of the two traced CTAs this one is (0, 1), or -1
__device__ __forceinline__ int js_trace_who(const RunArgs &r)
{
    if (blockIdx.x == 0) return 0;
    const unsigned second = r.trace_cta >= 0 && r.trace_cta < (int)gridDim.x ? (unsigned)r.trace_cta : gridDim.x - 1;
    return blockIdx.x == second ? 1 : -1;
}

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int ld_volatile_i32(const int *p)
{
    int v;
    asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Grid-wide barrier for a cooperative (co-resident) launch.  Every CTA calls it
// the same number of times; `epoch` counts the calls.  The wait is bounded: after
// spin_limit polls, or when another CTA has given up, the CTA raises `abort` and
// the function returns false in every thread of the CTA; the caller must then
// leave the kernel.  Returns true when all CTAs have arrived.
__device__ __forceinline__ bool grid_barrier(JsCtl *ctl, unsigned &epoch, unsigned spin_limit)
{
    __syncthreads();
    epoch += 1;
    if (gridDim.x == 1) return true;      // a single CTA: the block-wide barrier above is all there is to wait for
    int ok = 1;
    if (threadIdx.x == 0) {
        const unsigned target = epoch * gridDim.x;
        // arrive: a release at gpu scope (it also covers the other threads' writes, ordered before it
        // by the __syncthreads above) with no value to wait for; the polls below are acquires
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(&ctl->bar_count) : "memory");
        unsigned polls = 0;
        while (ld_acquire_u32(&ctl->bar_count) < target) {
            if (++polls > spin_limit || ld_volatile_i32(&ctl->abort) != 0) {
                atomicExch(&ctl->abort, 1);
                ok = 0;
                break;
            }
            if (polls > 64) __nanosleep(64);
        }
        if (ok && ld_volatile_i32(&ctl->abort) != 0) ok = 0;
    }
    return __syncthreads_and(ok) != 0;
}

__device__ __forceinline__ float js_act_fn(int act, float v)
{
    if (act == JS_ACT_RELU) return fmaxf(v, 0.0f);
    const float y = 0.7978845608028654f * (v + 0.044715f * v * v * v);
    return 0.5f * v * (1.0f + tanhf(y));
}

// x_t from the logits of position t and its reserved noise (Appendix A.3), binary kinds
__device__ __forceinline__ int js_sample_binary(int nk, float z, float noise)
{
    if (nk == JS_NOISE_UNIFORM_ICDF) {
        const float p = 1.0f / (1.0f + expf(-z));
        return noise < p ? 1 : 0;
    }
    return (z + noise) > 0.0f ? 1 : 0;
}

// x_t of a C-way position, computed by one warp from the position's logits (Appendix A.3).
//   JS_NOISE_GUMBEL       noise = C Gumbel numbers: argmax_c (z_c + g_c), lowest index among equals
//   JS_NOISE_UNIFORM_CAT  noise = one uniform number u: the first class c with u * S < sum_{i<=c} e_i,
//                         e_i = exp(z_i - max z), S = sum of all e_i (inverse CDF of the softmax)
// Every lane returns the class; a row without a finite score gives class 0.
__device__ __forceinline__ int js_warp_sample_cat(int nk, const float *zz, const float *noise, int C, int lane)
{
    if (nk == JS_NOISE_UNIFORM_CAT) {
        float mx = -INFINITY;
        for (int c = lane; c < C; c += 32) mx = fmaxf(mx, zz[c]);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
        // two passes over the classes in chunks of 32 (lane = class inside the chunk): the total,
        // then the running sums; a chunk's running sums are an inclusive scan across the lanes
        float total = 0.0f;
        for (int c0 = 0; c0 < C; c0 += 32) {
            float e = (c0 + lane < C) ? expf(zz[c0 + lane] - mx) : 0.0f;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const float o = __shfl_up_sync(0xffffffffu, e, off);
                if (lane >= off) e += o;
            }
            total += __shfl_sync(0xffffffffu, e, 31);
        }
        const float target = noise[0] * total;
        float carry = 0.0f;
        int found = INT_MAX;
        for (int c0 = 0; c0 < C && found == INT_MAX; c0 += 32) {
            float e = (c0 + lane < C) ? expf(zz[c0 + lane] - mx) : 0.0f;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const float o = __shfl_up_sync(0xffffffffu, e, off);
                if (lane >= off) e += o;
            }
            const float run = carry + e;
            const unsigned hit = __ballot_sync(0xffffffffu, c0 + lane < C && target < run);
            if (hit) found = c0 + __ffs((int)hit) - 1;
            carry += __shfl_sync(0xffffffffu, e, 31);
        }
        if (found == INT_MAX) found = (total == total) ? C - 1 : 0;      // u at the very top, or no finite score
        return found;
    }
    float best = -INFINITY;
    int bi = INT_MAX;
    for (int c = lane; c < C; c += 32) {
        const float v = zz[c] + noise[c];
        if (v > best) { best = v; bi = c; }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, off);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
        if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
    }
    if ((unsigned)bi >= (unsigned)C) bi = 0;      // no finite score in the row: class 0
    return bi;
}

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// host-side launchers implemented by the kernel files
int js_launch_made_generic(const MadeDev &m, const RunArgs &r, int grid_limit, cudaStream_t stream);
int js_made_generic_max_grid(int prec);
