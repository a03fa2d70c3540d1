// Device-side solver loops shared by the masked-MLP kernels.  An engine supplies
// the phases (grid barrier, initialisation, one windowed forward pass with the
// sampling step); the driver is the control logic of Algorithms 1-3 and of the
// strict feedforward order, executed identically by every thread of every CTA.
//
// Window bookkeeping.  fin_x = number of leading positions of the current
// iterate known to be final; fin_h = hidden units of degree <= fin_h hold their
// final values.  The proof of Proposition 1 gives fin_x >= k after k Jacobi
// iterations; more sharply, if an iteration left positions < j unchanged they
// solve their equations, so positions <= j are final.  A forward pass on an
// iterate with fin_x final positions makes hidden units of degree <= fin_x final.
#pragma once
#include <limits.h>

#include "js_common.cuh"

struct Win {
    int hdeg_lo;   // hidden units of degree <= hdeg_lo are final: not recomputed
    int hdeg_hi;   // hidden units of degree >  hdeg_hi are not needed yet
    int plo, phi;  // output positions [plo, phi) are sampled and committed
    int olo, ohi;  // output positions [olo, ohi) are computed (>= the committed range)
};

__device__ __forceinline__ Win make_win(int hlo, int hhi, int plo, int phi)
{
    Win w = {hlo, hhi, plo, phi, plo, phi};
    return w;
}

__device__ __forceinline__ void note_change(const RunArgs &r, int parity, int b, int d)
{
    atomicOr(&r.smp_changed[parity * r.batch + b], 1);
    atomicMin(&r.ctl->agg_minfirst[parity], d);
    atomicOr(&r.ctl->agg_any[parity], 1);
}

// After the barrier that ends an iteration: CTA 0 clears the other parity's flags.
// Safe because every CTA read that parity before it passed at least one later
// barrier, and nobody writes it again before at least one more barrier.
__device__ __forceinline__ void reset_other_parity(const RunArgs &r, int parity)
{
    if (blockIdx.x != 0) return;
    const int o = parity ^ 1;
    for (int i = threadIdx.x; i < r.batch; i += blockDim.x) r.smp_changed[o * r.batch + i] = 0;
    if (threadIdx.x == 0) {
        r.ctl->agg_any[o] = 0;
        r.ctl->agg_minfirst[o] = INT_MAX;
    }
}

// CTA 0: a sample whose iterate did not change (or that hit the cap) stops counting.
__device__ __forceinline__ void book_samples(const RunArgs &r, int parity, int k, bool at_cap, bool add,
                                             bool final_write)
{
    if (blockIdx.x != 0) return;
    int *done = r.smp_state, *count = r.smp_state + r.batch;
    for (int b = threadIdx.x; b < r.batch; b += blockDim.x) {
        if (!done[b] && (r.smp_changed[parity * r.batch + b] == 0 || at_cap)) {
            done[b] = 1;
            count[b] = add ? count[b] + k : k;
            if (final_write && r.out_iters) r.out_iters[b] = count[b];
            atomicMax(&r.ctl->iters_max, count[b]);
        }
    }
}

struct DriverResult {
    int status, iterations, frontier;
    bool alive;
};

// The solver loops are written as ONE loop with ONE call of the engine's forward pass: the
// engines inline their whole pipeline into that call, and a copy per solver would multiply the
// kernel's code size (the persistent kernels are instruction-cache sensitive).
template <class E>
__device__ DriverResult made_driver(E &e, int T_, const RunArgs &r)
{
    DriverResult res = {JS_OK, 0, 0, true};
    JsCtl *ctl = r.ctl;
    const int mode = r.kmode;

    if (mode == KM_JACOBI_GS) {
        e.init(r.init);
        if (!e.barrier()) { res.alive = false; return res; }
        if constexpr (E::has_jgs) {
            // Algorithm 2: all blocks in parallel, a sequential sweep inside each.
            const int B = r.block, M = (T_ + B - 1) / B;
            const int cap = (r.max_iters > 0 && r.max_iters < M) ? r.max_iters : M;
            int fin_x = 0, fin_h = 0;
            for (int k = 1;; ++k) {
                const int p = k & 1;
                if (!e.jgs_outer(p, r.frontier_skip ? fin_h : 0, r.frontier_skip ? fin_x / B : 0, res.iterations)) {
                    res.alive = false;
                    return res;
                }
                const int any = ld_volatile_i32(&ctl->agg_any[p]);
                const int mf = ld_volatile_i32(&ctl->agg_minfirst[p]);
                book_samples(r, p, k, k == cap, false, true);
                reset_other_parity(r, p);
                fin_h = max(fin_h, fin_x);
                // after outer iteration k the first k blocks are final (proof of Prop. 2)
                fin_x = any ? max(min(k * B, T_), min(mf + 1, T_)) : T_;
                if (!any || k == cap) {
                    if (any && cap < M) res.status = JS_NOT_CONVERGED;
                    break;
                }
            }
            res.frontier = fin_x;
        } else {
            res.status = JS_ERR_UNSUPPORTED;
        }
        return res;
    }
    if (mode != KM_FORWARD && mode != KM_HIDDEN && mode != KM_SEQ && mode != KM_JACOBI && mode != KM_GS_JACOBI) {
        res.status = JS_ERR_ARG;
        return res;
    }

    e.init((mode == KM_FORWARD || mode == KM_HIDDEN) ? r.x_in : mode == KM_SEQ ? (const uint8_t *)nullptr : r.init);
    if (!e.barrier()) { res.alive = false; return res; }

    // state shared by the modes
    const int B = mode == KM_GS_JACOBI ? r.block : T_;     // Jacobi = one block of all positions
    int fin_x = 0, fin_h = 0;      // see the header comment
    int a = 0;                     // start of the current block (GS-Jacobi) / position (sequential order)
    int lo = 0;                    // positions of the current block below lo are settled
    int k = 0;                     // iteration inside the current block
    int tick = 0;                  // forward passes with change flags so far (parity of the flag buffers)
    for (;;) {
        Win w;
        bool flag = false;
        float *zout = nullptr;
        const int bend = min(a + B, T_), len = bend - a;
        if (mode == KM_FORWARD) {
            w = make_win(0, T_, 0, T_);
            zout = r.logits_out;
        } else if (mode == KM_HIDDEN) {
            w = make_win(r.hid_lo, T_, 0, 0);               // no output position: the hidden layers alone
        } else if (mode == KM_SEQ) {
            // Eq. 1 in strict order: step a keeps position a of a forward pass
            w = make_win(0, T_, a, a + 1);
            if (r.seq_skip) w.hdeg_lo = a - 1, w.hdeg_hi = a;     // only the units that became computable
            else w.olo = 0, w.ohi = T_;                           // the whole network, every step
        } else {
            // Algorithm 1 (one block) or the inner loop of Algorithm 3 (block [a, bend))
            k += 1;
            tick += 1;
            flag = true;
            w = r.frontier_skip ? make_win(fin_h, bend - 1 + (mode == KM_JACOBI), lo, bend)
                                : make_win(0, T_, a, bend);
        }
        const int p = tick & 1;
        if (!e.step(w, flag, p, zout)) { res.alive = false; return res; }
        res.iterations++;

        if (mode == KM_FORWARD || mode == KM_HIDDEN) break;
        if (mode == KM_SEQ) {
            if (++a == T_) break;
            continue;
        }
        const int cap = (r.max_iters > 0 && r.max_iters < len) ? r.max_iters : len;
        const int any = ld_volatile_i32(&ctl->agg_any[p]);
        const int mf = ld_volatile_i32(&ctl->agg_minfirst[p]);
        book_samples(r, p, k, k == cap, mode == KM_GS_JACOBI, mode == KM_JACOBI);
        reset_other_parity(r, p);
        fin_h = max(fin_h, min(fin_x, mode == KM_JACOBI ? T_ : bend - 1));
        lo = any ? max(lo + 1, min(mf + 1, bend)) : bend;
        fin_x = max(fin_x, lo);
        if (any && k < cap) {
            // samples that stopped changing are at their fixed point: drop them from the working
            // batch when that frees a whole tile of rows (hidden rows are then recomputed)
            if (mode == KM_JACOBI && r.compact) {
                const int c = e.compact(p);
                if (c < 0) { res.alive = false; return res; }
                if (c > 0) fin_h = 0;
            }
            continue;
        }
        // the block is finished: unchanged, or at its cap
        if (any && cap < len) res.status = JS_NOT_CONVERGED;
        if (mode == KM_JACOBI) break;
        fin_x = bend;          // positions < bend are never touched again: settled
        if (blockIdx.x == 0)   // new block: nobody is done (same threads wrote these entries)
            for (int b = threadIdx.x; b < r.batch; b += blockDim.x) r.smp_state[b] = 0;
        a = bend;
        lo = a;
        k = 0;
        if (a >= T_) break;
    }
    if (mode == KM_SEQ) {
        res.frontier = T_;
        if (blockIdx.x == 0 && r.out_iters)
            for (int b = threadIdx.x; b < r.batch; b += blockDim.x) r.out_iters[b] = 1;
    } else if (mode == KM_GS_JACOBI) {
        res.frontier = T_;
        if (blockIdx.x == 0 && r.out_iters)
            for (int b = threadIdx.x; b < r.batch; b += blockDim.x) r.out_iters[b] = r.smp_state[r.batch + b];
    } else if (mode == KM_JACOBI) {
        res.frontier = fin_x;
    }
    return res;
}

// Every CTA adds its statistics; the last one to leave copies the control block to the caller's
// mapped host memory (so that the host needs no device-to-host copy) and zeroes it, ready for
// the next launch (so that the host needs no memset either, unless a call ended abnormally).
__device__ __forceinline__ void driver_finish(const RunArgs &r, const DriverResult &res, unsigned long long issued,
                                              unsigned long long skipped, unsigned long long mma_flops = 0,
                                              unsigned long long weight_bytes = 0)
{
    if (threadIdx.x != 0) return;
    JsCtl *c = r.ctl;
    atomicAdd(&c->tiles_issued, issued);
    atomicAdd(&c->tiles_skipped, skipped);
    if (mma_flops) atomicAdd(&c->mma_flops, mma_flops);
    if (weight_bytes) atomicAdd(&c->weight_bytes, weight_bytes);
    if (blockIdx.x == 0) {
        c->iterations = res.iterations;
        c->frontier = res.frontier;
    }
    if (!res.alive) atomicExch(&c->abort, 1);
    __threadfence();
    if (atomicAdd(&c->exit_count, 1u) != gridDim.x - 1) return;
    __threadfence();
    // word-wise through volatile pointers: the block was written by other CTAs
    constexpr int NW = sizeof(JsCtl) / 4;
    unsigned w[NW];
    volatile unsigned *cw = reinterpret_cast<volatile unsigned *>(c);
    for (int i = 0; i < NW; ++i) w[i] = cw[i];
    JsCtl *o = reinterpret_cast<JsCtl *>(w);
    o->status = o->abort != 0 ? JS_ERR_TIMEOUT : res.status;     // res.status is the same in every CTA
    if (r.result) {
        volatile unsigned *rw = reinterpret_cast<volatile unsigned *>(r.result);
        for (int i = 0; i < NW; ++i) rw[i] = w[i];
        __threadfence_system();
    }
    for (int i = 0; i < NW; ++i) cw[i] = 0u;
}
