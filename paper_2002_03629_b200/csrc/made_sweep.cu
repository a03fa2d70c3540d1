// Cached sequential sweeps of a masked MLP with binary positions, on the sm_100a tensor cores.
//
// A sweep computes positions a .. b-1 of a block strictly in order (Eq. 1 of arXiv 2002.03629),
// each from the positions before it: positions < a are given (their hidden activations come from
// a forward pass on the previous iterate), positions inside the block are the fresh ones.  That is
// the inner loop of Jacobi-GS (Algorithm 2: all blocks in parallel, a sweep inside each) and, with
// one block covering every position, the feedforward pass itself with every hidden unit evaluated
// once (the cached sampler of Section 4.2).
//
// Work decomposition.  A job is (128 samples, one block); jobs never talk to each other, so the
// kernel needs no grid-wide synchronisation at all.  Inside a job the positions are taken in
// groups of G.  With sorted degrees, everything a group needs from before the group - inputs and
// hidden units of degree <= t0, the group's first position - is a PREFIX of every layer's units,
// so its contribution to the group's G output logits and to the handful of hidden units of degree
// t0+1 .. t0+G is a GEMM  [128 samples x prefix] x [prefix x (<= 32 units)]  per layer: TMA feeds
// the prefix of the activations (from the previous iterate's activations up to the block's start,
// from the job's own buffer F after it) and 16-row weight boxes, tcgen05.mma accumulates in tensor
// memory.  What the units of the group contribute to one another is a triangular system of at most
// 32 x 32 weights per layer, solved position by position with thread = sample row: logit, sample
// against the fixed noise (Appendix A.3), then the hidden units that the new symbol makes
// computable.  The group's activations then go to F, where the next group's GEMMs find them.
//
// Every value is a fixed function of the iterate: the split into prefix and group depends on the
// block size and the position alone.  Waits are bounded as in the other tensor-core kernels.
#include <cuda.h>

#include <algorithm>
#include <vector>

#include "js_common.cuh"
#include "js_model.h"
#include "made_driver.cuh"
#include "tc_common.cuh"

namespace {

constexpr int BM = TC_BM, BK = TC_BK;
constexpr int NTH = 192;
constexpr int NUP = 32;                      // most units of one layer inside a group
constexpr int GMAX = 32;                     // most positions per group
constexpr int A_BYTES = BM * BK * 2;
constexpr int NB = 128;                      // units per chunk of a base GEMM
constexpr int GPB = 8;                       // groups per base: a base GEMM serves the next GPB groups
constexpr int W_BYTES = NB * BK * 2;
constexpr int STAGE_BYTES = A_BYTES + W_BYTES;          // 32 KB, a multiple of 1 KB
constexpr int BASE_COL = 256;                // tensor-memory columns of the two base accumulators (NB each)
constexpr int XS = BM + 1;                    // row stride of X and Nz: a lane per position writes without bank conflicts
constexpr int MAX_STAGES = 10;
constexpr int SMEM_DYN_MAX = 227 * 1024 - 4 * 1024;

struct SwShared {
    uint64_t full[MAX_STAGES], empty[MAX_STAGES], tfull, tempty, gdone, bfull[2], bempty[2];
    int kbs[JS_MAXL + 1], ub0[JS_MAXL + 1];  // current base: its K blocks per layer (0: none), its first unit
    uint32_t tmem_base;
    int stop;
    float lut_s[2];
    // geometry of the current group, per GEMM l (activations a[l] -> a[l+1])
    int kin0[JS_MAXL + 1], nin[JS_MAXL + 1], u0[JS_MAXL + 1], nu[JS_MAXL + 1], kb_n[JS_MAXL + 1];
    int cs[JS_MAXL + 1][GMAX + 2];           // cs[l][i] = units of a[l] with degree <= t0 + i   (l >= 1)
    float bias_s[JS_MAXL + 1][NUP];
};

struct Geo { int kin0, kb_n, nin, u0, nu, npad; };
struct Base { int kbs, ub0, nb; };           // K blocks [0, kbs), units [ub0, ub0 + nb)

// shared-memory accesses by 32-bit shared address: the position loop runs on one warp per scheduler, and
// a generic load (which is what a pointer kept in a structure compiles to) waits much longer than ld.shared
__device__ __forceinline__ float4 lds_f4(uint32_t a)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ void sts_f4(uint32_t a, float4 v)
{
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(a), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ float lds_f(uint32_t a)
{
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ void sts_f(uint32_t a, float v) { asm volatile("st.shared.f32 [%0], %1;" ::"r"(a), "f"(v) : "memory"); }

// Position i of the group when every hidden layer gains exactly one unit there (byte l of jn_packed: its index among
// the group's units of a[l+1]).  The chain  symbol -> unit of a[1] -> ... -> unit of a[L]  is one scalar
// fused multiply-add and one activation per layer: the unit's running sum and the one weight are
// loaded beforehand, so no shared-memory round trip sits between two layers.  The additions to the
// running sums of everything else in the group (32 per layer) come after the chain, the loads of one
// layer issued before the arithmetic of the layer below: a warp issues in order, and with one warp
// per scheduler nothing else hides a load.  Every running sum receives exactly the operations, in
// exactly the order, of the general path (SweepEngine::scatter).  vbase: the thread's row in slot 0 of V.
template <int L>
__device__ __forceinline__ void position_one_each(uint32_t wbase, uint32_t vbase, int act, int i, float enc, int row,
                                               uint32_t jn_packed)
{
    const int sw7 = row & 7;
    int jn[L];
#pragma unroll
    for (int l = 0; l < L; ++l) jn[l] = (int)((jn_packed >> (8 * l)) & 255u);
    float p[L], ws[L], val[L + 1];
    uint32_t w4[L + 1], pa[L];
    int kw7[L + 1];                                                 // the weight rows' chunk permutation
#pragma unroll
    for (int l = 0; l <= L; ++l) {
        const int k = l == 0 ? i : jn[l - 1];                      // this position's source in a[l]
        w4[l] = wbase + 4u * (uint32_t)((l * NUP + k) * NUP);
        kw7[l] = k & 7;
    }
#pragma unroll
    for (int l = 0; l < L; ++l) {
        pa[l] = vbase + 4u * (uint32_t)(l * BM * NUP + ((((jn[l] >> 2) ^ sw7) << 2) | (jn[l] & 3)));
        p[l] = lds_f(pa[l]);
        ws[l] = lds_f(w4[l] + 4u * (uint32_t)((((jn[l] >> 2) ^ kw7[l]) << 2) | (jn[l] & 3)));
    }
    val[0] = enc;
#pragma unroll
    for (int l = 0; l < L; ++l)
        val[l + 1] = __bfloat162float(__float2bfloat16_rn(tc_act_fn(act, fmaf(ws[l], val[l], p[l]))));
    // half a layer (four 16-byte chunks, 16 targets) at a time, two register buffers in turn
    constexpr int HC = NUP / 8;
    float4 w[2][HC], x[2][HC];
    // a half whose 16 targets all lie below the first unit that may read the source is left out (the
    // same for every thread: the targets' masked weights are zero)
    bool live[2 * (L + 1)];
#pragma unroll
    for (int l = 0; l <= L; ++l) {
        const int jmin = l < L ? jn[l] : i + 1;
        live[2 * l] = jmin < 4 * HC;
        live[2 * l + 1] = true;
    }
#pragma unroll
    for (int h = 0; h <= 2 * (L + 1); ++h) {
        if (h < 2 * (L + 1) && live[h]) {
            // loads of half-step h, issued before the arithmetic of half-step h - 1
            const int l = h >> 1, cb = (h & 1) * HC;
            const uint32_t v4 = vbase + 4u * (uint32_t)(l * BM * NUP);
#pragma unroll
            for (int c = 0; c < HC; ++c)
                w[h & 1][c] = lds_f4(w4[l] + 16u * (uint32_t)((cb + c) ^ kw7[l]));
#pragma unroll
            for (int c = 0; c < HC; ++c)
                x[h & 1][c] = lds_f4(v4 + 16u * (uint32_t)((cb + c) ^ sw7));
        }
        if (h >= 1 && live[h - 1]) {
            const int g = h - 1, l = g >> 1, cb = (g & 1) * HC;
            const uint32_t v4 = vbase + 4u * (uint32_t)(l * BM * NUP);
            const float s = val[l];
#pragma unroll
            for (int c = 0; c < HC; ++c) {
                float4 xv = x[g & 1][c];
                const float4 wv = w[g & 1][c];
                xv.x = fmaf(wv.x, s, xv.x);
                xv.y = fmaf(wv.y, s, xv.y);
                xv.z = fmaf(wv.z, s, xv.z);
                xv.w = fmaf(wv.w, s, xv.w);
                sts_f4(v4 + 16u * (uint32_t)((cb + c) ^ sw7), xv);
            }
        }
        // the unit's activation replaces its running sum (after both halves of its layer are stored)
        if (h >= 1 && ((h - 1) & 1) == 1 && (h - 1) / 2 < L) sts_f(pa[(h - 1) / 2 < L ? (h - 1) / 2 : 0], val[(h - 1) / 2 + 1]);
    }
}

struct SweepEngine {
    const MadeDev &m;
    const SweepDev &sw;
    const RunArgs &r;
    SwShared &sh;
    uint8_t *ring;
    float *V;            // [L+1][128 rows][NUP]: running sums, then activations, of the group's units; a row's
                         // eight 16-byte chunks are permuted by the row number (conflict-free 16-byte accesses)
    float *X;            // [NUP][XS]: encodings of the group's positions
    float *Wg;           // [L+1][NUP][NUP]: weights between the group's units
    float *Nz;           // [GMAX][XS]: the group's noise
    int warp, lane;
    int stage = 0;
    uint32_t spar = 0;
    uint32_t tf_par = 0, te_par = 0, gd_par = 0;
    int bbuf = 0;                  // base accumulator in turn; bit b of bb_par: parity of its next use
    uint32_t bb_par = 0;
    bool dead = false;
    uint32_t tmem_base = 0;
    unsigned long long mma_flops = 0;

    __device__ SweepEngine(const MadeDev &m_, const SweepDev &sw_, const RunArgs &r_, SwShared &sh_, uint8_t *ring_)
        : m(m_), sw(sw_), r(r_), sh(sh_), ring(ring_)
    {
        warp = threadIdx.x >> 5;
        lane = threadIdx.x & 31;
        // The running sums V live in the operand ring's memory: the ring is idle from the moment a group's
        // prefix sums are complete until the next group's loads start, which is exactly when V is in use
        // (the threads fence their accesses against the asynchronous proxy before they let the loads go).
        V = reinterpret_cast<float *>(ring);
        uint8_t *p = ring + (size_t)sw.ring_bytes;
        X = reinterpret_cast<float *>(p);
        p += (size_t)NUP * XS * 4;
        Wg = reinterpret_cast<float *>(p);
        p += (size_t)(m.L + 1) * NUP * NUP * 4;
        Nz = reinterpret_cast<float *>(p);
    }

    // optional device timeline (JS_OPT_TRACE, js_get_trace) of the first CTA: one row of stamps per group;
    // slots: 0 operands may be loaded, 1 last MMA issued, 2 group tables ready, 3 prefix sums complete,
    // 4 prefix sums read, 5 positions done, 6 activations stored, 7 group geometry ready, 8 the group's
    // weights staged
    int group_no = 0;
    __device__ void trace(int slot) const
    {
        if (r.trace == nullptr || blockIdx.x != 0 || group_no >= JS_TRACE_PHASES) return;
        r.trace[(size_t)group_no * JS_TRACE_SLOTS + slot] = global_ns();
    }

    // units of a[l] with degree <= d (a[0]: the positions themselves, degree = position + 1)
    __device__ int cnt(int l, int d) const { return l == 0 ? d : __ldg(&sw.cnt[l][d]); }

    // group [t0, t1) of a block ending at b: hidden degrees (t0, hi] are evaluated inside it
    __device__ Geo geo(int l, int t0, int t1, int hi) const
    {
        Geo g;
        g.kin0 = cnt(l, t0);
        g.kb_n = (g.kin0 + BK - 1) / BK;
        g.nin = cnt(l, hi) - g.kin0;
        if (l < m.L) {
            g.u0 = cnt(l + 1, t0);
            g.nu = cnt(l + 1, hi) - g.u0;
        } else {
            g.u0 = t0;
            g.nu = t1 - t0;
        }
        g.npad = (g.nu + 15) & ~15;
        return g;
    }

    // Base of the GPB groups that start at position s0 (block ends at b): per layer, the sums over all FULL
    // K blocks below the first group's prefix boundary, for every unit those groups will evaluate.  The
    // groups' own GEMMs then run only over the K blocks from there on.
    __device__ Base base_of(int l, int s0, int b) const
    {
        const int sE = min(s0 + GPB * sw.G, b), hiS = min(sE, b - 1);
        Base g;
        g.kbs = cnt(l, s0) / BK;
        if (l < m.L) {
            g.ub0 = cnt(l + 1, s0);
            g.nb = cnt(l + 1, hiS) - g.ub0;
        } else {
            g.ub0 = s0;
            g.nb = sE - s0;
        }
        if (g.nb <= 0) g.kbs = 0;
        return g;
    }
    __device__ int base_start(int a, int t0) const { return a + ((t0 - a) / (GPB * sw.G)) * (GPB * sw.G); }

    __device__ uint8_t *stage_a(int s) const { return ring + (size_t)s * STAGE_BYTES; }
    __device__ uint8_t *stage_b(int s) const { return ring + (size_t)s * STAGE_BYTES + A_BYTES; }
    __device__ uint32_t stage_parity() const { return (spar >> stage) & 1u; }
    __device__ void advance_stage()
    {
        spar ^= 1u << stage;
        if (++stage == sw.n_stages) stage = 0;
    }

    // ------------------------------------------------------------------ roles
    __device__ void producer(int rt, int slot, int a, int b)
    {
        int kb_old[JS_MAXL + 1];
        for (int l = 0; l <= m.L; ++l) kb_old[l] = cnt(l, a) / BK;
        for (int t0 = a; t0 < b && !dead; t0 += sw.G) {
            const int t1 = min(t0 + sw.G, b), hi = min(t1, b - 1);
            // the previous group's activations (or the job's start values) are in F
            if (!mbar_wait_idle(&sh.gdone, gd_par, r.ctl)) { dead = true; break; }
            gd_par ^= 1u;
            fence_proxy_async();
            trace(0);
            const int s0 = base_start(a, t0);
            if (t0 == s0) {
                // the base GEMMs of the next GPB groups: NB units at a time over the full K blocks of the prefix
                for (int l = 0; l <= m.L && !dead; ++l) {
                    const Base bs = base_of(l, s0, b);
                    for (int c = 0; c * NB < bs.nb && bs.kbs > 0 && !dead; ++c) {
                        mma_flops += 2ull * BM * BK * NB * (unsigned long long)bs.kbs;
                        for (int kb = 0; kb < bs.kbs; ++kb) {
                            if (!mbar_wait(&sh.empty[stage], stage_parity() ^ 1u, r.ctl)) { dead = true; break; }
                            mbar_expect_tx(&sh.full[stage], A_BYTES + NB * BK * 2);
                            if (kb < kb_old[l])
                                tma_load_2d(smem_u32(stage_a(stage)), sw.tmAold + l, &sh.full[stage], kb * BK, rt * BM);
                            else
                                tma_load_3d(smem_u32(stage_a(stage)), sw.tmF + l, &sh.full[stage], (kb - kb_old[l]) * BK, 0, slot);
                            tma_load_2d(smem_u32(stage_b(stage)), sw.tmW16 + 2 * (m.L + 1) + l, &sh.full[stage], kb * BK,
                                        bs.ub0 + c * NB);
                            advance_stage();
                        }
                    }
                }
            }
            for (int l = 0; l <= m.L && !dead; ++l) {
                const Geo g = geo(l, t0, t1, hi);
                if (g.nu == 0) continue;
                const uint32_t bytes = A_BYTES + (uint32_t)g.npad * BK * 2;
                const int kbs = base_of(l, s0, b).kbs;
                mma_flops += 2ull * BM * BK * (unsigned long long)g.npad * (unsigned long long)(g.kb_n - kbs);
                for (int kb = kbs; kb < g.kb_n; ++kb) {
                    if (!mbar_wait(&sh.empty[stage], stage_parity() ^ 1u, r.ctl)) { dead = true; break; }
                    mbar_expect_tx(&sh.full[stage], bytes);
                    if (kb < kb_old[l])
                        tma_load_2d(smem_u32(stage_a(stage)), sw.tmAold + l, &sh.full[stage], kb * BK, rt * BM);
                    else
                        tma_load_3d(smem_u32(stage_a(stage)), sw.tmF + l, &sh.full[stage], (kb - kb_old[l]) * BK, 0, slot);
                    // one box of 16 or of 32 weight rows (a load per 16 rows cost a fifth of the K loop)
                    tma_load_2d(smem_u32(stage_b(stage)), sw.tmW16 + (g.npad == 32 ? m.L + 1 : 0) + l, &sh.full[stage],
                                kb * BK, g.u0);
                    advance_stage();
                }
            }
            group_no++;
        }
    }

    __device__ void mma_issuer(int a, int b)
    {
        for (int t0 = a; t0 < b && !dead; t0 += sw.G) {
            const int t1 = min(t0 + sw.G, b), hi = min(t1, b - 1);
            // the epilogue has read the previous group's accumulators
            if (!mbar_wait_idle(&sh.tempty, te_par ^ 1u, r.ctl)) { dead = true; break; }
            te_par ^= 1u;
            tc_fence_after();
            bool any = false;
            const int s0 = base_start(a, t0);
            if (t0 == s0) {
                const uint32_t idescb = instr_desc_bf16(NB);
                for (int l = 0; l <= m.L && !dead; ++l) {
                    const Base bs = base_of(l, s0, b);
                    for (int c = 0; c * NB < bs.nb && bs.kbs > 0 && !dead; ++c) {
                        // the epilogue has copied this accumulator's previous chunk away
                        if (!mbar_wait(&sh.bempty[bbuf], ((bb_par >> bbuf) & 1u) ^ 1u, r.ctl)) { dead = true; break; }
                        tc_fence_after();
                        const uint32_t d_base = tmem_base + (uint32_t)(BASE_COL + bbuf * NB);
                        for (int kb = 0; kb < bs.kbs; ++kb) {
                            if (!mbar_wait(&sh.full[stage], stage_parity(), r.ctl)) { dead = true; break; }
                            tc_fence_after();
                            const uint64_t adesc = smem_desc_sw128(smem_u32(stage_a(stage)));
                            const uint64_t bdesc = smem_desc_sw128(smem_u32(stage_b(stage)));
#pragma unroll
                            for (int k = 0; k < BK / 16; ++k)
                                umma_bf16(d_base, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idescb,
                                          (kb > 0 || k > 0) ? 1u : 0u);
                            umma_commit(&sh.empty[stage]);
                            advance_stage();
                        }
                        if (dead) break;
                        umma_commit(&sh.bfull[bbuf]);
                        bb_par ^= 1u << bbuf;
                        bbuf ^= 1;
                    }
                }
                if (dead) break;
            }
            for (int l = 0; l <= m.L && !dead; ++l) {
                const Geo g = geo(l, t0, t1, hi);
                if (g.nu == 0) continue;
                const uint32_t idesc = instr_desc_bf16(g.npad);
                const uint32_t d_tmem = tmem_base + (uint32_t)(l * NUP);
                const int kbs = base_of(l, s0, b).kbs;
                for (int kb = kbs; kb < g.kb_n; ++kb) {
                    if (!mbar_wait(&sh.full[stage], stage_parity(), r.ctl)) { dead = true; break; }
                    tc_fence_after();
                    const uint64_t adesc = smem_desc_sw128(smem_u32(stage_a(stage)));
                    const uint64_t bdesc = smem_desc_sw128(smem_u32(stage_b(stage)));
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        umma_bf16(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc,
                                  (kb > kbs || k > 0) ? 1u : 0u);
                    umma_commit(&sh.empty[stage]);
                    advance_stage();
                    any = true;
                }
            }
            if (dead) break;
            if (any) umma_commit(&sh.tfull);
            else mbar_arrive(&sh.tfull);          // a group with empty prefixes (the very first positions)
            trace(1);
            group_no++;
        }
    }

    // row k (a source among the group's units of a[l]) of the table of weights inside the group: 32 targets
    // as eight 16-byte chunks, chunk c stored at position c ^ (k & 7)
    __device__ uint32_t wrow(int l, int k) const { return smem_u32(Wg) + 4u * (uint32_t)((l * NUP + k) * NUP); }

    __device__ void ep_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

    // unit j of the group in layer slot l, sample row `row`: its shared-memory address
    __device__ uint32_t vat(int l, int j, int row) const
    {
        return smem_u32(V) + 4u * (uint32_t)(((l * BM + row) * NUP) + ((((j >> 2) ^ (row & 7)) << 2) | (j & 3)));
    }

    // source k of a[l] has the value `val`: add its contribution to the running sums of the group's units
    // of a[l+1] (masked weights are zero where the target may not read the source)
    // Targets below jmin cannot read this source (their degree is lower, their masked weight zero): their
    // 16-byte chunks are left alone, which halves the shared-memory traffic that bounds the position loop.
    __device__ void scatter(int l, int k, float val, int row, int jmin)
    {
        const int c0 = jmin >> 2;
        // the row's 32 running sums as eight 16-byte accesses, all loads before all stores: one warp per
        // scheduler cannot hide the latency of a load that waits behind a store it might alias
        const uint32_t w4 = wrow(l, k);
        const uint32_t v4 = smem_u32(V) + 4u * (uint32_t)((l * BM + row) * NUP);
        const int sw7 = row & 7, kw7 = k & 7;
        float4 w[NUP / 4], x[NUP / 4];
#pragma unroll
        for (int c = 0; c < NUP / 4; ++c)
            if (c >= c0) w[c] = lds_f4(w4 + 16u * (uint32_t)(c ^ kw7));
#pragma unroll
        for (int c = 0; c < NUP / 4; ++c)
            if (c >= c0) x[c] = lds_f4(v4 + 16u * (uint32_t)(c ^ sw7));
#pragma unroll
        for (int c = 0; c < NUP / 4; ++c) {
            if (c < c0) continue;
            x[c].x = fmaf(w[c].x, val, x[c].x);
            x[c].y = fmaf(w[c].y, val, x[c].y);
            x[c].z = fmaf(w[c].z, val, x[c].z);
            x[c].w = fmaf(w[c].w, val, x[c].w);
        }
#pragma unroll
        for (int c = 0; c < NUP / 4; ++c)
            if (c >= c0) sts_f4(v4 + 16u * (uint32_t)(c ^ sw7), x[c]);
    }

    // n consecutive values (unit j = 0..n-1 of layer slot l, or the group's encodings when l < 0) of this
    // thread's row as bf16 to dst[0..n): single elements up to a 16-byte boundary, then eight at a time
    __device__ float run_val(int l, int j, int row) const { return l < 0 ? X[j * XS + row] : lds_f(vat(l, j, row)); }
    __device__ void store_run(__nv_bfloat16 *dst, int l, int row, int n)
    {
        int j = 0;
        for (; j < n && (reinterpret_cast<uintptr_t>(dst + j) & 15u) != 0; ++j) dst[j] = __float2bfloat16_rn(run_val(l, j, row));
        for (; j + 8 <= n; j += 8) {
            float x[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) x[i] = run_val(l, j + i, row);
            *reinterpret_cast<uint4 *>(dst + j) = make_uint4(pack_bf16x2(x[0], x[1]), pack_bf16x2(x[2], x[3]),
                                                             pack_bf16x2(x[4], x[5]), pack_bf16x2(x[6], x[7]));
        }
        for (; j < n; ++j) dst[j] = __float2bfloat16_rn(run_val(l, j, row));
    }

    // start of a job: the job's buffer F holds, per layer, the units from the K block that contains
    // the block's first old unit onwards: copies of the old activations up to degree a, zeros after
    __device__ void job_init(int rt, int slot, int a, int b)
    {
        const int row = (warp & 3) * 32 + lane;
        const size_t esz = 2;
        for (int l = 0; l <= m.L; ++l) {
            const int k_old = cnt(l, a), kb0 = (k_old / BK) * BK;
            const int ncopy = k_old - kb0;
            const int cols = min(sw.WF[l], ((cnt(l, min(b, m.T)) - kb0 + BK - 1) / BK) * BK);
            __nv_bfloat16 *f = sw.F[l] + ((size_t)slot * BM + row) * sw.WF[l];
            const __nv_bfloat16 *old = (const __nv_bfloat16 *)m.a[l] + (size_t)(rt * BM + row) * m.n[l] + kb0;
            for (int c = 0; c < cols; c += 8) {
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (c + 8 <= ncopy) {
                    v = __ldcg(reinterpret_cast<const uint4 *>(old + c));
                } else if (c < ncopy) {
                    __nv_bfloat16 tmp[8];
                    for (int i = 0; i < 8; ++i) tmp[i] = c + i < ncopy ? old[c + i] : __float2bfloat16_rn(0.0f);
                    v = *reinterpret_cast<const uint4 *>(tmp);
                }
                *reinterpret_cast<uint4 *>(f + c) = v;
            }
            (void)esz;
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.gdone);
    }

    // LT: the number of hidden layers if the one-unit-per-layer path is compiled for it (1 .. 4), else 0
    template <int LT>
    __device__ void epilogue(int rt, int slot, int a, int b, bool &row_changed)
    {
        const int q = warp & 3, row = q * 32 + lane, tid = threadIdx.x - 64;
        const int smp = rt * BM + row;
        const bool valid = smp < r.batch;
        const int L = m.L;
        int kb_old[JS_MAXL + 1];
        for (int l = 0; l <= L; ++l) kb_old[l] = cnt(l, a) / BK;
        job_init(rt, slot, a, b);
        for (int t0 = a; t0 < b && !dead; t0 += sw.G) {
            const int t1 = min(t0 + sw.G, b), hi = min(t1, b - 1), ng = t1 - t0;
            // ---- geometry, small tables, the weights between the group's units, noise (while the GEMMs run)
            ep_sync();                                   // everybody is done with the previous group's tables
            const int s0 = base_start(a, t0);
            if (tid <= L) {
                const Geo g = geo(tid, t0, t1, hi);
                sh.kin0[tid] = g.kin0; sh.nin[tid] = g.nin; sh.u0[tid] = g.u0; sh.nu[tid] = g.nu; sh.kb_n[tid] = g.kb_n;
                const Base bs = base_of(tid, s0, b);
                sh.kbs[tid] = bs.kbs; sh.ub0[tid] = bs.ub0;
            }
            for (int i = tid; i < (L + 1) * (GMAX + 2); i += 128) {
                const int l = i / (GMAX + 2), k = i % (GMAX + 2);
                if (l >= 1) sh.cs[l][k] = cnt(l, min(t0 + k, m.T));
            }
            ep_sync();
            if (tid == 0) trace(7);
            {
                // Every global load of the thread first, the stores to shared memory after them: the compiler
                // may not move a load across a store it cannot tell apart, and one round trip per layer and
                // per table would cost more than the group's GEMMs.
                // thread = (source k = lane, chunk of four targets): four loads (each coalesced over the
                // warp's sources), one 16-byte store to row k of the source-major table, chunks permuted by
                // the row number like the running sums (a new activation updates all its targets)
                constexpr int LB = 3;            // layers per round trip
                for (int l0 = 0; l0 <= L; l0 += LB) {
                    __nv_bfloat16 wv[LB][2][4];
                    float bv[LB];
#pragma unroll
                    for (int dl = 0; dl < LB; ++dl) {
                        const int l = min(l0 + dl, L);
                        const int nu = sh.nu[l], nin = sh.nin[l], u0 = sh.u0[l], kin0 = sh.kin0[l];
                        const __nv_bfloat16 *Wl = (const __nv_bfloat16 *)m.W[l];
                        const int K = m.n[l];
#pragma unroll
                        for (int e = 0; e < 2; ++e)
#pragma unroll
                            for (int jj = 0; jj < 4; ++jj) {
                                const int j = 4 * (q + 4 * e) + jj;
                                wv[dl][e][jj] = (j < nu && lane < nin) ? Wl[(size_t)(u0 + j) * K + kin0 + lane]
                                                                       : __float2bfloat16_rn(0.0f);
                            }
                        bv[dl] = (tid < NUP && tid < nu) ? m.bias[l][u0 + tid] : 0.0f;
                    }
#pragma unroll
                    for (int dl = 0; dl < LB; ++dl) {
                        const int l = min(l0 + dl, L);           // past the last layer: the last layer again
#pragma unroll
                        for (int e = 0; e < 2; ++e)
                            sts_f4(wrow(l, lane) + 16u * (uint32_t)((q + 4 * e) ^ (lane & 7)),
                                   make_float4(__bfloat162float(wv[dl][e][0]), __bfloat162float(wv[dl][e][1]),
                                               __bfloat162float(wv[dl][e][2]), __bfloat162float(wv[dl][e][3])));
                        if (tid < NUP) sh.bias_s[l][tid] = bv[dl];
                    }
                }
            }
            if (tid == 0) trace(8);
            {
                // noise and the symbols the group's positions hold now (for the change flags; 255 where there
                // is none): a warp takes its 32 rows in turn, lane = position, so that a load instruction
                // touches one line instead of 32; eight rows' loads before their stores
#pragma unroll 1
                for (int r0 = 0; r0 < 32; r0 += 8) {
                    float nv[8];
                    uint8_t xo[8];
#pragma unroll
                    for (int rr = 0; rr < 8; ++rr) {
                        const int s2 = rt * BM + q * 32 + r0 + rr;
                        const bool in = s2 < r.batch && lane < ng;
                        nv[rr] = in ? __ldg(r.noise + (size_t)s2 * m.T + t0 + lane) : 0.0f;
                        xo[rr] = in ? r.x[(size_t)s2 * m.T + t0 + lane] : (uint8_t)255;
                    }
#pragma unroll
                    for (int rr = 0; rr < 8; ++rr) {
                        Nz[lane * XS + q * 32 + r0 + rr] = nv[rr];
                        X[lane * XS + q * 32 + r0 + rr] = (float)xo[rr];
                    }
                }
            }
            ep_sync();
            if (tid == 0) trace(2);
            // ---- a new base: its sums go from tensor memory to this job's part of S, chunk by chunk, as the
            // MMAs deliver them; thread = sample row writes, and later reads, only its own row
            if (t0 == s0) {
                for (int l = 0; l <= L && !dead; ++l) {
                    const Base bs = base_of(l, s0, b);
                    float *Sl = sw.S + (((size_t)slot * (L + 1) + l) * sw.nbs) * BM + row;
                    for (int c = 0; c * NB < bs.nb && bs.kbs > 0; ++c) {
                        if (!mbar_wait(&sh.bfull[bbuf], (bb_par >> bbuf) & 1u, r.ctl)) { dead = true; break; }
                        tc_fence_after();
#pragma unroll 1
                        for (int h = 0; h < NB; h += 32) {
                            float v[32];
                            tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(BASE_COL + bbuf * NB + h), v);
#pragma unroll
                            for (int i = 0; i < 32; ++i) Sl[(size_t)(c * NB + h + i) * BM] = v[i];
                        }
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&sh.bempty[bbuf]);
                        bb_par ^= 1u << bbuf;
                        bbuf ^= 1;
                    }
                }
                if (dead) break;
            }
            // ---- the next group's tables (weights between its units, noise, symbols) are touched once per
            // sweep and would come from DRAM, two dependent round trips of 2.5 us each: ask for them now
            if (t1 < b) {
                const int t2 = min(t1 + sw.G, b), hi2 = min(t2, b - 1);
                for (int i = tid; i < (L + 1) * NUP; i += 128) {
                    const int l = i / NUP, j = i % NUP;
                    const Geo g = geo(l, t1, t2, hi2);
                    if (j < g.nu && g.nin > 0) {
                        const __nv_bfloat16 *pw = (const __nv_bfloat16 *)m.W[l] + (size_t)(g.u0 + j) * m.n[l] + g.kin0;
                        prefetch_l2(pw);
                        prefetch_l2(pw + g.nin - 1);
                    }
                }
                if (valid) {
                    const float *np = r.noise + (size_t)smp * m.T + t1;
                    prefetch_l2(np);
                    prefetch_l2(np + (t2 - t1) - 1);
                    prefetch_l2(r.x + (size_t)smp * m.T + t1);
                }
            }
            // ---- prefix sums out of tensor memory
            if (!mbar_wait(&sh.tfull, tf_par, r.ctl)) { dead = true; break; }
            tf_par ^= 1u;
            tc_fence_after();
            if (tid == 0) trace(3);
            for (int l = 0; l <= L; ++l) {
                float v[32];
                if (sh.nu[l] > 0 && sh.kb_n[l] > sh.kbs[l]) {
                    tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(l * NUP), v);
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = 0.0f;
                }
                if (sh.kbs[l] > 0 && sh.nu[l] > 0) {
                    // base + the group's own K blocks (in that order, always)
                    const float *Sl = sw.S + (((size_t)slot * (L + 1) + l) * sw.nbs + (sh.u0[l] - sh.ub0[l])) * BM + row;
                    const int nuv = sh.nu[l];
                    float sv[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) sv[i] = i < nuv ? __ldcg(Sl + (size_t)i * BM) : 0.0f;
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = sv[i] + v[i];
                }
                // running pre-activation of every unit of the group: prefix sum + bias; the group's own
                // contributions are added below, each as soon as its source exists
                const uint32_t v4 = smem_u32(V) + 4u * (uint32_t)((l * BM + row) * NUP);
#pragma unroll
                for (int c = 0; c < NUP / 4; ++c)
                    sts_f4(v4 + 16u * (uint32_t)(c ^ (row & 7)),
                           make_float4(v[4 * c] + sh.bias_s[l][4 * c], v[4 * c + 1] + sh.bias_s[l][4 * c + 1],
                                       v[4 * c + 2] + sh.bias_s[l][4 * c + 2], v[4 * c + 3] + sh.bias_s[l][4 * c + 3]));
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.tempty);
            if (tid == 0) trace(4);
            // ---- the group's positions in order, thread = sample row.  A value that becomes known (a
            // sampled symbol, then the hidden units it completes, layer by layer) is added at once to
            // the running sums of everything in the group that reads it: the additions of one source
            // are independent of each other, and each target receives its sources in index order.
            for (int i = 0; i < ng; ++i) {
                const int t = t0 + i;
                // the units this position completes, per hidden layer (looked up before the sampling,
                // which hides the loads)
                int jn[LT > 0 ? LT : 1];
                bool one_each = true;
#pragma unroll
                for (int l = 0; l < (LT > 0 ? LT : 1); ++l) {
                    if (LT == 0) break;
                    const int ca = sh.cs[l + 1][i], cb = sh.cs[l + 1][i + 1];
                    jn[l] = ca - sh.u0[l];
                    one_each = one_each && cb - ca == 1;
                }
                const float z = lds_f(vat(L, i, row));
                const uint32_t xa = smem_u32(X) + 4u * (uint32_t)(i * XS + row);
                const int xn = js_sample_binary(r.nk, z, lds_f(smem_u32(Nz) + 4u * (uint32_t)(i * XS + row)));
                if (valid && (int)lds_f(xa) != xn) {
                    r.x[(size_t)smp * m.T + t] = (uint8_t)xn;
                    row_changed = true;
                }
                const float enc = sh.lut_s[xn];
                sts_f(xa, enc);
                if (t + 1 > hi) continue;
                if constexpr (LT > 0) {
                    if (one_each) {
                        uint32_t pk = 0;                   // indices below 32, one byte each
#pragma unroll
                        for (int l = 0; l < LT; ++l) pk |= (uint32_t)jn[l] << (8 * l);
                        position_one_each<LT>(smem_u32(Wg), smem_u32(V) + 4u * (uint32_t)(row * NUP), m.act, i, enc, row, pk);
                        continue;
                    }
                }
                scatter(0, i, enc, row, L > 0 ? sh.cs[1][i] - sh.u0[0] : i + 1);
                // the hidden units that position t makes computable: degree t + 1
                for (int l = 0; l < L; ++l) {
                    const int j0 = sh.cs[l + 1][i] - sh.u0[l], j1 = sh.cs[l + 1][i + 1] - sh.u0[l];
                    for (int j = j0; j < j1; ++j) {
                        const uint32_t pv = vat(l, j, row);
                        const float val = __bfloat162float(__float2bfloat16_rn(tc_act_fn(m.act, lds_f(pv))));
                        sts_f(pv, val);
                        scatter(l + 1, j, val, row, l + 1 < L ? sh.cs[l + 2][i] - sh.u0[l + 1] : i + 1);
                    }
                }
            }
            if (tid == 0) trace(5);
            // ---- the group's activations into F, for the GEMMs of the groups that follow
            if (t1 < b) {
                // the symbols' encodings by thread = row (their table is position-major); the hidden
                // units by warp: its 32 rows in turn, lane = unit, so that a store instruction writes one
                // run of 2-byte values instead of touching 32 lines
                store_run(sw.F[0] + ((size_t)slot * BM + row) * sw.WF[0] + (t0 - kb_old[0] * BK), -1, row, ng);
                __syncwarp();
                for (int l = 1; l <= L; ++l) {
                    const int n = sh.nin[l];
                    __nv_bfloat16 *dst = sw.F[l] + ((size_t)slot * BM + q * 32) * sw.WF[l] + (sh.kin0[l] - kb_old[l] * BK) + lane;
                    if (lane < n) {
#pragma unroll 1
                        for (int r0 = 0; r0 < 32; r0 += 8) {
                            float v[8];
#pragma unroll
                            for (int rr = 0; rr < 8; ++rr) v[rr] = lds_f(vat(l - 1, lane, q * 32 + r0 + rr));
#pragma unroll
                            for (int rr = 0; rr < 8; ++rr) dst[(size_t)(r0 + rr) * sw.WF[l]] = __float2bfloat16_rn(v[rr]);
                        }
                    }
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.gdone);
            } else {
                fence_proxy_async();          // the next job's loads will overwrite the running sums
            }
            if (tid == 0) trace(6);
            group_no++;
        }
    }
};

// LT = the model's number of hidden layers where the one-unit-per-layer path of the position loop is
// compiled for it (1 .. 4), else 0.
template <int LT>
__global__ void __launch_bounds__(NTH, 1)
made_sweep_kernel(const __grid_constant__ MadeDev m, const __grid_constant__ SweepDev sw, const __grid_constant__ RunArgs r)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ SwShared sh;
    uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_STAGES; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
        mbar_init(&sh.tfull, 1);
        mbar_init(&sh.tempty, 4);
        mbar_init(&sh.gdone, 4);
        for (int i = 0; i < 2; ++i) { mbar_init(&sh.bfull[i], 1); mbar_init(&sh.bempty[i], 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
        sh.lut_s[0] = m.lut[0];
        sh.lut_s[1] = m.lut[1];
    }
    if (warp == 1) tmem_alloc(&sh.tmem_base, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    SweepEngine e(m, sw, r, sh, ring);
    e.tmem_base = sh.tmem_base;
    // jobs: (row tile, block), the blocks with the longest prefixes first
    const int B = r.block, nblk = (m.T + B - 1) / B, MT = (r.batch + BM - 1) / BM;
    const int njobs = MT * (nblk - r.blk_lo);
    for (int job = blockIdx.x; job < njobs; job += gridDim.x) {
        const int blk = nblk - 1 - job / MT, rt = job % MT;
        const int a = blk * B, b = min(a + B, m.T);
        // The accumulators and the ring are idle between jobs; the roles meet here so that a job's
        // start values are never written while the previous job is still being read, and so that
        // all of them see the same answer to "has a wait given up".
        __syncthreads();
        if (threadIdx.x == 0) sh.stop = ld_volatile_i32(&r.ctl->abort);
        __syncthreads();
        if (sh.stop) break;
        if (warp == 0) {
            if (e.lane == 0) e.producer(rt, blockIdx.x, a, b);
        } else if (warp == 1) {
            if (e.lane == 0) e.mma_issuer(a, b);
        } else {
            bool row_changed = false;
            e.template epilogue<LT>(rt, blockIdx.x, a, b, row_changed);
            const int smp = rt * BM + (warp & 3) * 32 + e.lane;
            if (row_changed && smp < r.batch) r.smp_changed[smp] = 1;
        }
        __syncwarp();
    }
    DriverResult res = {JS_OK, 0, m.T, !e.dead};
    tc_fence_before();
    __syncthreads();
    if (!res.alive || ld_volatile_i32(&r.ctl->abort) != 0) {
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);      // let copies still in flight land
        res.alive = false;
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(e.tmem_base, 512);
    }
    driver_finish(r, res, 0, 0, e.mma_flops, 0);
}

// Per-sample bookkeeping of Jacobi-GS after outer iteration k (one CTA): a sample whose iterate did
// not change stops counting; the flags are cleared for the next iteration and the host learns
// whether anything changed.
__global__ void jgs_book_kernel(int batch, int k, int at_cap, int *changed, int *done, int32_t *out_iters, int *any_out)
{
    __shared__ int any;
    if (threadIdx.x == 0) any = 0;
    __syncthreads();
    for (int b = threadIdx.x; b < batch; b += blockDim.x) {
        const int c = changed[b];
        if (c) any = 1;
        if (!done[b] && (c == 0 || at_cap)) {
            done[b] = 1;
            if (out_iters) out_iters[b] = k;
        }
        changed[b] = 0;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        *any_out = any;
        __threadfence_system();
    }
}

}  // namespace

// --------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn sweep_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (fn) return fn;
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
        return nullptr;
    fn = (EncodeTiledFn)p;
    return fn;
}

static bool sweep_encode(CUtensorMap *out, const void *base, int rank, const cuuint64_t *dims, const cuuint64_t *strides,
                         const cuuint32_t *box)
{
    EncodeTiledFn fn = sweep_encode_fn();
    if (!fn) return false;
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

typedef void (*SweepKernelFn)(const MadeDev, const SweepDev, const RunArgs);
static SweepKernelFn sweep_kernel_of(int L)
{
    switch (L) {
    case 1: return made_sweep_kernel<1>;
    case 2: return made_sweep_kernel<2>;
    case 3: return made_sweep_kernel<3>;
    case 4: return made_sweep_kernel<4>;
    default: return made_sweep_kernel<0>;
    }
}

// Builds what the sweeps need beside the tensor-core view of the model: prefix counts per degree,
// the group size, the jobs' buffers F and the tensor maps.  Returns 1 if the model qualifies
// (binary positions, sorted degrees, bf16), 0 if not, negative on CUDA errors.  Called on first use.
int js_sweep_prepare(js_model *mo)
{
    if (mo->sweep_state != 0) return mo->sweep_state > 0 ? 1 : 0;
    mo->sweep_state = -1;
    const MadeDev &v = mo->made;
    SweepDev &s = mo->sweep;
    if (!mo->tc_ok || v.C != 1 || v.prec != JS_BF16 || !sweep_encode_fn()) return 0;
    if ((v.L + 1) * NUP > BASE_COL) return 0;              // the groups' accumulators end where the base's begin
    const int L = v.L, T = v.T;
    // prefix counts; the group size is the largest one that keeps every layer's units of a group within NUP
    std::vector<std::vector<int>> cnt(L + 1);
    for (int l = 1; l <= L; ++l) {
        cnt[l].assign(T + 1, 0);
        const std::vector<int> &dg = mo->host_deg[l];
        for (size_t i = 1; i < dg.size(); ++i)
            if (dg[i] < dg[i - 1]) return 0;                       // needs sorted degrees
        size_t p = 0;
        for (int d = 0; d <= T; ++d) {
            while (p < dg.size() && dg[p] <= d) ++p;
            cnt[l][d] = (int)p;
        }
    }
    int G = GMAX;
    for (; G >= 1; --G) {
        bool ok = true;
        for (int l = 1; l <= L && ok; ++l)
            for (int d = 0; d < T && ok; ++d)
                if (cnt[l][std::min(d + G, T)] - cnt[l][d] > NUP) ok = false;
        if (ok) break;
    }
    if (G < 1) return 0;
    s.G = G;
    const int v_bytes = (L + 1) * NUP * BM * 4;            // shares the ring's memory
    const int fixed = NUP * XS * 4 + (L + 1) * NUP * NUP * 4 + GMAX * XS * 4;
    s.n_stages = std::min(MAX_STAGES, (SMEM_DYN_MAX - 1024 - fixed) / STAGE_BYTES);
    if (s.n_stages < 2) return 0;
    s.ring_bytes = std::max(s.n_stages * STAGE_BYTES, (v_bytes + 1023) / 1024 * 1024);
    if (1024 + s.ring_bytes + fixed > SMEM_DYN_MAX) return 0;
    s.smem_bytes = 1024 + s.ring_bytes + fixed;
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (sms < 1) return 0;
    s.slots = sms;
    auto fail = [&]() { cudaGetLastError(); return JS_ERR_CUDA; };
    std::vector<CUtensorMap> mapsF(L + 1), mapsW(3 * (L + 1));       // weights: boxes of 16, of 32 and of NB rows
    for (int l = 0; l <= L; ++l) {
        if (l >= 1) {
            void *p = nullptr;
            if (cudaMalloc(&p, (T + 1) * sizeof(int)) != cudaSuccess) return fail();
            mo->allocs.push_back(p);
            if (cudaMemcpy(p, cnt[l].data(), (T + 1) * sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess) return fail();
            s.cnt[l] = (const int *)p;
        } else {
            s.cnt[l] = nullptr;
        }
        s.WF[l] = (v.n[l] + BK - 1) / BK * BK + BK;
        void *f = nullptr;
        const size_t bytes = (size_t)s.slots * BM * s.WF[l] * 2;
        if (cudaMalloc(&f, bytes) != cudaSuccess) return fail();
        mo->allocs.push_back(f);
        if (cudaMemset(f, 0, bytes) != cudaSuccess) return fail();
        s.F[l] = (__nv_bfloat16 *)f;
        {
            const cuuint64_t dims[3] = {(cuuint64_t)s.WF[l], (cuuint64_t)BM, (cuuint64_t)s.slots};
            const cuuint64_t strides[2] = {(cuuint64_t)s.WF[l] * 2, (cuuint64_t)s.WF[l] * 2 * BM};
            const cuuint32_t box[3] = {(cuuint32_t)BK, (cuuint32_t)BM, 1};
            if (!sweep_encode(&mapsF[l], f, 3, dims, strides, box)) return 0;
        }
        for (int big = 0; big < 3; ++big) {
            const cuuint64_t dims[2] = {(cuuint64_t)v.n[l], (cuuint64_t)v.n[l + 1]};
            const cuuint64_t strides[1] = {(cuuint64_t)v.n[l] * 2};
            const cuuint32_t box[2] = {(cuuint32_t)BK, big == 2 ? (cuuint32_t)NB : 16u << big};
            if (!sweep_encode(&mapsW[big * (L + 1) + l], v.W[l], 2, dims, strides, box)) return 0;
        }
    }
    void *pf = nullptr, *pw = nullptr;
    if (cudaMalloc(&pf, (L + 1) * sizeof(CUtensorMap)) != cudaSuccess) return fail();
    mo->allocs.push_back(pf);
    if (cudaMalloc(&pw, 3 * (L + 1) * sizeof(CUtensorMap)) != cudaSuccess) return fail();
    mo->allocs.push_back(pw);
    if (cudaMemcpy(pf, mapsF.data(), (L + 1) * sizeof(CUtensorMap), cudaMemcpyHostToDevice) != cudaSuccess) return fail();
    if (cudaMemcpy(pw, mapsW.data(), 3 * (L + 1) * sizeof(CUtensorMap), cudaMemcpyHostToDevice) != cudaSuccess) return fail();
    s.tmF = (const CUtensorMap *)pf;
    s.tmW16 = (const CUtensorMap *)pw;
    s.tmAold = mo->tc.tmA;
    {
        // base sums: per slot and layer, room for the units of GPB groups (rounded up to whole chunks)
        int nbs = NB;
        for (int l = 1; l <= L; ++l)
            for (int d = 0; d < T; ++d) nbs = std::max(nbs, cnt[l][std::min(d + GPB * G, T)] - cnt[l][d]);
        nbs = std::max(nbs, GPB * G);
        s.nbs = (nbs + NB - 1) / NB * NB;
        void *p = nullptr;
        const size_t bytes = (size_t)s.slots * (L + 1) * s.nbs * BM * sizeof(float);
        if (cudaMalloc(&p, bytes) != cudaSuccess) return fail();
        mo->allocs.push_back(p);
        s.S = (float *)p;
    }
    {
        void *p = nullptr;
        if (cudaMalloc(&p, 2 * (size_t)mo->rows * sizeof(int)) != cudaSuccess) return fail();
        mo->allocs.push_back(p);
        if (cudaMemset(p, 0, 2 * (size_t)mo->rows * sizeof(int)) != cudaSuccess) return fail();
        mo->sw_flags = (int *)p;
        if (cudaHostAlloc((void **)&mo->h_any, sizeof(int), cudaHostAllocMapped) != cudaSuccess) return fail();
        if (cudaHostGetDevicePointer((void **)&mo->d_any, mo->h_any, 0) != cudaSuccess) return fail();
    }
    if (cudaFuncSetAttribute(sweep_kernel_of(L), cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN_MAX) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    mo->sweep_state = 1;
    return 1;
}

// One launch: sweeps of every block >= r.blk_lo (block size r.block) for every row tile.
int js_launch_made_sweep(const js_model *mo, const RunArgs &r, cudaStream_t stream)
{
    const SweepDev &s = mo->sweep;
    const int nblk = (mo->made.T + r.block - 1) / r.block, MT = (r.batch + BM - 1) / BM;
    const int njobs = MT * (nblk - r.blk_lo);
    if (njobs < 1) return (int)cudaErrorInvalidValue;
    const int grid = std::min(njobs, s.slots);
    sweep_kernel_of(mo->made.L)<<<grid, NTH, s.smem_bytes, stream>>>(mo->made, s, r);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? 0 : (int)e;
}

int js_launch_jgs_book(const js_model *mo, int batch, int k, int at_cap, int32_t *out_iters, cudaStream_t stream)
{
    jgs_book_kernel<<<1, 256, 0, stream>>>(batch, k, at_cap, mo->sw_flags, mo->sw_flags + mo->rows, out_iters, mo->d_any);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? 0 : (int)e;
}
