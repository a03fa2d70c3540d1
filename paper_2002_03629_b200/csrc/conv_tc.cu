// Masked-convolution sampler (PixelCNN-style stack) on the sm_100a tensor cores.
//
// Every masked 3x3 convolution is an implicit GEMM: M = 128 consecutive pixels of one
// image (whole rows), N = output channels, K = live taps x input channels.  Only the
// five taps the causal mask keeps are visited (row above: left, centre, right; same
// row: left, centre); the centre tap's colour-group mask is already folded into the
// packed weights.  The A operand of tap (ky, kx) is the activation tensor shifted by
// (ky-1, kx-1): one 4-D TMA box {64 channels, width, rows, 1 image} whose start
// coordinate may lie outside the image, where TMA fills zeros - that is the zero
// padding.  The 1x1 head is a plain GEMM with one 256-class sub-pixel per N tile, and
// its epilogue is the sampling step (Gumbel-max against the fixed noise, compare,
// re-encode), as in the masked-MLP kernel.  Solver loops: made_driver.cuh.
#include <cuda.h>

#include <vector>

#include "js_common.cuh"
#include "js_model.h"
#include "made_driver.cuh"
#include "tc_common.cuh"

namespace {

constexpr int BM = TC_BM, BK = TC_BK;
constexpr int NTH = 320;          // warp 0 loads, warp 1 MMA, warps 2-9 epilogue: two per tensor-memory lane quadrant
constexpr int ACC_COLS = 256;
constexpr int A_BYTES = BM * BK * 2;
constexpr int STAGE_BYTES = A_BYTES + 256 * BK * 2;   // A tile + up to 256 weight rows
constexpr int N_STAGES = 3;
constexpr int RING_BYTES = N_STAGES * STAGE_BYTES;    // 144 KB
constexpr int STAGING_BYTES = 32 * 1024;
constexpr int SMEM_BYTES = RING_BYTES + STAGING_BYTES + 1024;
constexpr int MAX_IMAGES = 256;

enum { EPI_HIDDEN = 0, EPI_LOGITS = 1, EPI_CAT = 3 };
// which activations a layer reads and writes.  SRC_NEW: the working set.  SRC_OLD: the set of the previous
// outer iterate (Jacobi-GS).  SRC_MIXED: the row above from the previous outer iterate, the own row from
// the working set - the view a one-row block has in Algorithm 2.
enum { SRC_NEW = 0, SRC_OLD = 1, SRC_MIXED = 2 };

// the five taps a causal 3x3 kernel keeps, in the order the packed weights use
__device__ __constant__ int c_tap_ky[5] = {0, 0, 0, 1, 1};
__device__ __constant__ int c_tap_kx[5] = {0, 1, 2, 0, 1};

struct ConvShared {
    uint64_t full[N_STAGES], empty[N_STAGES], tfull[2], tempty[2];
    uint32_t tmem_base;
    float bias_s[4][256];
    float xbest[2][4][32];    // head: the upper class half's best score and class, by tile parity and quadrant
    int xbi[2][4][32];
    float lut_s[256];         // input encoding table
    int img[MAX_IMAGES];      // images still iterating
    unsigned char keep[MAX_IMAGES];
    int n_img;
};

struct ConvEngine {
    static constexpr bool has_jgs = true;
    const ConvDev &m;
    const RunArgs &r;
    ConvShared &sh;
    uint8_t *ring, *staging;
    unsigned epoch = 0;
    unsigned long long issued = 0, skipped = 0, mma_flops = 0, weight_bytes = 0;
    int warp, lane;
    int stage = 0;
    uint32_t sphase = 0;
    int acc = 0;
    uint32_t aphase = 0;
    bool dead = false;
    uint32_t tmem_base = 0;

    __device__ ConvEngine(const ConvDev &m_, const RunArgs &r_, ConvShared &sh_, uint8_t *ring_)
        : m(m_), r(r_), sh(sh_), ring(ring_), staging(ring_ + RING_BYTES)
    {
        warp = threadIdx.x >> 5;
        lane = threadIdx.x & 31;
    }

    // optional device timeline (JS_OPT_TRACE, js_get_trace): first and last CTA, one row of stamps per
    // phase: 0 producer starts, 1 first operands have landed, 2 last MMA issued, 3 last accumulator
    // complete, 4 epilogues done, 5 grid barrier passed
    int phase_no = 0;
    int raised_img = -1, raised_phase = -1;      // last (image, phase) this warp reported a change for
    __device__ void trace(int slot) const
    {
        if (r.trace == nullptr || phase_no >= JS_TRACE_PHASES) return;
        const int who = js_trace_who(r);
        if (who < 0) return;
        r.trace[((size_t)who * JS_TRACE_PHASES + phase_no) * JS_TRACE_SLOTS + slot] = global_ns();
    }

    __device__ bool barrier()
    {
        fence_proxy_async();      // epilogue stores are read by the next layer's TMA loads
        const bool ok = grid_barrier(r.ctl, epoch, r.spin_limit);
        fence_proxy_async();
        if (threadIdx.x == 0) trace(5);
        return ok;
    }

    __device__ void init(const uint8_t *src)
    {
        const size_t n = (size_t)r.batch * m.T;
        __nv_bfloat16 *a0 = (__nv_bfloat16 *)m.act[0];
        for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
            const uint8_t v = src ? src[i] : (uint8_t)0;
            if (r.x) r.x[i] = v;
            const size_t pix = i / m.in_ch;                 // global pixel index (image-major)
            a0[pix * 64 + (i % m.in_ch)] = __float2bfloat16_rn(m.lut[v]);
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
        for (int i = threadIdx.x; i < r.batch; i += blockDim.x) sh.img[i] = i;
        if (threadIdx.x == 0) sh.n_img = r.batch;
        __syncthreads();
    }

    // Images whose iterate did not change are at their fixed point: they drop out of the
    // tile lists.  Every CTA derives the same list from the per-sample flags; rows do not
    // move, so nothing has to be rebuilt.  Always returns 0 (no remapping).
    __device__ int compact(int parity)
    {
        __syncthreads();
        // the flags are fetched by as many threads as there are images (one thread reading them one after
        // the other paid an L2 round trip per image, 7 us per pass on a batch of 16), then one thread packs
        for (int i = threadIdx.x; i < sh.n_img; i += blockDim.x)
            sh.keep[i] = ld_volatile_i32(&r.smp_changed[parity * r.batch + sh.img[i]]) != 0 ? 1 : 0;
        __syncthreads();
        if (threadIdx.x == 0) {
            int k = 0;
            for (int i = 0; i < sh.n_img; ++i)
                if (sh.keep[i]) sh.img[k++] = sh.img[i];
            sh.n_img = k;
            if (blockIdx.x == 0) { r.ctl->compactions += 1; r.ctl->live = k; }
        }
        __syncthreads();
        return 0;
    }

    __device__ uint8_t *stage_a(int s) const { return ring + (size_t)s * STAGE_BYTES; }
    __device__ uint8_t *stage_b(int s) const { return ring + (size_t)s * STAGE_BYTES + A_BYTES; }
    __device__ void advance_stage()
    {
        if (++stage == N_STAGES) { stage = 0; sphase ^= 1u; }
    }
    __device__ void advance_acc()
    {
        acc ^= 1;
        if (acc == 0) aphase ^= 1u;
    }

    // row tiles (of every image) that the window touches.  A hidden unit of colour group g at
    // pixel p reads positions < 3p + g ("degree"); position t = 3p + c.
    __device__ void live_rows(bool head, const Win &w, int &yt_lo, int &yt_hi) const
    {
        const int lo_key = head ? w.olo : w.hdeg_lo + 1;      // live iff largest degree/position >= lo_key
        const int hi_key = head ? w.ohi - 1 : w.hdeg_hi;      // live iff smallest degree/position <= hi_key
        yt_lo = m.nyt;
        yt_hi = 0;
        for (int yt = 0; yt < m.nyt; ++yt) {
            const int p0 = yt * m.R * m.width;
            const int p1 = min(m.height, (yt + 1) * m.R) * m.width - 1;
            const int dmin = p0 * m.in_ch, dmax = p1 * m.in_ch + m.in_ch - 1;
            if (dmax >= lo_key && dmin <= hi_key) { yt_lo = min(yt_lo, yt); yt_hi = max(yt_hi, yt + 1); }
        }
        if (yt_hi < yt_lo) yt_lo = yt_hi = 0;
    }

    // tile id -> (image, row tile, sub-pixel); `per` = 1 for conv layers, in_ch for the head
    __device__ void locate(int id, int nyl, int yt_lo, int per, int &n, int &yt, int &c) const
    {
        c = id % per;
        const int t2 = id / per;
        yt = yt_lo + t2 % nyl;
        n = sh.img[t2 / nyl];
    }

    __device__ int kblocks(int l) const
    {
        return l < m.n_conv ? 5 * (m.cin_pad[l] / BK) : m.ch / BK;
    }

    __device__ void producer(int l, int yt_lo, int nyl, int ntiles, int src)
    {
        const bool head = (l == m.n_conv);
        const int per = head ? m.in_ch : 1;
        const int bn = head ? 256 : m.ch;
        const CUtensorMap *ma_new = m.tmAct + l, *ma_old = m.tmActOld + l, *mw = m.tmW + l;
        const uint32_t bytes = A_BYTES + bn * BK * 2;
        const int kcs = head ? m.ch / BK : m.cin_pad[l] / BK;
        trace(0);
        for (int id = blockIdx.x; id < ntiles && !dead; id += gridDim.x) {
            int n, yt, c;
            locate(id, nyl, yt_lo, per, n, yt, c);
            const int y0 = yt * m.R;
            const int ntaps = head ? 1 : 5;
            for (int tap = 0; tap < ntaps && !dead; ++tap) {
                const int dy = head ? 0 : c_tap_ky[tap] - 1, dx = head ? 0 : c_tap_kx[tap] - 1;
                const CUtensorMap *ma = (src == SRC_OLD || (src == SRC_MIXED && dy < 0)) ? ma_old : ma_new;
                for (int kc = 0; kc < kcs; ++kc) {
                    if (!mbar_wait(&sh.empty[stage], sphase ^ 1u, r.ctl)) { dead = true; break; }
                    mbar_expect_tx(&sh.full[stage], bytes);
                    tma_load_4d(smem_u32(stage_a(stage)), ma, &sh.full[stage], kc * BK, dx, y0 + dy, n);
                    tma_load_2d(smem_u32(stage_b(stage)), mw, &sh.full[stage], kc * BK,
                                head ? c * 256 : tap * m.ch);
                    advance_stage();
                }
            }
        }
    }

    __device__ void mma_issuer(int l, int ntiles)
    {
        const bool head = (l == m.n_conv);
        const uint32_t idesc = instr_desc_bf16(head ? 256 : m.ch);
        const int nkb = kblocks(l);
        for (int id = blockIdx.x; id < ntiles && !dead; id += gridDim.x) {
            if (!mbar_wait(&sh.tempty[acc], aphase ^ 1u, r.ctl)) { dead = true; break; }
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(acc * ACC_COLS);
            for (int kb = 0; kb < nkb; ++kb) {
                if (!mbar_wait(&sh.full[stage], sphase, r.ctl)) { dead = true; break; }
                tc_fence_after();
                if (kb == 0 && id == (int)blockIdx.x) trace(1);
                const uint64_t adesc = smem_desc_sw128(smem_u32(stage_a(stage)));
                const uint64_t bdesc = smem_desc_sw128(smem_u32(stage_b(stage)));
#pragma unroll
                for (int k = 0; k < BK / 16; ++k)
                    umma_bf16(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc,
                              (kb > 0 || k > 0) ? 1u : 0u);
                umma_commit(&sh.empty[stage]);
                advance_stage();
            }
            if (dead) break;
            umma_commit(&sh.tfull[acc]);
            advance_acc();
        }
        trace(2);
    }

    __device__ void release_acc()
    {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.tempty[acc]);
    }

    // conv layer: ReLU(acc + bias) -> bf16, through the staging buffer so that the NHWC stores
    // are coalesced (see the masked-MLP kernel for the layout of the staging rows)
    __device__ void epi_hidden_tile(int l, int n, int y0, uint32_t tbase, int src)
    {
        uint8_t *stg = staging + (size_t)(warp - 2) * 8192;
        const float *bs = sh.bias_s[warp - 2];
        const int bn = m.ch;
#pragma unroll 1
        for (int c0 = 0; c0 < bn; c0 += 32) {
            float v[32];
            tmem_ld32(tbase + (uint32_t)c0, v);
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 32; i += 2)
                pk[i / 2] = pack_bf16x2(fmaxf(v[i] + bs[c0 + i], 0.0f), fmaxf(v[i + 1] + bs[c0 + i + 1], 0.0f));
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int chunk = c0 / 8 + i;
                *reinterpret_cast<uint4 *>(stg + lane * 256 + ((chunk ^ (lane & 15)) << 4)) =
                    make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
            }
        }
        release_acc();
        __nv_bfloat16 *out = (__nv_bfloat16 *)(src == SRC_OLD ? m.act_old[l + 1] : m.act[l + 1]);
        const int q = warp & 3, ch = lane & 15;
        const int col = ch * 8;
        const int rows_valid = (min(m.height, y0 + m.R) - y0) * m.width;     // pixels of the tile inside the image
        const size_t pix0 = (size_t)n * m.height * m.width + (size_t)y0 * m.width;
#pragma unroll 4
        for (int it = 0; it < 16; ++it) {
            const int rl = it * 2 + (lane >> 4);
            const uint4 val = *reinterpret_cast<const uint4 *>(stg + rl * 256 + ((ch ^ (rl & 15)) << 4));
            const int prow = q * 32 + rl;
            if (prow < rows_valid && col < bn) *reinterpret_cast<uint4 *>(out + (pix0 + prow) * bn + col) = val;
        }
        __syncwarp();
    }

    // Inverse CDF of the softmax from one uniform number u: the first class c with u * S < sum_{i<=c} e_i,
    // e_i = exp(z_i - max z).  Three readings of the thread's 256 logits out of tensor memory: the maximum,
    // the running sums (kept at the chunk ends), the class inside the chunk found.  Kept out of line: it
    // must not cost the Gumbel path registers.
    __device__ __noinline__ int head_icdf(uint32_t tbase, const float *bias, float u)
    {
        float mx = -INFINITY;
        for (int c0 = 0; c0 < 256; c0 += 32) {
            float v[32];
            __syncwarp();
            tmem_ld32(tbase + (uint32_t)c0, v);
#pragma unroll
            for (int i = 0; i < 32; ++i) mx = fmaxf(mx, v[i] + __ldg(bias + c0 + i));
        }
        float run = 0.0f, cum[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            float v[32];
            __syncwarp();
            tmem_ld32(tbase + (uint32_t)(k * 32), v);
#pragma unroll
            for (int i = 0; i < 32; ++i) run += __expf((v[i] + __ldg(bias + k * 32 + i)) - mx);
            cum[k] = run;
        }
        const float target = u * run;
        int ck = 8;
        float base = 0.0f;
#pragma unroll
        for (int k = 7; k >= 0; --k)
            if (target < cum[k]) { ck = k; base = k > 0 ? cum[k - 1] : 0.0f; }
        int bi = (run == run) ? 255 : 0;          // u at the very top of the range; no finite score: class 0
        for (int k = 0; k < 8; ++k) {
            float v[32];
            __syncwarp();
            tmem_ld32(tbase + (uint32_t)(k * 32), v);         // warp-wide load: every lane takes part
            if (k != ck) continue;
            float s2 = base;
            int hit = -1;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                s2 += __expf((v[i] + __ldg(bias + k * 32 + i)) - mx);
                hit = (hit < 0 && target < s2) ? i : hit;
            }
            bi = k * 32 + (hit < 0 ? 31 : hit);
        }
        return bi;
    }

    __device__ void epilogue(int l, int kind, const Win &w, bool flag, int parity, float *zout, int yt_lo, int nyl,
                             int ntiles, int src)
    {
        const bool head = (l == m.n_conv);
        const int per = head ? m.in_ch : 1;
        const int q = warp & 3;
        // Two warps share a quadrant (a warp reaches only the tensor-memory lanes of its own quadrant).  The
        // second one takes the upper 128 classes of a 256-way head tile: the argmax is bound by instruction
        // issue, one warp per scheduler was not enough; elsewhere it only hands the accumulator back.
        const int half = (warp - 2) >> 2;
        int tile_par = 0;
        bool any_changed = false;
        int first = INT_MAX;
        for (int id = blockIdx.x; id < ntiles && !dead; id += gridDim.x) {
            int n, yt, c;
            locate(id, nyl, yt_lo, per, n, yt, c);
            const int y0 = yt * m.R;
            const bool split_head = head && kind == EPI_CAT && r.nk == JS_NOISE_GUMBEL;
            if (half == 1 && !(head && (split_head || kind == EPI_LOGITS))) {
                if (!mbar_wait(&sh.tfull[acc], aphase, r.ctl)) { dead = true; break; }
                tc_fence_after();
                release_acc();
                advance_acc();
                continue;
            }
            if (!head) {
                float *bs = sh.bias_s[warp - 2];
                __syncwarp();
                for (int i = lane; i < m.ch; i += 32) bs[i] = m.bias[l][i];
                __syncwarp();
            }
            if (!mbar_wait(&sh.tfull[acc], aphase, r.ctl)) { dead = true; break; }
            tc_fence_after();
            if (warp == 4 && lane == 0) trace(3);
            const uint32_t tbase = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * ACC_COLS);
            if (!head) {
                epi_hidden_tile(l, n, y0, tbase, src);
            } else {
                // thread = one pixel of the tile; 256 logits of sub-pixel c
                const int prow = q * 32 + lane;
                const int rows_valid = (min(m.height, y0 + m.R) - y0) * m.width;
                const bool valid = prow < rows_valid;
                const int pix = y0 * m.width + prow;
                const int t = pix * m.in_ch + c;
                const size_t at = (size_t)n * m.T + t;
                const float *bias = m.bias[m.n_conv] + (size_t)c * 256;
                float best = -INFINITY;
                int bi = 0;
                // the current symbol, asked for now: its latency passes while the classes are reduced
                const bool commit = kind == EPI_CAT && valid && t >= w.plo && t < w.phi;
                int xold = 0;
                if (commit) xold = (int)__ldcg(r.x + at);
                if (kind == EPI_CAT && r.nk == JS_NOISE_UNIFORM_CAT) {
                    bi = head_icdf(tbase, bias, commit ? __ldg(r.noise + at) : 0.5f);
                } else
                for (int c0 = half * 128; c0 < half * 128 + 128; c0 += 32) {
                    float v[32];
                    __syncwarp();
                    tmem_ld32(tbase + (uint32_t)c0, v);
                    if (!valid) continue;
                    if (kind == EPI_LOGITS) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) zout[at * 256 + c0 + i] = v[i] + bias[c0 + i];
                    } else {
                        const float *gg = r.noise + at * 256 + c0;
                        float sc[32];
#pragma unroll
                        for (int i = 0; i < 32; i += 4) {
                            const float4 b4 = __ldg(reinterpret_cast<const float4 *>(bias + c0 + i));
                            const float4 g4 = __ldg(reinterpret_cast<const float4 *>(gg + i));
                            sc[i] = (v[i] + b4.x) + g4.x;
                            sc[i + 1] = (v[i + 1] + b4.y) + g4.y;
                            sc[i + 2] = (v[i + 2] + b4.z) + g4.z;
                            sc[i + 3] = (v[i + 3] + b4.w) + g4.w;
                        }
                        argmax_chunk32(sc, c0, best, bi);
                    }
                }
                release_acc();        // the accumulator has been read: the next tile's MMAs may have it
                if (split_head) {
                    // the two halves meet: the upper half's result wins only if strictly larger (lowest index on ties)
                    if (half == 1) {
                        sh.xbest[tile_par][q][lane] = best;
                        sh.xbi[tile_par][q][lane] = bi;
                    }
                    asm volatile("bar.sync %0, 64;" ::"r"(1 + q) : "memory");
                    if (half == 0) {
                        const float b1 = sh.xbest[tile_par][q][lane];
                        if (b1 > best) { best = b1; bi = sh.xbi[tile_par][q][lane]; }
                    }
                    tile_par ^= 1;
                }
                if (half == 1) { advance_acc(); continue; }
                bool ch = false;
                if (commit && xold != bi) {
                    r.x[at] = (uint8_t)bi;
                    ((__nv_bfloat16 *)m.act[0])[((size_t)n * m.height * m.width + pix) * 64 + c] =
                        __float2bfloat16_rn(sh.lut_s[bi]);
                    ch = true;
                }
                if (flag) {
                    // every pixel of the tile belongs to image n: one lane reports for the warp, with a
                    // plain store (a load to look first would be an L2 round trip per tile), and only
                    // once per image and phase
                    if (__any_sync(0xffffffffu, ch) && (raised_img != n || raised_phase != phase_no)) {
                        if (lane == 0) r.smp_changed[parity * r.batch + n] = 1;
                        raised_img = n;
                        raised_phase = phase_no;
                    }
                    if (ch) {
                        any_changed = true;
                        first = min(first, t);
                    }
                }
            }
            advance_acc();
        }
        if (warp == 4 && lane == 0) trace(4);
        if (flag) {
            const bool wany = __any_sync(0xffffffffu, any_changed);
            if (wany) {
                const int wmin = __reduce_min_sync(0xffffffffu, first);
                if (lane == 0) {
                    atomicMin(&r.ctl->agg_minfirst[parity], wmin);
                    atomicOr(&r.ctl->agg_any[parity], 1);
                }
            }
        }
    }

    __device__ bool layer_phase(int l, int kind, const Win &w, bool flag, int parity, float *zout, int src = SRC_NEW)
    {
        const bool head = (l == m.n_conv);
        int yt_lo, yt_hi;
        live_rows(head, w, yt_lo, yt_hi);
        const int nyl = yt_hi - yt_lo;
        const int ntiles = sh.n_img * nyl * (head ? m.in_ch : 1);
        if (threadIdx.x == 0) {
            for (int id = blockIdx.x; id < ntiles; id += gridDim.x) {
                issued++;
                mma_flops += 2ull * BM * BK * (unsigned long long)(head ? 256 : m.ch) * (unsigned long long)kblocks(l);
            }
            // a layer's packed weights serve every tile: the pass streams them once
            if (blockIdx.x == 0 && ntiles > 0)
                weight_bytes += 2ull * BK * (unsigned long long)kblocks(l) * (unsigned long long)(head ? 256 * m.in_ch : m.ch);
            if (blockIdx.x == 0) skipped += (unsigned long long)(r.batch * m.nyt - sh.n_img * nyl) * (head ? m.in_ch : 1);
        }
        if (ntiles == 0) return false;
        phase_no++;
        if (warp == 0) {
            if (lane == 0) producer(l, yt_lo, nyl, ntiles, src);
        } else if (warp == 1) {
            if (lane == 0) mma_issuer(l, ntiles);
        } else {
            epilogue(l, kind, w, flag, parity, zout, yt_lo, nyl, ntiles, src);
        }
        return true;
    }

    __device__ bool step(const Win &w, bool flag, int parity, float *zout, int src = SRC_NEW)
    {
        const int l_end = src == SRC_OLD ? m.n_conv - 1 : m.n_conv;      // the old set needs no head
        for (int l = 0; l <= l_end; ++l) {
            const bool last = (l == m.n_conv);
            const bool did = layer_phase(l, last ? (zout ? EPI_LOGITS : EPI_CAT) : EPI_HIDDEN, w, last && flag, parity, zout, src);
            if (did || l == l_end)
                if (!barrier()) return false;
        }
        return true;
    }

    // One outer iteration of Algorithm 2 with one-image-row blocks.  A block's sequential sweep yields the
    // unique solution of the block's own triangular system given the rows above at the previous outer
    // iterate; Jacobi iterations on that sub-system reach the very same solution in at most |B| steps
    // (Proposition 1 applied to the block), and they can run for all rows of all images at once as
    // forward passes in which every layer reads the row above from the activations of x^{k-1} and its
    // own row from the working activations.  So: the hidden layers once on x^{k-1} (the "old" set),
    // then mixed passes until no symbol changes, then the comparison with x^{k-1} for the outer flags,
    // which are left in the flag slot `parity`.
    __device__ bool jgs_outer(int parity, int, int, int &iterations)
    {
        const size_t n = (size_t)r.batch * m.T;
        const size_t npix64 = (size_t)r.batch * m.height * m.width * 64 / 8;       // uint4 units of the padded image
        for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
            r.x_old[i] = r.x[i];
        {
            const uint4 *src = reinterpret_cast<const uint4 *>(m.act[0]);
            uint4 *dst = reinterpret_cast<uint4 *>(m.act_old[0]);
            for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < npix64; i += (size_t)gridDim.x * blockDim.x)
                dst[i] = src[i];
        }
        if (!barrier()) return false;
        // every CTA has read the previous outer iteration's flags by now: both slots start clean
        if (blockIdx.x == 0) {
            for (int i = threadIdx.x; i < 2 * r.batch; i += blockDim.x) r.smp_changed[i] = 0;
            if (threadIdx.x == 0) {
                r.ctl->agg_any[0] = r.ctl->agg_any[1] = 0;
                r.ctl->agg_minfirst[0] = r.ctl->agg_minfirst[1] = INT_MAX;
            }
        }
        const Win w = make_win(0, m.T, 0, m.T);
        if (!step(w, false, 0, nullptr, SRC_OLD)) return false;
        iterations++;
        const int cap = m.width * m.in_ch;
        int q = parity;
        for (int k = 1; k <= cap; ++k) {
            q ^= 1;
            if (!step(w, true, q, nullptr, SRC_MIXED)) return false;
            iterations++;
            const int any = ld_volatile_i32(&r.ctl->agg_any[q]);
            reset_other_parity(r, q);
            if (!barrier()) return false;
            if (!any) break;
        }
        // both flag slots start clean, then the outer comparison fills slot `parity`
        if (blockIdx.x == 0) {
            for (int i = threadIdx.x; i < 2 * r.batch; i += blockDim.x) r.smp_changed[i] = 0;
            if (threadIdx.x == 0) {
                r.ctl->agg_any[0] = r.ctl->agg_any[1] = 0;
                r.ctl->agg_minfirst[0] = r.ctl->agg_minfirst[1] = INT_MAX;
            }
        }
        if (!barrier()) return false;
        for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
            if (r.x[i] != r.x_old[i]) note_change(r, parity, (int)(i / m.T), (int)(i % m.T));
        return barrier();
    }
};

__global__ void __launch_bounds__(NTH, 1)
conv_tc_kernel(const __grid_constant__ ConvDev m, const __grid_constant__ RunArgs r)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ ConvShared sh;
    uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        for (int s = 0; s < N_STAGES; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&sh.tfull[a], 1); mbar_init(&sh.tempty[a], 8); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    for (int i = threadIdx.x; i < 256; i += blockDim.x) sh.lut_s[i] = m.lut[i];
    if (warp == 1) tmem_alloc(&sh.tmem_base, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    ConvEngine e(m, r, sh, ring);
    e.tmem_base = sh.tmem_base;
    DriverResult res = made_driver(e, m.T, r);
    if (e.dead) res.alive = false;

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
    driver_finish(r, res, e.issued, e.skipped, e.mma_flops, e.weight_bytes);
}

}  // namespace

// --------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn conv_encode_fn()
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

static bool encode_nd(CUtensorMap *out, const void *base, int rank, const cuuint64_t *dims, const cuuint64_t *strides,
                      const cuuint32_t *box)
{
    EncodeTiledFn fn = conv_encode_fn();
    if (!fn) return false;
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <typename T>
static bool upload(js_model *mo, const T *host, size_t count, T **dev)
{
    void *p = nullptr;
    if (cudaMalloc(&p, std::max<size_t>(count * sizeof(T), 16)) != cudaSuccess) return false;
    mo->allocs.push_back(p);
    if (host) {
        if (cudaMemcpy(p, host, count * sizeof(T), cudaMemcpyHostToDevice) != cudaSuccess) return false;
    } else if (cudaMemset(p, 0, count * sizeof(T)) != cudaSuccess) {
        return false;
    }
    *dev = (T *)p;
    return true;
}

// Builds the device model of a masked-conv stack.  JS_OK, JS_ERR_UNSUPPORTED for shapes the
// kernel does not cover, JS_ERR_CUDA on runtime failures.
int js_conv_build(js_model *mo, const js_conv_desc *d)
{
    ConvDev &v = mo->conv;
    if (d->prec != JS_BF16 || d->C != 256 || d->n_lut != 256) return JS_ERR_UNSUPPORTED;
    if (d->in_ch < 1 || d->in_ch > 8 || (d->ch != 64 && d->ch != 128)) return JS_ERR_UNSUPPORTED;
    if (d->width < 8 || d->width > 128 || (128 % d->width) != 0 || d->height < 1) return JS_ERR_UNSUPPORTED;
    if (d->n_conv < 1 || d->n_conv > JS_MAXL || d->max_batch > MAX_IMAGES) return JS_ERR_UNSUPPORTED;
    if (!conv_encode_fn()) return JS_ERR_UNSUPPORTED;
    v.height = d->height; v.width = d->width; v.in_ch = d->in_ch; v.ch = d->ch; v.n_conv = d->n_conv; v.C = d->C;
    v.T = d->height * d->width * d->in_ch;
    v.R = 128 / d->width;
    v.nyt = (d->height + v.R - 1) / v.R;
    const int ch = d->ch, nb = mo->max_batch;
    const size_t npix = (size_t)nb * d->height * d->width;
    auto group = [&](int k) { return (int)(((long long)d->in_ch * k) / ch); };

    std::vector<CUtensorMap> mapsA(d->n_conv + 1), mapsAold(d->n_conv + 1), mapsW(d->n_conv + 1);
    for (int l = 0; l <= d->n_conv; ++l) {
        const int c_l = l == 0 ? 64 : ch;                 // channels of act[l] (the image is padded to 64)
        if (l < d->n_conv) v.cin_pad[l] = c_l;
        // two sets: the working activations, and those of the previous outer iterate (Jacobi-GS)
        for (int set = 0; set < 2; ++set) {
            __nv_bfloat16 *a = nullptr;
            if (!upload<__nv_bfloat16>(mo, nullptr, npix * c_l, &a)) return JS_ERR_CUDA;
            (set == 0 ? v.act[l] : v.act_old[l]) = a;
            const cuuint64_t dims[4] = {(cuuint64_t)c_l, (cuuint64_t)d->width, (cuuint64_t)d->height, (cuuint64_t)nb};
            const cuuint64_t strides[3] = {(cuuint64_t)c_l * 2, (cuuint64_t)d->width * c_l * 2,
                                           (cuuint64_t)d->height * d->width * c_l * 2};
            const cuuint32_t box[4] = {(cuuint32_t)BK, (cuuint32_t)d->width, (cuuint32_t)v.R, 1};
            if (!encode_nd(set == 0 ? &mapsA[l] : &mapsAold[l], a, 4, dims, strides, box)) return JS_ERR_UNSUPPORTED;
        }
    }
    static const int tky[5] = {0, 0, 0, 1, 1}, tkx[5] = {0, 1, 2, 0, 1};
    for (int l = 0; l < d->n_conv; ++l) {
        const int cin = l == 0 ? d->in_ch : ch, cpad = v.cin_pad[l];
        std::vector<__nv_bfloat16> wp((size_t)5 * ch * cpad, __float2bfloat16_rn(0.0f));
        for (int tap = 0; tap < 5; ++tap)
            for (int co = 0; co < ch; ++co)
                for (int ci = 0; ci < cin; ++ci) {
                    bool keep = true;
                    if (tap == 4) {                       // centre tap: colour-group mask, type A then type B
                        const int gi = l == 0 ? ci : group(ci), go = group(co);
                        keep = l == 0 ? (gi < go) : (gi <= go);
                    }
                    const float w = keep ? d->W[l][(((size_t)co * 3 + tky[tap]) * 3 + tkx[tap]) * cin + ci] : 0.0f;
                    wp[((size_t)tap * ch + co) * cpad + ci] = __float2bfloat16_rn(w);
                }
        __nv_bfloat16 *wd = nullptr;
        if (!upload<__nv_bfloat16>(mo, wp.data(), wp.size(), &wd)) return JS_ERR_CUDA;
        const cuuint64_t dims[2] = {(cuuint64_t)cpad, (cuuint64_t)5 * ch};
        const cuuint64_t strides[1] = {(cuuint64_t)cpad * 2};
        const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)ch};
        if (!encode_nd(&mapsW[l], wd, 2, dims, strides, box)) return JS_ERR_UNSUPPORTED;
        float *bd = nullptr;
        if (!upload<float>(mo, d->b[l], ch, &bd)) return JS_ERR_CUDA;
        v.bias[l] = bd;
    }
    {
        const int nout = d->in_ch * d->C;
        std::vector<__nv_bfloat16> wh((size_t)nout * ch);
        for (int o = 0; o < nout; ++o)
            for (int ci = 0; ci < ch; ++ci)
                wh[(size_t)o * ch + ci] =
                    __float2bfloat16_rn(group(ci) <= o / d->C ? d->W[d->n_conv][(size_t)o * ch + ci] : 0.0f);
        __nv_bfloat16 *wd = nullptr;
        if (!upload<__nv_bfloat16>(mo, wh.data(), wh.size(), &wd)) return JS_ERR_CUDA;
        const cuuint64_t dims[2] = {(cuuint64_t)ch, (cuuint64_t)nout};
        const cuuint64_t strides[1] = {(cuuint64_t)ch * 2};
        const cuuint32_t box[2] = {(cuuint32_t)BK, 256};
        if (!encode_nd(&mapsW[d->n_conv], wd, 2, dims, strides, box)) return JS_ERR_UNSUPPORTED;
        float *bd = nullptr;
        if (!upload<float>(mo, d->b[d->n_conv], nout, &bd)) return JS_ERR_CUDA;
        v.bias[d->n_conv] = bd;
    }
    {
        std::vector<float> lut(d->lut, d->lut + d->n_lut);
        for (auto &f : lut) f = __bfloat162float(__float2bfloat16_rn(f));
        float *ld = nullptr;
        if (!upload<float>(mo, lut.data(), lut.size(), &ld)) return JS_ERR_CUDA;
        v.lut = ld;
    }
    CUtensorMap *pa = nullptr, *pw = nullptr, *pao = nullptr;
    if (!upload<CUtensorMap>(mo, mapsAold.data(), mapsAold.size(), &pao)) return JS_ERR_CUDA;
    v.tmActOld = pao;
    if (!upload<CUtensorMap>(mo, mapsA.data(), mapsA.size(), &pa)) return JS_ERR_CUDA;
    if (!upload<CUtensorMap>(mo, mapsW.data(), mapsW.size(), &pw)) return JS_ERR_CUDA;
    v.tmAct = pa;
    v.tmW = pw;
    if (cudaFuncSetAttribute(conv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess) {
        cudaGetLastError();
        return JS_ERR_UNSUPPORTED;
    }
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    mo->conv_max_grid = sms;
    mo->conv_T = v.T;
    mo->conv_C = v.C;
    return JS_OK;
}

int js_launch_conv_tc(const js_model *mo, const RunArgs &r, cudaStream_t stream)
{
    const ConvDev &v = mo->conv;
    const int tiles = r.batch * v.nyt * v.in_ch;
    const int grid = std::max(1, std::min(mo->conv_max_grid, tiles));
    void *args[2] = {(void *)&v, (void *)&r};
    cudaError_t e = cudaLaunchCooperativeKernel((const void *)conv_tc_kernel, dim3(grid), dim3(NTH), args, SMEM_BYTES,
                                                stream);
    return e == cudaSuccess ? 0 : (int)e;
}
