// Tensor-core path of the masked-MLP sampler for sm_100a.
//
// One persistent cooperative kernel runs the whole solver.  Every layer of the
// masked network is a GEMM  D[128 samples x BN units] = A[128 x K] * W[BN x K]^T
// on the 5th-generation tensor cores: operands arrive in shared memory by TMA
// (128-byte swizzle, K-major), one elected thread issues tcgen05.mma with the
// fp32 accumulator in tensor memory, and four epilogue warps read it back with
// tcgen05.ld.  Masked (all-zero) K blocks beyond a tile's last live input are
// never loaded; adding exact zeros would not change the fp32 sum, so h_t stays
// the same function whatever is skipped.  The output layer's epilogue is the
// sampling step itself (Appendix A.3 of arXiv 2002.03629): bias, fixed noise,
// threshold or 256-way argmax, compare with the previous iterate, per-sample
// change flags; logits never reach global memory.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM
// owner, warps 2-5 = epilogue (TMEM lane quadrant = warp index mod 4).
// All waits are bounded; a wait that gives up raises the abort flag, every role
// drains, TMEM is freed and the kernel returns JS_ERR_TIMEOUT.
#include <cuda.h>

#include <algorithm>

#include "js_common.cuh"
#include "js_model.h"
#include "made_driver.cuh"
#include "tc_common.cuh"

namespace {

constexpr int BM = TC_BM;          // samples per tile (UMMA M)
constexpr int BK = TC_BK;          // bf16 elements per K block
constexpr int NTH = 192;
constexpr int ACC_COLS = 256;      // TMEM columns per accumulator slot (two slots)
constexpr int A_BYTES = BM * BK * 2;
constexpr int STAGING_BYTES = 32 * 1024;   // epilogue transposition buffer, 8 KB per epilogue warp
constexpr int MAX_STAGES = 6;
// binary output tiles: per sample row 128 noise values and 128 symbols, rows padded by 16 bytes
constexpr int BIN_NZ_ROW = 512 + 16, BIN_XS_ROW = 128 + 16;
constexpr int BIN_NZ_BYTES = BM * BIN_NZ_ROW, BIN_XS_BYTES = BM * BIN_XS_ROW;
constexpr int CAT_ROW = 1024 + 16;     // 256-way output tiles: a sample row's noise, padded
// Shared memory after the 1 KB alignment slack: operand ring | auxiliary buffer | tile metadata.
// The auxiliary buffer is the staging area of the hidden-layer epilogues and, in models with
// binary outputs, also holds the noise and symbol rows of an output tile (never both at once).
constexpr int SMEM_DYN_MAX = 227 * 1024 - 6 * 1024;      // what a CTA may ask for beside its static part

enum { EPI_HIDDEN = 0, EPI_LOGITS = 1, EPI_BINARY = 2, EPI_CAT = 3 };

struct TcShared {
    uint64_t full[MAX_STAGES], empty[MAX_STAGES], tfull[2], tempty[2];
    uint64_t nzbar[4];             // per epilogue warp: bulk copies of a binary tile's noise and symbols
    uint32_t tmem_base;
    int off[JS_MAXL + 1];          // start of layer l's tile metadata inside `meta`
    float lut_s[256];              // input encoding table (a lookup per committed symbol would be an L2 round trip)
    alignas(16) float bias_s[4][256];   // per epilogue warp: bias of the current tile's columns (read as float4)
    int wcnt[NTH / 32];            // compaction: per-warp counts
    int cbase;                     // compaction: rows kept so far
};

// ------------------------------------------------------------------ engine
struct TcEngine {
    static constexpr bool has_jgs = false;
    const MadeDev &m;
    const TcDev &t;
    const RunArgs &r;
    TcShared &sh;
    uint8_t *ring;
    uint8_t *staging;
    const int *meta;               // tile metadata in shared memory: per layer kb_end[nt], dmin[nt], dmax[nt]
    unsigned epoch = 0;
    unsigned long long issued = 0, skipped = 0, mma_flops = 0, weight_bytes = 0;
    int warp, lane;
    // pipeline state, advanced identically by the roles that share it
    int stage = 0;
    uint32_t spar = 0;             // bit s: parity of the next use of ring stage s
    int cur_stages = 1, cur_stage_bytes = 0;      // ring geometry of the current layer
    int acc = 0;
    uint32_t aphase = 0;
    uint32_t nzphase = 0;
    bool noise_here = false;       // the uploaded noise has been seen to be complete
    bool dead = false;
    uint32_t tmem_base = 0;
    // working batch: rows [0, live) of the activation buffers hold samples perm[pcur][row]
    int live = 0;
    int pcur = 0;

    __device__ TcEngine(const MadeDev &m_, const TcDev &t_, const RunArgs &r_, TcShared &sh_, uint8_t *ring_,
                        const int *meta_)
        : m(m_), t(t_), r(r_), sh(sh_), ring(ring_), staging(ring_ + t_.ring_bytes), meta(meta_)
    {
        warp = threadIdx.x >> 5;
        lane = threadIdx.x & 31;
        live = r.batch;
    }
    __device__ const int *perm_cur() const { return r.perm + (size_t)pcur * r.perm_stride; }

    int phase_no = 0;              // counts gemm phases, for the optional timeline
    unsigned stamp = 0;            // phase counter: marks this phase's partial-sum flags
    // partial sums the tile being finished has to add (owner chunk): set per tile by the epilogue
    int cur_parts = 0;
    const float *cur_pbase = nullptr;
    size_t cur_tile_floats = 0;
    __device__ void trace(int slot) const
    {
        if (r.trace == nullptr || phase_no >= JS_TRACE_PHASES) return;
        const int who = js_trace_who(r);
        if (who < 0) return;
        r.trace[((size_t)who * JS_TRACE_PHASES + phase_no) * JS_TRACE_SLOTS + slot] = global_ns();
    }

    __device__ bool barrier()
    {
        // epilogue stores of this phase must be visible to the TMA reads of the next one
        fence_proxy_async();
        const bool ok = grid_barrier(r.ctl, epoch, r.spin_limit);
        fence_proxy_async();
        if (threadIdx.x == 0) trace(5);
        return ok;
    }

    __device__ void init(const uint8_t *src)
    {
        const size_t n = (size_t)r.batch * m.T;
        __nv_bfloat16 *a0 = (__nv_bfloat16 *)m.a[0];
        if (n % 16 == 0 && ((uintptr_t)src & 15u) == 0) {
            // sixteen positions per step (the buffers are 16-byte aligned)
            for (size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 16; i < n; i += (size_t)gridDim.x * blockDim.x * 16) {
                const uint4 xv = src ? __ldcg(reinterpret_cast<const uint4 *>(src + i)) : make_uint4(0u, 0u, 0u, 0u);
                if (r.x) *reinterpret_cast<uint4 *>(r.x + i) = xv;
                const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w};
                uint32_t o[8];
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    o[k] = pack_bf16x2(m.lut[(xw[k >> 1] >> (16 * (k & 1))) & 0xffu],
                                       m.lut[(xw[k >> 1] >> (16 * (k & 1) + 8)) & 0xffu]);
                uint4 *dst = reinterpret_cast<uint4 *>(a0 + i);
                dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
                dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
            }
        } else {
            for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
                const uint8_t v = src ? src[i] : (uint8_t)0;
                if (r.x) r.x[i] = v;
                a0[i] = __float2bfloat16_rn(m.lut[v]);
            }
        }
        for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < (size_t)t.n_pflags;
             i += (size_t)gridDim.x * blockDim.x)
            t.pflags[i] = 0u;
        if (blockIdx.x == 0) {
            for (int i = threadIdx.x; i < 2 * r.batch; i += blockDim.x) {
                r.smp_changed[i] = 0;
                r.smp_state[i] = 0;
            }
            for (int i = threadIdx.x; i < r.batch; i += blockDim.x) r.perm[i] = i;
            if (threadIdx.x == 0) {
                r.ctl->agg_any[0] = r.ctl->agg_any[1] = 0;
                r.ctl->agg_minfirst[0] = r.ctl->agg_minfirst[1] = INT_MAX;
            }
        }
    }

    // Compaction of the working batch after an iteration of parity `parity`.  Every CTA computes
    // the same list (rows whose sample changed, in order) from the per-sample flags, so no exchange
    // is needed to agree on it.  It is adopted only when it frees at least one 128-row tile; then
    // the encoded iterate is rebuilt for the new rows and a grid barrier makes it visible.
    // Returns 1 if rows were remapped, 0 if not, -1 if the barrier gave up.
    __device__ int compact(int parity)
    {
        const int *pc = perm_cur();
        int *pn = r.perm + (size_t)(pcur ^ 1) * r.perm_stride;
        const int *chg = r.smp_changed + (size_t)parity * r.batch;
        if (threadIdx.x == 0) sh.cbase = 0;
        __syncthreads();
        // four rows per thread and round, their loads in flight together
        for (int base = 0; base < live; base += 4 * NTH) {
            int b[4];
            bool keep[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int row = base + i * NTH + threadIdx.x;
                b[i] = row < live ? __ldcg(&pc[row]) : -1;
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) keep[i] = b[i] >= 0 && ld_volatile_i32(&chg[b[i]]) != 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (base + i * NTH >= live) break;
                const unsigned bal = __ballot_sync(0xffffffffu, keep[i]);
                if (lane == 0) sh.wcnt[warp] = __popc(bal);
                __syncthreads();
                int off = sh.cbase;
                for (int w2 = 0; w2 < warp; ++w2) off += sh.wcnt[w2];
                if (keep[i]) pn[off + __popc(bal & ((1u << lane) - 1u))] = b[i];
                int tot = 0;
                for (int w2 = 0; w2 < NTH / 32; ++w2) tot += sh.wcnt[w2];
                __syncthreads();
                if (threadIdx.x == 0) sh.cbase += tot;
                __syncthreads();
            }
        }
        const int nlive = sh.cbase;
        __syncthreads();
        if ((nlive + BM - 1) / BM >= (live + BM - 1) / BM) return 0;
        live = nlive;
        pcur ^= 1;
        if (blockIdx.x == 0 && threadIdx.x == 0) { r.ctl->compactions += 1; r.ctl->live = nlive; }
        __threadfence_block();
        __nv_bfloat16 *a0 = (__nv_bfloat16 *)m.a[0];
        if (m.T % 16 == 0) {
            // sixteen positions per step: one 16-byte load of symbols, two 16-byte stores of encodings
            const int per_row = m.T / 16;
            const size_t n = (size_t)live * per_row;
            for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
                const int row = (int)(i / per_row), d = (int)(i % per_row) * 16;
                const uint4 xv = __ldcg(reinterpret_cast<const uint4 *>(r.x + (size_t)pn[row] * m.T + d));
                const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w};
                uint32_t o[8];
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    o[k] = pack_bf16x2(m.lut[(xw[k >> 1] >> (16 * (k & 1))) & 0xffu],
                                       m.lut[(xw[k >> 1] >> (16 * (k & 1) + 8)) & 0xffu]);
                uint4 *dst = reinterpret_cast<uint4 *>(a0 + (size_t)row * m.T + d);
                dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
                dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
            }
        } else {
            const size_t n = (size_t)live * m.T;
            for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
                const int row = (int)(i / m.T), d = (int)(i % m.T);
                a0[i] = __float2bfloat16_rn(m.lut[r.x[(size_t)pn[row] * m.T + d]]);
            }
        }
        return barrier() ? 1 : -1;
    }

    __device__ int kb_end_of(int l, int nt) const { return meta[sh.off[l] + nt]; }
    // a 256-way output tile is one position: its degrees need no table
    __device__ bool one_pos_tiles(int l) const { return l == m.L && m.C == 256; }
    __device__ int dmin_of(int l, int nt) const { return one_pos_tiles(l) ? nt + 1 : meta[sh.off[l] + t.lay[l].nt + nt]; }
    __device__ int dmax_of(int l, int nt) const { return one_pos_tiles(l) ? nt + 1 : meta[sh.off[l] + 2 * t.lay[l].nt + nt]; }

    // The ring is cut anew for every layer: narrower weight tiles give more, smaller stages in the
    // same memory.  That is safe because the ring is drained at every phase boundary, and because
    // the parity of a stage's barriers is kept per stage (the u-th use of stage s waits for
    // completion u of full[s] and for completion u-1 of empty[s], whatever the order of use).
    __device__ void ring_for_layer(int l)
    {
        cur_stages = t.lay[l].n_stages;
        cur_stage_bytes = t.lay[l].stage_bytes;
        stage = 0;
    }
    __device__ uint8_t *stage_a(int s) const { return ring + (size_t)s * cur_stage_bytes; }
    __device__ uint8_t *stage_b(int s) const { return ring + (size_t)s * cur_stage_bytes + A_BYTES; }
    __device__ uint32_t stage_parity() const { return (spar >> stage) & 1u; }
    __device__ void advance_stage()
    {
        spar ^= 1u << stage;
        if (++stage == cur_stages) stage = 0;
    }
    __device__ void advance_acc()
    {
        acc ^= 1;
        if (acc == 0) aphase ^= 1u;
    }

    // live tile range of layer l under the window (tile degrees are monotone)
    __device__ void live_range(int l, const Win &w, int &nt_lo, int &nt_hi) const
    {
        const TcLayer &ly = t.lay[l];
        const bool is_out = (l == m.L);
        const int lo_key = is_out ? w.olo + 1 : w.hdeg_lo + 1;   // live iff dmax >= lo_key
        const int hi_key = is_out ? w.ohi : w.hdeg_hi;           // live iff dmin <= hi_key
        int a = 0, b = ly.nt;
        while (a < b) { const int mid = (a + b) >> 1; if (dmax_of(l, mid) >= lo_key) b = mid; else a = mid + 1; }
        nt_lo = a;
        a = nt_lo; b = ly.nt;
        while (a < b) { const int mid = (a + b) >> 1; if (dmin_of(l, mid) > hi_key) b = mid; else a = mid + 1; }
        nt_hi = a;
    }

    // ---- work units.  The K blocks of a tile are cut into chunks of ly.ch blocks (a property of
    // the layer and the tile alone, never of the window, so that every value is always summed
    // in the same order).  Each chunk is a unit; the host gave every CTA its list of units,
    // balanced by K length, non-owning chunks first.  The chunk with the highest K blocks owns
    // the tile: it adds the other chunks' fp32 partial sums in chunk order and runs the epilogue.
    // Because every CTA works through partial chunks before owners, an owner's wait always ends.
    struct Unit {
        int mt, nt, kb0, kb1;
        int nparts;        // owner: partial sums to add (>= 0); non-owner: -1
        int slot;          // non-owner: its slot; owner: slot of the tile's first partial
    };
    __device__ bool next_unit(int l, int &e, int e_end, int nt_lo, int nt_hi, int MT, Unit &u) const
    {
        const TcLayer &ly = t.lay[l];
        while (e < e_end) {
            const int v = ly.sched[e++];
            u.mt = v >> 24;
            u.nt = (v >> 8) & 0xffff;
            const int chunk = v & 0xff;
            if (u.mt >= MT || u.nt < nt_lo || u.nt >= nt_hi) continue;
            // nc chunks of nearly equal length: the first `rem` of them hold one K block more
            const int kbe = kb_end_of(l, u.nt);
            const int nc = (kbe + ly.ch - 1) / ly.ch;
            const int base = kbe / nc, rem = kbe - base * nc;
            u.kb0 = chunk * base + min(chunk, rem);
            u.kb1 = u.kb0 + base + (chunk < rem ? 1 : 0);
            const bool owner = (chunk == nc - 1);
            u.nparts = owner ? nc - 1 : -1;
            u.slot = u.mt * ly.slots_per_mt + ly.slot_base[u.nt] + (owner ? 0 : chunk);
            return true;
        }
        return false;
    }
    // this CTA's unit list of layer l for a working batch of MT row tiles
    __device__ void unit_list(int l, int MT, int &e, int &e_end) const
    {
        const TcLayer &ly = t.lay[l];
        const int *so = ly.sched_off + (size_t)(ly.n_sched > 1 ? MT - 1 : 0) * (gridDim.x + 1);
        e = so[blockIdx.x];
        e_end = so[blockIdx.x + 1];
    }

    __device__ void producer(int l, int nt_lo, int nt_hi, int MT)
    {
        const TcLayer &ly = t.lay[l];
        const CUtensorMap *ma = t.tmA + l, *mw = t.tmW + l;
        const uint32_t bytes = A_BYTES + ly.bn * BK * 2;
        ring_for_layer(l);
        trace(0);
        int e, e_end;
        unit_list(l, MT, e, e_end);
        Unit u;
        while (!dead && next_unit(l, e, e_end, nt_lo, nt_hi, MT, u)) {
            issued++;
            mma_flops += 2ull * BM * BK * (unsigned long long)ly.bn * (unsigned long long)(u.kb1 - u.kb0);
            if (u.mt == 0) weight_bytes += 2ull * BK * (unsigned long long)ly.bn * (unsigned long long)(u.kb1 - u.kb0);
            for (int kb = u.kb0; kb < u.kb1; ++kb) {
                if (!mbar_wait(&sh.empty[stage], stage_parity() ^ 1u, r.ctl)) { dead = true; break; }
                mbar_expect_tx(&sh.full[stage], bytes);
                tma_load_2d(smem_u32(stage_a(stage)), ma, &sh.full[stage], kb * BK, u.mt * BM);
                tma_load_2d(smem_u32(stage_b(stage)), mw, &sh.full[stage], 0, kb * ly.npad + u.nt * ly.bn);
                advance_stage();
            }
        }
        // The next phase starts with a round trip to HBM for its first weight blocks, while every
        // CTA waits.  Ask L2 for them now: weights depend on nothing, and this thread is idle until
        // the grid barrier.  (The same tile range is assumed for the next layer; a wrong guess only
        // wastes the hint.)
        {
            const int ln = (l == m.L) ? 0 : l + 1;
            const TcLayer &nx = t.lay[ln];
            int e2, e2_end, lo2 = 0, hi2 = nx.nt;
            unit_list(ln, MT, e2, e2_end);
            Unit v;
            if (next_unit(ln, e2, e2_end, lo2, hi2, MT, v))
                for (int kb = v.kb0; kb < v.kb1 && kb < v.kb0 + nx.n_stages; ++kb)
                    tma_prefetch_2d(t.tmW + ln, 0, kb * nx.npad + v.nt * nx.bn);
        }
    }

    __device__ void mma_issuer(int l, int nt_lo, int nt_hi, int MT)
    {
        const TcLayer &ly = t.lay[l];
        const uint32_t idesc = instr_desc_bf16(ly.bn);
        ring_for_layer(l);
        int e, e_end;
        unit_list(l, MT, e, e_end);
        Unit u;
        bool first = true;
        while (!dead && next_unit(l, e, e_end, nt_lo, nt_hi, MT, u)) {
            if (!mbar_wait(&sh.tempty[acc], aphase ^ 1u, r.ctl)) { dead = true; break; }
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(acc * ACC_COLS);
            for (int kb = u.kb0; kb < u.kb1; ++kb) {
                if (!mbar_wait(&sh.full[stage], stage_parity(), r.ctl)) { dead = true; break; }
                tc_fence_after();
                if (first) { trace(1); first = false; }
                const uint64_t adesc = smem_desc_sw128(smem_u32(stage_a(stage)));
                const uint64_t bdesc = smem_desc_sw128(smem_u32(stage_b(stage)));
#pragma unroll
                for (int k = 0; k < BK / 16; ++k)       // 16 bf16 = 32 bytes per instruction along K
                    umma_bf16(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc,
                              (kb > u.kb0 || k > 0) ? 1u : 0u);
                umma_commit(&sh.empty[stage]);          // frees the stage once these MMAs have read it
                advance_stage();
            }
            if (dead) break;
            umma_commit(&sh.tfull[acc]);                // accumulator complete
            advance_acc();
        }
        trace(2);
    }

    // ---- partial sums.  Layout of a slot: [column / 4][128 rows] float4, written and read with
    // thread = row, so stores and loads are coalesced without any transposition.
    __device__ size_t tile_floats(int l) const { return (size_t)BM * t.lay[l].bn; }

    // non-owning chunk: accumulator -> its slot, then raise the slot's flag for this row quadrant
    __device__ void store_partial(int l, int slot, uint32_t tbase)
    {
        const int q = warp & 3, row = q * 32 + lane;
        float4 *base = reinterpret_cast<float4 *>(t.partials + (size_t)slot * tile_floats(l)) + row;
#pragma unroll 1
        for (int c0 = 0; c0 < t.lay[l].bn; c0 += 32) {
            uint32_t ra[32];
            tmem_ld32_issue(tbase + (uint32_t)c0, ra);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 8; ++i)
                base[(size_t)(c0 / 4 + i) * BM] = make_float4(__uint_as_float(ra[4 * i]), __uint_as_float(ra[4 * i + 1]),
                                                              __uint_as_float(ra[4 * i + 2]), __uint_as_float(ra[4 * i + 3]));
        }
        release_acc();
        __threadfence();
        __syncwarp();
        if (lane == 0) {
            unsigned *f = t.pflags + (size_t)slot * 4 + q;
            asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(f), "r"(stamp) : "memory");
        }
    }

    // owner: bounded wait until this warp's row quadrant of every partial of the tile is stored
    __device__ bool wait_partials(int slot, int nparts)
    {
        // lane p polls the flag of partial p: one round trip for all of them instead of one each
        const int q = warp & 3;
        int ok = 1;
        for (int p0 = 0; p0 < nparts && ok; p0 += 32) {
            const bool mine = p0 + lane < nparts;
            const unsigned *f = t.pflags + (size_t)(slot + p0 + (mine ? lane : 0)) * 4 + q;
            uint64_t t0 = 0;
            for (unsigned i = 0;; ++i) {
                const bool set = !mine || ld_acquire_u32(f) == stamp;
                if (__all_sync(0xffffffffu, set)) break;
                if ((i & 15u) == 15u) {
                    if (t0 == 0) t0 = global_ns();
                    const bool give_up = ld_volatile_i32(&r.ctl->abort) != 0 || global_ns() - t0 > MBAR_WAIT_NS;
                    if (__any_sync(0xffffffffu, give_up)) {
                        if (lane == 0) atomicExch(&r.ctl->abort, 1);
                        ok = 0;
                        break;
                    }
                }
            }
        }
        __threadfence();
        return ok != 0;
    }

    // the same for 64 columns held in two register groups, with all sixteen loads of a partial in
    // flight together (one memory latency per partial instead of two)
    __device__ void add_partials64(uint32_t (&ra)[32], uint32_t (&rb)[32], int c0) const
    {
        const int row = (warp & 3) * 32 + lane;
        for (int p = 0; p < cur_parts; ++p) {
            const float4 *base = reinterpret_cast<const float4 *>(cur_pbase + (size_t)p * cur_tile_floats) + row;
            float4 v[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = __ldcg(base + (size_t)(c0 / 4 + i) * BM);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                ra[4 * i] = __float_as_uint(__uint_as_float(ra[4 * i]) + v[i].x);
                ra[4 * i + 1] = __float_as_uint(__uint_as_float(ra[4 * i + 1]) + v[i].y);
                ra[4 * i + 2] = __float_as_uint(__uint_as_float(ra[4 * i + 2]) + v[i].z);
                ra[4 * i + 3] = __float_as_uint(__uint_as_float(ra[4 * i + 3]) + v[i].w);
                rb[4 * i] = __float_as_uint(__uint_as_float(rb[4 * i]) + v[i + 8].x);
                rb[4 * i + 1] = __float_as_uint(__uint_as_float(rb[4 * i + 1]) + v[i + 8].y);
                rb[4 * i + 2] = __float_as_uint(__uint_as_float(rb[4 * i + 2]) + v[i + 8].z);
                rb[4 * i + 3] = __float_as_uint(__uint_as_float(rb[4 * i + 3]) + v[i + 8].w);
            }
        }
    }

    // add the tile's partial sums, in chunk order, to 32 accumulator columns starting at c0
    __device__ void add_partials(uint32_t (&ra)[32], int c0) const
    {
        const int row = (warp & 3) * 32 + lane;
        for (int p = 0; p < cur_parts; ++p) {
            const float4 *base = reinterpret_cast<const float4 *>(cur_pbase + (size_t)p * cur_tile_floats) + row;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float4 v = __ldcg(base + (size_t)(c0 / 4 + i) * BM);
                ra[4 * i] = __float_as_uint(__uint_as_float(ra[4 * i]) + v.x);
                ra[4 * i + 1] = __float_as_uint(__uint_as_float(ra[4 * i + 1]) + v.y);
                ra[4 * i + 2] = __float_as_uint(__uint_as_float(ra[4 * i + 2]) + v.z);
                ra[4 * i + 3] = __float_as_uint(__uint_as_float(ra[4 * i + 3]) + v.w);
            }
        }
    }

    // ---- chunk-wise epilogues: thread = one sample row of the tile, 32 columns at a time
    __device__ void epi_logits(float *zout, int row, int n0, int c0, const float (&v)[32])
    {
        const int N = m.n[m.L + 1];
        if (row >= r.batch) return;
        const float *bias = m.bias[m.L];
        const int col = n0 + c0;
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (col + i < N) zout[(size_t)row * N + col + i] = v[i] + bias[col + i];
    }

    // ---- whole-tile epilogues that go through shared memory so that global accesses are
    // coalesced.  Each epilogue warp owns 32 rows of the tile and an 8 KB staging area holding
    // 32 rows x 256 bytes; 16-byte chunk c of row r sits at chunk c ^ (r & 15) (conflict-free both
    // for the row-per-lane writes and for the row-wise reads).
    // (at the end of the auxiliary buffer: the part before it serves hidden layers as extra ring stages)
    __device__ uint8_t *my_staging() const { return staging + (t.aux_bytes - STAGING_BYTES) + (size_t)(warp - 2) * 8192; }

    __device__ void load_bias_tile(int l, int n0, int bn)
    {
        float *bs = sh.bias_s[warp - 2];
        const int N = m.n[l + 1];
        __syncwarp();
        for (int i = lane; i < bn; i += 32) bs[i] = (n0 + i < N) ? m.bias[l][n0 + i] : 0.0f;
        __syncwarp();
    }

    __device__ void release_acc()
    {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.tempty[acc]);
    }

    // accumulator columns [half*64, half*64+64) of this warp's 32 rows -> staging, raw fp32,
    // row-per-lane (thread = TMEM lane), 16-byte chunks swizzled by row
    __device__ void stage_half(uint32_t tbase, int half)
    {
        uint8_t *stg = my_staging();
        uint32_t ra[32], rb[32];
        tmem_ld32_issue(tbase + (uint32_t)(half * 64), ra);       // two loads in flight per wait
        tmem_ld32_issue(tbase + (uint32_t)(half * 64 + 32), rb);
        tmem_wait_ld();
        if (cur_parts > 0) add_partials64(ra, rb, half * 64);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            *reinterpret_cast<uint4 *>(stg + lane * 256 + ((i ^ (lane & 15)) << 4)) =
                make_uint4(ra[4 * i], ra[4 * i + 1], ra[4 * i + 2], ra[4 * i + 3]);
            *reinterpret_cast<uint4 *>(stg + lane * 256 + (((i + 8) ^ (lane & 15)) << 4)) =
                make_uint4(rb[4 * i], rb[4 * i + 1], rb[4 * i + 2], rb[4 * i + 3]);
        }
    }

    // The row-wise passes below give half a warp to each row: lane -> row pair member (lane >> 4)
    // and 16-byte chunk (lane & 15) = four consecutive columns.  Their loops are kept rolled: these
    // kernels are instruction-cache bound when every path is unrolled.

    // hidden layer: act(acc + bias) -> bf16, 64 columns at a time
    __device__ void epi_hidden_tile(int l, int mt, int n0, uint32_t tbase)
    {
        uint8_t *stg = my_staging();
        const float *bs = sh.bias_s[warp - 2];
        const int N = m.n[l + 1];
        __nv_bfloat16 *out = (__nv_bfloat16 *)m.a[l + 1];
        const int q = warp & 3, ch = lane & 15, rsel = lane >> 4;
        const int act = m.act;
        const int halves = t.lay[l].bn / 64;
#pragma unroll 1
        for (int half = 0; half < halves; ++half) {
            stage_half(tbase, half);
            if (half == halves - 1) { release_acc(); if (warp == 4 && lane == 0) trace(6); } else __syncwarp();
            const int cb = half * 64 + ch * 4;
            const float b0 = bs[cb], b1 = bs[cb + 1], b2 = bs[cb + 2], b3 = bs[cb + 3];
            const int col = n0 + cb;
#pragma unroll 4
            for (int it = 0; it < 16; ++it) {
                const int rl = it * 2 + rsel;
                const float4 v = *reinterpret_cast<const float4 *>(stg + rl * 256 + ((ch ^ (rl & 15)) << 4));
                const int row = mt * BM + q * 32 + rl;
                const uint32_t p0 = pack_bf16x2(tc_act_fn(act, v.x + b0), tc_act_fn(act, v.y + b1));
                const uint32_t p1 = pack_bf16x2(tc_act_fn(act, v.z + b2), tc_act_fn(act, v.w + b3));
                if (row < live && col < N) *reinterpret_cast<uint2 *>(out + (size_t)row * N + col) = make_uint2(p0, p1);
            }
            __syncwarp();
        }
    }

    // Raise the per-sample change flag.  Thousands of tiles report on the same few words, and
    // accesses to one address serialise in L2; a load to look first would put an L2 round trip at
    // the end of every tile's epilogue.  So: a plain store, and each thread remembers the last
    // (sample, phase) it raised, which keeps it to one store per row and phase in the common case
    // of a thread that meets the same row in tile after tile.
    int raised_sample = -1;
    unsigned raised_stamp = 0;
    __device__ void raise_flag(int parity, int sample)
    {
        if (raised_sample == sample && raised_stamp == stamp) return;
        r.smp_changed[parity * r.batch + sample] = 1;
        raised_sample = sample;
        raised_stamp = stamp;
    }

    // ---- binary output layer (128 positions per tile), thread = one sample row of the tile.
    // The row's noise (512 bytes) and current symbols (128 bytes) are brought into shared memory by
    // bulk copies that are issued before the accumulator is waited for, so they travel while the
    // K loop still runs; rows are padded by 16 bytes, which makes the row-per-lane 16-byte accesses
    // conflict-free.  The new symbols replace the old ones in place, the new encodings (bf16)
    // overwrite the part of the noise row that has been consumed, and a row in which something
    // changed goes back to global memory as two bulk stores.
    __device__ uint8_t *nz_row() const { return staging + (size_t)((warp & 3) * 32 + lane) * BIN_NZ_ROW; }
    __device__ uint8_t *xs_row() const { return staging + BIN_NZ_BYTES + (size_t)((warp & 3) * 32 + lane) * BIN_XS_ROW; }

    __device__ void bin_fetch_rows(int smp, int n0, int ncols)
    {
        const int q = warp & 3;
        bulk_wait_read();                     // this thread's earlier bulk stores no longer read the rows
        __syncwarp();
        if (t.bin_bulk) {
            const uint32_t bytes = smp >= 0 ? (uint32_t)ncols * 5u : 0u;
            const uint32_t tot = __reduce_add_sync(0xffffffffu, bytes);
            if (lane == 0) mbar_expect_tx(&sh.nzbar[q], tot);
            __syncwarp();
            if (smp >= 0) {
                const size_t at = (size_t)smp * m.T + n0;
                bulk_load(smem_u32(nz_row()), r.noise + at, (uint32_t)ncols * 4u, &sh.nzbar[q]);
                bulk_load(smem_u32(xs_row()), r.x + at, (uint32_t)ncols, &sh.nzbar[q]);
            }
        } else if (smp >= 0) {
            // widths that are not multiples of 16: plain loads (8 positions at a time)
            const size_t at = (size_t)smp * m.T + n0;
            uint8_t *nz = nz_row(), *xs = xs_row();
            for (int c = 0; c < ncols; c += 8) {
                const float4 v0 = ld_nc_f4_now(r.noise + at + c), v1 = ld_nc_f4_now(r.noise + at + c + 4);
                const uint2 xv = __ldcg(reinterpret_cast<const uint2 *>(r.x + at + c));
                *reinterpret_cast<float4 *>(nz + c * 4) = v0;
                *reinterpret_cast<float4 *>(nz + c * 4 + 16) = v1;
                *reinterpret_cast<uint2 *>(xs + c) = xv;
            }
        }
    }

    // NK: the noise kind as a compile-time constant (a per-element branch on it halves the speed
    // of this loop, which a single warp per scheduler runs)
    template <int NK>
    __device__ bool epi_binary_tile(const Win &w, int smp, int rw, int n0, int ncols, uint32_t tbase, bool flag,
                                    int parity, bool &wany, int &wfirst)
    {
        const float *bs = sh.bias_s[warp - 2];
        uint8_t *nz = nz_row(), *xs = xs_row();
        const float lut0 = sh.lut_s[0], lut1 = sh.lut_s[1];
        // columns [clo, chi) of the tile are sampled; the others keep their symbol
        const int clo = max(w.plo - n0, 0), chi = min(min(w.phi, m.T) - n0, ncols);
        if (t.bin_bulk) {
            if (!mbar_wait(&sh.nzbar[warp & 3], nzphase, r.ctl)) return false;
            nzphase ^= 1u;
        }
        uint32_t diff_any = 0, fdiff = 0;
        int fword = INT_MAX;
        const bool tr = (warp == 4 && lane == 0);
        if (tr) trace(6);
#pragma unroll 1
        for (int c0 = 0; c0 < BM; c0 += 32) {
            uint32_t ra[32];
            __syncwarp();
            tmem_ld32_issue(tbase + (uint32_t)c0, ra);
            tmem_wait_ld();
            if (c0 == BM - 32) release_acc();
            if (cur_parts > 0) add_partials(ra, c0);
            if (smp >= 0 && c0 < ncols) {
                // everything the 32 columns need is read before anything is written: the stores below
                // go to the same rows, and a load may not overtake a store it might alias
                float4 e4[8], b4[8];
                uint4 xo4[2];
#pragma unroll
                for (int i = 0; i < 8; ++i) e4[i] = *reinterpret_cast<const float4 *>(nz + (c0 + i * 4) * 4);
#pragma unroll
                for (int i = 0; i < 2; ++i) xo4[i] = *reinterpret_cast<const uint4 *>(xs + c0 + i * 16);
#pragma unroll
                for (int i = 0; i < 8; ++i) b4[i] = *reinterpret_cast<const float4 *>(bs + c0 + i * 4);
                uint32_t xn[8];
                uint2 en[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int c = c0 + i * 4;
                    const uint32_t xw = (i & 3) == 0 ? xo4[i >> 2].x : (i & 3) == 1 ? xo4[i >> 2].y
                                      : (i & 3) == 2 ? xo4[i >> 2].z : xo4[i >> 2].w;
                    const float e[4] = {e4[i].x, e4[i].y, e4[i].z, e4[i].w};
                    const float bb[4] = {b4[i].x, b4[i].y, b4[i].z, b4[i].w};
                    uint32_t nw = 0;
                    float enc[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint32_t o = (xw >> (8 * k)) & 0xffu;
                        const float z = __uint_as_float(ra[i * 4 + k]) + bb[k];
                        const bool in = (unsigned)(c + k - clo) < (unsigned)(chi - clo);
                        const uint32_t nv = in ? (uint32_t)js_sample_binary(NK, z, e[k]) : o;
                        nw |= nv << (8 * k);
                        enc[k] = nv ? lut1 : lut0;
                    }
                    const uint32_t df = nw ^ xw;
                    // first word with a change and its difference, by selects; the position follows below
                    const bool newfirst = df != 0u && fword == INT_MAX;
                    fword = newfirst ? c : fword;
                    fdiff = newfirst ? df : fdiff;
                    diff_any |= df;
                    xn[i] = nw;
                    en[i] = make_uint2(pack_bf16x2(enc[0], enc[1]), pack_bf16x2(enc[2], enc[3]));
                }
                // new symbols in place; encodings over noise that has been consumed (bytes [2c, 2c+8)
                // of the row lie below the noise of column c+4 and beyond)
                *reinterpret_cast<uint4 *>(xs + c0) = make_uint4(xn[0], xn[1], xn[2], xn[3]);
                *reinterpret_cast<uint4 *>(xs + c0 + 16) = make_uint4(xn[4], xn[5], xn[6], xn[7]);
#pragma unroll
                for (int i = 0; i < 8; i += 2)
                    *reinterpret_cast<uint4 *>(nz + (c0 + i * 4) * 2) = make_uint4(en[i].x, en[i].y, en[i + 1].x, en[i + 1].y);
            }
        }
        __syncwarp();
        if (tr) trace(7);
        const bool changed = diff_any != 0u;
        const int first = changed ? n0 + fword + ((__ffs((int)fdiff) - 1) >> 3) : INT_MAX;
        if (t.bin_bulk) {
            fence_proxy_async_smem();         // the rows were written through the generic proxy
            if (changed) {
                bulk_store(r.x + (size_t)smp * m.T + n0, smem_u32(xs), (uint32_t)ncols);
                bulk_store((__nv_bfloat16 *)m.a[0] + (size_t)rw * m.T + n0, smem_u32(nz), (uint32_t)ncols * 2u);
                bulk_commit();
            }
        } else if (changed) {
            uint8_t *xg = r.x + (size_t)smp * m.T + n0;
            __nv_bfloat16 *ag = (__nv_bfloat16 *)m.a[0] + (size_t)rw * m.T + n0;
            for (int c = 0; c < ncols; c += 8) {
                *reinterpret_cast<uint2 *>(xg + c) = *reinterpret_cast<const uint2 *>(xs + c);
                *reinterpret_cast<uint4 *>(ag + c) = *reinterpret_cast<const uint4 *>(nz + c * 2);
            }
        }
        if (flag) {
            if (changed) raise_flag(parity, smp);
            if (__any_sync(0xffffffffu, changed)) {
                wany = true;
                wfirst = min(wfirst, __reduce_min_sync(0xffffffffu, first));
            }
        }
        return true;
    }

    // ---- 256-way output layer: one position per tile, thread = one sample row.  Running argmax of
    // logit + Gumbel noise over eight chunks of 32 classes, lowest index first among equals.
    // This layer is bound by HBM and by its epilogues, and few threads own a valid row when the batch
    // is small, so plain loads leave little in flight.  Therefore: a row's noise (1 KB) is asked into
    // L2 one tile ahead, and the rows of the first t.cat_rows rows of the tile (whole warps) come
    // into shared memory by one bulk copy each, issued before the accumulator is waited for; rows
    // are padded by 16 bytes so that the row-per-lane reads are conflict-free.  Rows beyond that
    // load their noise directly, one chunk ahead of the reduction.
    __device__ void cat_prefetch(int sample, int d)
    {
        if (sample < 0) return;
        const float *gg = r.noise + ((size_t)sample * m.T + d) * 256;
#pragma unroll
        for (int i = 0; i < 8; ++i) prefetch_l2(gg + i * 32);
    }
    __device__ bool cat_in_smem() const { return (warp & 3) * 32 + 32 <= t.cat_rows; }
    __device__ uint8_t *cat_row() const { return staging + (size_t)((warp & 3) * 32 + lane) * CAT_ROW; }
    __device__ void cat_fetch_rows(int sample, int d)
    {
        if (!cat_in_smem()) return;
        const int q = warp & 3;
        __syncwarp();                         // every lane is done with the previous tile's rows
        const uint32_t tot = __reduce_add_sync(0xffffffffu, sample >= 0 ? 1024u : 0u);
        if (lane == 0) mbar_expect_tx(&sh.nzbar[q], tot);
        __syncwarp();
        if (sample >= 0)
            bulk_load(smem_u32(cat_row()), r.noise + ((size_t)sample * m.T + d) * 256, 1024u, &sh.nzbar[q]);
    }
    __device__ bool epi_cat_tile(int sample, int row, int d, uint32_t tbase, const Win &w, bool flag, int parity,
                                 bool &any_changed, int &first)
    {
        const float *bs = sh.bias_s[warp - 2];
        const bool smem_rows = cat_in_smem();
        const float *gg = smem_rows ? reinterpret_cast<const float *>(cat_row())
                                    : r.noise + ((size_t)max(sample, 0) * m.T + d) * 256;
        if (smem_rows) {
            if (!mbar_wait(&sh.nzbar[warp & 3], nzphase, r.ctl)) return false;
            nzphase ^= 1u;
        }
        float best = -INFINITY;
        int bi = 0;
        // the current symbol, asked for now: its latency passes while the classes are reduced
        const bool commit = sample >= 0 && d >= w.plo && d < w.phi;
        int xold = 0;
        if (commit) xold = (int)__ldcg(r.x + (size_t)sample * m.T + d);
        float4 g4[8], gn[8];
        if (sample >= 0 && !smem_rows) {
#pragma unroll
            for (int i = 0; i < 8; ++i) g4[i] = ld_nc_f4_now(gg + i * 4);
        }
#pragma unroll 1
        for (int c0 = 0; c0 < 256; c0 += 32) {
            uint32_t ra[32];
            __syncwarp();
            tmem_ld32_issue(tbase + (uint32_t)c0, ra);
            if (sample >= 0) {
                if (smem_rows) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) g4[i] = *reinterpret_cast<const float4 *>(gg + c0 + i * 4);
                } else if (c0 + 32 < 256) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) gn[i] = ld_nc_f4_now(gg + c0 + 32 + i * 4);
                }
            }
            tmem_wait_ld();
            if (c0 == 256 - 32) release_acc();
            if (cur_parts > 0) add_partials(ra, c0);
            if (sample >= 0) {
                float sc[32];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float4 b4 = *reinterpret_cast<const float4 *>(bs + c0 + i * 4);
                    sc[4 * i] = (__uint_as_float(ra[4 * i]) + b4.x) + g4[i].x;
                    sc[4 * i + 1] = (__uint_as_float(ra[4 * i + 1]) + b4.y) + g4[i].y;
                    sc[4 * i + 2] = (__uint_as_float(ra[4 * i + 2]) + b4.z) + g4[i].z;
                    sc[4 * i + 3] = (__uint_as_float(ra[4 * i + 3]) + b4.w) + g4[i].w;
                }
                argmax_chunk32(sc, c0, best, bi);
                if (!smem_rows) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) g4[i] = gn[i];
                }
            }
        }
        bool ch = false;
        if (commit && xold != bi) {
            r.x[(size_t)sample * m.T + d] = (uint8_t)bi;
            ((__nv_bfloat16 *)m.a[0])[(size_t)row * m.T + d] = __float2bfloat16_rn(sh.lut_s[bi]);
            ch = true;
        }
        if (flag && ch) {
            raise_flag(parity, sample);
            any_changed = true;
            first = min(first, d);
        }
        return true;
    }

    // ---- 256-way output layer with ONE uniform number per position (inverse CDF of the softmax):
    // the first class c with  u * S < sum_{i<=c} e_i,  e_i = exp(z_i - max z), S their total.  The
    // thread's 256 logits stay in tensor memory and are read three times in chunks of 32: the
    // maximum, the running sums (remembered at the chunk ends, which tells the chunk that holds the
    // answer), and once more for the class inside that chunk.  The running sum is carried in class
    // order with the same instructions in the second and third reading, so both see the same values.
    __device__ bool epi_icdf_tile(int sample, int row, int d, uint32_t tbase, const Win &w, bool flag, int parity,
                                  bool &any_changed, int &first)
    {
        const float *bs = sh.bias_s[warp - 2];
        const bool commit = sample >= 0 && d >= w.plo && d < w.phi;
        int xold = 0;
        float u = 0.5f;
        if (commit) {
            xold = (int)__ldcg(r.x + (size_t)sample * m.T + d);
            u = __ldg(r.noise + (size_t)sample * m.T + d);
        }
        float mx = -INFINITY;
#pragma unroll 1
        for (int c0 = 0; c0 < 256; c0 += 32) {
            uint32_t ra[32];
            __syncwarp();
            tmem_ld32_issue(tbase + (uint32_t)c0, ra);
            tmem_wait_ld();
            if (cur_parts > 0) add_partials(ra, c0);
#pragma unroll
            for (int i = 0; i < 32; ++i) mx = fmaxf(mx, __uint_as_float(ra[i]) + bs[c0 + i]);
        }
        float run = 0.0f, cum[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            uint32_t ra[32];
            __syncwarp();
            tmem_ld32_issue(tbase + (uint32_t)(k * 32), ra);
            tmem_wait_ld();
            if (cur_parts > 0) add_partials(ra, k * 32);
#pragma unroll
            for (int i = 0; i < 32; ++i) run += __expf((__uint_as_float(ra[i]) + bs[k * 32 + i]) - mx);
            cum[k] = run;
        }
        const float target = u * run;
        int ck = 8;                       // the first chunk whose closing sum exceeds the target
        float base = 0.0f;
#pragma unroll
        for (int k = 7; k >= 0; --k) {
            if (target < cum[k]) { ck = k; base = k > 0 ? cum[k - 1] : 0.0f; }
        }
        int bi = (run == run) ? 255 : 0;  // u at the very top of the range; no finite score: class 0
#pragma unroll 1
        for (int k = 0; k < 8; ++k) {
            uint32_t ra[32];
            __syncwarp();
            tmem_ld32_issue(tbase + (uint32_t)(k * 32), ra);      // every lane reads (the load is warp-wide) ...
            tmem_wait_ld();
            if (k == 7) release_acc();
            if (k != ck) continue;                                // ... the lanes whose answer lies elsewhere skip the rest
            if (cur_parts > 0) add_partials(ra, k * 32);
            float s2 = base;
            int hit = -1;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                s2 += __expf((__uint_as_float(ra[i]) + bs[k * 32 + i]) - mx);
                hit = (hit < 0 && target < s2) ? i : hit;
            }
            bi = k * 32 + (hit < 0 ? 31 : hit);
        }
        bool ch = false;
        if (commit && xold != bi) {
            r.x[(size_t)sample * m.T + d] = (uint8_t)bi;
            ((__nv_bfloat16 *)m.a[0])[(size_t)row * m.T + d] = __float2bfloat16_rn(sh.lut_s[bi]);
            ch = true;
        }
        if (flag && ch) {
            raise_flag(parity, sample);
            any_changed = true;
            first = min(first, d);
        }
        return true;
    }

    __device__ void epilogue(int l, int kind, const Win &w, bool flag, int parity, float *zout, int nt_lo,
                             int nt_hi, int MT)
    {
        const TcLayer &ly = t.lay[l];
        const int q = warp & 3;
        // noise that is still on its way from the host (jacobi_sample_host): the first sampling
        // epilogue waits for it, bounded
        if (r.noise_ready != nullptr && !noise_here && (kind == EPI_BINARY || kind == EPI_CAT)) {
            int ok = 1;
            if (lane == 0) {
                uint64_t t0 = 0;
                for (unsigned i = 0;; ++i) {
                    unsigned v;
                    asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(r.noise_ready) : "memory");
                    if (v == r.noise_stamp) break;
                    if ((i & 15u) == 15u) {
                        if (t0 == 0) t0 = global_ns();
                        if (ld_volatile_i32(&r.ctl->abort) != 0 || global_ns() - t0 > MBAR_WAIT_NS) {
                            atomicExch(&r.ctl->abort, 1);
                            ok = 0;
                            break;
                        }
                    }
                    __nanosleep(200);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) dead = true;
            noise_here = true;
        }
        bool any_changed = false;
        int first = INT_MAX;
        bool cat_ahead = false;        // the current tile's noise was asked into L2 during the previous tile
        int e, e_end;
        unit_list(l, MT, e, e_end);
        Unit u;
        while (!dead && next_unit(l, e, e_end, nt_lo, nt_hi, MT, u)) {
            const int nt = u.nt, mt = u.mt;
            const bool owner = u.nparts >= 0;
            if (owner && kind != EPI_LOGITS) load_bias_tile(l, nt * ly.bn, ly.bn);
            int csmp = -1;
            if (owner && kind == EPI_CAT && r.nk != JS_NOISE_GUMBEL) {
                const int rw = mt * BM + q * 32 + lane;
                csmp = rw < live ? perm_cur()[rw] : -1;
            }
            if (owner && kind == EPI_CAT && r.nk == JS_NOISE_GUMBEL) {
                const int rw = mt * BM + q * 32 + lane;
                csmp = rw < live ? perm_cur()[rw] : -1;
                if (!cat_ahead) cat_prefetch(csmp, nt);          // first tile of the phase
                cat_fetch_rows(csmp, nt);
                // the next tile's noise towards L2 while this tile is reduced
                Unit nx;
                int e2 = e;
                cat_ahead = next_unit(l, e2, e_end, nt_lo, nt_hi, MT, nx) && nx.nparts >= 0;
                if (cat_ahead) {
                    const int rn = nx.mt * BM + q * 32 + lane;
                    cat_prefetch(rn < live ? perm_cur()[rn] : -1, nx.nt);
                }
            }
            int bsmp = -1, bcols = 0;
            if (owner && kind == EPI_BINARY) {
                const int rw = mt * BM + q * 32 + lane;
                bsmp = rw < live ? perm_cur()[rw] : -1;
                bcols = min(BM, m.T - nt * ly.bn);
                bin_fetch_rows(bsmp, nt * ly.bn, bcols);     // in flight while the tile is still being computed
            }
            if (owner) {
                cur_parts = u.nparts;
                cur_pbase = t.partials + (size_t)u.slot * tile_floats(l);
                cur_tile_floats = tile_floats(l);
                // partial sums do not depend on this CTA's accumulator: wait for them first
                if (cur_parts > 0 && !wait_partials(u.slot, cur_parts)) { dead = true; break; }
            }
            if (!mbar_wait(&sh.tfull[acc], aphase, r.ctl)) { dead = true; break; }
            tc_fence_after();
            if (warp == 4 && lane == 0) trace(3);
            const int row = mt * BM + q * 32 + lane;
            const int n0 = nt * ly.bn;
            const uint32_t tbase = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * ACC_COLS);
            if (!owner) {
                store_partial(l, u.slot, tbase);
                advance_acc();
                continue;
            }
            if (kind == EPI_HIDDEN) {
                epi_hidden_tile(l, mt, n0, tbase);
            } else if (kind == EPI_BINARY) {
                bool wany = false;
                int wfirst = INT_MAX;
                const bool fine = r.nk == JS_NOISE_LOGISTIC
                    ? epi_binary_tile<JS_NOISE_LOGISTIC>(w, bsmp, row, n0, bcols, tbase, flag, parity, wany, wfirst)
                    : epi_binary_tile<JS_NOISE_UNIFORM_ICDF>(w, bsmp, row, n0, bcols, tbase, flag, parity, wany, wfirst);
                if (!fine) { dead = true; break; }
                if (wany) { any_changed = true; first = min(first, wfirst); }
            } else if (kind == EPI_CAT) {
                const bool fine = r.nk == JS_NOISE_GUMBEL ? epi_cat_tile(csmp, row, nt, tbase, w, flag, parity, any_changed, first)
                                                          : epi_icdf_tile(csmp, row, nt, tbase, w, flag, parity, any_changed, first);
                if (!fine) { dead = true; break; }
            } else {
                for (int c0 = 0; c0 < ly.bn; c0 += 32) {
                    float v[32];
                    {
                        uint32_t ra[32];
                        tmem_ld32_issue(tbase + (uint32_t)c0, ra);
                        tmem_wait_ld();
                        if (cur_parts > 0) add_partials(ra, c0);
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(ra[i]);
                    }
                    epi_logits(zout, row, n0, c0, v);
                }
                release_acc();
            }
            advance_acc();
        }
        bulk_wait_all();          // bulk stores of this phase are complete before the grid barrier
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

    // one layer over the window; returns false when there was nothing to do (no barrier needed)
    __device__ bool gemm_phase(int l, int kind, const Win &w, bool flag, int parity, float *zout)
    {
        int nt_lo, nt_hi;
        live_range(l, w, nt_lo, nt_hi);
        const int MT = (live + BM - 1) / BM;
        const int nlive = max(0, nt_hi - nt_lo);
        if (threadIdx.x == 0 && blockIdx.x == 0) skipped += (unsigned long long)(t.lay[l].nt - nlive) * MT;
        stamp += 1;
        if (nlive == 0) return false;
        phase_no++;
        if (warp == 0) {
            if (lane == 0) producer(l, nt_lo, nt_hi, MT);
        } else if (warp == 1) {
            if (lane == 0) mma_issuer(l, nt_lo, nt_hi, MT);
        } else {
            epilogue(l, kind, w, flag, parity, zout, nt_lo, nt_hi, MT);
        }
        return true;
    }

    // one forward pass over the window: a single loop and a single call site, so that the whole
    // pipeline is instantiated once in the kernel
    __device__ bool step(const Win &w, bool flag, int parity, float *zout)
    {
        const int out_kind = zout ? EPI_LOGITS : (m.C == 1 ? EPI_BINARY : EPI_CAT);
        for (int l = 0; l <= m.L; ++l) {
            const bool last = (l == m.L);
            const bool did = gemm_phase(l, last ? out_kind : EPI_HIDDEN, w, last && flag, parity, zout);
            if (did || last)
                if (!barrier()) return false;
        }
        return true;
    }
};

__global__ void __launch_bounds__(NTH, 1)
made_tc_kernel(const __grid_constant__ MadeDev m, const __grid_constant__ TcDev t, const __grid_constant__ RunArgs r)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ TcShared sh;
    uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);

    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0 && r.trace != nullptr && js_trace_who(r) >= 0)
        r.trace[((size_t)js_trace_who(r) * JS_TRACE_PHASES) * JS_TRACE_SLOTS + 2] = global_ns();   // kernel entry
    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_STAGES; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&sh.tfull[a], 1); mbar_init(&sh.tempty[a], 4); }
        for (int a = 0; a < 4; ++a) mbar_init(&sh.nzbar[a], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    for (int i = threadIdx.x; i < (m.C == 1 ? 2 : m.C) && i < 256; i += blockDim.x) sh.lut_s[i] = m.lut[i];
    if (warp == 1) tmem_alloc(&sh.tmem_base, 512);
    // tile metadata of every layer into shared memory (the range searches and the K-loop bounds
    // would otherwise be chains of dependent global loads in every phase)
    int *meta = reinterpret_cast<int *>(ring + t.ring_bytes + t.aux_bytes);
    {
        int off = 0;
        for (int l = 0; l <= m.L; ++l) {
            const int nt = t.lay[l].nt;
            if (threadIdx.x == 0) sh.off[l] = off;
            const bool one_pos = (l == m.L && m.C == 256);
            for (int i = threadIdx.x; i < nt; i += blockDim.x) {
                meta[off + i] = t.lay[l].kb_end[i];
                if (!one_pos) {
                    meta[off + nt + i] = t.lay[l].dmin[i];
                    meta[off + 2 * nt + i] = t.lay[l].dmax[i];
                }
            }
            off += one_pos ? nt : 3 * nt;
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    TcEngine e(m, t, r, sh, ring, meta);
    e.tmem_base = sh.tmem_base;
    if (threadIdx.x == 0) e.trace(0);
    DriverResult res = made_driver(e, m.T, r);
    if (e.dead) res.alive = false;
    if (threadIdx.x == 0) { e.phase_no = 0; e.trace(1); }

    // leave: let copies still in flight land (only possible after an aborted wait), free TMEM
    tc_fence_before();
    __syncthreads();
    if (!res.alive || ld_volatile_i32(&r.ctl->abort) != 0) {
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
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

// Weight layout of this kernel: K-block major, [K block][padded unit][64 inputs], so that the
// bn x 64 box of one TMA load is one contiguous piece of memory (bn x 128 bytes) instead of bn
// pieces of 128 bytes a whole weight row apart: a stream of such boxes reads DRAM pages in full.
__global__ void tile_major_weights(const __nv_bfloat16 *__restrict__ W, __nv_bfloat16 *__restrict__ Wp, int N, int K,
                                   int npad, int nkb)
{
    const size_t total = (size_t)nkb * npad * (BK / 8);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int j8 = (int)(i % (BK / 8));
        const size_t rowp = i / (BK / 8);
        const int n = (int)(rowp % npad), kb = (int)(rowp / npad);
        const int k = kb * BK + j8 * 8;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (n < N && k < K) v = *reinterpret_cast<const uint4 *>(W + (size_t)n * K + k);     // K is a multiple of 8
        *reinterpret_cast<uint4 *>(Wp + rowp * BK + j8 * 8) = v;
    }
}

// --------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn()
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

// 2-D bf16 row-major tensor [rows][cols], box = 64 columns x box_rows rows, 128-byte swizzle
static bool encode_map(CUtensorMap *out, const void *base, int rows, int cols, int box_rows)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Builds the tensor-core view of a model.  Returns 1 if the model qualifies, 0 if it
// does not (the CUDA-core path then serves it), negative on CUDA errors.
int js_tc_prepare(js_model *mo)
{
    const MadeDev &v = mo->made;
    TcDev &t = mo->tc;
    mo->tc_ok = 0;
    if (v.prec != JS_BF16) return 0;
    if (!(v.C == 1 || v.C == 256)) return 0;
    for (int l = 0; l <= v.L; ++l)
        if (v.n[l] % 8 != 0) return 0;
    if (!get_encode_fn()) return 0;
    const int L = v.L;
    bool wide = (v.C == 256);
    t.stage_bytes = A_BYTES + (wide ? 256 : 128) * BK * 2;
    // Output-tile width per layer: 256 for 256-way outputs (one position per tile), else 128; hidden
    // layers with so few 128-wide tiles that three quarters of the SMs would idle use 64 (shorter K
    // blocks, half the epilogue per CTA, twice the CTAs).
    int sms_now = 0;
    {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms_now, cudaDevAttrMultiProcessorCount, dev);
    }
    std::vector<int> bns(L + 1);
    for (int l = 0; l <= L; ++l) {
        bns[l] = (l == L && wide) ? 256 : 128;
        if (l < L && (long long)((v.n[l + 1] + 127) / 128) * (mo->rows / BM) * 4 <= sms_now) bns[l] = 64;
    }
    int meta_ints = 0;
    for (int l = 0; l <= L; ++l)
        meta_ints += (l == L && wide) ? (v.n[l + 1] + 255) / 256 : 3 * ((v.n[l + 1] + bns[l] - 1) / bns[l]);
    const int meta_bytes = (meta_ints * 4 + 127) & ~127;
    t.aux_bytes = std::max(STAGING_BYTES, BIN_NZ_BYTES + BIN_XS_BYTES);
    t.cat_rows = 0;
    if (wide) {
        // three operand stages; the rest holds as many whole warps of noise rows as fit
        const int left = SMEM_DYN_MAX - 1024 - 3 * t.stage_bytes - meta_bytes;
        t.cat_rows = std::min(BM, std::max(0, left / (32 * CAT_ROW)) * 32);
        t.aux_bytes = std::max(STAGING_BYTES, t.cat_rows * CAT_ROW);
    }
    t.bin_bulk = (!wide && v.T % 16 == 0) ? 1 : 0;
    t.n_stages = (SMEM_DYN_MAX - 1024 - t.aux_bytes - meta_bytes) / t.stage_bytes;
    if (t.n_stages > (wide ? 3 : 4)) t.n_stages = wide ? 3 : 4;
    if (t.n_stages < 2) return 0;
    t.ring_bytes = t.n_stages * t.stage_bytes;
    std::vector<CUtensorMap> mapsA(L + 1), mapsW(L + 1);
    std::vector<std::vector<int>> kb_all(L + 1);
    for (int l = 0; l <= L; ++l) {
        const int bn = bns[l];
        const int N = v.n[l + 1], K = v.n[l], nt = (N + bn - 1) / bn;
        std::vector<int> kb(nt), dmin(nt), dmax(nt);
        const std::vector<int> &dout = mo->host_deg[l + 1], &din = mo->host_deg[l];
        for (int i = 0; i < nt; ++i) {
            int lo = INT32_MAX, hi = 0;
            for (int u = i * bn; u < std::min(N, (i + 1) * bn); ++u) { lo = std::min(lo, dout[u]); hi = std::max(hi, dout[u]); }
            int ke = K;
            while (ke > 0 && !(l == L ? din[ke - 1] < hi : din[ke - 1] <= hi)) --ke;
            kb[i] = std::max(1, (ke + BK - 1) / BK);
            dmin[i] = lo; dmax[i] = hi;
            if (i > 0 && (dmin[i] < dmin[i - 1] || dmax[i] < dmax[i - 1])) return 0;   // needs sorted degrees
        }
        void *p = nullptr;
        for (std::vector<int> *src : {&kb, &dmin, &dmax}) {
            if (cudaMalloc(&p, nt * sizeof(int)) != cudaSuccess) return JS_ERR_CUDA;
            mo->allocs.push_back(p);
            if (cudaMemcpy(p, src->data(), nt * sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess) return JS_ERR_CUDA;
            if (src == &kb) t.lay[l].kb_end = (const int *)p;
            else if (src == &dmin) t.lay[l].dmin = (const int *)p;
            else t.lay[l].dmax = (const int *)p;
        }
        t.lay[l].bn = bn;
        t.lay[l].nt = nt;
        t.lay[l].stage_bytes = A_BYTES + bn * BK * 2;
        // hidden layers need only the staging area at the end of the auxiliary buffer: the ring may
        // run into the rest of it (an SM keeps about three stages in flight, and 96 KB in flight are
        // not quite enough to saturate its 108 GB/s)
        const int ring_cap = t.ring_bytes + (l < L ? t.aux_bytes - STAGING_BYTES : 0);
        t.lay[l].n_stages = std::min(MAX_STAGES, ring_cap / t.lay[l].stage_bytes);
        kb_all[l] = kb;
        if (!encode_map(&mapsA[l], v.a[l], mo->rows, K, BM)) return 0;
        {
            const int nkb = (K + BK - 1) / BK, npad = nt * bn;
            void *wp = nullptr;
            if (cudaMalloc(&wp, (size_t)nkb * npad * BK * sizeof(__nv_bfloat16)) != cudaSuccess) return JS_ERR_CUDA;
            mo->allocs.push_back(wp);
            tile_major_weights<<<1184, 256>>>((const __nv_bfloat16 *)v.W[l], (__nv_bfloat16 *)wp, N, K, npad, nkb);
            if (cudaGetLastError() != cudaSuccess) return JS_ERR_CUDA;
            t.lay[l].npad = npad;
            if (!encode_map(&mapsW[l], wp, nkb * npad, BK, bn)) return 0;
        }
    }
    if (cudaDeviceSynchronize() != cudaSuccess) return JS_ERR_CUDA;     // the tile-major copies are complete
    // ---- split-K work units and their static assignment to CTAs (longest processing time first)
    int sms = 0;
    {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (sms < 1) return 0;
    }
    const int MTmax = mo->rows / BM;
    std::vector<int> chs(L + 1);
    int G = 1;
    for (int l = 0; l <= L; ++l) {
        const std::vector<int> &kb = kb_all[l];
        long long total_kb = 0;
        for (int x : kb) total_kb += (long long)x * MTmax;
        int ch = 1 << 20;                                              // enough tiles: no split
        int kb_longest = 1;
        for (int x : kb) kb_longest = std::max(kb_longest, x);
        // splitting pays only for long K loops: handing a partial sum over costs about as much
        // as ten K blocks of loading
        // The chain  longest K loop -> hand-over -> owner's epilogue  is what a phase has to wait for,
        // so the longest tiles are cut into three chunks (measured on K loops of 64 blocks: chunks
        // of 18 to 24 blocks are within 3 % of each other, 32 and 12 are each 12 % slower).
        if ((long long)kb.size() * MTmax < 2LL * sms && kb_longest >= 40)
            ch = std::max(4, (kb_longest + 2) / 3);
        chs[l] = ch;
        long long units = 0;
        for (int x : kb) units += (long long)((x + ch - 1) / ch) * MTmax;
        G = (int)std::max<long long>(G, std::min<long long>(sms, units));
    }
    t.grid = G;
    size_t part_floats = 0;
    int max_slots = 0;
    // One schedule per size of the working batch (compaction shrinks it), as long as that is a
    // handful; the chunks themselves never depend on it, only who computes them.
    const int n_sched = MTmax <= 16 ? MTmax : 1;
    for (int l = 0; l <= L; ++l) {
        const std::vector<int> &kb = kb_all[l];
        const int ch = chs[l], nt = (int)kb.size(), bn = t.lay[l].bn;
        std::vector<int> slot_base(nt);
        int slots = 0;
        for (int i = 0; i < nt; ++i) { slot_base[i] = slots; slots += (kb[i] + ch - 1) / ch - 1; }
        auto chunk_len = [&](int i, int c) {
            const int nc = (kb[i] + ch - 1) / ch, base = kb[i] / nc, rem = kb[i] - base * nc;
            return base + (c < rem ? 1 : 0);
        };
        auto nparts_of_tile = [&](int i) { return (kb[i] + ch - 1) / ch - 1; };
        std::vector<int> off, flat;
        for (int si = 0; si < n_sched; ++si) {
            const int MT = n_sched > 1 ? si + 1 : MTmax;
            // units: non-owning chunks first, then owners
            struct U { int mt, nt, chunk, size; };
            std::vector<U> part, own;
            for (int mt = 0; mt < MT; ++mt)
                for (int i = 0; i < nt; ++i) {
                    const int nc = nparts_of_tile(i) + 1;
                    for (int c = 0; c + 1 < nc; ++c) part.push_back({mt, i, c, chunk_len(i, c)});
                    own.push_back({mt, i, nc - 1, chunk_len(i, nc - 1)});
                }
            // List scheduling on a small model of a CTA, in units of one K block's load time
            // (about 0.35 us): the K loops of a CTA's units run back to back; a unit's epilogue
            // starts when its K loop is done, the previous epilogue is done and (for an owner) the
            // tile's partial sums have been stored.  Units are taken longest first and put where
            // the CTA finishes earliest.  Inside a CTA: partial chunks first (owners elsewhere
            // wait for them), then owners that wait for nobody, then owners that add partial sums.
            const int FILL = 6, EPI_PART = 5, EPI_OWN = (l == L ? (bn == 256 ? 5 : 9) : 4), EPI_ADD = 8;
            struct Item { int code, size, epi, ready; };
            std::vector<std::vector<Item>> lp(G), lo0(G), lo1(G);
            auto finish = [&](int c, const Item *extra, int where) {
                long long M = FILL, E = 0;
                auto run = [&](const Item &it) {
                    M += it.size;
                    const long long start = std::max<long long>(std::max(M, E), it.ready);
                    E = start + it.epi;
                };
                for (const Item &it : lp[c]) run(it);
                if (extra && where == 0) run(*extra);
                for (const Item &it : lo0[c]) run(it);
                if (extra && where == 1) run(*extra);
                for (const Item &it : lo1[c]) run(it);
                if (extra && where == 2) run(*extra);
                return E;
            };
            auto place = [&](const Item &it, int where) {
                int best = 0;
                long long bt = -1;
                for (int c = 0; c < G; ++c) {
                    const long long f = finish(c, &it, where);
                    if (bt < 0 || f < bt) { bt = f; best = c; }
                }
                (where == 0 ? lp : where == 1 ? lo0 : lo1)[best].push_back(it);
                return best;
            };
            std::stable_sort(part.begin(), part.end(), [](const U &a, const U &b) { return a.size > b.size; });
            std::vector<long long> ready((size_t)MT * nt, 0);          // when a tile's partial sums are all stored
            for (const U &u : part) {
                const Item it = {(u.mt << 24) | (u.nt << 8) | u.chunk, u.size, EPI_PART, 0};
                const int c = place(it, 0);
                long long M = FILL, E = 0;                             // completion of this chunk in its CTA
                for (const Item &x : lp[c]) { M += x.size; E = std::max(M, E) + x.epi; }
                ready[(size_t)u.mt * nt + u.nt] = std::max(ready[(size_t)u.mt * nt + u.nt], E);
            }
            std::stable_sort(own.begin(), own.end(), [&](const U &a, const U &b) {
                return a.size + EPI_ADD * nparts_of_tile(a.nt) > b.size + EPI_ADD * nparts_of_tile(b.nt);
            });
            for (const U &u : own) {
                const int np = nparts_of_tile(u.nt);
                const Item it = {(u.mt << 24) | (u.nt << 8) | u.chunk, u.size, EPI_OWN + EPI_ADD * np,
                                 np > 0 ? (int)ready[(size_t)u.mt * nt + u.nt] + 3 : 0};
                place(it, np > 0 ? 2 : 1);
            }
            // Where a CTA has several whole tiles whose epilogue lasts longer than a short K loop (the
            // 256-way argmax), a run of short tiles at the end of its list leaves their epilogues in
            // the open.  Order such lists short, long, short, long ...: every short tile's epilogue
            // hides behind the long K loop that follows, and only the last tile's shows.
            if (ch == (1 << 20) && bn == 256)
                for (int c = 0; c < G; ++c) {
                    std::vector<Item> &v0 = lo0[c];
                    std::stable_sort(v0.begin(), v0.end(), [](const Item &a, const Item &b) { return a.size < b.size; });
                    std::vector<Item> mix;
                    for (size_t i = 0, j = v0.size(); i < j;) {
                        mix.push_back(v0[i++]);
                        if (i < j) mix.push_back(v0[--j]);
                    }
                    // short, longest, next short, next longest ...; the middle of the sorted list comes last
                    v0 = mix;
                }
            for (int c = 0; c < G; ++c) {
                off.push_back((int)flat.size());
                for (const Item &it : lp[c]) flat.push_back(it.code);
                for (const Item &it : lo0[c]) flat.push_back(it.code);
                for (const Item &it : lo1[c]) flat.push_back(it.code);
            }
            off.push_back((int)flat.size());
        }
        auto up = [&](const std::vector<int> &h, const int **dst) -> bool {
            void *q = nullptr;
            if (cudaMalloc(&q, std::max<size_t>(h.size(), 1) * sizeof(int)) != cudaSuccess) return false;
            mo->allocs.push_back(q);
            if (!h.empty() && cudaMemcpy(q, h.data(), h.size() * sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess) return false;
            *dst = (const int *)q;
            return true;
        };
        if (!up(slot_base, &t.lay[l].slot_base) || !up(off, &t.lay[l].sched_off) || !up(flat, &t.lay[l].sched)) return JS_ERR_CUDA;
        t.lay[l].ch = ch;
        t.lay[l].n_sched = n_sched;
        t.lay[l].slots_per_mt = slots;
        max_slots = std::max(max_slots, slots * MTmax);
        part_floats = std::max(part_floats, (size_t)slots * MTmax * BM * bn);
    }
    {
        void *q = nullptr;
        if (cudaMalloc(&q, std::max<size_t>(part_floats, 4) * sizeof(float)) != cudaSuccess) return JS_ERR_CUDA;
        mo->allocs.push_back(q);
        t.partials = (float *)q;
        t.n_pflags = std::max(max_slots, 1) * 4;
        if (cudaMalloc(&q, (size_t)t.n_pflags * sizeof(unsigned)) != cudaSuccess) return JS_ERR_CUDA;
        mo->allocs.push_back(q);
        if (cudaMemset(q, 0, (size_t)t.n_pflags * sizeof(unsigned)) != cudaSuccess) return JS_ERR_CUDA;
        t.pflags = (unsigned *)q;
    }
    void *pa = nullptr, *pw = nullptr;
    if (cudaMalloc(&pa, (L + 1) * sizeof(CUtensorMap)) != cudaSuccess) return JS_ERR_CUDA;
    mo->allocs.push_back(pa);
    if (cudaMalloc(&pw, (L + 1) * sizeof(CUtensorMap)) != cudaSuccess) return JS_ERR_CUDA;
    mo->allocs.push_back(pw);
    if (cudaMemcpy(pa, mapsA.data(), (L + 1) * sizeof(CUtensorMap), cudaMemcpyHostToDevice) != cudaSuccess) return JS_ERR_CUDA;
    if (cudaMemcpy(pw, mapsW.data(), (L + 1) * sizeof(CUtensorMap), cudaMemcpyHostToDevice) != cudaSuccess) return JS_ERR_CUDA;
    t.tmA = (const CUtensorMap *)pa;
    t.tmW = (const CUtensorMap *)pw;

    t.smem_bytes = 1024 + t.ring_bytes + t.aux_bytes + meta_bytes;
    // the attribute belongs to the function, not to a model: always allow the largest request
    const int smem = SMEM_DYN_MAX;
    if (cudaFuncSetAttribute(made_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
        cudaGetLastError();      // not sticky: the CUDA-core kernels will serve this model
        return 0;
    }
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, made_tc_kernel, NTH, smem) != cudaSuccess || per_sm < 1)
        return 0;
    mo->tc_max_grid = sms;      // one CTA per SM: each owns all 512 TMEM columns
    mo->tc_ok = 1;
    return 1;
}

int js_launch_made_tc(const js_model *mo, const RunArgs &r, cudaStream_t stream)
{
    const MadeDev &v = mo->made;
    const TcDev &t = mo->tc;
    (void)r.batch;
    const int grid = std::min(t.grid, mo->tc_max_grid);
    if (grid != t.grid) return (int)cudaErrorInvalidConfiguration;     // the schedules need exactly t.grid CTAs
    void *args[3] = {(void *)&v, (void *)&t, (void *)&r};
    cudaError_t e = cudaLaunchCooperativeKernel((const void *)made_tc_kernel, dim3(grid), dim3(NTH), args,
                                                t.smem_bytes, stream);
    return e == cudaSuccess ? 0 : (int)e;
}
