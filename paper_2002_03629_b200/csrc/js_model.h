// Host-side model object behind the opaque js_model handle.
#pragma once
#include <cuda.h>

#include <vector>

#include "js_common.cuh"

// Tensor-core view of a masked MLP: per layer the output-tile width, the tile
// metadata (last live K block, smallest / largest degree) and the TMA descriptors.
struct TcLayer {
    const int *kb_end;
    const int *dmin;
    const int *dmax;
    int bn;
    int nt;
    int stage_bytes, n_stages;   // this layer's cut of the operand ring
    int npad;                    // units padded to whole tiles: rows per K block of the tile-major weight copy
    // split-K: the K blocks of tile nt are cut into chunks of `ch` blocks, each chunk a work unit
    // of its own; the last chunk owns the tile and adds the others' fp32 partial sums in order
    int ch;
    int slots_per_mt;            // partial-sum slots per row tile = sum over nt of (chunks - 1)
    const int *slot_base;        // [nt] first slot of tile nt inside a row tile
    int n_sched;                 // schedules: one per number of live row tiles (1..n_sched), or a single one
    const int *sched_off;        // [n_sched][grid + 1] work units of CTA c: sched[sched_off[c] .. sched_off[c+1])
    const int *sched;            // units packed as (row tile << 24) | (n tile << 8) | chunk
};
struct TcDev {
    const CUtensorMap *tmA;      // [L+1] activations a[l], box 64 x 128
    const CUtensorMap *tmW;      // [L+1] masked weights W[l], box 64 x bn
    TcLayer lay[JS_MAXL + 1];
    int stage_bytes, n_stages, smem_bytes;
    int ring_bytes, aux_bytes;   // shared memory: operand ring, then the epilogues' auxiliary buffer
    int cat_rows;                // 256-way outputs: the first cat_rows rows of a tile get their noise through shared memory
    int bin_bulk;                // binary output rows are 16-byte granular: moved by bulk copies
    int grid;                    // CTAs the schedules were built for (the launch uses exactly this)
    float *partials;             // [slot][columns/4][128 rows] float4: fp32 partial sums of non-owning chunks
    unsigned *pflags;            // [slot][4 row quadrants]: phase stamp once the partial is stored
    int n_pflags;
};

// What the cached sweeps (made_sweep.cu) need beside the tensor-core view.
struct SweepDev {
    const CUtensorMap *tmAold;          // [L+1] activations a[l] of the previous iterate, box 64 x 128 (= TcDev::tmA)
    const CUtensorMap *tmF;             // [L+1] the jobs' buffers F[l], 3-D {column, row, slot}, box 64 x 128 x 1
    const CUtensorMap *tmW16;           // [3][L+1] masked weights W[l]: boxes of 64 x 16, 64 x 32 and 64 x 64 (columns x rows)
    float *S;                           // [slot][L+1][nbs][128 rows] fp32: base sums of a job's next groups
    int nbs;
    __nv_bfloat16 *F[JS_MAXL + 1];      // [slot][128 rows][WF[l]]: a job's fresh activations of a[l]
    int WF[JS_MAXL + 1];
    const int *cnt[JS_MAXL + 1];        // cnt[l][d], d = 0..T: units of a[l] with degree <= d (l >= 1)
    int G;                              // positions per group
    int n_stages, ring_bytes, smem_bytes, slots;
};

// Device view of a masked-convolution stack (tensor-core kernel only).
struct ConvDev {
    int height, width, in_ch, ch, n_conv, C, T;
    int R;                              // image rows per 128-pixel tile
    int nyt;                            // row tiles per image
    int cin_pad[JS_MAXL];               // input channels of conv layer l, padded to a multiple of 64
    void *act[JS_MAXL + 1];             // NHWC bf16; act[0] = encoded image padded to 64 channels
    void *act_old[JS_MAXL + 1];         // the same for the previous outer iterate (Jacobi-GS)
    const float *bias[JS_MAXL + 1];     // conv biases, head bias at [n_conv]
    const float *lut;
    const CUtensorMap *tmAct;           // [n_conv+1] 4-D maps {channel, x, y, image}, box 64 x width x R x 1
    const CUtensorMap *tmActOld;        // the same over act_old
    const CUtensorMap *tmW;             // [n_conv+1] 2-D maps of the packed weights
};

struct js_model {
    int kind = 0;                 // 0 masked MLP, 1 masked-conv stack
    int max_batch = 0;
    int rows = 0;                 // max_batch rounded up to a multiple of 128
    MadeDev made{};
    int conv_T = 0, conv_C = 0;
    std::vector<void *> allocs;   // every device allocation, freed by js_model_destroy
    std::vector<std::vector<int>> host_deg;
    JsCtl *ctl = nullptr;
    JsCtl *h_result = nullptr;    // pinned host memory, mapped: the kernels report here
    JsCtl *d_result = nullptr;    // the same memory as the device sees it
    bool ctl_clean = false;       // the last call left the control block zeroed
    // host-buffer entry point: device staging, copy stream, "noise has arrived" word
    float *st_noise = nullptr;
    uint8_t *st_x = nullptr, *st_init = nullptr;
    int32_t *st_iters = nullptr;
    unsigned *d_nflag = nullptr, *h_nflag = nullptr;
    unsigned n_uploads = 0;
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ev_main = nullptr, ev_copy = nullptr;
    int *smp_changed = nullptr, *smp_state = nullptr, *perm = nullptr;
    uint8_t *x_old = nullptr, *x_tmp = nullptr;
    unsigned long long *trace = nullptr;
    int opt_frontier_skip = 1, opt_seq_skip = 2, opt_spin_limit = 1 << 22, opt_path = 0, opt_compact = 1, opt_trace = 0;
    int max_grid_generic = 0;
    TcDev tc{};
    int tc_ok = 0, tc_max_grid = 0;
    ConvDev conv{};
    int conv_max_grid = 0;
    SweepDev sweep{};
    int sweep_state = 0;          // 0 not prepared yet, 1 ready, -1 the model does not qualify
    int *sw_flags = nullptr;      // [2][rows]: per-sample change flags and done flags of the sweeps
    int *h_any = nullptr, *d_any = nullptr;      // mapped host word: did anything change in this outer iteration
    js_stats stats{};
};

int js_tc_prepare(js_model *m);
int js_launch_made_tc(const js_model *m, const RunArgs &r, cudaStream_t stream);
int js_conv_build(js_model *m, const js_conv_desc *d);
int js_launch_conv_tc(const js_model *m, const RunArgs &r, cudaStream_t stream);
int js_sweep_prepare(js_model *m);
int js_launch_made_sweep(const js_model *m, const RunArgs &r, cudaStream_t stream);
int js_launch_jgs_book(const js_model *m, int batch, int k, int at_cap, int32_t *out_iters, cudaStream_t stream);
