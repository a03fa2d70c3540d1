// Host-side model object behind the opaque js_model handle.
#pragma once
#include <vector>

#include "js_common.cuh"

struct js_model {
    int kind = 0;                 // 0 masked MLP, 1 masked-conv stack
    int max_batch = 0;
    int rows = 0;                 // max_batch rounded up to a multiple of 128
    MadeDev made{};
    int conv_T = 0, conv_C = 0;
    std::vector<void *> allocs;   // every device allocation, freed by js_model_destroy
    std::vector<std::vector<int>> host_deg;
    JsCtl *ctl = nullptr;
    int *smp_changed = nullptr, *smp_state = nullptr;
    uint8_t *x_old = nullptr, *x_tmp = nullptr;
    int opt_frontier_skip = 1, opt_seq_skip = 0, opt_spin_limit = 1 << 22, opt_path = 0, opt_compact = 1;
    int max_grid_generic = 0;
    js_stats stats{};
};
