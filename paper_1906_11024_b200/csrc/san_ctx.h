// The context behind the opaque san_ctx handle: host-side tables plus pointers into the
// caller's device buffers.  Nothing here owns device memory.
#pragma once

#include <stddef.h>
#include <stdint.h>

#include "../../include/san.h"
#include "san_policy.h"

struct san_ctx {
    san_config cfg;
    san::Policy self_pol, enc_pol;
    int elem_bytes = 0, n_seqs = 0, sm_count = 0;

    // cache arena (caller-owned)
    char* cache = nullptr;
    size_t cache_bytes_needed = 0;
    size_t self_plane_bytes = 0, mem_plane_bytes = 0, aan_plane_bytes = 0;
    int n_self_k_planes = 0, n_self_v_planes = 0, n_enc_k_planes = 0, n_enc_v_planes = 0;
    size_t off_self_k = 0, off_self_v = 0, off_mem_k = 0, off_mem_v = 0, off_aan = 0;

    // workspace (caller-owned): error words, tickets of split rows, their partial sums
    char* ws = nullptr;
    size_t ws_bytes_needed = 0, ws_off_tickets = 0, ws_off_part = 0;
    size_t n_tickets = 0, part_floats = 0;
    int* err = nullptr;
    int* tickets = nullptr;
    float* part = nullptr;
    bool fused_attr_set = false;   // shared-memory opt-in of the one-launch step kernel done
    bool team_attr_set = false;    // the same for the team-pipeline step kernel
    bool rows_attr_set = false;    // and for the short-rows step kernel
    int step_kernel = 0;           // 0: automatic, 1: per-warp pipeline kernel, 2: team-pipeline kernel, 3: short-rows kernel (san_step_kernel_select)
    int team_cut_override[4] = {-1, 4, 64, 0};   // spans per row (log2; -1: automatic), heads per unit, positions per tile, layers per unit (0: automatic)
    int team_grab_mult = 1;
    int last_step_kernel = 0;      // which kernel the last san_decode_step launched (0: none yet)
    int last_rows_per_unit[2] = {0, 0};   // team pipeline: heads per unit for self / enc-dec attention in that launch

    // How the one-launch step cuts long rows (positions per item, layers per item), remembered
    // per launch shape: the search that balances the items over the warps costs more than a
    // short step, and a decode loop repeats the same shape for many steps.
    struct StepPlan {
        bool valid = false;
        unsigned epoch = 0;                      // policy_epoch it was made for
        int n_seqs = 0, n_sent = 0, len_bound = 0, src_bound = 0;
        int span_self = 0, lg_self = 0, span_enc = 0, lg_enc = 0;
    };
    static constexpr int kPlans = 8;
    StepPlan plans[kPlans];
    int plan_next = 0;
    unsigned policy_epoch = 0;     // raised whenever a sharing policy changes
};
