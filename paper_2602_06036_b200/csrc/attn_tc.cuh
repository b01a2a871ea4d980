// Interface of the bf16 tensor-core block-attention kernel.
#pragma once

#include "dflash_internal.h"

namespace dflash {

// head_dim 128, 64-token pages, rows * (Hq/Hkv) <= 128
bool attn_tc_supported(const dflash_config& c, int rows);
int64_t attn_tc_part_bytes(const dflash_config& c, int batch, int rows, int sm_count);
int64_t attn_tc_counter_bytes(const dflash_config& c, int batch);
// How the keys of a call are split into ranges, and what that needs of the partials buffer (host arithmetic only).
struct AttnPlan {
    int tiles_per_unit;        // 64-key tiles per range
    int n_chunks;              // ranges per (sequence, kv head) at max_ctx_len
    int64_t units;             // partial slots the kernels index: batch * Hkv * n_chunks
    int64_t capacity_units;    // slots attn_tc_part_bytes provides for this batch (units never exceeds it)
};
AttnPlan attn_tc_plan(const dflash_config& c, int batch, int max_ctx_len, int sm_count);
// `part`: split-KV scratch of the size above. `counters` is not used by the current kernels (the
// partials are merged by a second kernel, not by a last arriver).
// `early_kv`: the layer's cached context was complete before the kernel preceding this one started waiting
// (true for layers after the first of a draft block: the first layer's wait covered the context
// projection); its first tiles are then requested before this kernel's own grid dependency resolves.
// `early_len` [device, batch] or nullptr: with early_kv, only pages wholly below this many rows per sequence
// are requested early (the rows from there on are written inside the same call, by a kernel whose end
// only this kernel's grid dependency covers).
// `first_of_call`: no kernel of the same call precedes this one; it then starts in plain stream order,
// because lengths and page numbers (possibly outputs of the caller's previous call) are read early.
int launch_attention_tc(const Launch& L, const dflash_attn_args& a, float* part, int32_t* counters, bool early_kv = false,
                        const int32_t* early_len = nullptr, bool first_of_call = false);

// Backward of the block attention (tensor-core path): rows * (Hq/Hkv) <= 64, head_dim 128, 64-token pages.
// `D`: fp32 scratch [batch * rows * Hq] (rowsum(dO * O), handed from the first kernel to the second).
bool attn_bwd_supported(const dflash_config& c, int rows);
int launch_attention_bwd(const Launch& L, const dflash_attn_bwd_args& a, float* D);

}  // namespace dflash
