// Internal to the library: pieces of the closed-form plan that the launcher re-applies when a
// caller overrides the tile shape.
#pragma once
#include "attn.h"

namespace attn_internal {
// Grid size for `heads` heads of `q_tiles` Q tiles, `steps` KV steps along the whole key axis and
// `ratio` = Q-tile rows / KV-tile rows.  Non-causal: one CTA per tile when there are at least as many
// tiles as compute units, otherwise the cheaper of a uniform and a balanced split of the key axis.
// Causal (tiles need unequal numbers of steps): always equal ranges of the unit line, one per unit.
int grid_size(const attn_hw_desc& h, int heads, int q_tiles, int steps, int ratio, int causal);
// Work units (KV steps summed over Q tiles) of one head.
long long head_units(int q_tiles, int steps, int ratio, int causal);
}  // namespace attn_internal
