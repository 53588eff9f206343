// Internal to the library: pieces of the closed-form plan that the launcher re-applies when a
// caller overrides the tile shape.
#pragma once
#include "attn.h"

namespace attn_internal {
// Grid size for `tiles` Q tiles of `steps` KV steps each: one CTA per tile when there are at least as
// many tiles as compute units; otherwise the cheaper of a uniform and a balanced split of the key axis.
int grid_size(const attn_hw_desc& h, int tiles, int steps);
}  // namespace attn_internal
