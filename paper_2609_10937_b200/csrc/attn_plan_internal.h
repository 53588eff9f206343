// Internal to the library: pieces of the closed-form plan that the launcher re-applies when a
// caller overrides the tile shape.
#pragma once
#include "attn.h"

namespace attn_internal {
// Grid size for `heads` heads of `q_tiles` Q tiles, `steps` KV steps along the whole key axis and
// `ratio` = Q-tile rows / KV-tile rows; `kv_bytes_per_head` = bytes of K and V of one head.
// Non-causal, fewer tiles than compute units: the cheapest of one CTA per tile, k CTAs per tile along the key
// axis (as one cluster each where `groups` 32-row groups of `part_floats_per_row` fp32 values per row fit the
// landing areas -- the Q buffer for two parts, `ring_bytes` of K/V ring otherwise -- and the descriptor says
// that many clusters can be resident; else through the workspace) and equal ranges of the unit line.
// Non-causal, more tiles than units: one CTA per tile, or one persistent CTA per unit walking an
// equal range of the (tile, step) line when that is cheaper and the K/V of the heads in flight fit the cache.
// Causal (tiles need unequal numbers of steps): equal ranges of the unit line, or k = 2..4 CTAs per tile as one cluster.
// Returns the grid and its cost: KV steps on the longest CTA's path plus the descriptor's ovh_* term of the winner.
struct Grid { int ctas; long long cost; };
Grid grid_size(const attn_hw_desc& h, int heads, int q_tiles, int steps, int ratio, int causal,
              long long kv_bytes_per_head, int groups, int part_floats_per_row, long long ring_bytes);
// The derivation for Lq query rows and Lk keys per head (attn_plan_ex is the case Lq == Lk).
int plan_qk(const attn_hw_desc* desc, int B, int H, int Lq, int Lk, int d, int causal, attn_tiles* out);
// Work units (KV steps summed over Q tiles) of one head.
long long head_units(int q_tiles, int steps, int ratio, int causal);
}  // namespace attn_internal
