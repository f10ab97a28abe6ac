// Host side of the attention step of a pass.
#pragma once
#include "common.cuh"
struct s2d2_ctx;
int attention_init(s2d2_ctx* c);
void attention_destroy(s2d2_ctx* c);
// Attention of one layer over the rows of the pass; reads c->q / c->k_rows / c->v_rows and the KV
// pool, writes c->attn.  max_ctx / max_rows: largest cached length and row count of a sequence.
int attention(s2d2_ctx* c, const s2d2::PassView& pv, int layer, int max_ctx, int max_rows);

namespace s2d2 { namespace att { struct AttnParams; } }
// Geometry of the tensor-core attention of a pass (query tiles, key splits sized for about
// target_items work items; 0 = twice the SM count); false when only the plain kernel applies.
// *map_kv receives the host copy of the KV pool's tensor map.
bool attention_plan(s2d2_ctx* c, const s2d2::PassView& pv, int max_ctx, int max_rows, int target_items,
                    s2d2::att::AttnParams* out, const void** map_kv);
