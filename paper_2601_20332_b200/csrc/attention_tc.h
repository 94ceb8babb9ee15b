// Tensor-core windowed attention (tcgen05 / TMEM / TMA) interface: bf16, head_dim 128,
// visible set of every sequence a range [0, n_vis).
#pragma once
#include "wd_internal.h"

// TMA descriptors over a state's whole K cache [L][BH][S][dh] and transposed V cache
// [L][BH][dh][Sp] (BH = batch * n_kv_heads).
wd_status wd_attn_tc_encode_cache(CUtensorMap* map_k, CUtensorMap* map_vt, const void* kcache, const void* vcache,
                                  int L, int BH, int S, int Sp, int dh);

// q: [n_rows][Hq*dh] bf16.  Query tiles: tile t covers rows [qtile_row0[t], +qtile_n[t]) of
// sequence qtile_seq[t] (at most 128 rows, never crossing a sequence boundary); seq_nvis[b] =
// number of visible positions of sequence b.  All four are device arrays.
wd_status wd_attn_tc_launch(const void* q, int n_rows, int n_tiles, const int32_t* qtile_seq, const int32_t* qtile_row0,
                            const int32_t* qtile_n, const int32_t* seq_nvis, const CUtensorMap* map_k,
                            const CUtensorMap* map_vt, void* out, float* tap, int Hq, int Hkv, int dh, int layer,
                            int max_vis, int sm_count, int32_t* status, cudaStream_t stream, int max_tile_rows = 0,
                            size_t* smem_used = nullptr);
// max_vis = most visible positions of any sequence (sizes the split of the keys over a cluster).
// max_tile_rows = most valid rows of any query tile when the caller knows it (0: unknown): with grouped-query
// heads and at most 64 (32) rows per tile, two (four) query heads of one KV head share a tile.
// smem_used (optional): the dynamic shared memory of one CTA of the launch (the single-key-tile form takes less than
// half an SM's, so that the next kernel's CTAs can be resident beside it).
