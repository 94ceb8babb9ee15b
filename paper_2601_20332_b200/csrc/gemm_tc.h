// Tensor-core GEMM (tcgen05 / TMEM / TMA) interface, bf16 only.
#pragma once
#include <vector>

#include "wd_internal.h"

#define WD_TC_MAX_SPLIT 16          // most split-K slices
#define WD_TC_SPLITK_MAX_ROWS 256   // split-K only while the token tile count is 1

enum { WD_TC_WQ = 0, WD_TC_WK, WD_TC_WV, WD_TC_WO, WD_TC_WG, WD_TC_WU, WD_TC_WD, WD_TC_LM, WD_TC_KINDS };

// One weight matrix [n, K] taking part in a GEMM (its rows become output columns).
struct WdTcSeg {
    const void* w;
    int n;
    const CUtensorMap* map;   // TMA descriptor, box 64 (K) x 128 (n), 128-byte swizzle; null on the plain path
};

// Activation operand [rows, K]; its TMA descriptor depends on rows and on the token tile, so it
// is encoded per launch.
struct WdTcX {
    const void* ptr = nullptr;
    int K = 0;
};

struct WdTcWeights {
    std::vector<CUtensorMap> maps;      // [kind][layer]
    int n_layers = 0;
    WdTcX x_map_d, x_map_attn, x_map_h;
    const CUtensorMap* get(int kind, int l) const {
        return maps.empty() ? nullptr : &maps[(size_t)kind * n_layers + l];
    }
};

wd_status wd_tc_weights_init(WdTcWeights* tc, const wd_model_dims* d, const void* tok_embed, const void* lm_head,
                             const std::vector<const void*>& wq, const std::vector<const void*>& wk,
                             const std::vector<const void*>& wv, const std::vector<const void*>& wo,
                             const std::vector<const void*>& wg, const std::vector<const void*>& wu,
                             const std::vector<const void*>& wd, const void* xn, const void* attn, const void* h);

// y[split][rows][sum n_i] = x * [w_0; w_1; ...]^T, split-K partial sums side by side
// (split_stride = rows * sum n_i floats).  The consumer adds the slices.
wd_status wd_tc_gemm(const WdTcX* x, const WdTcSeg* segs, int nseg, int rows, int K, float* y, size_t y_floats,
                     int sm_count, int32_t* status, cudaStream_t stream, int* n_split_out,
                     bool force_single_split = false);

size_t wd_tc_scratch_bytes(int rows, int n_out, int k_in);
wd_status wd_tc_gemm_standalone(const void* x, const void* w, float* y, int rows, int n_out, int k_in, void* scratch,
                                size_t scratch_bytes, cudaStream_t stream);
