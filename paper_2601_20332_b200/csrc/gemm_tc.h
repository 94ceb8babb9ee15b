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
    int fp8 = 0;             // byte matrix of e4m3 codes
    // descriptors already encoded for this operand, keyed by (rows, token tile): the same few
    // shapes come back every step
    struct Entry { int rows, bn; CUtensorMap map; };
    mutable std::vector<Entry> cache;
    bool keep = true;        // false: one-off operand (single operations): encode on the stack, remember nothing
    // > 0: most dynamic shared memory a CTA of the GEMM over this operand may take (fewer ring stages), so that it
    // fits on an SM beside a CTA of the kernel that produces the operand and can fetch weights while that runs
    mutable int smem_cap = 0;
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

// What the CTA that completes an output tile does with the summed tile ("fused epilogue").
// The tile sums still pass through the partial-sum slices in y; these modes only add the
// consumer's work to the GEMM so that no separate kernel (and no dependency bubble) follows.
enum { WD_FUSE_NONE = 0, WD_FUSE_QKV = 1, WD_FUSE_RESID = 2, WD_FUSE_SWIGLU = 3, WD_FUSE_LMSTATS = 4 };

struct WdTcFuse {
    int mode = WD_FUSE_NONE;
    int32_t* counters = nullptr;      // zeroed ints, one per output tile (left zeroed again on return)
    int rows_total = 0;
    // QKV and SWIGLU: the input rows were not normalised; scale by 1/rms from these partial sums of squares
    const float* sumsq_in = nullptr;  // [n_prev_tiles][rows_total]
    int n_prev_tiles = 0;
    float inv_d = 0.f, eps = 0.f;
    // QKV: rotate q/k heads, write q and the K / transposed-V cache rows (head_dim 128 = one tile per head)
    const int32_t* row_seq = nullptr;
    const int32_t* row_pos = nullptr;
    const float2* rope_tab = nullptr;
    __nv_bfloat16* q = nullptr;
    __nv_bfloat16* kcache = nullptr;
    __nv_bfloat16* vcache = nullptr;
    int Hq = 0, Hkv = 0, S = 0, Sp = 0;
    int batch = 1;                    // sequences of the state (index check of row_seq)
    int cluster = 0;                  // 1: take the cluster split-K kernel (gemm_ck.cu) where it can serve the shape
    // RESID: x += tile; xg = bf16(x * gain_next) for the next GEMM; partial sums of squares of the new x
    float* x = nullptr;
    const float* gain_next = nullptr; // null: no xg (after the last block)
    __nv_bfloat16* xg = nullptr;
    float* sumsq_out = nullptr;       // [d/128][rows_total]
    float* tap = nullptr;
    // SWIGLU: h = silu(gate) * up, gate tile t and up tile t complete together
    __nv_bfloat16* h = nullptr;
    int F = 0;
    // LMSTATS (LM head, whole tiles per CTA, rows <= 256): per (row, CTA) maximum, lowest argmax and
    // sum of exp(l - max) over the vocabulary tiles the CTA covered, [rows][n_chunks] with n_chunks
    // (= grid size) filled in by wd_tc_gemm; the logits themselves are written only if write_logits
    // is set (parity tests)
    mutable int n_chunks = 0;
    float* st_max = nullptr;
    int32_t* st_idx = nullptr;
    double* st_sum = nullptr;
    int write_logits = 0;
};

// FP8 operands (e4m3 codes, one float scale per weight row and per activation row): the maps of
// the segments and of x then describe byte matrices (box 128 (K) x rows), K is still the number
// of elements, and every output is multiplied by sw[segment][n] * sx[row] in the epilogue.
struct WdTcFp8 {
    const float* sw[3] = {nullptr, nullptr, nullptr};
    const float* sx = nullptr;
};

// Gate/up launches (two weight matrices of the same height): where the GEMM can keep the gate tile and
// the up tile of the same columns in two accumulators, its epilogue writes h = silu(gate) * up as bf16
// [rows, n] and nothing goes to y.  `done` tells the caller whether that happened; if not, y holds the
// partial sums as usual and the caller runs the SwiGLU kernel.
struct WdTcSwiglu {
    __nv_bfloat16* h = nullptr;
    mutable bool done = false;
};

// y[split][rows][sum n_i] = x * [w_0; w_1; ...]^T, split-K partial sums side by side
// (split_stride = rows * sum n_i floats).  The consumer adds the slices.
wd_status wd_tc_gemm(const WdTcX* x, const WdTcSeg* segs, int nseg, int rows, int K, float* y, size_t y_floats,
                     int sm_count, int32_t* status, cudaStream_t stream, int* n_split_out,
                     bool force_single_split = false, const WdTcFuse* fuse = nullptr, const WdTcFp8* fp8 = nullptr,
                     const WdTcSwiglu* sg = nullptr);
// Chain kernel (few rows): up to four consecutive fused GEMMs (modes QKV / RESID / SWIGLU) in one persistent
// launch whose weight stream never stops; each GEMM's input is the previous one's finished tiles.
struct WdTcChainItem {
    const WdTcX* x;
    const WdTcSeg* segs;
    int nseg, K;
    WdTcFuse fuse;
};
// Device counters of finished tiles (counted up across launches) and the host's running totals.  After a
// device-side error the two may disagree: zero both before the next launch.
struct WdTcChainState {
    int32_t* ready_dev = nullptr;     // [4], zero-initialised
    int32_t ready_host[4] = {0, 0, 0, 0};
};
bool wd_tc_chain_rows_ok(int rows);
// WD_ERR_CAPACITY: the partial sums do not fit y (the caller launches the GEMMs one by one instead)
wd_status wd_tc_chain(const WdTcChainItem* items, int n, int rows, float* y, size_t y_floats, int sm_count,
                      int32_t* status, WdTcChainState* cs, cudaStream_t stream);

// Few tokens (rows <= 128), fused modes QKV / RESID / SWIGLU: split-K over the four CTAs of a thread-block
// cluster, the partial tiles summed through distributed shared memory, the consumer's work done by the
// CTAs that own the result (gemm_ck.cu).  Nothing is written to a partial-sum buffer.
bool wd_ck_usable(int rows, int K, const WdTcSeg* segs, int nseg, const WdTcFuse* fuse);
int wd_ck_max_rows();      // most rows for which every mode fits its buffers beside a ring deep enough to stream
wd_status wd_ck_gemm(const WdTcX* x, const WdTcSeg* segs, int nseg, int rows, int K, int sm_count, int32_t* status,
                     cudaStream_t stream, const WdTcFuse* fuse);

// TMA descriptor of a [n_rows, K] byte matrix for the FP8 path (box 128 x box_rows)
wd_status wd_tc_encode_fp8(CUtensorMap* m, const void* ptr, int n_rows, int K, int box_rows);
// TMA descriptor of a [n_rows, K] bf16 matrix (box 64 x box_rows, 128-byte swizzle)
wd_status wd_tc_encode_bf16(CUtensorMap* m, const void* ptr, int n_rows, int K, int box_rows);

size_t wd_tc_scratch_bytes(int rows, int n_out, int k_in);
wd_status wd_tc_gemm_standalone(const void* x, const void* w, float* y, int rows, int n_out, int k_in, void* scratch,
                                size_t scratch_bytes, cudaStream_t stream);
wd_status wd_tc_gemm_standalone_fp8(const uint8_t* xq, const float* sx, const uint8_t* wq, const float* sw, float* y,
                                    int rows, int n_out, int k_in, float* slices, size_t slice_floats, cudaStream_t stream);

// ---- NVFP4 (gemm_fp4.cu): e2m1 codes packed two per byte, one unsigned e4m3 scale per 16 elements along K,
// one float scale per row
size_t wd_fp4_operand_bytes(int n_rows, int K);                       // device bytes of one quantised operand
void wd_fp4_operand_split(void* mem, int n_rows, int K, WdFp4Operand* op);
// quantises a [n_rows, K] matrix of `dtype` (taken as bfloat16), K a multiple of 16
void wd_launch_quantize_nvfp4(int dtype, const void* x, int n_rows, int K, const WdFp4Operand* op, cudaStream_t st);
// y[split][rows][n] = x * w^T on the block-scaled tensor-core path (K a multiple of 256); K slices side by side.
// w_static: the weights were quantised before the previous kernel on the stream started, so the kernel may
// fetch them ahead of its dependency wait.
wd_status wd_fp4_gemm(const WdFp4Operand* x, const WdFp4Operand* w, float* y, size_t y_floats, int sm_count, int32_t* status,
                      cudaStream_t stream, int* n_split_out, bool force_single_split, bool w_static);
// adds the K slices of a GEMM result: y[i] = sum_s part[s * stride + i]
void wd_launch_reduce_slices(const float* part, int n_split, size_t stride, float* y, size_t total, cudaStream_t st);
