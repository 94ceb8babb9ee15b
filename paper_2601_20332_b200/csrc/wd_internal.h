// Internal declarations shared by the translation units of libwd.so.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda.h>
#include <stdint.h>
#include <stddef.h>
#include <vector>

#include "../../include/wd.h"

#define WD_CUDA_TRY(expr)                               \
    do {                                                \
        cudaError_t _e = (expr);                        \
        if (_e != cudaSuccess) { wd_note_cuda_error(_e, __FILE__, __LINE__); return WD_ERR_CUDA; } \
    } while (0)

void wd_note_cuda_error(cudaError_t e, const char* file, int line);

// kernels launched by this thread so far (every launcher below counts itself)
extern thread_local long long wd_launch_counter;

static inline size_t wd_align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static inline int wd_ceil_div(int a, int b) { return (a + b - 1) / b; }
static inline size_t wd_elt_size(int dtype) { return dtype == WD_F32 ? 4 : 2; }

// ---------------------------------------------------------------------------
// host planner (planner.cpp): pure integer logic, no CUDA
// ---------------------------------------------------------------------------
struct WdSeq {
    std::vector<int32_t> ids;
    std::vector<uint8_t> decoded;
    std::vector<int32_t> dec_step;
    std::vector<int32_t> wex;       // external window of the current phase
    int32_t t = 0;                  // diffusion step index
    int32_t since = 0;              // steps since the last refresh
    int32_t phase_start = 0;
    int32_t eos_id = -1;            // adaptive termination: id of the end-of-sequence token, -1 = off
    int32_t refresh_mode = 0;       // WD_REFRESH_FULL (the paper's refresh) or WD_REFRESH_WINDOW (variant)
    int32_t stagger_i = 0, stagger_n = 0;   // staggered refresh (variant): sequence i of n, n = 0: off
};

// steps by which sequence i of n shifts its phase clock when refresh steps are staggered (0: not at all)
static inline int32_t wd_stagger_offset(int32_t i, int32_t n, int32_t R) {
    return n > 0 ? (int32_t)(((int64_t)i * R) / n) : 0;
}

struct WdSeqPlan {
    bool done = false, refresh = false, vis_contiguous = false;
    std::vector<int32_t> wex, active, buffer, decoded, transient, far_field, rows, vis;
};

// Pure: does not modify `s`.
wd_status wd_plan_seq(const WdSeq& s, int32_t A, int32_t B, int32_t R, int32_t T, WdSeqPlan* out);
// Apply a step's update set and advance the phase counters.
void wd_commit_seq(WdSeq& s, const WdSeqPlan& plan, const int32_t* positions,
                   const int32_t* token_ids, int32_t n);

// Count-level shadow of a sequence's planner state.  Which positions a step unmasks is only
// known on the device, but HOW MANY rows, active rows and visible positions the following steps
// have does not depend on it (k tokens leave the window per step), so the host can size the
// launches of several steps ahead while the device plans the index lists.
struct WdCount {
    int32_t undecoded = 0, decoded = 0;   // |U|, |Dec|
    int32_t wex_size = 0, w_alive = 0;    // external window: size at phase start, still undecoded
    int32_t t = 0, since = 0;
    int32_t refresh_mode = 0;
    int32_t stagger_i = 0, stagger_n = 0;
    std::vector<int32_t> hist;            // tokens unmasked at each step of the current phase
};
struct WdCountPlan {
    bool done = false, refresh = false;
    bool window_refresh = false;          // refresh that computes only the new window and the previous phase's tokens
    int32_t prev_phase_start = 0;
    int32_t n_active = 0, n_transient = 0, n_vis = 0, n_rows = 0, n_wex = 0, n_unmask = 0;
};
void wd_count_init(WdCount& c, const WdSeq& s);
wd_status wd_count_plan(const WdCount& c, int32_t A, int32_t B, int32_t R, int32_t T, int32_t k, WdCountPlan* out);
void wd_count_commit(WdCount& c, const WdCountPlan& p);

// ---------------------------------------------------------------------------
// kernel launchers.  Every pointer is a device pointer unless stated.
// `status` is a device int32: kernels store WD_ERR_* there on a failed check.
// ---------------------------------------------------------------------------

// x[r,:] = embed[ids[row_seq[r]*S + row_pos[r]], :]  (float residual stream); also fills the
// rotary table rope_tab[r][j] = (cos, sin)(row_pos[r] * theta^(-2j/dh)), j < dh/2
void wd_launch_embed(int dtype, const void* embed, const int32_t* ids, const int32_t* row_seq,
                     const int32_t* row_pos, float* x, float2* rope_tab, int n_rows, int d, int S, int vocab, int dh,
                     float theta, int32_t* status, cudaStream_t st);

// fused pipeline (bf16): x, xg = bf16(x * gain), sumsq[d/128][n_rows] partial sums of squares, rope_tab
void wd_launch_embed_fused(const void* embed, const int32_t* ids, const int32_t* row_seq, const int32_t* row_pos,
                           float* x, void* xg, const float* gain, float* sumsq, float2* rope_tab, int n_rows, int d, int S,
                           int vocab, int dh, float theta, int32_t* status, cudaStream_t st);

// An operand in the NVFP4 format: e2m1 codes packed two per byte (element 2j in the low nibble), one unsigned
// e4m3 scale per 16 elements along K, one float scale per row.
struct WdFp4Operand {
    uint8_t* codes = nullptr;    // [n_rows][K / 2]
    uint8_t* sf = nullptr;       // [n_rows][K / 16]
    float* g = nullptr;          // [n_rows]
    int n_rows = 0, K = 0;
};

// x += sum_s part[s] (if part != null); xn = rmsnorm(x) * gain, written as `dtype`.
// With row_idx != null the rows x[row_idx[i]] are read (no partial add, x not written)
// and xn[i] is written: used for the final norm over the active rows only.  d % 4 == 0.
void wd_launch_rmsnorm(int dtype, float* x, const float* part, int n_split, size_t split_stride,
                       const float* gain, float eps, void* xn, const int32_t* row_idx, int n_rows,
                       int d, cudaStream_t st, uint8_t* xq = nullptr, float* sx = nullptr, const WdFp4Operand* x4 = nullptr);
// (xq != null: FP8 output instead of xn: e4m3 codes [n_rows][d] and one scale per row;
//  x4 != null: NVFP4 output instead of xn, quantised from the bfloat16 rounding of the normalised row; d % 16 == 0)

// plain GEMM: y[rows, n] (float) = x[rows,k] * w[n,k]^T
void wd_launch_gemm_plain(int dtype, const void* x, const void* w, float* y, int rows, int n, int k,
                          int ldy, cudaStream_t st);

// qkv partials -> RoPE -> q (dtype) and K/V cache rows.
//   part: [n_split][n_rows][(Hq+2Hkv)*dh] float, columns = [q | k | v]
//   kcache: [batch][Hkv][S][dh]; vcache: [batch][Hkv][dh][Sp] (this layer's slices)
void wd_launch_rope_scatter(int dtype, const float* part, int n_split, size_t split_stride,
                            const int32_t* row_seq, const int32_t* row_pos, const float2* rope_tab, void* q,
                            void* kcache, void* vcache, int n_rows, int Hq, int Hkv, int dh, int S, int Sp,
                            int batch, int32_t* status, cudaStream_t st);
// (a row whose position or sequence index is outside the state records WD_ERR_BOUNDS and writes no cache row)

// general (index-list) attention, CUDA cores.
//   row_seq[r]: sequence of row r (null: one sequence)
//   vis_idx: concatenated visible positions, sequence b at [vis_off[b], vis_off[b+1])
//            (vis_off null: one sequence seeing vis_idx[0, max_vis))
void wd_launch_attention_plain(int dtype, const void* q, const void* kcache, const void* vcache,
                               const int32_t* row_seq, const int32_t* vis_idx, const int32_t* vis_off,
                               void* out, float* tap, int n_rows, int max_vis, int Hq, int Hkv, int dh,
                               int S, int Sp, int batch, int32_t* status, cudaStream_t st);
// (a visible index outside [0, S) or a sequence index outside [0, batch) records WD_ERR_BOUNDS and is not dereferenced)

// h = silu(gate) * up from partials [n_split][n_rows][2F] (columns = [gate | up]); F % 4 == 0
void wd_launch_swiglu(int dtype, const float* part, int n_split, size_t split_stride, void* h,
                      int n_rows, int F, cudaStream_t st);

// FP8: h as e4m3 codes [n_rows][F] with one scale per row (F <= 32768)
wd_status wd_launch_swiglu_fp8(const float* part, int n_split, size_t split_stride, uint8_t* hq, float* sh, int n_rows,
                               int F, cudaStream_t st);
// NVFP4: the bfloat16 rounding of h in the NVFP4 format (F % 64 == 0, F <= 32768)
wd_status wd_launch_swiglu_fp4(const float* part, int n_split, size_t split_stride, const WdFp4Operand* h4, int n_rows,
                               int F, cudaStream_t st);
// per-row e4m3 quantisation of a [n_rows, K] matrix of `dtype` (K % 4 == 0): codes and scales
void wd_launch_quantize_rows(int dtype, const void* w, int n_rows, int K, uint8_t* q, float* s, cudaStream_t st);

// x += sum_s part[s]; optionally copy x to tap.
void wd_launch_residual_add(float* x, const float* part, int n_split, size_t split_stride,
                            float* tap, int n_rows, int d, cudaStream_t st);

// unmask stage 1: per (row, vocabulary chunk) maximum, lowest argmax, sum exp(l - max) in double;
// outputs are [n][wd_unmask_chunks(V)]
#define WD_UNMASK_MAX_CHUNKS 64
int wd_unmask_chunks(int V);
void wd_launch_rowstats(const float* logits, int n, int V, float* ch_max, int32_t* ch_idx, double* ch_sum,
                        cudaStream_t st);

// unmask stage 2, per sequence: merge the chunks of each row into (token, sum exp), rank the
// rows by (sum exp ascending, position ascending), emit the first min(k, n_b); optionally write
// the chosen ids into ids[b*S + pos].  act_off == null: one sequence holding rows [0, n_single).
void wd_launch_select(const float* ch_max, const int32_t* ch_idx, const double* ch_sum, int n_chunks,
                      int32_t* row_token, double* row_sumexp, const int32_t* act_pos, const int32_t* act_off,
                      int n_single, int batch, int k, int32_t* ids, int S, int32_t* n_sel, int32_t* sel_pos,
                      int32_t* sel_token, float* sel_conf, float* row_conf, uint8_t* decoded, int32_t* dec_step,
                      const int32_t* step_of_seq, cudaStream_t st);

// Device-side planner (one block per sequence): builds the step's index lists from the device
// copy of the state; the host supplies counts and offsets only.  Up to WD_PLAN_MAX_BATCH sequences.
#define WD_PLAN_MAX_BATCH 16
struct WdPlanLaunch {
    int32_t batch, S, A, T;
    int32_t refresh[WD_PLAN_MAX_BATCH], done[WD_PLAN_MAX_BATCH], n_wex[WD_PLAN_MAX_BATCH], n_vis[WD_PLAN_MAX_BATCH],
        t[WD_PLAN_MAX_BATCH];
    int32_t window_refresh[WD_PLAN_MAX_BATCH], prev_phase_start[WD_PLAN_MAX_BATCH];   // the window-only refresh variant
    int32_t row_off[WD_PLAN_MAX_BATCH + 1], act_off[WD_PLAN_MAX_BATCH + 1], vis_off[WD_PLAN_MAX_BATCH + 1],
        qt_off[WD_PLAN_MAX_BATCH + 1];
    const uint8_t* decoded;       // [batch][S] device
    const int32_t* dec_step;      // [batch][S] device
    int32_t* wex;                 // [batch][S] device: external window of the phase
    int32_t *row_seq, *row_pos, *act_row, *act_pos, *act_off_dev, *vis_off_dev, *vis_idx, *qt_seq, *qt_row0, *qt_n, *nvis_dev,
        *tseq_dev;
    int32_t* status;
};
void wd_launch_plan(const WdPlanLaunch& h, cudaStream_t st);

// query-tile lists of one sequence for the tensor-core attention (single operation): see the kernel
void wd_launch_fill_qtiles(int32_t* lists, int n_rows, int n_vis, cudaStream_t st);

wd_status wd_launch_wait_expire(cudaStream_t st);
int32_t* wd_op_status_ptr();   // device address of the single-operation status word
extern bool wd_pdl_enabled;    // programmatic dependent launch on every kernel (default on)
