/*
 * wd.h — C ABI of the windowed denoising step (Window-Diffusion) for NVIDIA B200.
 *
 * One call of wd_step() runs one diffusion step of a masked diffusion language
 * model over only the tokens the method says must be computed:
 *   - the sequence is a fixed-length state of decoded tokens and [MASK]
 *     placeholders (paper Section 3.1);
 *   - undecoded tokens are split into an external window (a fixed-length prefix
 *     of the undecoded region), its front part the internal window of ACTIVE
 *     tokens, the BUFFER tokens (external minus active minus tokens decoded in
 *     this phase) and the pruned FAR-FIELD tokens (Section 4.2);
 *   - steps are grouped into phases of one REFRESH step (full forward over the
 *     decoded tokens and the external window, all K/V written to the cache)
 *     followed by NORMAL steps (only active tokens and recently decoded tokens
 *     are computed; buffer and earlier decoded tokens are read from the cache)
 *     (Section 4.3);
 *   - logits exist only for active tokens, and the step ends by unmasking the
 *     k active tokens with the highest prediction confidence (Section 4.1,
 *     Observation 1 of Section 3.2).
 *
 * Conventions
 *   - Every function returns a wd_status (0 = WD_OK, positive = informational,
 *     negative = error).  Nothing aborts, traps or throws across this boundary.
 *   - "device" pointers are CUDA device memory of the current device, "host"
 *     pointers are ordinary host memory.  The library never allocates device
 *     memory: the caller passes workspaces whose sizes the *_bytes functions
 *     report.  All device pointers must be 256-byte aligned.
 *   - Borrowed memory (weights, workspaces, debug taps) stays owned by the
 *     caller and must outlive the object that borrows it.
 *   - The library is sm_100a only and has no CPU fallback.
 */
#ifndef WD_H
#define WD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define WD_API __attribute__((visibility("default")))
#else
#define WD_API
#endif

typedef int wd_status;

enum {
    WD_OK = 0,
    WD_DONE = 1,                      /* no undecoded token left anywhere      */
    WD_ERR_NULL = -1,                 /* a required pointer is NULL            */
    WD_ERR_INVALID_DIMS = -2,
    WD_ERR_WORKSPACE_TOO_SMALL = -3,
    WD_ERR_UNSUPPORTED_ARCH = -4,     /* current device is not sm_100          */
    WD_ERR_BAD_PARAM = -5,            /* A<1, B<0, R<1, T<0, k<0, bad index... */
    WD_ERR_CAPACITY = -6,             /* a caller-sized buffer is too short    */
    WD_ERR_PENDING = -7,              /* wd_step without wd_step_sync before   */
    WD_ERR_CUDA = -8,                 /* a CUDA runtime/driver call failed     */
    WD_ERR_DEVICE_TIMEOUT = -9,       /* a bounded device-side wait ran out    */
    WD_ERR_BOUNDS = -10,              /* a device-side index check failed      */
    WD_ERR_NOT_PENDING = -11,         /* wd_step_sync without wd_step before   */
    WD_ERR_MISALIGNED = -12,
    WD_ERR_INTERNAL = -13,            /* host and device planners disagree (a bug)   */
    WD_ERR_POISONED = -14             /* an earlier device-side error left this state inconsistent */
};

enum { WD_F32 = 0, WD_BF16 = 1 };     /* element type of weights, activations, K/V cache */

/* What a refresh step computes (wd_state_set_refresh_mode, wd_plan_raw). */
enum {
    WD_REFRESH_FULL = 0,              /* every visible position: Section 4.3 of the paper           */
    WD_REFRESH_WINDOW = 1             /* variant, NOT in the paper: only the new external window and
                                         the tokens decoded during the phase that just ended; older
                                         context keeps its cached K/V.  Exact for one block, an
                                         approximation beyond.  The first step is always full.   */
};

/* GEMM implementation selector (wd_set_gemm_impl, wd_op_gemm). */
enum {
    WD_GEMM_AUTO = 0,                 /* tensor-core kernel for bf16, plain for f32 */
    WD_GEMM_PLAIN = 1,                /* CUDA-core kernel (any dtype)               */
    WD_GEMM_TCGEN05 = 2               /* tcgen05/TMEM/TMA kernel (bf16 only)        */
};

/* Model shape.  The paper runs the pretrained model unmodified (Section 4.1),
 * so the block is the usual one: pre-norm residual blocks with RMSNorm, rotary
 * embedding at the absolute position, bidirectional grouped-query attention,
 * SwiGLU feed-forward, final RMSNorm, untied LM head, no biases. */
typedef struct wd_model_dims {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
    float   rope_theta, rms_eps;
    int32_t dtype;                    /* WD_F32 or WD_BF16                                  */
    int32_t mask_id;                  /* id of the [MASK] placeholder (Section 3.1)         */
    int32_t max_batch;                /* sequences per state                                */
    int32_t max_seq;                  /* S: positions per sequence                          */
    int32_t max_rows;                 /* most rows computed in one step, whole batch        */
    int32_t max_active;               /* most active rows in one step, whole batch          */
} wd_model_dims;

/* Device pointers to the weights, row-major with the reduction dimension
 * contiguous ("[out, in]").  Per-layer members are HOST arrays of n_layers
 * device pointers.  Matrices have the model dtype; norm gains are float.
 * Borrowed, never written. */
typedef struct wd_weights {
    const void*         tok_embed;    /* [vocab, d_model]                     */
    const void* const*  wq;           /* [n_q_heads*head_dim, d_model]        */
    const void* const*  wk;           /* [n_kv_heads*head_dim, d_model]       */
    const void* const*  wv;           /* [n_kv_heads*head_dim, d_model]       */
    const void* const*  wo;           /* [d_model, n_q_heads*head_dim]        */
    const void* const*  w_gate;       /* [d_ffn, d_model]                     */
    const void* const*  w_up;         /* [d_ffn, d_model]                     */
    const void* const*  w_down;       /* [d_model, d_ffn]                     */
    const float* const* attn_norm;    /* [d_model]                            */
    const float* const* ffn_norm;     /* [d_model]                            */
    const float*        final_norm;   /* [d_model]                            */
    const void*         lm_head;      /* [vocab, d_model]                     */
} wd_weights;

typedef struct wd_ctx wd_ctx;         /* model + step workspace               */
typedef struct wd_state wd_state;     /* a batch of sequences + their K/V cache */

/* Index sets of one sequence for the next step (Section 4.2; the buffer-set
 * equation; Section 4.3 for which rows are computed).  The caller allocates
 * every list with `capacity` entries (capacity >= sequence length is always
 * enough); lists come back ascending. */
typedef struct wd_index_sets {
    int32_t  capacity;
    int32_t* active;       int32_t n_active;      /* internal window A^(t)                       */
    int32_t* buffer;       int32_t n_buffer;      /* B^(t): undecoded context read from the cache */
    int32_t* decoded;      int32_t n_decoded;     /* every decoded position                      */
    int32_t* transient;    int32_t n_transient;   /* decoded in this phase and still recomputed  */
    int32_t* far_field;    int32_t n_far_field;   /* pruned undecoded positions                  */
    int32_t* rows;         int32_t n_rows;        /* positions computed this step                */
    int32_t* vis;          int32_t n_vis;         /* positions whose K/V are attended            */
    int32_t* ext_window;   int32_t n_ext_window;  /* W_ex^(p) as fixed at the phase start        */
    int32_t  is_refresh;                          /* 1 = refresh step, 0 = normal step           */
    int32_t  vis_contiguous;                      /* 1 if vis == [0, n_vis)                      */
    int32_t  done;                                /* 1 if the sequence has no undecoded token    */
} wd_index_sets;

/* Result of a step, host memory, caller-allocated: n_unmasked[batch];
 * positions / token_ids / confidence [batch * k] with sequence i at offset i*k,
 * ranked by confidence (highest first; equal confidence: lowest position). */
typedef struct wd_step_out {
    int32_t* n_unmasked;
    int32_t* positions;
    int32_t* token_ids;
    float*   confidence;
} wd_step_out;

/* Optional device buffers that receive intermediate values of the next steps
 * (for parity tests; leave unset in timed runs).  Any member may be NULL.
 * With n_rows computed rows and n_act active rows in the step (whole batch,
 * sequences concatenated in order, positions ascending inside a sequence):
 *   layer_out [n_layers][n_rows][d_model]   block outputs (residual stream)
 *   attn_out  [n_layers][n_rows][n_q_heads*head_dim]   attention outputs before
 *             the output projection
 *   logits    [n_act][vocab]   logits of the active rows
 * all float.  Capacities are for max_rows / max_active. */
typedef struct wd_debug_taps {
    float* layer_out;
    float* attn_out;
    float* logits;
} wd_debug_taps;

/* Per-step counters filled by wd_step (host). */
typedef struct wd_step_info {
    int32_t is_refresh;      /* any sequence refreshed (sequences of a state share the phase clock) */
    int32_t n_rows;          /* rows computed, whole batch   */
    int32_t n_active;        /* active rows, whole batch     */
    int32_t n_vis;           /* visible positions, summed    */
    int32_t n_launches;      /* kernels enqueued by the step */
    int32_t gemm_impl;       /* WD_GEMM_PLAIN or WD_GEMM_TCGEN05 actually used */
} wd_step_info;

/* ---- sizes -------------------------------------------------------------- */

/* Bytes of device workspace wd_create needs for these dims (0 if invalid). */
WD_API size_t wd_workspace_bytes(const wd_model_dims* dims);
/* Bytes of device memory one state of `batch` sequences of `seq_len` positions
 * needs (token ids + K/V cache of every layer; 0 if invalid). */
WD_API size_t wd_state_bytes(const wd_model_dims* dims, int32_t batch, int32_t seq_len);
/* Library version: major*10000 + minor*100 + patch. */
WD_API int32_t wd_version(void);
/* Bytes of that state memory taken by the K/V cache of every layer (Section 4.3: the cache the
 * refresh step writes and the normal steps read): K rows plus the transposed V rows, whose
 * positions are padded to a multiple of 8.  0 if invalid. */
WD_API size_t wd_kv_bytes(const wd_model_dims* dims, int32_t batch, int32_t seq_len);
/* Static text for a status code. */
WD_API const char* wd_status_string(wd_status s);
/* Text of the last CUDA runtime / driver error a call of this thread ran into ("" if none), with
 * the source line that saw it: the detail behind a WD_ERR_CUDA return.  Valid until the thread's
 * next failing call. */
WD_API const char* wd_last_error(void);

/* ---- context ------------------------------------------------------------ */

/* Build a context on the current CUDA device for the model whose forward pass the step runs
 * (Section 3.1: a bidirectional transformer; Section 4.1: the pretrained model is used without
 * architectural change, so `weights` are its matrices as they are).  Validates dims (head_dim even,
 * n_q_heads a multiple of n_kv_heads, bf16 needs d_model, d_ffn and
 * n_q_heads*head_dim to be multiples of 64, ...), borrows weights and
 * workspace, creates the TMA descriptors of the weights.
 * Errors: WD_ERR_NULL, WD_ERR_INVALID_DIMS, WD_ERR_WORKSPACE_TOO_SMALL,
 * WD_ERR_MISALIGNED, WD_ERR_UNSUPPORTED_ARCH, WD_ERR_CUDA. */
WD_API wd_status wd_create(const wd_model_dims* dims, const wd_weights* weights,
                    void* workspace /*device*/, size_t workspace_bytes, wd_ctx** out);
/* Frees host objects only. */
WD_API wd_status wd_destroy(wd_ctx* ctx);
/* Choose the GEMM kernel used by later steps (default WD_GEMM_AUTO). */
WD_API wd_status wd_set_gemm_impl(wd_ctx* ctx, int32_t impl);

/* Where the element-wise consumers of the projections run (the 1/rms scaling of the normalised
 * input, RoPE and the K/V cache write of Section 4.3, the residual adds, SwiGLU).  Every mode
 * computes the same step (Sections 3.1 and 4.3) within rounding; they differ in kernel structure only.
 *   WD_FUSION_AUTO     (default) the library's choice for the step's row count
 *   WD_FUSION_NONE     separate kernels after each GEMM (nine kernels per block)
 *   WD_FUSION_TILE     the GEMM CTA that completes an output tile finishes it (five kernels per block)
 *   WD_FUSION_CLUSTER  few rows (<= 128): the K slices of a tile are summed inside a thread-block
 *                      cluster through distributed shared memory and finished by the CTAs that own
 *                      the result; other row counts fall back to WD_FUSION_NONE
 *   WD_FUSION_CHAIN    few rows: the projections between two attention calls run as one persistent
 *                      kernel that never stops streaming weights; other row counts fall back
 * The fused modes need bf16, head_dim 128 and d_model, d_ffn multiples of 128 (else WD_FUSION_NONE).
 * Errors: WD_ERR_NULL, WD_ERR_BAD_PARAM. */
enum { WD_FUSION_AUTO = -1, WD_FUSION_NONE = 0, WD_FUSION_TILE = 1, WD_FUSION_CLUSTER = 2, WD_FUSION_CHAIN = 3 };
WD_API wd_status wd_set_fusion(wd_ctx* ctx, int32_t mode);

/* CUDA graphs for the kernels of a step (Section 4.3: the normal steps of a phase repeat the same
 * launch configuration).  On by default.  A step that the device plans (see wd_step) and whose launch
 * configuration — batch, computed rows, active rows, query tiles, key tiles, projection mode — recurs is
 * recorded into a graph (a normal step with full active windows at once, any other step the second time its
 * configuration occurs) and replayed
 * from then on (at most 8 graphs per context, least recently used replaced); the planner kernel and the
 * copy of the result block stay ordinary launches on the caller's stream.  Graphs need the tensor-core
 * kernels (bf16, head_dim 128) and are used only while earlier steps are still queued: a caller that calls
 * wd_step_sync after every step gets direct launches, which are faster then.  Steps with debug taps, with
 * profiling on, with a fused-consumer mode, planned on the host, or issued on a stream that is itself being
 * captured or that cannot be captured (the legacy default stream) are launched directly.  Results are
 * bit-identical either way.  wd_debug_graph_stats reports how many graphs were recorded and how many steps
 * were replayed since the context was created. */
WD_API wd_status wd_set_graphs(wd_ctx* ctx, int32_t on);
WD_API wd_status wd_debug_graph_stats(const wd_ctx* ctx, int32_t* captured, int32_t* replayed);

/* GEMM timing for benchmarks.  While enabled, wd_step brackets every GEMM launch
 * (one launch covers all weight matrices that share an input: q/k/v, gate/up)
 * with CUDA events on the step's stream and wd_step_sync adds up their device
 * time and their algorithmic bytes (weights once + activations in + result
 * out).  Enabling resets the totals.  Off by default; leave it off in runs
 * whose step time is reported. */
WD_API wd_status wd_profile_enable(wd_ctx* ctx, int32_t on);
WD_API wd_status wd_profile_read(const wd_ctx* ctx, double* gemm_ms, double* gemm_bytes, int64_t* gemm_launches);

/* ---- sequence state (Section 3.1: the fixed-length state x^(t)) ---------- */

/* token_ids: host [batch, seq_len].  decoded: host [batch, seq_len] of 0/1, or
 * NULL meaning decoded = (id != mask_id).  Decoded-ness is tracked by these
 * flags afterwards, never by comparing ids with mask_id.  state_mem is device
 * memory of wd_state_bytes(); its K/V cache part is set to zero here (the first
 * step is a refresh and writes every row whose value it uses, but the key tiles
 * of the tensor-core attention also cover far-field rows, masked, which must hold
 * finite numbers).  Copies ids to the device on the legacy default stream and
 * waits for it.
 * Errors: WD_ERR_NULL, WD_ERR_BAD_PARAM (batch/seq_len out of range),
 * WD_ERR_WORKSPACE_TOO_SMALL, WD_ERR_CUDA. */
WD_API wd_status wd_state_create(wd_ctx* ctx, int32_t batch, int32_t seq_len,
                          const int32_t* token_ids, const uint8_t* decoded,
                          void* state_mem /*device*/, size_t state_mem_bytes, wd_state** out);
/* Start over with new ids/flags (same batch and seq_len): step counter 0, next
 * step is a refresh.  The host->device copies of the ids and flags are enqueued on
 * `stream` from pinned staging buffers inside the state: the steps that follow must
 * be enqueued on the same stream (or be ordered after it by the caller), and a
 * second reset first waits until the previous reset's copies have left the staging
 * buffers.  Also clears WD_ERR_POISONED. */
WD_API wd_status wd_state_reset(wd_state* st, const int32_t* token_ids, const uint8_t* decoded,
                         void* stream /*cudaStream_t*/);
WD_API wd_status wd_state_destroy(wd_state* st);
/* Host mirror of one sequence: any of the outputs may be NULL.
 * token_ids/decoded/dec_step have seq_len entries; dec_step is the step at
 * which a token was unmasked, INT32_MIN for tokens that were given. */
WD_API wd_status wd_state_read(const wd_state* st, int32_t seq, int32_t* token_ids, uint8_t* decoded,
                        int32_t* dec_step, int32_t* step_index, int32_t* steps_since_refresh);
WD_API wd_status wd_debug_taps_set(wd_state* st, const wd_debug_taps* taps /*NULL = off*/);

/* Checkpoint / resume of the sequence state x^(t) of Section 3.1 with the phase bookkeeping of
 * Section 4.3 (token ids, decoded flags, decode steps, step index, steps since the last refresh,
 * the external window of the running phase, end-of-sequence id, refresh mode), as one flat host
 * blob of wd_state_export_bytes().  The K/V cache is not part of the blob: it lives in the
 * caller's own state memory (wd_kv_bytes() of it), which the caller may copy and restore itself.
 *   wd_state_import(st, blob, bytes, cache_valid, stream): `st` must have the blob's batch and
 *   seq_len.  cache_valid != 0: the caller has restored the state memory the blob was taken with,
 *   and the trajectory continues exactly where it stopped.  cache_valid == 0: the cache is taken
 *   as lost, the stored external window is dropped, and the next step is a refresh step, which
 *   rewrites every cache row it reads (Section 4.3); the phase clock restarts there (only for
 *   states in WD_REFRESH_FULL mode: the window-only variant's refresh does not rebuild the cache).  A resumed
 *   state is planned on the host (one wd_step_sync per wd_step).  Copies are enqueued on `stream`
 *   and waited for.  Clears WD_ERR_POISONED.
 * Errors: WD_ERR_NULL, WD_ERR_PENDING, WD_ERR_CAPACITY (export buffer too short), WD_ERR_BAD_PARAM
 * (foreign, damaged or mismatching blob: nothing is changed), WD_ERR_CUDA. */
WD_API size_t wd_state_export_bytes(const wd_state* st);
WD_API wd_status wd_state_export(const wd_state* st, void* blob /*host*/, size_t bytes);
WD_API wd_status wd_state_import(wd_state* st, const void* blob /*host*/, size_t bytes, int32_t cache_valid,
                          void* stream /*cudaStream_t*/);

/* Test hook for the device-side index checks: overwrites ONE entry of the DEVICE copy of the
 * token ids with `id`, unchecked, leaving the host mirror alone.  An id outside [0, vocab) makes
 * the next step's embedding kernel skip that row's gather and record WD_ERR_BOUNDS, which
 * wd_step_sync then reports (no fault: the bad index is never dereferenced). */
WD_API wd_status wd_debug_poke_id(wd_state* st, int32_t seq, int32_t pos, int32_t id, void* stream /*cudaStream_t*/);
/* Adaptive termination (Section 4.2, "Adaptive termination"): once a step has unmasked the
 * token `eos_id` at some position, undecoded positions after the first such position are never
 * activated again (they stay far-field and are ignored) and a sequence is done when nothing
 * undecoded is left before it.  An eos id that was part of the given tokens does not count.
 * eos_id < 0 switches it off (the default; the paper's main results also run with a fixed
 * length).  Kept across wd_state_reset.  Errors: WD_ERR_NULL, WD_ERR_PENDING, WD_ERR_BAD_PARAM. */
WD_API wd_status wd_state_set_eos(wd_state* st, int32_t eos_id);
/* What the refresh steps of this state compute: WD_REFRESH_FULL (default, the paper's refresh)
 * or WD_REFRESH_WINDOW (the variant described at the enum; no counterpart in the paper).
 * Kept across wd_state_reset.  Errors: WD_ERR_NULL, WD_ERR_PENDING, WD_ERR_BAD_PARAM. */
WD_API wd_status wd_state_set_refresh_mode(wd_state* st, int32_t mode);
/* Staggered refresh steps for a batch (no counterpart in the paper, which describes one sequence:
 * Section 4.3 gives every phase one refresh step followed by normal steps, and with one phase clock
 * per batch all sequences would run their compute-heavy refresh step in the same call).  With
 * on != 0, sequence i of a batch of n shifts its phase clock by o = i * R / n steps (integer
 * division): every sequence still refreshes at its first step (nothing is cached yet), a sequence
 * with 0 < o < R refreshes again at step o, which makes its first phase o steps long, and all
 * later phases have R steps.  Every phase is a phase of Section 4.3; only where the phases of
 * different sequences begin differs, so that each call of wd_step carries about n / R refresh
 * steps and the step time is flat.  Off by default.  Kept across wd_state_reset.
 * Errors: WD_ERR_NULL, WD_ERR_PENDING. */
WD_API wd_status wd_state_set_stagger(wd_state* st, int32_t on);

/* ---- FP8 mode (no counterpart in the paper, which calls quantisation orthogonal to the method) ----
 * The projections q/k/v, gate/up, down and the LM head then take both operands in 8-bit floating
 * point e4m3: every weight row once (wd_fp8_enable) and every activation row at every step is
 * divided by its own scale s = max|row| / 448 (1 for a zero row), rounded to the nearest e4m3
 * value (ties to even), multiplied on the tensor cores (tcgen05 kind::f8f6f4, fp32 accumulation)
 * and scaled back by the two row scales.  The output projection, attention, the residual stream
 * and the K/V cache stay as they are.  Halves the weight bytes a normal step streams; changes the
 * numbers (relative error of a projection about 3-4 %).  bf16 models on the tensor-core path only.
 *   wd_fp8_bytes   size of the device memory block wd_fp8_enable needs (0 for invalid dims / fp32)
 *   wd_fp8_enable  quantises the weights on `stream` into `mem` (caller-owned, 256-byte aligned,
 *                  must outlive the context) and switches the mode on for later steps.
 *                  d_model and d_ffn must be multiples of 16, d_ffn <= 32768.
 *   wd_fp8_set     switches the mode off / on again (on needs a prior wd_fp8_enable).
 * Errors: WD_ERR_NULL, WD_ERR_BAD_PARAM, WD_ERR_MISALIGNED, WD_ERR_WORKSPACE_TOO_SMALL, WD_ERR_CUDA. */
WD_API size_t wd_fp8_bytes(const wd_model_dims* dims);
WD_API wd_status wd_fp8_enable(wd_ctx* ctx, void* mem, size_t mem_bytes, void* stream /*cudaStream_t*/);
WD_API wd_status wd_fp8_set(wd_ctx* ctx, int32_t on);

/* NVFP4 mode (outside the paper, which calls quantisation orthogonal to its method; bf16 models with
 * d_model and d_ffn multiples of 256).  The same projections as in the FP8 mode (q/k/v, gate/up, down and
 * the LM head; the attention output projection stays bf16) take both operands in the NVFP4 format:
 * 4-bit e2m1 elements, one unsigned e4m3 scale per block of 16 elements along the inner dimension,
 * one float scale per row (row maximum / (6 * 448)).  Every weight row is quantised once
 * (wd_fp4_enable), every activation row (the bf16 output of the RMSNorm / SwiGLU kernels) at every
 * step; the product runs on the block-scaled tensor-core path with fp32 accumulation.  The two quantised
 * modes exclude each other: enabling one switches the other off.
 *   wd_fp4_bytes   size of the device memory block wd_fp4_enable needs (0 for invalid dims)
 *   wd_fp4_enable  quantises the weights on `stream` into `mem` (caller-owned, 256-byte aligned, must
 *                  outlive the context's use of the mode) and switches the mode on
 *   wd_fp4_set     switches the mode off / on again (on needs a prior wd_fp4_enable).
 * Errors: WD_ERR_NULL, WD_ERR_BAD_PARAM (dtype or widths), WD_ERR_MISALIGNED, WD_ERR_WORKSPACE_TOO_SMALL. */
WD_API size_t wd_fp4_bytes(const wd_model_dims* dims);
WD_API wd_status wd_fp4_enable(wd_ctx* ctx, void* mem, size_t mem_bytes, void* stream /*cudaStream_t*/);
WD_API wd_status wd_fp4_set(wd_ctx* ctx, int32_t on);

/* ---- the step ----------------------------------------------------------- */

/* Preview of the index sets the next wd_step(st, A, B, R, T, ...) will use for
 * sequence `seq`.  Pure host function, no GPU work, does not change the state.
 *   A  size of the internal (active) window, >= 1
 *   B  number of buffer tokens: the external window holds A+B undecoded tokens
 *   R  phase length in steps: 1 refresh + (R-1) normal steps, >= 1
 *   T  a token unmasked at step s is recomputed at steps s+1..s+T of the same
 *      phase (the post-decode transient of Section 4.3), >= 0
 * Errors: WD_ERR_NULL, WD_ERR_BAD_PARAM, WD_ERR_CAPACITY. */
WD_API wd_status wd_plan(const wd_state* st, int32_t seq, int32_t A, int32_t B, int32_t R, int32_t T,
                  wd_index_sets* out);

/* The same planner on explicit state arrays (no wd_state, no GPU, usable in a
 * process without a CUDA device): decoded[seq_len] 0/1 flags, dec_step[seq_len]
 * (step at which a token was unmasked, INT32_MIN if it was given), token_ids and
 * eos_id for adaptive termination (see wd_state_set_eos; token_ids may be NULL
 * when eos_id < 0), step_index t, steps_since_refresh, and the external window
 * stored at the last refresh (ext_window[n_ext_window], ascending; empty before
 * the first step), refresh_mode (WD_REFRESH_FULL or WD_REFRESH_WINDOW), and the staggered-refresh
 * identity of the sequence (stagger_i of stagger_n, see wd_state_set_stagger; stagger_n = 0: off).
 * Errors: as wd_plan, plus WD_ERR_BAD_PARAM for an index outside the sequence. */
WD_API wd_status wd_plan_raw(const uint8_t* decoded, const int32_t* dec_step, const int32_t* token_ids,
                             int32_t eos_id, int32_t seq_len, int32_t step_index,
                             int32_t steps_since_refresh, const int32_t* ext_window, int32_t n_ext_window,
                             int32_t A, int32_t B, int32_t R, int32_t T, int32_t refresh_mode,
                             int32_t stagger_i, int32_t stagger_n, wd_index_sets* out);

/* Enqueue one step for every sequence of the state on `stream` and return
 * without waiting.  k = tokens unmasked per sequence (at most the number of
 * active tokens; 0 = compute only).  Needs max_active >= batch * A.  `info` may
 * be NULL.
 *
 * Steps may be enqueued back to back, up to 32 without a wd_step_sync in
 * between, while the device can plan them itself: every sequence started from
 * a decoded prefix (prompt then masks), at most 16 sequences, adaptive
 * termination and GEMM profiling off.  A device kernel then builds the index
 * lists from the device copy of the state (the sets of Section 4.2 and the
 * phase structure of Section 4.3, the same planner as wd_plan, bit for bit) and
 * the host only supplies counts, which do not depend on which tokens were
 * unmasked.  Otherwise (arbitrary decoded patterns, adaptive termination) the
 * host plans each step and wd_step_sync must come before the next wd_step.
 * wd_plan, wd_state_read, wd_state_reset and the setters need an empty queue.
 * Returns WD_OK, WD_DONE (nothing left to decode: nothing enqueued),
 * WD_ERR_PENDING (queue full, or this state needs a sync between steps),
 * WD_ERR_BAD_PARAM, WD_ERR_CAPACITY (a dims.max_* limit), WD_ERR_INTERNAL,
 * WD_ERR_CUDA. */
WD_API wd_status wd_step(wd_state* st, int32_t A, int32_t B, int32_t R, int32_t T, int32_t k,
                  void* stream /*cudaStream_t*/, wd_step_info* info);

/* Wait for every enqueued step, read the results and the device status word,
 * apply the update sets U^(t) (Section 3.1: the few positions a step changes) to the
 * host mirror of the state in order and advance the phase counters (Section 4.3:
 * steps since the refresh that opened the phase).  `out` (host, may be NULL)
 * receives the result of the NEWEST step.  Returns WD_OK, WD_ERR_NOT_PENDING,
 * WD_ERR_DEVICE_TIMEOUT, WD_ERR_BOUNDS, WD_ERR_INTERNAL, WD_ERR_CUDA.
 * After WD_ERR_DEVICE_TIMEOUT or WD_ERR_BOUNDS the steps up to the failing one are
 * committed, the rest of the queue is dropped, and, because queued steps behind the
 * failing one have already run on the device, the state is marked inconsistent:
 * wd_step, wd_plan and wd_generate return WD_ERR_POISONED until wd_state_reset or
 * wd_state_import.  The context and other states stay usable. */
WD_API wd_status wd_step_sync(wd_state* st, wd_step_out* out);

/* The same, returning every enqueued step's result: outs[0] is the oldest.
 * `capacity` = entries of outs (0 with outs NULL just commits); WD_ERR_CAPACITY
 * if more steps are pending (nothing is consumed then).  *n_steps (may be NULL)
 * = steps completed. */
WD_API wd_status wd_step_sync_all(wd_state* st, wd_step_out* outs, int32_t capacity, int32_t* n_steps);

/* Whole-generation driver: the decoding loop of Section 4 (repeat windowed
 * denoising steps, a refresh step opening every phase, until no masked position
 * is left inside the reach of the window) run by the library.  Steps are enqueued
 * back to back on `stream` and drained in groups, so the host only waits when
 * the queue is full; a state that needs a host plan per step (see wd_step) is
 * stepped and synchronised one step at a time instead.  Stops when wd_step
 * reports WD_DONE (with adaptive termination: once the end-of-sequence token is
 * out and nothing before it is masked) or after max_steps steps (max_steps <= 0:
 * no limit).  On return the queue is empty and the host mirror is current
 * (wd_state_read gives the tokens).  *n_steps (may be NULL) = steps run,
 * *n_tokens (may be NULL) = tokens unmasked over all sequences.  Needs an empty
 * queue (WD_ERR_PENDING).  Returns WD_DONE when generation finished, WD_OK when
 * max_steps stopped it, else the first error of wd_step / wd_step_sync. */
WD_API wd_status wd_generate(wd_state* st, int32_t A, int32_t B, int32_t R, int32_t T, int32_t k,
                      int32_t max_steps, void* stream /*cudaStream_t*/, int32_t* n_steps, int32_t* n_tokens);

/* ---- single operations (unit parity tests, micro-benchmarks) -------------- */

/* y[rows, n_out] (float, device) = x[rows, k_in] * w[n_out, k_in]^T, x and w of
 * `dtype`, fp32 accumulation.  `scratch` (device, scratch_bytes) holds split-K
 * partial sums for WD_GEMM_TCGEN05 (wd_op_gemm_scratch_bytes); unused for
 * WD_GEMM_PLAIN.  Section 3.1's transformer forward is made of these.
 * Errors: WD_ERR_NULL, WD_ERR_BAD_PARAM, WD_ERR_WORKSPACE_TOO_SMALL, WD_ERR_CUDA,
 * WD_ERR_DEVICE_TIMEOUT (only after the caller synchronises: see wd_op_status). */
WD_API wd_status wd_op_gemm(int32_t dtype, int32_t impl, const void* x, const void* w, float* y,
                     int32_t rows, int32_t n_out, int32_t k_in,
                     void* scratch, size_t scratch_bytes, void* stream);
WD_API size_t wd_op_gemm_scratch_bytes(int32_t rows, int32_t n_out, int32_t k_in);

/* The FP8 projection of the FP8 mode as a single operation (see wd_fp8_enable): both bf16
 * operands are quantised row by row to e4m3 (scale = max|row| / 448) into `scratch`, multiplied
 * on the tensor cores and scaled back; y[rows, n_out] float.  k_in a multiple of 16; scratch
 * 256-byte aligned, wd_op_gemm_fp8_scratch_bytes large.  Errors as wd_op_gemm. */
WD_API wd_status wd_op_gemm_fp8(const void* x, const void* w, float* y, int32_t rows, int32_t n_out, int32_t k_in,
                         void* scratch, size_t scratch_bytes, void* stream /*cudaStream_t*/);
WD_API size_t wd_op_gemm_fp8_scratch_bytes(int32_t rows, int32_t n_out, int32_t k_in);

/* The NVFP4 projection of the NVFP4 mode as a single operation (see wd_fp4_enable; no counterpart in the
 * paper): both bf16 operands are quantised into `scratch` (4-bit e2m1 codes, one unsigned e4m3 scale per
 * block of 16 elements along k, one float scale per row), multiplied on the block-scaled tensor-core
 * path (tcgen05 kind::mxf4nvf4, block scales applied by the hardware from tensor memory, fp32
 * accumulation) and scaled back by the row scales; y[rows, n_out] float.  k_in a multiple of 256;
 * scratch 256-byte aligned, wd_op_gemm_fp4_scratch_bytes large.  Errors as wd_op_gemm. */
WD_API wd_status wd_op_gemm_fp4(const void* x, const void* w, float* y, int32_t rows, int32_t n_out, int32_t k_in,
                         void* scratch, size_t scratch_bytes, void* stream /*cudaStream_t*/);
WD_API size_t wd_op_gemm_fp4_scratch_bytes(int32_t rows, int32_t n_out, int32_t k_in);

/* The two halves of wd_op_gemm_fp4 for callers that quantise an operand once and multiply it many times
 * (no counterpart in the paper).  wd_op_nvfp4_quantize writes the NVFP4 form of the bf16 matrix
 * x[rows, k_in] (k_in a multiple of 16) into `out` (device, 256-byte aligned, wd_op_nvfp4_bytes large:
 * codes [rows][k_in / 2], then block scales [rows][k_in / 16], then float row scales [rows], each part
 * starting on a 256-byte boundary).  wd_op_gemm_nvfp4 multiplies two such operands: y[rows, n_out] float;
 * k_in a multiple of 256; scratch 256-byte aligned, wd_op_gemm_scratch_bytes(rows, n_out, k_in) large.
 * Errors as wd_op_gemm. */
WD_API size_t wd_op_nvfp4_bytes(int32_t rows, int32_t k_in);
WD_API wd_status wd_op_nvfp4_quantize(const void* x, int32_t rows, int32_t k_in, void* out, size_t out_bytes,
                               void* stream /*cudaStream_t*/);
WD_API wd_status wd_op_gemm_nvfp4(const void* xq, const void* wq, float* y, int32_t rows, int32_t n_out, int32_t k_in,
                           void* scratch, size_t scratch_bytes, void* stream /*cudaStream_t*/);

/* (No counterpart in the paper: a packaging variant of wd_op_gemm.)
 * The same bf16 tensor-core GEMM, y[rows, n_out] (float) = x[rows, k_in] * w[n_out, k_in]^T,
 * for callers that cannot hand over scratch memory because they may not allocate
 * where they call from: code living inside another framework's memory pool, a
 * serving loop that bans allocator calls once it is running, a process whose device
 * memory is already fully committed.  The split-K partial sums go to a fixed
 * 16 MiB array that is part of the library image (wd_op_gemm_noalloc_max_floats()
 * floats; each GPU that loads the library keeps it until the process exits).  This
 * call allocates nothing, on the host or on the device (the operands' TMA descriptors
 * are built on the stack).
 *   - Limit: rows * n_out must not exceed wd_op_gemm_noalloc_max_floats(), otherwise
 *     WD_ERR_CAPACITY and nothing is launched.  Fewer K slices are used when the
 *     array cannot hold more, so large shapes run slower than with wd_op_gemm.
 *   - The first call on each device does the set-up for that device, with that device
 *     current: it looks up the device addresses of the array and of the operations'
 *     status word and sets the kernels' shared-memory limit, and remembers all three
 *     per device.  Make that first call before any stream capture begins.
 *   - All calls share the one array and it keeps whatever the last call left in it.
 *     Nothing needs clearing (every partial sum that is read is written first by
 *     the same call), but two calls that overlap on the GPU, e.g. on different
 *     streams, race on it: keep calls on one stream or order them with events.
 * Pointers are device pointers; x, w bf16 row-major with k_in contiguous, 16-byte
 * aligned, k_in a multiple of 8.  Errors: WD_ERR_NULL, WD_ERR_BAD_PARAM,
 * WD_ERR_CAPACITY, WD_ERR_MISALIGNED, WD_ERR_CUDA; a device-side time-out is
 * reported by wd_op_status(). */
WD_API wd_status wd_op_gemm_noalloc(const void* x, const void* w, float* y, int32_t rows, int32_t n_out,
                                    int32_t k_in, void* stream);
WD_API size_t wd_op_gemm_noalloc_max_floats(void);

/* Bidirectional grouped-query attention (Section 3.1: no causal mask) of
 * n_rows query rows over n_vis cached positions of one sequence:
 * out[r, h, :] = softmax_j(q[r,h,:] . K[kvh(h), vis[j], :] / sqrt(head_dim)) V[kvh(h), vis[j], :].
 * q, out: [n_rows, n_q_heads, head_dim]; kcache: [n_kv_heads, seq_len, head_dim];
 * vcache TRANSPOSED: [n_kv_heads, head_dim, seq_len] (the layout the step keeps V in, so
 * that V tiles are read with the key position contiguous); vis: device int32 [n_vis];
 * all of `dtype`. */
WD_API wd_status wd_op_attention(int32_t dtype, const void* q, const void* kcache, const void* vcache,
                          const int32_t* vis, void* out, int32_t n_rows, int32_t n_vis,
                          int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int32_t seq_len,
                          void* stream);

/* The same attention (Section 3.1, no causal mask) through the tensor-core kernel the step uses when
 * the visible set of a sequence is a range: n_rows query rows of one sequence over the cached
 * positions [0, n_vis), bf16, head_dim 128.  q, out: [n_rows, n_q_heads, 128] bf16; kcache:
 * [n_kv_heads, seq_len, 128]; vcache_t TRANSPOSED: [n_kv_heads, 128, seq_len], seq_len a multiple
 * of 8; rows of the caches at or beyond n_vis are never used as values (they may hold anything,
 * NaN included).  max_vis >= n_vis sizes the split of the keys over the CTAs of a thread-block
 * cluster exactly as the step does for its longest sequence (max_vis = n_vis: this sequence is the
 * longest; larger: some CTAs of a cluster get no key tile, as for the shorter sequences of a
 * batch).  scratch: device, 4-byte aligned, wd_op_attention_tc_scratch_bytes(n_rows) (the query-tile
 * lists, written by a small kernel on `stream`).  All pointers device, 16-byte aligned.
 * Errors: WD_ERR_NULL, WD_ERR_BAD_PARAM, WD_ERR_MISALIGNED, WD_ERR_WORKSPACE_TOO_SMALL, WD_ERR_CUDA;
 * a device-side time-out is reported by wd_op_status(). */
WD_API wd_status wd_op_attention_tc(const void* q, const void* kcache, const void* vcache_t, void* out,
                             int32_t n_rows, int32_t n_vis, int32_t max_vis, int32_t n_q_heads,
                             int32_t n_kv_heads, int32_t seq_len, void* scratch, size_t scratch_bytes,
                             void* stream /*cudaStream_t*/);
WD_API size_t wd_op_attention_tc_scratch_bytes(int32_t n_rows);

/* The unmask rule on given logits (device float [n, vocab]) of one sequence:
 * token = lowest index of the maximal logit, confidence = its softmax
 * probability; the min(k, n) rows of highest confidence are returned (equal
 * confidence: lowest position).  positions: device int32 [n] ascending.
 * Outputs are device arrays: row_token[n], row_sumexp[n] (sum_v exp(logit_v - max)
 * accumulated in double, the reciprocal of the confidence and the ranking key),
 * row_conf[n], sel_pos[k], sel_token[k], sel_conf[k], n_sel[1]; none may overlap. */
WD_API wd_status wd_op_unmask(const float* logits, const int32_t* positions, int32_t n, int32_t vocab,
                       int32_t k, int32_t* row_token, double* row_sumexp, float* row_conf,
                       int32_t* sel_pos, int32_t* sel_token, float* sel_conf, int32_t* n_sel,
                       void* scratch, size_t scratch_bytes, void* stream);
/* Device scratch the unmask operation needs (per-chunk partial statistics), 8-byte aligned. */
WD_API size_t wd_op_unmask_scratch_bytes(int32_t n, int32_t vocab);

/* Logits and the unmask rule in one pass, as the step does it for its active rows (Section 4.1:
 * logits only for the active tokens, decoding decided by prediction confidence): logits[n, vocab]
 * (float) = x[n, k_in] * w[vocab, k_in]^T on the tensor cores (x = the normalised active rows, w =
 * the LM head, both bf16, k_in a multiple of 8), whose epilogue reduces every CTA's logits to
 * per-row (maximum, lowest index of the maximum, sum of exp(logit - maximum) in double); a second
 * kernel merges the CTAs' entries of a row in a fixed order and ranks the rows.  Same outputs and
 * tie rules as wd_op_unmask; `logits` (device, required) also receives the logits themselves, so
 * that a test can hand the very same numbers to another implementation of the rule.  n <= 1024.
 * scratch: device, 8-byte aligned, wd_op_lm_unmask_scratch_bytes(n, vocab).
 * Errors: WD_ERR_NULL, WD_ERR_BAD_PARAM, WD_ERR_CAPACITY (n), WD_ERR_MISALIGNED,
 * WD_ERR_WORKSPACE_TOO_SMALL, WD_ERR_CUDA; device-side time-outs through wd_op_status(). */
WD_API wd_status wd_op_lm_unmask(const void* x, const void* w, const int32_t* positions, int32_t n, int32_t vocab,
                          int32_t k_in, int32_t k, float* logits, int32_t* row_token, double* row_sumexp,
                          float* row_conf, int32_t* sel_pos, int32_t* sel_token, float* sel_conf, int32_t* n_sel,
                          void* scratch, size_t scratch_bytes, void* stream /*cudaStream_t*/);
WD_API size_t wd_op_lm_unmask_scratch_bytes(int32_t n, int32_t vocab);

/* Device status word shared by the single operations: 0, or the first
 * WD_ERR_DEVICE_TIMEOUT / WD_ERR_BOUNDS raised by a kernel since the last
 * call.  Synchronises the device. */
WD_API wd_status wd_op_status(void);

/* Exercises the library's error path for device-side waits without any fault: one
 * thread waits, with the same bounded wait every kernel of the library uses, on a
 * shared-memory barrier that nothing ever signals.  The wait gives up after its
 * time limit (two seconds), the kernel records
 * WD_ERR_DEVICE_TIMEOUT in the operations' status word and returns normally; the
 * context stays usable.  wd_op_status() then reports and clears the code.
 * `stream`: a CUDA stream handle or NULL.  Errors: WD_ERR_CUDA. */
WD_API wd_status wd_debug_wait_expire(void* stream);

#ifdef __cplusplus
}
#endif
#endif /* WD_H */
