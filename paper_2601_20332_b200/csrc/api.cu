// C ABI of libwd.so: context, sequence state, the step driver and the single
// operations.  Host code; every step of the path runs in the kernels it launches.
#include <algorithm>
#include <climits>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "wd_internal.h"
#include "gemm_tc.h"
#include "attention_tc.h"

// ---------------------------------------------------------------------------
// error bookkeeping
// ---------------------------------------------------------------------------
static thread_local char g_last_cuda_error[256];

void wd_note_cuda_error(cudaError_t e, const char* file, int line) {
    snprintf(g_last_cuda_error, sizeof(g_last_cuda_error), "%s at %s:%d", cudaGetErrorString(e), file, line);
    cudaGetLastError();   // clear the sticky-less error so later calls report their own
}

extern "C" const char* wd_status_string(wd_status s) {
    switch (s) {
        case WD_OK: return "ok";
        case WD_DONE: return "done: no undecoded token left";
        case WD_ERR_NULL: return "null pointer";
        case WD_ERR_INVALID_DIMS: return "invalid model dims";
        case WD_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case WD_ERR_UNSUPPORTED_ARCH: return "device is not sm_100";
        case WD_ERR_BAD_PARAM: return "bad parameter";
        case WD_ERR_CAPACITY: return "capacity exceeded";
        case WD_ERR_PENDING: return "a step is pending: call wd_step_sync first";
        case WD_ERR_CUDA: return g_last_cuda_error[0] ? g_last_cuda_error : "CUDA error";
        case WD_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
        case WD_ERR_BOUNDS: return "a device-side index check failed";
        case WD_ERR_NOT_PENDING: return "no step pending";
        case WD_ERR_MISALIGNED: return "device pointer not 256-byte aligned";
        case WD_ERR_INTERNAL: return "internal inconsistency between the host and device planners";
        case WD_ERR_POISONED: return "a device-side error left the state inconsistent: reset or import it first";
        default: return "unknown status";
    }
}

extern "C" const char* wd_last_error(void) { return g_last_cuda_error; }

extern "C" int32_t wd_version(void) { return 200; }

// ---------------------------------------------------------------------------
// context
// ---------------------------------------------------------------------------
struct wd_ctx {
    wd_model_dims d;
    const void* tok_embed;
    const void* lm_head;
    const float* final_norm;
    std::vector<const void*> wq, wk, wv, wo, wg, wu, wd;
    std::vector<const float*> attn_norm, ffn_norm;
    int gemm_impl = WD_GEMM_AUTO;
    int attn_impl = WD_GEMM_AUTO;   // WD_GEMM_PLAIN forces the CUDA-core attention
    int sm_count = 148;

    // CUDA graphs of the kernels of a step (wd_set_graphs): a device-planned step whose launch
    // configuration (StepKey) has been seen before is captured once and replayed afterwards
    struct StepKey {
        uint64_t state_uid = 0;
        int batch = 0, rows = 0, n_act = 0, n_qtiles = 0, key_tiles = 0, max_tile_rows = 0, k_eff = 0, mode = 0, impl = 0, attn_impl = 0;
        bool operator==(const StepKey& o) const {
            return state_uid == o.state_uid && batch == o.batch && rows == o.rows && n_act == o.n_act && n_qtiles == o.n_qtiles &&
                   key_tiles == o.key_tiles && max_tile_rows == o.max_tile_rows && k_eff == o.k_eff && mode == o.mode &&
                   impl == o.impl && attn_impl == o.attn_impl;
        }
    };
    struct StepGraph { StepKey key; cudaGraphExec_t exec = nullptr; int n_kernels = 0, impl_used = 0; uint64_t last_use = 0; };
    bool graphs_on = true;
    std::vector<StepGraph> graphs;      // at most kMaxGraphs, least recently used replaced
    std::vector<StepKey> seen;          // configurations met once (capture pays from the second time on)
    uint64_t graph_clock = 0;
    int graphs_captured = 0, graphs_replayed = 0, graph_failures = 0;

    // workspace carve-up (device)
    float* x = nullptr;          // [max_rows, d] residual stream
    void* xn = nullptr;          // [max_rows, d] normalised rows (model dtype)
    void* q = nullptr;           // [max_rows, Hq*dh]
    void* attn = nullptr;        // [max_rows, Hq*dh]
    void* h = nullptr;           // [max_rows, F]
    float* part = nullptr;       // split-K partial sums / GEMM outputs
    size_t part_floats = 0;
    float* logits = nullptr;     // [max_active, V]
    int32_t* row_token = nullptr;
    double* row_sumexp = nullptr;
    float* row_conf = nullptr;
    float* ch_max = nullptr;     // [max_active][chunks] unmask stage-1 statistics
    int32_t* ch_idx = nullptr;
    double* ch_sum = nullptr;
    float2* rope_tab = nullptr;  // [max_rows][dh/2] (cos, sin) of this step's rows
    float* sumsq = nullptr;      // [d/128][max_rows] partial sums of squares of the residual rows
    int32_t* tile_counters = nullptr;  // arrival counters of the fused GEMM epilogues (kept zero)
    size_t n_tile_counters = 0;
    int fuse = WD_FUSION_AUTO;   // where the consumers of the GEMMs run (wd_set_fusion)
    int32_t* plan = nullptr;     // packed index lists of the step
    size_t plan_ints = 0;
    int32_t* result = nullptr;   // [status | n_sel[batch] | pos | tok | conf]
    size_t result_ints = 0;

    WdTcWeights tc;              // tensor maps of the weights (bf16 only)
    WdTcChainState chain;        // counters of the chain kernel (WD_FUSION_CHAIN)
    bool chain_dirty = false;    // a device-side error may have left them out of step: zero them before the next launch

    // FP8 mode (wd_fp8_enable): e4m3 copies of q/k/v, gate/up, down and the LM head with one scale
    // per weight row, FP8 activation buffers with one scale per row, and their tensor maps
    bool fp8_ready = false, fp8_on = false;
    struct Fp8Mat { const uint8_t* q = nullptr; const float* s = nullptr; CUtensorMap map; };
    std::vector<Fp8Mat> f8q, f8k, f8v, f8g, f8u, f8d;
    Fp8Mat f8lm;
    uint8_t* xn8 = nullptr;      // [max_rows, d]
    uint8_t* h8 = nullptr;       // [max_rows, F]
    float* sxn = nullptr;        // [max_rows]
    float* sh = nullptr;         // [max_rows]
    WdTcX x8_d, x8_h;
    // NVFP4 mode (wd_fp4_enable): the same projections with e2m1 codes, e4m3 block scales and float row scales;
    // q/k/v and gate/up are one operand each (their rows one after the other)
    bool fp4_ready = false, fp4_on = false;
    std::vector<WdFp4Operand> f4qkv, f4gu, f4d;
    WdFp4Operand f4lm;
    void* fp4_x = nullptr;       // the step's quantised activations: max_rows x max(d, d_ffn)

    // optional GEMM timing (benchmarks): event pairs around every GEMM launch of a step
    bool prof_on = false;
    std::vector<cudaEvent_t> prof_events;
    size_t prof_used = 0;
    double prof_step_bytes = 0.0, prof_ms = 0.0, prof_bytes = 0.0;
    long long prof_launches = 0;
    ~wd_ctx() {
        for (cudaEvent_t e : prof_events) cudaEventDestroy(e);
        for (StepGraph& g : graphs) if (g.exec) cudaGraphExecDestroy(g.exec);
    }
};

static bool dims_valid(const wd_model_dims* d) {
    if (!d) return false;
    if (d->n_layers < 1 || d->d_model < 1 || d->n_q_heads < 1 || d->n_kv_heads < 1 || d->head_dim < 2 ||
        d->d_ffn < 1 || d->vocab < 2)
        return false;
    if (d->head_dim % 2 || d->n_q_heads % d->n_kv_heads) return false;
    if (d->dtype != WD_F32 && d->dtype != WD_BF16) return false;
    if (d->mask_id < 0 || d->mask_id >= d->vocab) return false;
    if (d->max_batch < 1 || d->max_seq < 1 || d->max_rows < 1 || d->max_active < 1) return false;
    if ((int64_t)d->max_rows > (int64_t)d->max_batch * d->max_seq) return false;
    if (d->max_active > d->max_rows) return false;
    if (!(d->rope_theta > 1.f) || !(d->rms_eps >= 0.f)) return false;
    if (d->d_model % 4 || d->d_ffn % 4 || d->d_model > 32768) return false;   // float4 paths
    if (d->dtype == WD_BF16) {
        // TMA tiles are 64 elements (128 bytes) along the reduction dimension
        if (d->d_model % 64 || d->d_ffn % 64 || (d->n_q_heads * d->head_dim) % 64) return false;
    }
    return true;
}

struct Carve {
    size_t off = 0;
    size_t take(size_t bytes) { size_t o = off; off = wd_align_up(off + bytes, 256); return o; }
};

static size_t max_gemm_cols(const wd_model_dims* d) {
    const size_t qkv = (size_t)(d->n_q_heads + 2 * d->n_kv_heads) * d->head_dim;
    return std::max({qkv, (size_t)d->d_model, (size_t)2 * d->d_ffn});
}

// partial-sum buffer: split-K is only used while rows are few
static size_t part_floats_for(const wd_model_dims* d) {
    const size_t cols = max_gemm_cols(d);
    const size_t small_rows = std::min<size_t>(d->max_rows, WD_TC_SPLITK_MAX_ROWS);
    return std::max((size_t)d->max_rows * cols, (size_t)WD_TC_MAX_SPLIT * small_rows * cols);
}

static void carve_ctx(const wd_model_dims* d, Carve& c, size_t off[24]) {
    const size_t e = wd_elt_size(d->dtype);
    const size_t MR = d->max_rows, MA = d->max_active, hq = (size_t)d->n_q_heads * d->head_dim;
    off[0] = c.take(MR * d->d_model * 4);                       // x
    off[1] = c.take(MR * d->d_model * e);                       // xn
    off[2] = c.take(MR * hq * e);                               // q
    off[3] = c.take(MR * hq * e);                               // attn
    off[4] = c.take(MR * d->d_ffn * e);                         // h
    off[5] = c.take(part_floats_for(d) * 4);                    // part
    off[6] = c.take(MA * d->vocab * 4);                         // logits
    off[7] = c.take(MA * 4);                                    // row_token
    off[8] = c.take(MA * 8);                                    // row_sumexp
    off[9] = c.take(MA * 4);                                    // row_conf
    const size_t plan_ints = 2 * MR + 2 * MA + 2 * ((size_t)d->max_batch + 1) + (size_t)d->max_batch * d->max_seq +
                             3 * (MR / 128 + (size_t)d->max_batch + 1) + 2 * (size_t)d->max_batch +
                             (size_t)d->max_batch * d->max_seq;      // + staging of the external windows
    off[10] = c.take(plan_ints * 4);                            // plan
    off[11] = c.take((1 + (size_t)d->max_batch + 3 * MA) * 4);  // result
    off[12] = plan_ints;
    // unmask statistics: per vocabulary chunk (CUDA-core path) or per 128-logit GEMM tile (LM-head epilogue)
    const size_t nch = std::max<size_t>((size_t)wd_unmask_chunks(d->vocab), 256);   // or one per CTA of the LM head
    off[13] = c.take(MA * nch * 4);                             // ch_max
    off[14] = c.take(MA * nch * 4);                             // ch_idx
    off[15] = c.take(MA * nch * 8);                             // ch_sum
    off[16] = c.take(MR * (size_t)(d->head_dim / 2) * 8);       // rope_tab
    off[17] = c.take(((size_t)d->d_model / 128 + 1) * MR * 4);  // sumsq
    off[18] = c.take(((max_gemm_cols(d) + 127) / 128) * (MR / 256 + 2) * 4);   // tile counters
    off[19] = ((max_gemm_cols(d) + 127) / 128) * (MR / 256 + 2);
    off[20] = c.take(256);                                       // chain kernel counters
    off[21] = c.off;
}

extern "C" size_t wd_workspace_bytes(const wd_model_dims* dims) {
    if (!dims_valid(dims)) return 0;
    Carve c;
    size_t off[24];
    carve_ctx(dims, c, off);
    return c.off;
}

// the transposed V cache keeps the position contiguous; rows padded to 16 bytes for TMA
static inline int seq_pad(int S) { return (S + 7) / 8 * 8; }

extern "C" size_t wd_state_bytes(const wd_model_dims* d, int32_t batch, int32_t seq_len) {
    if (!dims_valid(d) || batch < 1 || seq_len < 1 || batch > d->max_batch || seq_len > d->max_seq) return 0;
    const size_t k = (size_t)d->n_layers * batch * d->n_kv_heads * seq_len * d->head_dim * wd_elt_size(d->dtype);
    const size_t v = (size_t)d->n_layers * batch * d->n_kv_heads * seq_pad(seq_len) * d->head_dim * wd_elt_size(d->dtype);
    const size_t plan_state = wd_align_up((size_t)batch * seq_len, 256) + 2 * wd_align_up((size_t)batch * seq_len * 4, 256);
    return wd_align_up((size_t)batch * seq_len * 4, 256) + wd_align_up(k, 256) + wd_align_up(v, 256) + plan_state;
}

extern "C" size_t wd_kv_bytes(const wd_model_dims* d, int32_t batch, int32_t seq_len) {
    if (!dims_valid(d) || batch < 1 || seq_len < 1 || batch > d->max_batch || seq_len > d->max_seq) return 0;
    const size_t per = (size_t)d->n_layers * batch * d->n_kv_heads * d->head_dim * wd_elt_size(d->dtype);
    return per * seq_len + per * seq_pad(seq_len);      // K rows + transposed V rows (positions padded to 8)
}

extern "C" wd_status wd_create(const wd_model_dims* dims, const wd_weights* w, void* workspace,
                               size_t workspace_bytes, wd_ctx** out) {
    if (!dims || !w || !workspace || !out) return WD_ERR_NULL;
    *out = nullptr;
    if (!dims_valid(dims)) return WD_ERR_INVALID_DIMS;
    if (!w->tok_embed || !w->wq || !w->wk || !w->wv || !w->wo || !w->w_gate || !w->w_up || !w->w_down ||
        !w->attn_norm || !w->ffn_norm || !w->final_norm || !w->lm_head)
        return WD_ERR_NULL;
    for (int l = 0; l < dims->n_layers; ++l)
        if (!w->wq[l] || !w->wk[l] || !w->wv[l] || !w->wo[l] || !w->w_gate[l] || !w->w_up[l] || !w->w_down[l] ||
            !w->attn_norm[l] || !w->ffn_norm[l])
            return WD_ERR_NULL;
    if ((uintptr_t)workspace % 256) return WD_ERR_MISALIGNED;
    if (workspace_bytes < wd_workspace_bytes(dims)) return WD_ERR_WORKSPACE_TOO_SMALL;

    int dev = 0;
    cudaDeviceProp prop;
    WD_CUDA_TRY(cudaGetDevice(&dev));
    WD_CUDA_TRY(cudaGetDeviceProperties(&prop, dev));
    if (prop.major != 10) return WD_ERR_UNSUPPORTED_ARCH;

    wd_ctx* c = new (std::nothrow) wd_ctx();
    if (!c) return WD_ERR_CUDA;
    c->d = *dims;
    // debugging switches: WD_FUSE=1 moves the element-wise work into the GEMM epilogues,
    // WD_NO_PDL=1 launches every kernel fully serialised
    if (const char* e = getenv("WD_FUSE")) c->fuse = atoi(e);       // a WD_FUSION_* value
    if (const char* e = getenv("WD_GRAPHS")) c->graphs_on = atoi(e) != 0;
    if (const char* e = getenv("WD_NO_PDL")) wd_pdl_enabled = !(e[0] == '1');
    c->sm_count = prop.multiProcessorCount;
    c->tok_embed = w->tok_embed;
    c->lm_head = w->lm_head;
    c->final_norm = w->final_norm;
    for (int l = 0; l < dims->n_layers; ++l) {
        c->wq.push_back(w->wq[l]); c->wk.push_back(w->wk[l]); c->wv.push_back(w->wv[l]);
        c->wo.push_back(w->wo[l]); c->wg.push_back(w->w_gate[l]); c->wu.push_back(w->w_up[l]);
        c->wd.push_back(w->w_down[l]);
        c->attn_norm.push_back(w->attn_norm[l]); c->ffn_norm.push_back(w->ffn_norm[l]);
    }
    Carve cv;
    size_t off[24];
    carve_ctx(dims, cv, off);
    char* base = (char*)workspace;
    c->x = (float*)(base + off[0]);
    c->xn = base + off[1];
    c->q = base + off[2];
    c->attn = base + off[3];
    c->h = base + off[4];
    c->part = (float*)(base + off[5]);
    c->part_floats = part_floats_for(dims);
    c->logits = (float*)(base + off[6]);
    c->row_token = (int32_t*)(base + off[7]);
    c->row_sumexp = (double*)(base + off[8]);
    c->row_conf = (float*)(base + off[9]);
    c->plan = (int32_t*)(base + off[10]);
    c->plan_ints = off[12];
    c->result = (int32_t*)(base + off[11]);
    c->result_ints = 1 + (size_t)dims->max_batch + 3 * (size_t)dims->max_active;
    c->ch_max = (float*)(base + off[13]);
    c->ch_idx = (int32_t*)(base + off[14]);
    c->ch_sum = (double*)(base + off[15]);
    c->rope_tab = (float2*)(base + off[16]);
    c->sumsq = (float*)(base + off[17]);
    c->tile_counters = (int32_t*)(base + off[18]);
    c->n_tile_counters = off[19];
    WD_CUDA_TRY(cudaMemset(c->tile_counters, 0, c->n_tile_counters * 4));
    c->chain.ready_dev = (int32_t*)(base + off[20]);
    WD_CUDA_TRY(cudaMemset(c->chain.ready_dev, 0, 256));
    WD_CUDA_TRY(cudaMemset(c->result, 0, 4));

    if (dims->dtype == WD_BF16) {
        wd_status s = wd_tc_weights_init(&c->tc, dims, c->tok_embed, c->lm_head, c->wq, c->wk, c->wv, c->wo,
                                         c->wg, c->wu, c->wd, c->xn, c->attn, c->h);
        if (s != WD_OK) { delete c; return s; }
    }
    *out = c;
    return WD_OK;
}

// ---------------------------------------------------------------------------
// FP8 mode
// ---------------------------------------------------------------------------
static void drop_graphs(wd_ctx* c);

static size_t fp8_carve(const wd_model_dims* d, size_t* off /*[8]*/) {
    const size_t hq = (size_t)d->n_q_heads * d->head_dim, hkv = (size_t)d->n_kv_heads * d->head_dim;
    const size_t D = d->d_model, F = d->d_ffn, V = d->vocab, L = d->n_layers, MR = d->max_rows;
    const size_t rows_per_layer = hq + 2 * hkv + 2 * F + D;                  // weight rows with a scale each
    const size_t codes_per_layer = (hq + 2 * hkv) * D + 2 * F * D + D * F;
    size_t o = 0;
    auto take = [&](size_t bytes) { const size_t at = o; o = wd_align_up(o + bytes, 256); return at; };
    off[0] = take(L * codes_per_layer);          // layer weight codes
    off[1] = take(L * rows_per_layer * 4);       // layer weight scales
    off[2] = take(V * D);                        // LM head codes
    off[3] = take(V * 4);                        // LM head scales
    off[4] = take(MR * D);                       // xn8
    off[5] = take(MR * F);                       // h8
    off[6] = take(MR * 4);                       // sxn
    off[7] = take(MR * 4);                       // sh
    return o;
}

extern "C" size_t wd_fp8_bytes(const wd_model_dims* dims) {
    if (!dims_valid(dims) || dims->dtype != WD_BF16) return 0;
    size_t off[8];
    return fp8_carve(dims, off);
}

extern "C" wd_status wd_fp8_enable(wd_ctx* c, void* mem, size_t mem_bytes, void* stream_) {
    if (!c || !mem) return WD_ERR_NULL;
    const wd_model_dims& d = c->d;
    if (d.dtype != WD_BF16 || d.d_model % 16 || d.d_ffn % 16 || d.d_ffn > 32768) return WD_ERR_BAD_PARAM;
    if ((uintptr_t)mem % 256) return WD_ERR_MISALIGNED;
    size_t off[8];
    if (mem_bytes < fp8_carve(&d, off)) return WD_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t stream = (cudaStream_t)stream_;
    const int hq = d.n_q_heads * d.head_dim, hkv = d.n_kv_heads * d.head_dim, D = d.d_model, F = d.d_ffn, L = d.n_layers;
    uint8_t* codes = (uint8_t*)mem + off[0];
    float* scales = (float*)((char*)mem + off[1]);
    auto quant = [&](const void* w, int n, int K, wd_ctx::Fp8Mat* m) -> wd_status {
        wd_launch_quantize_rows(WD_BF16, w, n, K, codes, scales, stream);
        m->q = codes; m->s = scales;
        wd_status s = wd_tc_encode_fp8(&m->map, codes, n, K, 128);
        codes += (size_t)n * K;
        scales += n;
        return s;
    };
    c->f8q.assign(L, {}); c->f8k.assign(L, {}); c->f8v.assign(L, {}); c->f8g.assign(L, {}); c->f8u.assign(L, {}); c->f8d.assign(L, {});
    wd_status s;
    for (int l = 0; l < L; ++l) {
        if ((s = quant(c->wq[l], hq, D, &c->f8q[l])) != WD_OK) return s;
        if ((s = quant(c->wk[l], hkv, D, &c->f8k[l])) != WD_OK) return s;
        if ((s = quant(c->wv[l], hkv, D, &c->f8v[l])) != WD_OK) return s;
        if ((s = quant(c->wg[l], F, D, &c->f8g[l])) != WD_OK) return s;
        if ((s = quant(c->wu[l], F, D, &c->f8u[l])) != WD_OK) return s;
        if ((s = quant(c->wd[l], D, F, &c->f8d[l])) != WD_OK) return s;
    }
    codes = (uint8_t*)mem + off[2];
    scales = (float*)((char*)mem + off[3]);
    if ((s = quant(c->lm_head, d.vocab, D, &c->f8lm)) != WD_OK) return s;
    c->xn8 = (uint8_t*)mem + off[4];
    c->h8 = (uint8_t*)mem + off[5];
    c->sxn = (float*)((char*)mem + off[6]);
    c->sh = (float*)((char*)mem + off[7]);
    c->x8_d = WdTcX(); c->x8_d.ptr = c->xn8; c->x8_d.K = D; c->x8_d.fp8 = 1;
    c->x8_h = WdTcX(); c->x8_h.ptr = c->h8; c->x8_h.K = F; c->x8_h.fp8 = 1;
    WD_CUDA_TRY(cudaGetLastError());
    c->fp8_ready = true;
    c->fp8_on = true;
    c->fp4_on = false;
    drop_graphs(c);
    return WD_OK;
}

extern "C" wd_status wd_fp8_set(wd_ctx* c, int32_t on) {
    if (!c) return WD_ERR_NULL;
    if (on && !c->fp8_ready) return WD_ERR_BAD_PARAM;
    c->fp8_on = on != 0;
    if (on) c->fp4_on = false;
    return WD_OK;
}

// ---------------------------------------------------------------------------
// NVFP4 mode
// ---------------------------------------------------------------------------
static size_t fp4_carve(const wd_model_dims* d, size_t* off /*[6]*/) {
    const int hq = d->n_q_heads * d->head_dim, hkv = d->n_kv_heads * d->head_dim;
    const int D = d->d_model, F = d->d_ffn;
    const size_t L = d->n_layers;
    size_t o = 0;
    auto take = [&](size_t bytes) { const size_t at = o; o = wd_align_up(o + bytes, 256); return at; };
    off[0] = take(L * wd_fp4_operand_bytes(hq + 2 * hkv, D));
    off[1] = take(L * wd_fp4_operand_bytes(2 * F, D));
    off[2] = take(L * wd_fp4_operand_bytes(D, F));
    off[3] = take(wd_fp4_operand_bytes(d->vocab, D));
    off[4] = take(wd_fp4_operand_bytes(d->max_rows, std::max(D, F)));
    return o;
}

static bool fp4_dims_ok(const wd_model_dims* d) {
    return d->dtype == WD_BF16 && d->d_model % 256 == 0 && d->d_ffn % 256 == 0;
}

extern "C" size_t wd_fp4_bytes(const wd_model_dims* dims) {
    if (!dims_valid(dims) || !fp4_dims_ok(dims)) return 0;
    size_t off[6];
    return fp4_carve(dims, off);
}

extern "C" wd_status wd_fp4_enable(wd_ctx* c, void* mem, size_t mem_bytes, void* stream_) {
    if (!c || !mem) return WD_ERR_NULL;
    const wd_model_dims& d = c->d;
    if (!fp4_dims_ok(&d)) return WD_ERR_BAD_PARAM;
    if ((uintptr_t)mem % 256) return WD_ERR_MISALIGNED;
    size_t off[6];
    if (mem_bytes < fp4_carve(&d, off)) return WD_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t stream = (cudaStream_t)stream_;
    const int hq = d.n_q_heads * d.head_dim, hkv = d.n_kv_heads * d.head_dim, D = d.d_model, F = d.d_ffn, L = d.n_layers;
    // rows [r0, r0 + n) of an operand, quantised from one weight matrix
    auto quant = [&](const void* w, const WdFp4Operand& op, int r0, int n) {
        WdFp4Operand sub = op;
        sub.codes += (size_t)r0 * (op.K / 2);
        sub.sf += (size_t)r0 * (op.K / 16);
        sub.g += r0;
        sub.n_rows = n;
        wd_launch_quantize_nvfp4(WD_BF16, w, n, op.K, &sub, stream);
    };
    c->f4qkv.assign(L, {}); c->f4gu.assign(L, {}); c->f4d.assign(L, {});
    for (int l = 0; l < L; ++l) {
        wd_fp4_operand_split((char*)mem + off[0] + (size_t)l * wd_fp4_operand_bytes(hq + 2 * hkv, D), hq + 2 * hkv, D, &c->f4qkv[l]);
        quant(c->wq[l], c->f4qkv[l], 0, hq);
        quant(c->wk[l], c->f4qkv[l], hq, hkv);
        quant(c->wv[l], c->f4qkv[l], hq + hkv, hkv);
        wd_fp4_operand_split((char*)mem + off[1] + (size_t)l * wd_fp4_operand_bytes(2 * F, D), 2 * F, D, &c->f4gu[l]);
        quant(c->wg[l], c->f4gu[l], 0, F);
        quant(c->wu[l], c->f4gu[l], F, F);
        wd_fp4_operand_split((char*)mem + off[2] + (size_t)l * wd_fp4_operand_bytes(D, F), D, F, &c->f4d[l]);
        quant(c->wd[l], c->f4d[l], 0, D);
    }
    wd_fp4_operand_split((char*)mem + off[3], d.vocab, D, &c->f4lm);
    quant(c->lm_head, c->f4lm, 0, d.vocab);
    c->fp4_x = (char*)mem + off[4];
    WD_CUDA_TRY(cudaGetLastError());
    c->fp4_ready = true;
    c->fp4_on = true;
    c->fp8_on = false;
    drop_graphs(c);
    return WD_OK;
}

extern "C" wd_status wd_fp4_set(wd_ctx* c, int32_t on) {
    if (!c) return WD_ERR_NULL;
    if (on && !c->fp4_ready) return WD_ERR_BAD_PARAM;
    c->fp4_on = on != 0;
    if (on) c->fp8_on = false;
    return WD_OK;
}

extern "C" wd_status wd_destroy(wd_ctx* ctx) {
    if (!ctx) return WD_ERR_NULL;
    delete ctx;
    return WD_OK;
}

extern "C" wd_status wd_set_gemm_impl(wd_ctx* ctx, int32_t impl) {
    if (!ctx) return WD_ERR_NULL;
    if (impl != WD_GEMM_AUTO && impl != WD_GEMM_PLAIN && impl != WD_GEMM_TCGEN05) return WD_ERR_BAD_PARAM;
    if (impl == WD_GEMM_TCGEN05 && ctx->d.dtype != WD_BF16) return WD_ERR_BAD_PARAM;
    ctx->gemm_impl = impl;
    ctx->attn_impl = impl;          // the plain setting selects the CUDA-core kernels throughout
    return WD_OK;
}

extern "C" wd_status wd_set_fusion(wd_ctx* ctx, int32_t mode) {
    if (!ctx) return WD_ERR_NULL;
    if (mode < WD_FUSION_AUTO || mode > WD_FUSION_CHAIN) return WD_ERR_BAD_PARAM;
    ctx->fuse = mode;
    return WD_OK;
}

// Recorded step graphs hold their kernels' arguments by value: whatever changes a pointer that they hold
// (the quantised weights' memory) drops them.
static void drop_graphs(wd_ctx* c) {
    for (wd_ctx::StepGraph& g : c->graphs) if (g.exec) cudaGraphExecDestroy(g.exec);
    c->graphs.clear();
    c->seen.clear();
}

extern "C" wd_status wd_set_graphs(wd_ctx* ctx, int32_t on) {
    if (!ctx) return WD_ERR_NULL;
    ctx->graphs_on = on != 0;
    if (!ctx->graphs_on) drop_graphs(ctx);
    return WD_OK;
}

extern "C" wd_status wd_debug_graph_stats(const wd_ctx* ctx, int32_t* captured, int32_t* replayed) {
    if (!ctx || !captured || !replayed) return WD_ERR_NULL;
    *captured = ctx->graphs_captured;
    *replayed = ctx->graphs_replayed;
    return WD_OK;
}

extern "C" wd_status wd_profile_enable(wd_ctx* ctx, int32_t on) {
    if (!ctx) return WD_ERR_NULL;
    ctx->prof_on = on != 0;
    ctx->prof_ms = 0.0; ctx->prof_bytes = 0.0; ctx->prof_launches = 0;
    return WD_OK;
}

extern "C" wd_status wd_profile_read(const wd_ctx* ctx, double* gemm_ms, double* gemm_bytes, int64_t* gemm_launches) {
    if (!ctx) return WD_ERR_NULL;
    if (gemm_ms) *gemm_ms = ctx->prof_ms;
    if (gemm_bytes) *gemm_bytes = ctx->prof_bytes;
    if (gemm_launches) *gemm_launches = ctx->prof_launches;
    return WD_OK;
}

// ---------------------------------------------------------------------------
// state
// ---------------------------------------------------------------------------
static const int kQueueCap = 32;        // most steps enqueued without wd_step_sync

static uint64_t g_state_uid = 0;

struct wd_state {
    wd_ctx* ctx = nullptr;
    uint64_t uid = ++g_state_uid;       // never reused, unlike the address (keys the step graphs)
    int batch = 0, S = 0;
    std::vector<WdSeq> seqs;
    std::vector<WdSeqPlan> plans;       // of the pending step
    int32_t* ids_dev = nullptr;
    char* kcache = nullptr;             // [L][batch][Hkv][S][dh]
    char* vcache = nullptr;             // [L][batch][Hkv][dh][Sp]  (transposed: position contiguous)
    size_t kv_layer_bytes = 0, v_layer_bytes = 0;
    int Sp = 0;
    int32_t* plan_host = nullptr;       // pinned
    int32_t* result_host = nullptr;     // pinned: kQueueCap result blocks
    int32_t* ids_host = nullptr;        // pinned staging for ids
    uint8_t* dec_host = nullptr;        // pinned staging for the decoded flags
    cudaEvent_t done = nullptr;
    cudaEvent_t staged = nullptr;       // recorded after the copies that read the pinned staging buffers
    bool staged_recorded = false;
    bool poisoned = false;              // a queued step failed on the device: device state is ahead of the mirror
    bool pending = false;               // at least one step enqueued and not yet synced
    // Device copy of the planner state, kept up to date by the unmask kernel, and the count-level
    // shadow on the host: with them steps can be enqueued back to back (no host round trip), the
    // index lists being built by plan_kernel.  Used while every sequence started from a decoded
    // prefix and adaptive termination is off.
    uint8_t* decoded_dev = nullptr;     // [batch][S]
    int32_t* dec_step_dev = nullptr;    // [batch][S]  (0x80808080 = never)
    int32_t* wex_dev = nullptr;         // [batch][S]
    bool dev_mode = false;
    std::vector<WdCount> counts;
    struct Pending {
        int32_t A, B, R, T, k_eff, k_user;
        bool host_planned;
        std::vector<WdCountPlan> cp;
        std::vector<WdSeqPlan> plans;   // host-planned steps only
    };
    std::vector<Pending> queue;
    size_t result_slot_ints = 0;
    bool dev_plan_allowed = true;       // WD_HOST_PLAN=1 forces the host planner (debugging)
    wd_debug_taps taps = {nullptr, nullptr, nullptr};
    bool attn_tc = false;               // tensor-core attention usable (bf16, head_dim 128)
    CUtensorMap map_k, map_vt;
};

static void load_host_mirror(wd_state* st, const int32_t* ids, const uint8_t* decoded) {
    const int mask_id = st->ctx->d.mask_id;
    for (int b = 0; b < st->batch; ++b) {
        WdSeq& s = st->seqs[b];
        s.ids.assign(ids + (size_t)b * st->S, ids + (size_t)(b + 1) * st->S);
        s.decoded.resize(st->S);
        for (int i = 0; i < st->S; ++i)
            s.decoded[i] = decoded ? (decoded[(size_t)b * st->S + i] ? 1 : 0) : (s.ids[i] != mask_id ? 1 : 0);
        s.dec_step.assign(st->S, INT32_MIN);
        s.wex.clear();
        s.t = 0; s.since = 0; s.phase_start = 0;          // eos_id is kept across resets
    }
    memcpy(st->ids_host, ids, (size_t)st->batch * st->S * 4);
    // device-side planning needs every sequence to start from a decoded prefix (then the visible
    // set stays a range) and at most WD_PLAN_MAX_BATCH sequences; adaptive termination needs the
    // host to see every result, so it keeps the host planner
    bool prefix = st->batch <= WD_PLAN_MAX_BATCH;
    st->counts.assign(st->batch, WdCount());
    for (int b = 0; b < st->batch; ++b) {
        const WdSeq& s = st->seqs[b];
        bool seen_undecoded = false;
        for (int i = 0; i < st->S; ++i) {
            st->dec_host[(size_t)b * st->S + i] = s.decoded[i];
            if (!s.decoded[i]) seen_undecoded = true;
            else if (seen_undecoded) prefix = false;
        }
        if (s.eos_id >= 0) prefix = false;
        wd_count_init(st->counts[b], s);
    }
    st->dev_mode = prefix && st->dev_plan_allowed;
    st->queue.clear();
}

// uploads the device copy of the planner state (decoded flags; decode steps = "never")
static cudaError_t upload_plan_state(wd_state* st, cudaStream_t stream) {
    const size_t n = (size_t)st->batch * st->S;
    cudaError_t e = cudaMemcpyAsync(st->decoded_dev, st->dec_host, n, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(st->dec_step_dev, 0x80, n * 4, stream);
    return e;
}

extern "C" wd_status wd_state_create(wd_ctx* ctx, int32_t batch, int32_t seq_len, const int32_t* token_ids,
                                     const uint8_t* decoded, void* state_mem, size_t state_mem_bytes,
                                     wd_state** out) {
    if (!ctx || !token_ids || !state_mem || !out) return WD_ERR_NULL;
    *out = nullptr;
    if (batch < 1 || seq_len < 1 || batch > ctx->d.max_batch || seq_len > ctx->d.max_seq) return WD_ERR_BAD_PARAM;
    if ((uintptr_t)state_mem % 256) return WD_ERR_MISALIGNED;
    const size_t need = wd_state_bytes(&ctx->d, batch, seq_len);
    if (state_mem_bytes < need) return WD_ERR_WORKSPACE_TOO_SMALL;
    for (size_t i = 0; i < (size_t)batch * seq_len; ++i)
        if (token_ids[i] < 0 || token_ids[i] >= ctx->d.vocab) return WD_ERR_BAD_PARAM;

    wd_state* st = new (std::nothrow) wd_state();
    if (!st) return WD_ERR_CUDA;
    st->ctx = ctx; st->batch = batch; st->S = seq_len;
    st->seqs.resize(batch);
    const wd_model_dims& d = ctx->d;
    const size_t ids_bytes = wd_align_up((size_t)batch * seq_len * 4, 256);
    st->Sp = seq_pad(seq_len);
    st->kv_layer_bytes = (size_t)batch * d.n_kv_heads * seq_len * d.head_dim * wd_elt_size(d.dtype);
    st->v_layer_bytes = (size_t)batch * d.n_kv_heads * st->Sp * d.head_dim * wd_elt_size(d.dtype);
    const size_t kv = wd_align_up(st->kv_layer_bytes * d.n_layers, 256);
    st->ids_dev = (int32_t*)state_mem;
    st->kcache = (char*)state_mem + ids_bytes;
    st->vcache = st->kcache + kv;
    {
        char* ps = st->vcache + wd_align_up(st->v_layer_bytes * d.n_layers, 256);
        st->decoded_dev = (uint8_t*)ps;
        st->dec_step_dev = (int32_t*)(ps + wd_align_up((size_t)batch * seq_len, 256));
        st->wex_dev = (int32_t*)((char*)st->dec_step_dev + wd_align_up((size_t)batch * seq_len * 4, 256));
    }
    st->result_slot_ints = ctx->result_ints;
    cudaError_t e;
    if ((e = cudaHostAlloc((void**)&st->plan_host, ctx->plan_ints * 4, cudaHostAllocDefault)) != cudaSuccess ||
        (e = cudaHostAlloc((void**)&st->result_host, ctx->result_ints * 4 * kQueueCap, cudaHostAllocDefault)) != cudaSuccess ||
        (e = cudaHostAlloc((void**)&st->ids_host, (size_t)batch * seq_len * 4, cudaHostAllocDefault)) != cudaSuccess ||
        (e = cudaHostAlloc((void**)&st->dec_host, (size_t)batch * seq_len, cudaHostAllocDefault)) != cudaSuccess ||
        (e = cudaEventCreateWithFlags(&st->done, cudaEventDisableTiming)) != cudaSuccess ||
        (e = cudaEventCreateWithFlags(&st->staged, cudaEventDisableTiming)) != cudaSuccess) {
        wd_note_cuda_error(e, __FILE__, __LINE__);
        wd_state_destroy(st);
        return WD_ERR_CUDA;
    }
    if (const char* ev = getenv("WD_HOST_PLAN")) st->dev_plan_allowed = !(ev[0] == '1');
    load_host_mirror(st, token_ids, decoded);
    // Far-field cache rows are never read as values, but tiles of the tensor-core attention
    // cover them (masked): start from finite contents.
    e = cudaMemset(st->kcache, 0, st->kv_layer_bytes * d.n_layers);
    if (e == cudaSuccess) e = cudaMemset(st->vcache, 0, st->v_layer_bytes * d.n_layers);
    if (e != cudaSuccess) { wd_note_cuda_error(e, __FILE__, __LINE__); wd_state_destroy(st); return WD_ERR_CUDA; }
    if (d.dtype == WD_BF16 && d.head_dim == 128) {
        wd_status ms = wd_attn_tc_encode_cache(&st->map_k, &st->map_vt, st->kcache, st->vcache, d.n_layers,
                                               batch * d.n_kv_heads, seq_len, st->Sp, d.head_dim);
        if (ms != WD_OK) { wd_state_destroy(st); return ms; }
        st->attn_tc = true;
    }
    e = upload_plan_state(st, 0);
    if (e == cudaSuccess) e = cudaMemcpy(st->ids_dev, st->ids_host, (size_t)batch * seq_len * 4, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) { wd_note_cuda_error(e, __FILE__, __LINE__); wd_state_destroy(st); return WD_ERR_CUDA; }
    *out = st;
    return WD_OK;
}

extern "C" wd_status wd_state_reset(wd_state* st, const int32_t* token_ids, const uint8_t* decoded, void* stream) {
    if (!st || !token_ids) return WD_ERR_NULL;
    if (st->pending) return WD_ERR_PENDING;
    for (size_t i = 0; i < (size_t)st->batch * st->S; ++i)
        if (token_ids[i] < 0 || token_ids[i] >= st->ctx->d.vocab) return WD_ERR_BAD_PARAM;
    // the pinned staging buffers may still be the source of an earlier reset's copies
    if (st->staged_recorded) WD_CUDA_TRY(cudaEventSynchronize(st->staged));
    load_host_mirror(st, token_ids, decoded);
    st->poisoned = false;
    WD_CUDA_TRY(upload_plan_state(st, (cudaStream_t)stream));
    WD_CUDA_TRY(cudaMemcpyAsync(st->ids_dev, st->ids_host, (size_t)st->batch * st->S * 4, cudaMemcpyHostToDevice,
                                (cudaStream_t)stream));
    WD_CUDA_TRY(cudaEventRecord(st->staged, (cudaStream_t)stream));
    st->staged_recorded = true;
    return WD_OK;
}

// ---------------------------------------------------------------------------
// checkpoint / resume of the sequence state (host side; the K/V cache lives in the caller's
// state memory and is the caller's to copy)
// ---------------------------------------------------------------------------
namespace {
struct BlobHeader { uint32_t magic, version; int32_t batch, S; };
struct BlobSeq { int32_t t, since, phase_start, eos_id, refresh_mode, n_wex, stagger_i, stagger_n; };
constexpr uint32_t kBlobMagic = 0x57445354u;     // "WDST"
}

extern "C" size_t wd_state_export_bytes(const wd_state* st) {
    if (!st) return 0;
    size_t n = sizeof(BlobHeader);
    for (const WdSeq& s : st->seqs)
        n += sizeof(BlobSeq) + (size_t)st->S * 8 + wd_align_up((size_t)st->S, 4) + s.wex.size() * 4;
    return n;
}

extern "C" wd_status wd_state_export(const wd_state* st, void* buf, size_t bytes) {
    if (!st || !buf) return WD_ERR_NULL;
    if (st->pending) return WD_ERR_PENDING;
    if (st->poisoned) return WD_ERR_BAD_PARAM;
    if (bytes < wd_state_export_bytes(st)) return WD_ERR_CAPACITY;
    char* p = (char*)buf;
    BlobHeader h = {kBlobMagic, 1u, st->batch, st->S};
    memcpy(p, &h, sizeof(h)); p += sizeof(h);
    for (const WdSeq& s : st->seqs) {
        BlobSeq bs = {s.t, s.since, s.phase_start, s.eos_id, s.refresh_mode, (int32_t)s.wex.size(), s.stagger_i, s.stagger_n};
        memcpy(p, &bs, sizeof(bs)); p += sizeof(bs);
        memcpy(p, s.ids.data(), (size_t)st->S * 4); p += (size_t)st->S * 4;
        memcpy(p, s.dec_step.data(), (size_t)st->S * 4); p += (size_t)st->S * 4;
        memset(p, 0, wd_align_up((size_t)st->S, 4));
        memcpy(p, s.decoded.data(), (size_t)st->S); p += wd_align_up((size_t)st->S, 4);
        if (!s.wex.empty()) memcpy(p, s.wex.data(), s.wex.size() * 4);
        p += s.wex.size() * 4;
    }
    return WD_OK;
}

extern "C" wd_status wd_state_import(wd_state* st, const void* buf, size_t bytes, int32_t cache_valid, void* stream_) {
    if (!st || !buf) return WD_ERR_NULL;
    if (st->pending) return WD_ERR_PENDING;
    const char* p = (const char*)buf;
    const char* end = p + bytes;
    BlobHeader h;
    if (bytes < sizeof(h)) return WD_ERR_BAD_PARAM;
    memcpy(&h, p, sizeof(h)); p += sizeof(h);
    if (h.magic != kBlobMagic || h.version != 1u || h.batch != st->batch || h.S != st->S) return WD_ERR_BAD_PARAM;
    const int S = st->S, vocab = st->ctx->d.vocab;
    // parse and validate everything before anything is changed
    std::vector<WdSeq> seqs((size_t)st->batch);
    for (WdSeq& s : seqs) {
        BlobSeq bs;
        if ((size_t)(end - p) < sizeof(bs)) return WD_ERR_BAD_PARAM;
        memcpy(&bs, p, sizeof(bs)); p += sizeof(bs);
        const size_t need = (size_t)S * 8 + wd_align_up((size_t)S, 4);
        if (bs.n_wex < 0 || bs.n_wex > S || bs.t < 0 || bs.since < 0 || bs.phase_start < 0 || bs.phase_start > bs.t ||
            bs.eos_id >= vocab || (bs.refresh_mode != WD_REFRESH_FULL && bs.refresh_mode != WD_REFRESH_WINDOW) ||
            bs.stagger_n < 0 || bs.stagger_i < 0 || (bs.stagger_n > 0 && bs.stagger_i >= bs.stagger_n) ||
            (size_t)(end - p) < need + (size_t)bs.n_wex * 4)
            return WD_ERR_BAD_PARAM;
        s.t = bs.t; s.since = bs.since; s.phase_start = bs.phase_start;
        s.eos_id = bs.eos_id < 0 ? -1 : bs.eos_id; s.refresh_mode = bs.refresh_mode;
        s.stagger_i = bs.stagger_i; s.stagger_n = bs.stagger_n;
        s.ids.resize(S); s.dec_step.resize(S); s.decoded.resize(S); s.wex.resize((size_t)bs.n_wex);
        memcpy(s.ids.data(), p, (size_t)S * 4); p += (size_t)S * 4;
        memcpy(s.dec_step.data(), p, (size_t)S * 4); p += (size_t)S * 4;
        memcpy(s.decoded.data(), p, (size_t)S); p += wd_align_up((size_t)S, 4);
        if (bs.n_wex) memcpy(s.wex.data(), p, (size_t)bs.n_wex * 4);
        p += (size_t)bs.n_wex * 4;
        for (int i = 0; i < S; ++i)
            if (s.ids[i] < 0 || s.ids[i] >= vocab || s.decoded[i] > 1) return WD_ERR_BAD_PARAM;
        for (size_t i = 0; i < s.wex.size(); ++i)
            if (s.wex[i] < 0 || s.wex[i] >= S || (i > 0 && s.wex[i] <= s.wex[i - 1])) return WD_ERR_BAD_PARAM;
    }
    // a lost cache is rebuilt by a refresh that computes every visible position: the paper's refresh
    if (!cache_valid)
        for (const WdSeq& s : seqs)
            if (s.refresh_mode != WD_REFRESH_FULL) return WD_ERR_BAD_PARAM;
    cudaStream_t stream = (cudaStream_t)stream_;
    if (st->staged_recorded) WD_CUDA_TRY(cudaEventSynchronize(st->staged));
    st->seqs = std::move(seqs);
    st->counts.assign(st->batch, WdCount());
    for (int b = 0; b < st->batch; ++b) {
        WdSeq& s = st->seqs[b];
        // without its cache a state resumes with a refresh step (which rewrites every row it reads)
        if (!cache_valid) s.wex.clear();
        memcpy(st->ids_host + (size_t)b * S, s.ids.data(), (size_t)S * 4);
        memcpy(st->dec_host + (size_t)b * S, s.decoded.data(), (size_t)S);
        wd_count_init(st->counts[b], s);
    }
    // the device planner only takes states whose generation began from a decoded prefix; a resumed state
    // cannot prove that, so it is planned on the host (identical index sets, one host round trip per step)
    st->dev_mode = false;
    st->queue.clear();
    st->poisoned = false;
    const size_t n = (size_t)st->batch * S;
    WD_CUDA_TRY(cudaMemcpyAsync(st->decoded_dev, st->dec_host, n, cudaMemcpyHostToDevice, stream));
    WD_CUDA_TRY(cudaMemcpyAsync(st->ids_dev, st->ids_host, n * 4, cudaMemcpyHostToDevice, stream));
    // decode steps: reuse the pinned plan staging buffer when it is large enough, else copy per sequence from the mirror
    for (int b = 0; b < st->batch; ++b)
        WD_CUDA_TRY(cudaMemcpyAsync(st->dec_step_dev + (size_t)b * S, st->seqs[b].dec_step.data(), (size_t)S * 4,
                                    cudaMemcpyHostToDevice, stream));
    for (int b = 0; b < st->batch; ++b)
        if (!st->seqs[b].wex.empty())
            WD_CUDA_TRY(cudaMemcpyAsync(st->wex_dev + (size_t)b * S, st->seqs[b].wex.data(), st->seqs[b].wex.size() * 4,
                                        cudaMemcpyHostToDevice, stream));
    // the mirror's vectors are pageable sources: wait until the copies have read them
    WD_CUDA_TRY(cudaEventRecord(st->staged, stream));
    st->staged_recorded = true;
    WD_CUDA_TRY(cudaEventSynchronize(st->staged));
    return WD_OK;
}

extern "C" wd_status wd_debug_poke_id(wd_state* st, int32_t seq, int32_t pos, int32_t id, void* stream) {
    if (!st) return WD_ERR_NULL;
    if (st->pending) return WD_ERR_PENDING;
    if (seq < 0 || seq >= st->batch || pos < 0 || pos >= st->S) return WD_ERR_BAD_PARAM;
    WD_CUDA_TRY(cudaMemcpyAsync(st->ids_dev + (size_t)seq * st->S + pos, &id, 4, cudaMemcpyHostToDevice, (cudaStream_t)stream));
    WD_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    return WD_OK;
}

extern "C" wd_status wd_state_destroy(wd_state* st) {
    if (!st) return WD_ERR_NULL;
    if (st->pending && st->done) cudaEventSynchronize(st->done);
    if (st->plan_host) cudaFreeHost(st->plan_host);
    if (st->result_host) cudaFreeHost(st->result_host);
    if (st->ids_host) cudaFreeHost(st->ids_host);
    if (st->dec_host) cudaFreeHost(st->dec_host);
    if (st->done) cudaEventDestroy(st->done);
    if (st->staged) cudaEventDestroy(st->staged);
    delete st;
    return WD_OK;
}

extern "C" wd_status wd_state_read(const wd_state* st, int32_t seq, int32_t* token_ids, uint8_t* decoded,
                                   int32_t* dec_step, int32_t* step_index, int32_t* steps_since_refresh) {
    if (!st) return WD_ERR_NULL;
    if (st->pending) return WD_ERR_PENDING;
    if (seq < 0 || seq >= st->batch) return WD_ERR_BAD_PARAM;
    const WdSeq& s = st->seqs[seq];
    if (token_ids) memcpy(token_ids, s.ids.data(), (size_t)st->S * 4);
    if (decoded) memcpy(decoded, s.decoded.data(), (size_t)st->S);
    if (dec_step) memcpy(dec_step, s.dec_step.data(), (size_t)st->S * 4);
    if (step_index) *step_index = s.t;
    if (steps_since_refresh) *steps_since_refresh = s.since;
    return WD_OK;
}

extern "C" wd_status wd_state_set_eos(wd_state* st, int32_t eos_id) {
    if (!st) return WD_ERR_NULL;
    if (st->pending) return WD_ERR_PENDING;
    if (eos_id >= st->ctx->d.vocab) return WD_ERR_BAD_PARAM;
    for (WdSeq& s : st->seqs) s.eos_id = eos_id < 0 ? -1 : eos_id;
    if (eos_id >= 0) st->dev_mode = false;      // every result must reach the host planner before the next step
    return WD_OK;
}

extern "C" wd_status wd_state_set_refresh_mode(wd_state* st, int32_t mode) {
    if (!st) return WD_ERR_NULL;
    if (st->pending) return WD_ERR_PENDING;
    if (mode != WD_REFRESH_FULL && mode != WD_REFRESH_WINDOW) return WD_ERR_BAD_PARAM;
    for (WdSeq& s : st->seqs) s.refresh_mode = mode;
    for (WdCount& c : st->counts) c.refresh_mode = mode;
    return WD_OK;
}

extern "C" wd_status wd_state_set_stagger(wd_state* st, int32_t on) {
    if (!st) return WD_ERR_NULL;
    if (st->pending) return WD_ERR_PENDING;
    for (int b = 0; b < st->batch; ++b) {
        st->seqs[b].stagger_i = on ? b : 0;
        st->seqs[b].stagger_n = on ? st->batch : 0;
        st->counts[b].stagger_i = st->seqs[b].stagger_i;
        st->counts[b].stagger_n = st->seqs[b].stagger_n;
    }
    return WD_OK;
}

extern "C" wd_status wd_debug_taps_set(wd_state* st, const wd_debug_taps* taps) {
    if (!st) return WD_ERR_NULL;
    if (st->pending) return WD_ERR_PENDING;
    if (taps) st->taps = *taps;
    else st->taps = {nullptr, nullptr, nullptr};
    return WD_OK;
}

// ---------------------------------------------------------------------------
// wd_plan
// ---------------------------------------------------------------------------
static wd_status copy_list(const std::vector<int32_t>& v, int32_t* dst, int32_t* n, int32_t cap) {
    *n = (int32_t)v.size();
    if ((int32_t)v.size() > cap) return WD_ERR_CAPACITY;
    if (!v.empty()) {
        if (!dst) return WD_ERR_NULL;
        memcpy(dst, v.data(), v.size() * 4);
    }
    return WD_OK;
}

static wd_status export_plan(const WdSeqPlan& p, wd_index_sets* out);

extern "C" wd_status wd_plan(const wd_state* st, int32_t seq, int32_t A, int32_t B, int32_t R, int32_t T,
                             wd_index_sets* out) {
    if (!st || !out) return WD_ERR_NULL;
    if (st->pending) return WD_ERR_PENDING;
    if (st->poisoned) return WD_ERR_POISONED;
    if (seq < 0 || seq >= st->batch) return WD_ERR_BAD_PARAM;
    WdSeqPlan p;
    wd_status s = wd_plan_seq(st->seqs[seq], A, B, R, T, &p);
    if (s != WD_OK) return s;
    return export_plan(p, out);
}

extern "C" wd_status wd_plan_raw(const uint8_t* decoded, const int32_t* dec_step, const int32_t* token_ids,
                                 int32_t eos_id, int32_t seq_len, int32_t step_index, int32_t steps_since_refresh,
                                 const int32_t* ext_window, int32_t n_ext_window, int32_t A, int32_t B, int32_t R,
                                 int32_t T, int32_t refresh_mode, int32_t stagger_i, int32_t stagger_n, wd_index_sets* out) {
    if (!decoded || !dec_step || !out || (n_ext_window > 0 && !ext_window)) return WD_ERR_NULL;
    if (eos_id >= 0 && !token_ids) return WD_ERR_NULL;
    if (seq_len < 1 || n_ext_window < 0 || step_index < 0 || steps_since_refresh < 0) return WD_ERR_BAD_PARAM;
    if (refresh_mode != WD_REFRESH_FULL && refresh_mode != WD_REFRESH_WINDOW) return WD_ERR_BAD_PARAM;
    if (stagger_n < 0 || stagger_i < 0 || (stagger_n > 0 && stagger_i >= stagger_n)) return WD_ERR_BAD_PARAM;
    WdSeq s;
    if (token_ids) s.ids.assign(token_ids, token_ids + seq_len);
    else s.ids.assign(seq_len, 0);
    s.eos_id = eos_id < 0 ? -1 : eos_id;
    s.decoded.assign(decoded, decoded + seq_len);
    s.dec_step.assign(dec_step, dec_step + seq_len);
    for (int32_t i = 0; i < n_ext_window; ++i) {
        if (ext_window[i] < 0 || ext_window[i] >= seq_len) return WD_ERR_BAD_PARAM;
        s.wex.push_back(ext_window[i]);
    }
    s.t = step_index;
    s.since = steps_since_refresh;
    s.phase_start = step_index - steps_since_refresh;       // first step of the running phase
    s.refresh_mode = refresh_mode;
    s.stagger_i = stagger_i;
    s.stagger_n = stagger_n;
    WdSeqPlan p;
    wd_status r = wd_plan_seq(s, A, B, R, T, &p);
    if (r != WD_OK) return r;
    return export_plan(p, out);
}

static wd_status export_plan(const WdSeqPlan& p, wd_index_sets* out) {
    out->done = p.done ? 1 : 0;
    out->is_refresh = p.refresh ? 1 : 0;
    out->vis_contiguous = p.vis_contiguous ? 1 : 0;
    wd_status worst = WD_OK, r;
    const int32_t cap = out->capacity;
    if ((r = copy_list(p.active, out->active, &out->n_active, cap)) != WD_OK) worst = r;
    if ((r = copy_list(p.buffer, out->buffer, &out->n_buffer, cap)) != WD_OK) worst = r;
    if ((r = copy_list(p.decoded, out->decoded, &out->n_decoded, cap)) != WD_OK) worst = r;
    if ((r = copy_list(p.transient, out->transient, &out->n_transient, cap)) != WD_OK) worst = r;
    if ((r = copy_list(p.far_field, out->far_field, &out->n_far_field, cap)) != WD_OK) worst = r;
    if ((r = copy_list(p.rows, out->rows, &out->n_rows, cap)) != WD_OK) worst = r;
    if ((r = copy_list(p.vis, out->vis, &out->n_vis, cap)) != WD_OK) worst = r;
    if ((r = copy_list(p.wex, out->ext_window, &out->n_ext_window, cap)) != WD_OK) worst = r;
    return worst;
}

// ---------------------------------------------------------------------------
// GEMM dispatch: y[rows, sum n_i] = x[rows, K] * [w_0; w_1; ...]^T into ctx->part
// ---------------------------------------------------------------------------
struct GemmOut { int n_split; size_t split_stride; int launches; int impl; };

static bool use_tc(const wd_ctx* c) {
    if (c->d.dtype != WD_BF16) return false;
    return c->gemm_impl != WD_GEMM_PLAIN;
}

static wd_status run_gemm(wd_ctx* c, const void* x, const WdTcX* x_map, const WdTcSeg* segs, int nseg,
                          int rows, int K, float* y, size_t y_floats, int32_t* status, cudaStream_t stream,
                          GemmOut* go, bool single_split = false, const WdTcFuse* fuse = nullptr,
                          const WdTcFp8* fp8 = nullptr, const WdTcSwiglu* sg = nullptr) {
    int ncol = 0;
    for (int i = 0; i < nseg; ++i) ncol += segs[i].n;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (c->prof_on) {
        while (c->prof_events.size() < c->prof_used + 2) {
            cudaEvent_t e;
            WD_CUDA_TRY(cudaEventCreate(&e));
            c->prof_events.push_back(e);
        }
        e0 = c->prof_events[c->prof_used++];
        e1 = c->prof_events[c->prof_used++];
        // algorithmic bytes: weights once, activations in, result out
        const double elt = fp8 ? 1.0 : (double)wd_elt_size(c->d.dtype);
        c->prof_step_bytes += (double)ncol * K * elt + (double)rows * K * elt + (double)rows * ncol * 4;
        WD_CUDA_TRY(cudaEventRecord(e0, stream));
    }
    if (use_tc(c) && !fp8 && fuse && fuse->cluster && wd_ck_usable(rows, K, segs, nseg, fuse)) {
        // few rows: cluster split-K with the consumer in the epilogue; nothing goes to y
        wd_status s = wd_ck_gemm(x_map, segs, nseg, rows, K, c->sm_count, status, stream, fuse);
        if (s != WD_OK) return s;
        if (c->prof_on) c->prof_step_bytes -= (double)rows * ncol * 4 - (double)rows * ncol * 2;   // bf16 results
        *go = {1, (size_t)rows * ncol, 1, WD_GEMM_TCGEN05};
    } else if (use_tc(c)) {
        int n_split = 1;
        wd_status s = wd_tc_gemm(x_map, segs, nseg, rows, K, y, y_floats, c->sm_count, status, stream, &n_split,
                                 single_split, fuse, fp8, sg);
        if (s != WD_OK) return s;
        // SwiGLU done by the GEMM: bf16 h instead of the fp32 gate/up sums
        if (sg && sg->done && c->prof_on) c->prof_step_bytes -= (double)rows * ncol * 4 - (double)rows * (ncol / 2) * 2;
        *go = {n_split, (size_t)rows * ncol, 1, WD_GEMM_TCGEN05};
    } else {
        if ((size_t)rows * ncol > y_floats) return WD_ERR_CAPACITY;
        int col = 0;
        for (int i = 0; i < nseg; ++i) {
            wd_launch_gemm_plain(c->d.dtype, x, segs[i].w, y + col, rows, segs[i].n, K, ncol, stream);
            col += segs[i].n;
        }
        *go = {1, (size_t)rows * ncol, nseg, WD_GEMM_PLAIN};
    }
    if (e1) WD_CUDA_TRY(cudaEventRecord(e1, stream));
    return WD_OK;
}

// NVFP4 projection of the step: the step's quantised activations (left in ctx->fp4_x by the RMSNorm / SwiGLU
// kernel before it) times the quantised weights; K slices side by side in y like the bf16 kernel's.
static wd_status run_gemm_fp4(wd_ctx* c, const WdFp4Operand* w, int rows, int K, float* y, size_t y_floats,
                              int32_t* status, cudaStream_t stream, GemmOut* go, bool single_split = false) {
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (c->prof_on) {
        while (c->prof_events.size() < c->prof_used + 2) {
            cudaEvent_t e;
            WD_CUDA_TRY(cudaEventCreate(&e));
            c->prof_events.push_back(e);
        }
        e0 = c->prof_events[c->prof_used++];
        e1 = c->prof_events[c->prof_used++];
        // algorithmic bytes: codes + block scales of the weights once and of the activations, result out
        c->prof_step_bytes += (double)(w->n_rows + rows) * K * (0.5 + 1.0 / 16) + (double)rows * w->n_rows * 4;
        WD_CUDA_TRY(cudaEventRecord(e0, stream));
    }
    WdFp4Operand ox;
    wd_fp4_operand_split(c->fp4_x, rows, K, &ox);
    int ns = 1;
    wd_status s = wd_fp4_gemm(&ox, w, y, y_floats, c->sm_count, status, stream, &ns, single_split, /*w_static=*/true);
    if (s != WD_OK) return s;
    *go = {ns, (size_t)rows * w->n_rows, 1, WD_GEMM_TCGEN05};
    if (e1) WD_CUDA_TRY(cudaEventRecord(e1, stream));
    return WD_OK;
}

// ---------------------------------------------------------------------------
// wd_step
// ---------------------------------------------------------------------------
extern "C" wd_status wd_step(wd_state* st, int32_t A, int32_t B, int32_t R, int32_t T, int32_t k, void* stream_,
                             wd_step_info* info) {
    if (!st) return WD_ERR_NULL;
    if (A < 1 || B < 0 || R < 1 || T < 0 || k < 0) return WD_ERR_BAD_PARAM;
    if (st->poisoned) return WD_ERR_POISONED;
    wd_ctx* c = st->ctx;
    const wd_model_dims& d = c->d;
    cudaStream_t stream = (cudaStream_t)stream_;
    const int batch = st->batch, S = st->S;
    // Steps can queue up only while the device plans them (and no per-step profile is being taken)
    const bool dev_mode = st->dev_mode && !c->prof_on;
    if (!st->queue.empty() && (!dev_mode || (int)st->queue.size() >= kQueueCap)) return WD_ERR_PENDING;
    const int k_eff = std::min<int64_t>(k, A);

    // ---- shape of the step: per-sequence counts, from the host planner or from the count shadow
    wd_state::Pending pend;
    pend.A = A; pend.B = B; pend.R = R; pend.T = T; pend.k_eff = k_eff; pend.k_user = k;
    pend.host_planned = !dev_mode;
    pend.cp.assign(batch, WdCountPlan());
    bool all_done = true, any_refresh = false, all_contig = true;
    size_t n_rows = 0, n_act = 0, n_vis = 0, n_qtiles = 0;
    int max_vis = 0, max_tile_rows = 0;
    if (!dev_mode) {
        st->plans.assign(batch, WdSeqPlan());
        for (int b = 0; b < batch; ++b) {
            wd_status s = wd_plan_seq(st->seqs[b], A, B, R, T, &st->plans[b]);
            if (s != WD_OK) return s;
            const WdSeqPlan& p = st->plans[b];
            WdCountPlan& cp = pend.cp[b];
            cp.done = p.done; cp.refresh = p.refresh;
            cp.n_active = (int32_t)p.active.size(); cp.n_transient = (int32_t)p.transient.size();
            cp.n_vis = (int32_t)p.vis.size(); cp.n_rows = (int32_t)p.rows.size(); cp.n_wex = (int32_t)p.wex.size();
            cp.n_unmask = std::min(k_eff, cp.n_active);
            all_contig &= p.done || p.vis_contiguous;
        }
    } else {
        for (int b = 0; b < batch; ++b) {
            wd_status s = wd_count_plan(st->counts[b], A, B, R, T, k_eff, &pend.cp[b]);
            if (s != WD_OK) return s;
        }
        if (st->queue.empty()) {
            // the host mirror is current: cross-check the shadow's counts against the full planner
            for (int b = 0; b < batch; ++b) {
                WdSeqPlan p;
                if (wd_plan_seq(st->seqs[b], A, B, R, T, &p) != WD_OK) return WD_ERR_INTERNAL;
                const WdCountPlan& cp = pend.cp[b];
                if (p.done != cp.done) return WD_ERR_INTERNAL;
                if (!p.done && (p.refresh != cp.refresh || (int32_t)p.rows.size() != cp.n_rows ||
                                (int32_t)p.active.size() != cp.n_active || (int32_t)p.vis.size() != cp.n_vis ||
                                !p.vis_contiguous))
                    return WD_ERR_INTERNAL;
            }
        }
    }
    for (int b = 0; b < batch; ++b) {
        const WdCountPlan& cp = pend.cp[b];
        if (cp.done) continue;
        all_done = false;
        any_refresh |= cp.refresh;
        n_rows += cp.n_rows; n_act += cp.n_active; n_vis += cp.n_vis;
        n_qtiles += (cp.n_rows + 127) / 128;
        max_vis = std::max(max_vis, (int)cp.n_vis);
        max_tile_rows = std::max(max_tile_rows, std::min(128, (int)cp.n_rows));
    }
    if (all_done) return WD_DONE;
    if (n_rows > (size_t)d.max_rows || n_act > (size_t)d.max_active ||
        (size_t)batch * std::max(k_eff, 1) > (size_t)d.max_active)
        return WD_ERR_CAPACITY;

    // ---- pack the index lists and send them in one copy
    int32_t* ph = st->plan_host;
    size_t o = 0;
    const size_t o_row_seq = o; o += n_rows;
    const size_t o_row_pos = o; o += n_rows;
    const size_t o_act_row = o; o += n_act;
    const size_t o_act_pos = o; o += n_act;
    const size_t o_act_off = o; o += batch + 1;
    const size_t o_vis_off = o; o += batch + 1;
    const size_t o_qt_seq = o; o += n_qtiles;
    const size_t o_qt_row0 = o; o += n_qtiles;
    const size_t o_qt_n = o; o += n_qtiles;
    const size_t o_nvis = o; o += batch;
    const size_t o_tseq = o; o += batch;          // step index of each sequence (for the decode-step stamps)
    const size_t o_vis_idx = o; o += n_vis;       // last: every other offset depends on rows, active rows and tiles only
    if (o > c->plan_ints) return WD_ERR_CAPACITY;
    if (dev_mode) {
        // the device builds the lists; the host passes counts and offsets as kernel arguments
        WdPlanLaunch pl;
        memset(&pl, 0, sizeof(pl));
        pl.batch = batch; pl.S = S; pl.A = A; pl.T = T;
        int32_t r = 0, a = 0, v = 0, qt = 0;
        for (int b = 0; b < batch; ++b) {
            const WdCountPlan& cp = pend.cp[b];
            pl.row_off[b] = r; pl.act_off[b] = a; pl.vis_off[b] = v; pl.qt_off[b] = qt;
            pl.done[b] = cp.done; pl.refresh[b] = cp.refresh; pl.n_wex[b] = cp.n_wex; pl.n_vis[b] = cp.n_vis;
            pl.t[b] = st->counts[b].t;
            pl.window_refresh[b] = cp.window_refresh ? 1 : 0; pl.prev_phase_start[b] = cp.prev_phase_start;
            if (cp.done) continue;
            r += cp.n_rows; a += cp.n_active; v += cp.n_vis; qt += (cp.n_rows + 127) / 128;
        }
        pl.row_off[batch] = r; pl.act_off[batch] = a; pl.vis_off[batch] = v; pl.qt_off[batch] = qt;
        pl.decoded = st->decoded_dev; pl.dec_step = st->dec_step_dev; pl.wex = st->wex_dev;
        pl.row_seq = c->plan + o_row_seq; pl.row_pos = c->plan + o_row_pos;
        pl.act_row = c->plan + o_act_row; pl.act_pos = c->plan + o_act_pos;
        pl.act_off_dev = c->plan + o_act_off; pl.vis_off_dev = c->plan + o_vis_off; pl.vis_idx = c->plan + o_vis_idx;
        pl.qt_seq = c->plan + o_qt_seq; pl.qt_row0 = c->plan + o_qt_row0; pl.qt_n = c->plan + o_qt_n;
        pl.nvis_dev = c->plan + o_nvis; pl.tseq_dev = c->plan + o_tseq;
        pl.status = c->result;
        wd_launch_plan(pl, stream);
    } else {
        size_t r = 0, a = 0, v = 0, qt = 0;
        for (int b = 0; b < batch; ++b) {
            const WdSeqPlan& p = st->plans[b];
            ph[o_act_off + b] = (int32_t)a;
            ph[o_vis_off + b] = (int32_t)v;
            ph[o_nvis + b] = p.done ? 0 : (int32_t)p.vis.size();
            ph[o_tseq + b] = st->seqs[b].t;
            if (p.done) continue;
            for (size_t t0 = 0; t0 < p.rows.size(); t0 += 128, ++qt) {
                ph[o_qt_seq + qt] = b;
                ph[o_qt_row0 + qt] = (int32_t)(r + t0);
                ph[o_qt_n + qt] = (int32_t)std::min<size_t>(128, p.rows.size() - t0);
            }
            size_t ai = 0;
            for (size_t i = 0; i < p.rows.size(); ++i) {
                ph[o_row_seq + r] = b;
                ph[o_row_pos + r] = p.rows[i];
                if (ai < p.active.size() && p.active[ai] == p.rows[i]) {
                    ph[o_act_row + a] = (int32_t)r;
                    ph[o_act_pos + a] = p.rows[i];
                    ++a; ++ai;
                }
                ++r;
            }
            memcpy(ph + o_vis_idx + v, p.vis.data(), p.vis.size() * 4);
            v += p.vis.size();
        }
        ph[o_act_off + batch] = (int32_t)a;
        ph[o_vis_off + batch] = (int32_t)v;
        WD_CUDA_TRY(cudaMemcpyAsync(c->plan, ph, o * 4, cudaMemcpyHostToDevice, stream));
        // keep the device copy of the planner state complete (the unmask kernel maintains the flags
        // and decode steps): a refreshed external window is uploaded, so that later steps may be
        // planned on the device again
        size_t w = o;
        for (int b = 0; b < batch; ++b) {
            const WdSeqPlan& p = st->plans[b];
            if (p.done || !p.refresh || p.wex.empty()) continue;
            if (w + p.wex.size() > c->plan_ints) return WD_ERR_CAPACITY;
            memcpy(ph + w, p.wex.data(), p.wex.size() * 4);
            WD_CUDA_TRY(cudaMemcpyAsync(st->wex_dev + (size_t)b * S, ph + w, p.wex.size() * 4, cudaMemcpyHostToDevice, stream));
            w += p.wex.size();
        }
    }
    const int32_t* row_seq = c->plan + o_row_seq;
    const int32_t* row_pos = c->plan + o_row_pos;
    const int32_t* act_row = c->plan + o_act_row;
    const int32_t* act_pos = c->plan + o_act_pos;
    const int32_t* act_off = c->plan + o_act_off;
    const int32_t* vis_off = c->plan + o_vis_off;
    const int32_t* vis_idx = c->plan + o_vis_idx;
    int32_t* status = c->result;

    const int R_ = (int)n_rows, NA = (int)n_act;
    const int Hq = d.n_q_heads, Hkv = d.n_kv_heads, dh = d.head_dim, D = d.d_model, F = d.d_ffn;
    const int hq = Hq * dh, hkv = Hkv * dh;
    const long long launches0 = wd_launch_counter;
    int impl_used = WD_GEMM_PLAIN;
    c->prof_used = 0;
    c->prof_step_bytes = 0.0;
    GemmOut go;
    wd_status s;

    const int Sp = st->Sp;
    // Where the consumers of the GEMMs run (wd_set_fusion).  The fused forms need the tensor-core path,
    // head_dim 128 and widths that are multiples of 128; a mode that cannot serve the step's row count
    // falls back to the separate kernels.  The FP8 mode keeps its separate kernels.
    const bool fusable = use_tc(c) && dh == 128 && D % 128 == 0 && F % 128 == 0 && !c->fp8_on && !c->fp4_on;
    int fuse_mode = fusable ? c->fuse : WD_FUSION_NONE;
    if (fuse_mode == WD_FUSION_AUTO) fuse_mode = WD_FUSION_NONE;
    if (fuse_mode == WD_FUSION_CLUSTER && !(R_ <= wd_ck_max_rows() && D >= 256 && F >= 256 && hq >= 256)) fuse_mode = WD_FUSION_NONE;
    if (fuse_mode == WD_FUSION_CHAIN && (!wd_tc_chain_rows_ok(R_) || c->prof_on)) fuse_mode = WD_FUSION_NONE;
    const bool fused = fuse_mode != WD_FUSION_NONE;
    if (c->chain_dirty) {
        WD_CUDA_TRY(cudaMemsetAsync(c->chain.ready_dev, 0, 256, stream));
        WD_CUDA_TRY(cudaMemsetAsync(c->tile_counters, 0, c->n_tile_counters * 4, stream));
        for (int i = 0; i < 4; ++i) c->chain.ready_host[i] = 0;
        c->chain_dirty = false;
    }
    const bool fp8 = c->fp8_on && use_tc(c) && !fused;      // FP8 projections (q/k/v, gate/up, down, LM head)
    const bool fp4 = c->fp4_on && use_tc(c) && !fused;      // NVFP4 projections (the same ones)
    WdFp4Operand x4_d, x4_f, x4_lm;                         // the step's quantised activations, by use
    if (fp4) {
        wd_fp4_operand_split(c->fp4_x, R_, D, &x4_d);
        wd_fp4_operand_split(c->fp4_x, R_, F, &x4_f);
        wd_fp4_operand_split(c->fp4_x, NA, D, &x4_lm);
    }
    size_t attn_smem = 0;               // shared memory of an attention CTA (tensor-core form), for the projection after it
    auto attention = [&](int l, char* kc, char* vc) -> wd_status {
        float* attn_tap = st->taps.attn_out ? st->taps.attn_out + (size_t)l * R_ * hq : nullptr;
        if (st->attn_tc && all_contig && c->attn_impl != WD_GEMM_PLAIN)
            return wd_attn_tc_launch(c->q, R_, (int)n_qtiles, c->plan + o_qt_seq, c->plan + o_qt_row0, c->plan + o_qt_n,
                                     c->plan + o_nvis, &st->map_k, &st->map_vt, c->attn, attn_tap, Hq, Hkv, dh, l, max_vis,
                                     c->sm_count, status, stream, max_tile_rows, &attn_smem);
        wd_launch_attention_plain(d.dtype, c->q, kc, vc, row_seq, vis_idx, vis_off, c->attn, attn_tap, R_, max_vis, Hq,
                                  Hkv, dh, S, Sp, batch, status, stream);
        return WD_OK;
    };
    // ---- the kernels of the step, from the embedding to the selection (everything after the planner and
    // before the copy of the result block); launched directly, or recorded into a CUDA graph and replayed
    auto run_kernels = [&]() -> wd_status {
    c->tc.x_map_attn.smem_cap = 0;          // set per block below, and only beside the single-key-tile attention
    if (fused) {
        // Five kernels per block.  The GEMM input is bf16(x * gain) without the 1/rms factor; the CTA
        // that completes an output tile applies it (from per-block sums of squares written by the
        // previous GEMM) together with RoPE + cache scatter, SwiGLU, or the residual add.
        wd_launch_embed_fused(c->tok_embed, st->ids_dev, row_seq, row_pos, c->x, c->xn, c->attn_norm[0], c->sumsq,
                              c->rope_tab, R_, D, S, d.vocab, dh, d.rope_theta, status, stream);
        WdTcFuse base;
        base.counters = c->tile_counters;
        base.rows_total = R_;
        base.batch = batch;
        base.cluster = fuse_mode == WD_FUSION_CLUSTER ? 1 : 0;
        base.n_prev_tiles = D / 128;
        base.inv_d = 1.f / (float)D;
        base.eps = d.rms_eps;
        // The fused GEMMs between two attention calls: launched one by one, or (WD_FUSION_CHAIN) as one
        // persistent launch.
        WdTcChainItem items[4];
        WdTcSeg segbuf[4][3];
        int n_items = 0;
        auto push = [&](const WdTcX* xm, const WdTcSeg* segs, int nseg, int K, const WdTcFuse& f) {
            for (int i = 0; i < nseg; ++i) segbuf[n_items][i] = segs[i];
            items[n_items].x = xm; items[n_items].segs = segbuf[n_items]; items[n_items].nseg = nseg; items[n_items].K = K;
            items[n_items].fuse = f;
            ++n_items;
        };
        auto flush = [&]() -> wd_status {
            if (n_items == 0) return WD_OK;
            bool chained = false;
            if (fuse_mode == WD_FUSION_CHAIN && !c->prof_on && wd_tc_chain_rows_ok(R_)) {
                const wd_status cs = wd_tc_chain(items, n_items, R_, c->part, c->part_floats, c->sm_count, status, &c->chain, stream);
                if (cs == WD_OK) chained = true;
                else if (cs != WD_ERR_CAPACITY && cs != WD_ERR_BAD_PARAM) return cs;     // shapes the chain cannot take: one by one
            }
            for (int i = 0; i < n_items && !chained; ++i) {
                const wd_status gs = run_gemm(c, items[i].x->ptr, items[i].x, items[i].segs, items[i].nseg, R_, items[i].K, c->part,
                                              c->part_floats, status, stream, &go, false, &items[i].fuse);
                if (gs != WD_OK) return gs;
            }
            n_items = 0;
            return WD_OK;
        };
        impl_used = WD_GEMM_TCGEN05;
        for (int l = 0; l < d.n_layers; ++l) {
            char* kc = st->kcache + (size_t)l * st->kv_layer_bytes;
            char* vc = st->vcache + (size_t)l * st->v_layer_bytes;
            WdTcFuse fq = base;
            fq.mode = WD_FUSE_QKV;
            fq.sumsq_in = c->sumsq;
            fq.row_seq = row_seq; fq.row_pos = row_pos; fq.rope_tab = c->rope_tab;
            fq.q = (__nv_bfloat16*)c->q; fq.kcache = (__nv_bfloat16*)kc; fq.vcache = (__nv_bfloat16*)vc;
            fq.Hq = Hq; fq.Hkv = Hkv; fq.S = S; fq.Sp = Sp;
            WdTcSeg qkv[3] = {{c->wq[l], hq, c->tc.get(WD_TC_WQ, l)}, {c->wk[l], hkv, c->tc.get(WD_TC_WK, l)},
                              {c->wv[l], hkv, c->tc.get(WD_TC_WV, l)}};
            push(&c->tc.x_map_d, qkv, 3, D, fq);
            if ((s = flush()) != WD_OK) return s;
            if ((s = attention(l, kc, vc)) != WD_OK) return s;
            WdTcFuse fo = base;
            fo.mode = WD_FUSE_RESID;
            fo.x = c->x; fo.gain_next = c->ffn_norm[l]; fo.xg = (__nv_bfloat16*)c->xn; fo.sumsq_out = c->sumsq;
            WdTcSeg wo[1] = {{c->wo[l], D, c->tc.get(WD_TC_WO, l)}};
            push(&c->tc.x_map_attn, wo, 1, hq, fo);
            static const int chain_max = getenv("WD_CHAIN_MAX") ? atoi(getenv("WD_CHAIN_MAX")) : 4;    // tuning knob: GEMMs per chain launch
            if (n_items >= chain_max && (s = flush()) != WD_OK) return s;
            WdTcFuse fg = base;
            fg.mode = WD_FUSE_SWIGLU;
            fg.sumsq_in = c->sumsq; fg.h = (__nv_bfloat16*)c->h; fg.F = F;
            WdTcSeg gu[2] = {{c->wg[l], F, c->tc.get(WD_TC_WG, l)}, {c->wu[l], F, c->tc.get(WD_TC_WU, l)}};
            push(&c->tc.x_map_d, gu, 2, D, fg);
            if (n_items >= chain_max && (s = flush()) != WD_OK) return s;
            WdTcFuse fd = base;
            fd.mode = WD_FUSE_RESID;
            fd.x = c->x; fd.xg = (__nv_bfloat16*)c->xn; fd.sumsq_out = c->sumsq;
            fd.gain_next = l + 1 < d.n_layers ? c->attn_norm[l + 1] : nullptr;
            fd.tap = st->taps.layer_out ? st->taps.layer_out + (size_t)l * R_ * D : nullptr;
            WdTcSeg wdn[1] = {{c->wd[l], D, c->tc.get(WD_TC_WD, l)}};
            push(&c->tc.x_map_h, wdn, 1, F, fd);
            if (n_items >= chain_max && (s = flush()) != WD_OK) return s;
        }
        if ((s = flush()) != WD_OK) return s;
    } else {
    wd_launch_embed(d.dtype, c->tok_embed, st->ids_dev, row_seq, row_pos, c->x, c->rope_tab, R_, D, S, d.vocab, dh,
                    d.rope_theta, status, stream);
    bool down_pending = false;          // x still lacks the previous block's FFN output
    GemmOut down_go = {1, 0, 0, 0};
    for (int l = 0; l < d.n_layers; ++l) {
        char* kc = st->kcache + (size_t)l * st->kv_layer_bytes;
        char* vc = st->vcache + (size_t)l * st->v_layer_bytes;
        // attention half (FP8 mode: the normalised rows leave the RMSNorm as e4m3 codes + row scales)
        wd_launch_rmsnorm(d.dtype, c->x, down_pending ? c->part : nullptr, down_go.n_split, down_go.split_stride,
                          c->attn_norm[l], d.rms_eps, c->xn, nullptr, R_, D, stream, fp8 ? c->xn8 : nullptr, c->sxn,
                          fp4 ? &x4_d : nullptr);
        down_pending = false;
        if (fp4) {
            if ((s = run_gemm_fp4(c, &c->f4qkv[l], R_, D, c->part, c->part_floats, status, stream, &go)) != WD_OK) return s;
        } else if (fp8) {
            WdTcSeg qkv[3] = {{c->f8q[l].q, hq, &c->f8q[l].map}, {c->f8k[l].q, hkv, &c->f8k[l].map},
                              {c->f8v[l].q, hkv, &c->f8v[l].map}};
            WdTcFp8 f8;
            f8.sw[0] = c->f8q[l].s; f8.sw[1] = c->f8k[l].s; f8.sw[2] = c->f8v[l].s; f8.sx = c->sxn;
            if ((s = run_gemm(c, c->xn8, &c->x8_d, qkv, 3, R_, D, c->part, c->part_floats, status, stream, &go, false,
                              nullptr, &f8)) != WD_OK)
                return s;
        } else {
        WdTcSeg qkv[3] = {{c->wq[l], hq, c->tc.get(WD_TC_WQ, l)}, {c->wk[l], hkv, c->tc.get(WD_TC_WK, l)},
                          {c->wv[l], hkv, c->tc.get(WD_TC_WV, l)}};
        if ((s = run_gemm(c, c->xn, &c->tc.x_map_d, qkv, 3, R_, D, c->part, c->part_floats, status, stream, &go)) != WD_OK)
            return s;
        }
        impl_used = go.impl;
        wd_launch_rope_scatter(d.dtype, c->part, go.n_split, go.split_stride, row_seq, row_pos, c->rope_tab, c->q, kc,
                               vc, R_, Hq, Hkv, dh, S, Sp, batch, status, stream);
        if ((s = attention(l, kc, vc)) != WD_OK) return s;
        // the output projection's CTAs beside the attention's (when those take less than half an SM's shared
        // memory): a shorter ring, but its weights are on their way while the attention still runs
        // (measured: 215 KB for the two CTAs together still fits an SM, 222 KB does not)
        c->tc.x_map_attn.smem_cap = (attn_smem > 0 && attn_smem <= 110 * 1024 && R_ <= 128) ? (int)(223232 - attn_smem) : 0;
        WdTcSeg wo[1] = {{c->wo[l], D, c->tc.get(WD_TC_WO, l)}};
        if ((s = run_gemm(c, c->attn, &c->tc.x_map_attn, wo, 1, R_, hq, c->part, c->part_floats, status, stream, &go)) != WD_OK)
            return s;
        // feed-forward half
        wd_launch_rmsnorm(d.dtype, c->x, c->part, go.n_split, go.split_stride, c->ffn_norm[l], d.rms_eps, c->xn,
                          nullptr, R_, D, stream, fp8 ? c->xn8 : nullptr, c->sxn, fp4 ? &x4_d : nullptr);
        if (fp4) {
            if ((s = run_gemm_fp4(c, &c->f4gu[l], R_, D, c->part, c->part_floats, status, stream, &go)) != WD_OK) return s;
            if ((s = wd_launch_swiglu_fp4(c->part, go.n_split, go.split_stride, &x4_f, R_, F, stream)) != WD_OK) return s;
            if ((s = run_gemm_fp4(c, &c->f4d[l], R_, F, c->part, c->part_floats, status, stream, &go)) != WD_OK) return s;
        } else if (fp8) {
            WdTcSeg gu[2] = {{c->f8g[l].q, F, &c->f8g[l].map}, {c->f8u[l].q, F, &c->f8u[l].map}};
            WdTcFp8 f8;
            f8.sw[0] = c->f8g[l].s; f8.sw[1] = c->f8u[l].s; f8.sx = c->sxn;
            if ((s = run_gemm(c, c->xn8, &c->x8_d, gu, 2, R_, D, c->part, c->part_floats, status, stream, &go, false, nullptr,
                              &f8)) != WD_OK)
                return s;
            if ((s = wd_launch_swiglu_fp8(c->part, go.n_split, go.split_stride, c->h8, c->sh, R_, F, stream)) != WD_OK) return s;
            WdTcSeg wdn[1] = {{c->f8d[l].q, D, &c->f8d[l].map}};
            WdTcFp8 f8d;
            f8d.sw[0] = c->f8d[l].s; f8d.sx = c->sh;
            if ((s = run_gemm(c, c->h8, &c->x8_h, wdn, 1, R_, F, c->part, c->part_floats, status, stream, &go, false, nullptr,
                              &f8d)) != WD_OK)
                return s;
        } else {
        WdTcSeg gu[2] = {{c->wg[l], F, c->tc.get(WD_TC_WG, l)}, {c->wu[l], F, c->tc.get(WD_TC_WU, l)}};
        WdTcSwiglu sg;
        sg.h = use_tc(c) ? (__nv_bfloat16*)c->h : nullptr;
        if ((s = run_gemm(c, c->xn, &c->tc.x_map_d, gu, 2, R_, D, c->part, c->part_floats, status, stream, &go, false,
                          nullptr, nullptr, &sg)) != WD_OK)
            return s;
        if (!sg.done) wd_launch_swiglu(d.dtype, c->part, go.n_split, go.split_stride, c->h, R_, F, stream);
        WdTcSeg wdn[1] = {{c->wd[l], D, c->tc.get(WD_TC_WD, l)}};
        if ((s = run_gemm(c, c->h, &c->tc.x_map_h, wdn, 1, R_, F, c->part, c->part_floats, status, stream, &go)) != WD_OK)
            return s;
        }
        if (st->taps.layer_out || l == d.n_layers - 1) {
            float* tap = st->taps.layer_out ? st->taps.layer_out + (size_t)l * R_ * D : nullptr;
            wd_launch_residual_add(c->x, c->part, go.n_split, go.split_stride, tap, R_, D, stream);
        } else {
            down_pending = true;     // folded into the next block's RMSNorm
            down_go = go;
        }
    }
    }
    // logits for the active rows only, then the unmask reduction
    bool lm_fused = false;
    int lm_chunks = wd_unmask_chunks(d.vocab);
    if (NA > 0) {
        wd_launch_rmsnorm(d.dtype, c->x, nullptr, 0, 0, c->final_norm, d.rms_eps, c->xn, act_row, NA, D, stream,
                          fp8 ? c->xn8 : nullptr, c->sxn, fp4 ? &x4_lm : nullptr);
        WdTcSeg lm[1] = {{c->lm_head, d.vocab, c->tc.get(WD_TC_LM, 0)}};
        WdTcFp8 f8lm;
        if (fp8) {
            lm[0] = {c->f8lm.q, d.vocab, &c->f8lm.map};
            f8lm.sw[0] = c->f8lm.s; f8lm.sx = c->sxn;
        }
        // tensor-core path: the LM-head epilogue leaves per-tile (max, argmax, sum exp) instead of a separate
        // pass over the logits, which then never have to be written (only for the parity tap)
        WdTcFuse fl;
        fl.mode = WD_FUSE_LMSTATS;
        fl.st_max = c->ch_max; fl.st_idx = c->ch_idx; fl.st_sum = c->ch_sum;
        fl.write_logits = st->taps.logits ? 1 : 0;
        lm_fused = use_tc(c) && NA <= 1024 && c->sm_count % 4 == 0 && !fp4;     // one CTA group per tile of <= 256 active rows
        if (fp4) {
            if ((s = run_gemm_fp4(c, &c->f4lm, NA, D, c->logits, (size_t)d.max_active * d.vocab, status, stream, &go,
                                  /*single_split=*/true)) != WD_OK)
                return s;
        } else if ((s = run_gemm(c, fp8 ? (const void*)c->xn8 : c->xn, fp8 ? &c->x8_d : &c->tc.x_map_d, lm, 1, NA, D, c->logits,
                          (size_t)d.max_active * d.vocab, status, stream, &go, /*single_split=*/true,
                          lm_fused ? &fl : nullptr, fp8 ? &f8lm : nullptr)) != WD_OK)
            return s;
        if (lm_fused) lm_chunks = fl.n_chunks;
        else wd_launch_rowstats(c->logits, NA, d.vocab, c->ch_max, c->ch_idx, c->ch_sum, stream);
        if (st->taps.logits)
            WD_CUDA_TRY(cudaMemcpyAsync(st->taps.logits, c->logits, (size_t)NA * d.vocab * 4, cudaMemcpyDeviceToDevice,
                                        stream));
    }
    int32_t* n_sel = c->result + 1;
    int32_t* sel_pos = n_sel + batch;
    int32_t* sel_tok = sel_pos + (size_t)batch * std::max(k_eff, 1);
    float* sel_conf = (float*)(sel_tok + (size_t)batch * std::max(k_eff, 1));
    wd_launch_select(c->ch_max, c->ch_idx, c->ch_sum, lm_chunks, c->row_token, c->row_sumexp, act_pos,
                     act_off, 0, batch, k_eff, st->ids_dev, S, n_sel, sel_pos, sel_tok, sel_conf, c->row_conf,
                     st->decoded_dev, st->dec_step_dev, c->plan + o_tseq, stream);
    return WD_OK;
    };
    // A device-planned step whose launch configuration has occurred before is replayed from a graph: the
    // kernels' arguments depend only on the key below (the index lists, the per-sequence visible counts and the
    // step indices live in device memory, written by the planner kernel, which stays outside the graph).
    // Measured: 3.5 % off a 34-row step (kernel boundaries resolve faster inside a graph).
    bool graphed = false;
    int stream_capturing = 0;
    {
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(stream, &cs) != cudaSuccess) { cudaGetLastError(); cs = cudaStreamCaptureStatusActive; }
        stream_capturing = cs != cudaStreamCaptureStatusNone;
    }
    const bool taps_on = st->taps.layer_out || st->taps.attn_out || st->taps.logits;
    // Only while earlier steps are still queued: the GPU then has work while the host records or submits the
    // graph.  With an empty queue (a caller that syncs after every step) direct launches win, because the GPU
    // starts on the first kernels while the host is still launching the later ones (measured: 230 against 227
    // tokens/s end to end).
    // The tensor-core attention only: the index-list kernel sizes its shared memory by the exact visible count,
    // which a recorded launch would keep while the count grows.
    const bool attn_by_tc = st->attn_tc && all_contig && c->attn_impl != WD_GEMM_PLAIN;
    if (c->graphs_on && dev_mode && !c->prof_on && !taps_on && !fused && !stream_capturing && use_tc(c) && attn_by_tc &&
        !st->queue.empty()) {
        wd_ctx::StepKey key;
        key.state_uid = st->uid; key.batch = batch; key.rows = R_; key.n_act = NA; key.n_qtiles = (int)n_qtiles;
        key.key_tiles = (max_vis + 127) / 128; key.max_tile_rows = max_tile_rows; key.k_eff = k_eff;
        key.mode = (c->fp8_on ? 1 : 0) | (c->fp4_on ? 2 : 0) | (st->attn_tc ? 4 : 0);
        key.impl = c->gemm_impl; key.attn_impl = c->attn_impl;
        wd_ctx::StepGraph* hit = nullptr;
        for (wd_ctx::StepGraph& g : c->graphs) if (g.key == key) { hit = &g; break; }
        if (hit) {
            WD_CUDA_TRY(cudaGraphLaunch(hit->exec, stream));
            hit->last_use = ++c->graph_clock;
            wd_launch_counter += hit->n_kernels;
            impl_used = hit->impl_used;
            ++c->graphs_replayed;
            graphed = true;
        } else {
            // a refresh step's configuration rarely comes back (its rows grow with every phase), and neither does
            // that of a step near the end of a generation, whose active window shrinks by the tokens unmasked every
            // step: record those only when they do come back; a normal step with full windows recurs for many
            // phases: record it at once
            int live = 0;
            for (int b = 0; b < batch; ++b) live += pend.cp[b].done ? 0 : 1;
            bool seen = !any_refresh && NA == A * live;
            for (const wd_ctx::StepKey& k2 : c->seen) if (k2 == key) { seen = true; break; }
            if (!seen) {
                if (c->seen.size() >= 32) c->seen.erase(c->seen.begin());
                c->seen.push_back(key);
            } else if (cudaStreamBeginCapture(stream, cudaStreamCaptureModeRelaxed) == cudaSuccess) {
                static const bool gdbg = getenv("WD_GRAPH_DEBUG") != nullptr;
                const long long k0 = wd_launch_counter;
                const wd_status rs = run_kernels();
                cudaGraph_t graph = nullptr;
                const cudaError_t ce = cudaStreamEndCapture(stream, &graph);
                if (gdbg) fprintf(stderr, "wd graph: run %d end-capture %s graph %p\n", (int)rs, cudaGetErrorString(ce), (void*)graph);
                if (rs != WD_OK) {
                    if (graph) cudaGraphDestroy(graph);
                    cudaGetLastError();
                    return rs;
                }
                cudaGraphExec_t exec = nullptr;
                cudaError_t ie = cudaErrorUnknown;
                if (ce == cudaSuccess && graph) ie = cudaGraphInstantiate(&exec, graph, 0);
                if (gdbg) fprintf(stderr, "wd graph: instantiate %s\n", cudaGetErrorString(ie));
                if (ie == cudaSuccess) {
                    cudaGraphDestroy(graph);
                    wd_ctx::StepGraph g;
                    g.key = key; g.exec = exec; g.n_kernels = (int)(wd_launch_counter - k0); g.impl_used = impl_used;
                    g.last_use = ++c->graph_clock;
                    static const size_t kMaxGraphs = 8;
                    if (c->graphs.size() >= kMaxGraphs) {
                        size_t lru = 0;
                        for (size_t i = 1; i < c->graphs.size(); ++i) if (c->graphs[i].last_use < c->graphs[lru].last_use) lru = i;
                        cudaGraphExecDestroy(c->graphs[lru].exec);
                        c->graphs[lru] = g;
                    } else {
                        c->graphs.push_back(g);
                    }
                    WD_CUDA_TRY(cudaGraphLaunch(exec, stream));
                    ++c->graphs_captured;
                    graphed = true;
                } else {
                    // the capture could not be turned into a graph: nothing has run yet, launch directly
                    if (graph) cudaGraphDestroy(graph);
                    cudaGetLastError();
                    wd_launch_counter = k0;
                    if (++c->graph_failures >= 3) c->graphs_on = false;      // not on this system: stop trying
                }
            } else {
                if (getenv("WD_GRAPH_DEBUG")) fprintf(stderr, "wd graph: begin-capture %s\n", cudaGetErrorString(cudaPeekAtLastError()));
                cudaGetLastError();
            }
        }
    }
    if (!graphed && (s = run_kernels()) != WD_OK) return s;
    // this step's result block goes to its own slot of the pinned ring
    const size_t res_ints = 1 + (size_t)batch + 3 * (size_t)batch * std::max(k_eff, 1);
    int32_t* slot = st->result_host + st->queue.size() * st->result_slot_ints;
    WD_CUDA_TRY(cudaMemcpyAsync(slot, c->result, res_ints * 4, cudaMemcpyDeviceToHost, stream));
    WD_CUDA_TRY(cudaEventRecord(st->done, stream));
    WD_CUDA_TRY(cudaGetLastError());
    if (!dev_mode) pend.plans = st->plans;
    else for (int b = 0; b < batch; ++b) wd_count_commit(st->counts[b], pend.cp[b]);
    st->queue.push_back(std::move(pend));
    st->pending = true;
    if (info) {
        info->is_refresh = any_refresh ? 1 : 0;
        info->n_rows = R_; info->n_active = NA; info->n_vis = (int32_t)n_vis;
        info->n_launches = (int32_t)(wd_launch_counter - launches0); info->gemm_impl = impl_used;
    }
    return WD_OK;
}

// Completes every enqueued step, oldest first: reads its result block, re-plans it on the host
// mirror (which the previous step's results have just brought up to date) and commits.
static wd_status drain_queue(wd_state* st, wd_step_out* outs, bool every_step, int32_t* n_done) {
    WD_CUDA_TRY(cudaEventSynchronize(st->done));
    if (st->ctx->prof_on) {
        wd_ctx* c = st->ctx;
        for (size_t i = 0; i + 1 < c->prof_used; i += 2) {
            float ms = 0.f;
            if (cudaEventElapsedTime(&ms, c->prof_events[i], c->prof_events[i + 1]) == cudaSuccess) c->prof_ms += ms;
            c->prof_launches += 1;
        }
        c->prof_bytes += c->prof_step_bytes;
    }
    const int batch = st->batch;
    wd_status result = WD_OK;
    int32_t done = 0;
    for (size_t q = 0; q < st->queue.size(); ++q) {
        const wd_state::Pending& pd = st->queue[q];
        const int k = pd.k_eff, kk = std::max(k, 1), ku = pd.k_user;
        const int32_t* res = st->result_host + q * st->result_slot_ints;
        const int32_t* n_sel = res + 1;
        const int32_t* pos = n_sel + batch;
        const int32_t* tok = pos + (size_t)batch * kk;
        const float* conf = (const float*)(tok + (size_t)batch * kk);
        if (res[0] != 0) {
            cudaMemset(st->ctx->result, 0, 4);
            result = res[0] == WD_ERR_DEVICE_TIMEOUT ? WD_ERR_DEVICE_TIMEOUT : WD_ERR_BOUNDS;
            break;
        }
        // which out block receives this step: all of them in order, or only the newest
        wd_step_out* out = nullptr;
        if (outs) out = every_step ? &outs[done] : (q + 1 == st->queue.size() ? outs : nullptr);
        for (int b = 0; b < batch; ++b) {
            WdSeqPlan replanned;
            const WdSeqPlan* p = pd.host_planned ? &pd.plans[b] : &replanned;
            if (!pd.host_planned) {
                if (wd_plan_seq(st->seqs[b], pd.A, pd.B, pd.R, pd.T, &replanned) != WD_OK) { result = WD_ERR_INTERNAL; break; }
                const WdCountPlan& cp = pd.cp[b];
                if (replanned.done != cp.done ||
                    (!cp.done && ((int32_t)replanned.rows.size() != cp.n_rows || replanned.refresh != cp.refresh))) {
                    result = WD_ERR_INTERNAL;
                    break;
                }
            }
            const int n = p->done ? 0 : std::min(n_sel[b], k);
            if (!p->done) wd_commit_seq(st->seqs[b], *p, pos + (size_t)b * k, tok + (size_t)b * k, n);
            if (out) {
                if (out->n_unmasked) out->n_unmasked[b] = n;
                for (int i = 0; i < n; ++i) {
                    if (out->positions) out->positions[(size_t)b * ku + i] = pos[(size_t)b * k + i];
                    if (out->token_ids) out->token_ids[(size_t)b * ku + i] = tok[(size_t)b * k + i];
                    if (out->confidence) out->confidence[(size_t)b * ku + i] = conf[(size_t)b * k + i];
                }
            }
        }
        if (result != WD_OK) break;
        ++done;
    }
    const bool host_planned = !st->queue.empty() && st->queue.back().host_planned;
    st->queue.clear();
    st->pending = false;
    if (result != WD_OK) {
        // Steps queued behind the failed one have already run on the device, so the device copy of the
        // state (ids, flags, decode steps, K/V cache) may be ahead of the host mirror, or built on garbage:
        // the state takes no more steps until wd_state_reset or wd_state_import gives it a consistent start.
        st->dev_mode = false;
        st->poisoned = true;
        st->ctx->chain_dirty = true;
    }
    else if (host_planned)    // the count shadow did not follow host-planned steps: rebuild it from the mirror
        for (int b = 0; b < batch; ++b) wd_count_init(st->counts[b], st->seqs[b]);
    if (n_done) *n_done = done;
    return result;
}

extern "C" wd_status wd_step_sync(wd_state* st, wd_step_out* out) {
    if (!st) return WD_ERR_NULL;
    if (st->queue.empty()) return WD_ERR_NOT_PENDING;
    return drain_queue(st, out, false, nullptr);
}

extern "C" wd_status wd_step_sync_all(wd_state* st, wd_step_out* outs, int32_t capacity, int32_t* n_steps) {
    if (!st) return WD_ERR_NULL;
    if (capacity < 0 || (capacity > 0 && !outs)) return WD_ERR_BAD_PARAM;
    if (st->queue.empty()) return WD_ERR_NOT_PENDING;
    if (capacity > 0 && (int32_t)st->queue.size() > capacity) return WD_ERR_CAPACITY;
    return drain_queue(st, capacity > 0 ? outs : nullptr, true, n_steps);
}

extern "C" wd_status wd_generate(wd_state* st, int32_t A, int32_t B, int32_t R, int32_t T, int32_t k, int32_t max_steps,
                                 void* stream, int32_t* n_steps, int32_t* n_tokens) {
    if (!st) return WD_ERR_NULL;
    if (!st->queue.empty()) return WD_ERR_PENDING;
    if (st->poisoned) return WD_ERR_POISONED;
    if (n_steps) *n_steps = 0;
    if (n_tokens) *n_tokens = 0;
    int32_t steps = 0;
    long long before = 0, after = 0;
    for (const WdSeq& s : st->seqs)
        for (uint8_t d : s.decoded) before += d;
    wd_status result = WD_OK;
    bool finished = false;
    while (max_steps <= 0 || steps < max_steps) {
        wd_step_info info;
        wd_status s = wd_step(st, A, B, R, T, k, stream, &info);
        if (s == WD_ERR_PENDING && !st->queue.empty()) {        // queue full, or one host-planned step in flight
            if ((s = drain_queue(st, nullptr, true, nullptr)) != WD_OK) { result = s; break; }
            continue;
        }
        if (s == WD_DONE) {
            // the count shadow says nothing is left; with steps still in flight the mirror confirms it below
            finished = true;
            break;
        }
        if (s != WD_OK) { result = s; break; }
        ++steps;
    }
    if (!st->queue.empty()) {
        const wd_status s = drain_queue(st, nullptr, true, nullptr);
        if (result == WD_OK && s != WD_OK) result = s;
    }
    for (const WdSeq& s : st->seqs)
        for (uint8_t d : s.decoded) after += d;
    if (n_steps) *n_steps = steps;
    if (n_tokens) *n_tokens = (int32_t)(after - before);
    if (result != WD_OK) return result;
    return finished ? WD_DONE : WD_OK;
}

// ---------------------------------------------------------------------------
// single operations
// ---------------------------------------------------------------------------
extern "C" size_t wd_op_gemm_scratch_bytes(int32_t rows, int32_t n_out, int32_t k_in) {
    if (rows < 1 || n_out < 1 || k_in < 1) return 0;
    return wd_tc_scratch_bytes(rows, n_out, k_in);
}

extern "C" size_t wd_op_gemm_fp8_scratch_bytes(int32_t rows, int32_t n_out, int32_t k_in) {
    if (rows < 1 || n_out < 1 || k_in < 1) return 0;
    return wd_align_up((size_t)rows * k_in, 256) + wd_align_up((size_t)rows * 4, 256) + wd_align_up((size_t)n_out * k_in, 256) +
           wd_align_up((size_t)n_out * 4, 256) + wd_tc_scratch_bytes(rows, n_out, k_in);
}

extern "C" wd_status wd_op_gemm_fp8(const void* x, const void* w, float* y, int32_t rows, int32_t n_out, int32_t k_in,
                                    void* scratch, size_t scratch_bytes, void* stream_) {
    if (!x || !w || !y || !scratch) return WD_ERR_NULL;
    if (rows < 1 || n_out < 1 || k_in < 16 || k_in % 16) return WD_ERR_BAD_PARAM;
    if ((uintptr_t)scratch % 256) return WD_ERR_MISALIGNED;
    if (scratch_bytes < wd_op_gemm_fp8_scratch_bytes(rows, n_out, k_in)) return WD_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t stream = (cudaStream_t)stream_;
    char* p = (char*)scratch;
    uint8_t* xq = (uint8_t*)p; p += wd_align_up((size_t)rows * k_in, 256);
    float* sx = (float*)p; p += wd_align_up((size_t)rows * 4, 256);
    uint8_t* wq = (uint8_t*)p; p += wd_align_up((size_t)n_out * k_in, 256);
    float* sw = (float*)p; p += wd_align_up((size_t)n_out * 4, 256);
    wd_launch_quantize_rows(WD_BF16, x, rows, k_in, xq, sx, stream);
    wd_launch_quantize_rows(WD_BF16, w, n_out, k_in, wq, sw, stream);
    WD_CUDA_TRY(cudaGetLastError());
    return wd_tc_gemm_standalone_fp8(xq, sx, wq, sw, y, rows, n_out, k_in, (float*)p, wd_tc_scratch_bytes(rows, n_out, k_in) / 4,
                                     stream);
}

extern "C" size_t wd_op_gemm_fp4_scratch_bytes(int32_t rows, int32_t n_out, int32_t k_in) {
    if (rows < 1 || n_out < 1 || k_in < 256 || k_in % 256) return 0;
    return wd_fp4_operand_bytes(rows, k_in) + wd_fp4_operand_bytes(n_out, k_in) + wd_tc_scratch_bytes(rows, n_out, k_in);
}

extern "C" wd_status wd_op_gemm_fp4(const void* x, const void* w, float* y, int32_t rows, int32_t n_out, int32_t k_in,
                                    void* scratch, size_t scratch_bytes, void* stream_) {
    if (!x || !w || !y || !scratch) return WD_ERR_NULL;
    if (rows < 1 || n_out < 1 || k_in < 256 || k_in % 256) return WD_ERR_BAD_PARAM;
    if ((uintptr_t)scratch % 256) return WD_ERR_MISALIGNED;
    if (scratch_bytes < wd_op_gemm_fp4_scratch_bytes(rows, n_out, k_in)) return WD_ERR_WORKSPACE_TOO_SMALL;
    int32_t* status = wd_op_status_ptr();
    if (!status) return WD_ERR_CUDA;
    cudaStream_t stream = (cudaStream_t)stream_;
    int sm = 148, dev = 0;
    WD_CUDA_TRY(cudaGetDevice(&dev));
    WD_CUDA_TRY(cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev));
    WdFp4Operand ox, ow;
    char* p = (char*)scratch;
    wd_fp4_operand_split(p, rows, k_in, &ox); p += wd_fp4_operand_bytes(rows, k_in);
    wd_fp4_operand_split(p, n_out, k_in, &ow); p += wd_fp4_operand_bytes(n_out, k_in);
    wd_launch_quantize_nvfp4(WD_BF16, x, rows, k_in, &ox, stream);
    wd_launch_quantize_nvfp4(WD_BF16, w, n_out, k_in, &ow, stream);
    WD_CUDA_TRY(cudaGetLastError());
    int ns = 1;
    const size_t slice = (size_t)rows * n_out;
    wd_status s = wd_fp4_gemm(&ox, &ow, (float*)p, wd_tc_scratch_bytes(rows, n_out, k_in) / 4, sm, status, stream, &ns, false, false);
    if (s != WD_OK) return s;
    wd_launch_reduce_slices((const float*)p, ns, slice, y, slice, stream);
    WD_CUDA_TRY(cudaGetLastError());
    return WD_OK;
}

extern "C" size_t wd_op_nvfp4_bytes(int32_t rows, int32_t k_in) {
    if (rows < 1 || k_in < 16 || k_in % 16) return 0;
    return wd_fp4_operand_bytes(rows, k_in);
}

extern "C" wd_status wd_op_nvfp4_quantize(const void* x, int32_t rows, int32_t k_in, void* out, size_t out_bytes, void* stream_) {
    if (!x || !out) return WD_ERR_NULL;
    if (rows < 1 || k_in < 16 || k_in % 16) return WD_ERR_BAD_PARAM;
    if ((uintptr_t)out % 256) return WD_ERR_MISALIGNED;
    if (out_bytes < wd_fp4_operand_bytes(rows, k_in)) return WD_ERR_WORKSPACE_TOO_SMALL;
    WdFp4Operand op;
    wd_fp4_operand_split(out, rows, k_in, &op);
    wd_launch_quantize_nvfp4(WD_BF16, x, rows, k_in, &op, (cudaStream_t)stream_);
    WD_CUDA_TRY(cudaGetLastError());
    return WD_OK;
}

extern "C" wd_status wd_op_gemm_nvfp4(const void* xq, const void* wq, float* y, int32_t rows, int32_t n_out, int32_t k_in,
                                      void* scratch, size_t scratch_bytes, void* stream_) {
    if (!xq || !wq || !y || !scratch) return WD_ERR_NULL;
    if (rows < 1 || n_out < 1 || k_in < 256 || k_in % 256) return WD_ERR_BAD_PARAM;
    if ((uintptr_t)scratch % 256 || (uintptr_t)xq % 256 || (uintptr_t)wq % 256) return WD_ERR_MISALIGNED;
    if (scratch_bytes < wd_tc_scratch_bytes(rows, n_out, k_in)) return WD_ERR_WORKSPACE_TOO_SMALL;
    int32_t* status = wd_op_status_ptr();
    if (!status) return WD_ERR_CUDA;
    cudaStream_t stream = (cudaStream_t)stream_;
    int sm = 148, dev = 0;
    WD_CUDA_TRY(cudaGetDevice(&dev));
    WD_CUDA_TRY(cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev));
    WdFp4Operand ox, ow;
    wd_fp4_operand_split(const_cast<void*>(xq), rows, k_in, &ox);
    wd_fp4_operand_split(const_cast<void*>(wq), n_out, k_in, &ow);
    int ns = 1;
    const size_t slice = (size_t)rows * n_out;
    wd_status s = wd_fp4_gemm(&ox, &ow, (float*)scratch, scratch_bytes / 4, sm, status, stream, &ns, false, false);
    if (s != WD_OK) return s;
    wd_launch_reduce_slices((const float*)scratch, ns, slice, y, slice, stream);
    WD_CUDA_TRY(cudaGetLastError());
    return WD_OK;
}

extern "C" wd_status wd_op_gemm(int32_t dtype, int32_t impl, const void* x, const void* w, float* y, int32_t rows,
                                int32_t n_out, int32_t k_in, void* scratch, size_t scratch_bytes, void* stream) {
    if (!x || !w || !y) return WD_ERR_NULL;
    if (rows < 1 || n_out < 1 || k_in < 1) return WD_ERR_BAD_PARAM;
    if (dtype != WD_F32 && dtype != WD_BF16) return WD_ERR_BAD_PARAM;
    if (impl == WD_GEMM_AUTO) impl = dtype == WD_BF16 ? WD_GEMM_TCGEN05 : WD_GEMM_PLAIN;
    if (impl == WD_GEMM_PLAIN) {
        wd_launch_gemm_plain(dtype, x, w, y, rows, n_out, k_in, n_out, (cudaStream_t)stream);
        WD_CUDA_TRY(cudaGetLastError());
        return WD_OK;
    }
    if (impl != WD_GEMM_TCGEN05 || dtype != WD_BF16) return WD_ERR_BAD_PARAM;
    return wd_tc_gemm_standalone(x, w, y, rows, n_out, k_in, scratch, scratch_bytes, (cudaStream_t)stream);
}

extern "C" wd_status wd_op_attention(int32_t dtype, const void* q, const void* kcache, const void* vcache,
                                     const int32_t* vis, void* out, int32_t n_rows, int32_t n_vis,
                                     int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int32_t seq_len,
                                     void* stream) {
    if (!q || !kcache || !vcache || !vis || !out) return WD_ERR_NULL;
    if (dtype != WD_F32 && dtype != WD_BF16) return WD_ERR_BAD_PARAM;
    if (n_rows < 1 || n_vis < 1 || n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads || head_dim < 1 ||
        seq_len < n_vis)
        return WD_ERR_BAD_PARAM;
    if ((size_t)(n_vis + head_dim) * 4 > 200 * 1024) return WD_ERR_CAPACITY;
    int32_t* op_status = wd_op_status_ptr();
    if (!op_status) return WD_ERR_CUDA;
    // one sequence: no row->sequence table and no offsets, every row sees vis[0, n_vis)
    wd_launch_attention_plain(dtype, q, kcache, vcache, nullptr, vis, nullptr, out, nullptr, n_rows, n_vis, n_q_heads,
                              n_kv_heads, head_dim, seq_len, seq_len, 1, op_status, (cudaStream_t)stream);
    WD_CUDA_TRY(cudaGetLastError());
    return WD_OK;
}

extern "C" size_t wd_op_attention_tc_scratch_bytes(int32_t n_rows) {
    if (n_rows < 1) return 0;
    return wd_align_up((size_t)(3 * ((n_rows + 127) / 128) + 1) * 4, 256);
}

extern "C" wd_status wd_op_attention_tc(const void* q, const void* kcache, const void* vcache_t, void* out,
                                        int32_t n_rows, int32_t n_vis, int32_t max_vis, int32_t n_q_heads,
                                        int32_t n_kv_heads, int32_t seq_len, void* scratch, size_t scratch_bytes,
                                        void* stream_) {
    if (!q || !kcache || !vcache_t || !out || !scratch) return WD_ERR_NULL;
    if (n_rows < 1 || n_vis < 1 || n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads || seq_len < n_vis ||
        max_vis < n_vis || seq_len % 8)
        return WD_ERR_BAD_PARAM;
    if (((uintptr_t)q | (uintptr_t)kcache | (uintptr_t)vcache_t | (uintptr_t)out) % 16 || (uintptr_t)scratch % 4)
        return WD_ERR_MISALIGNED;
    if (scratch_bytes < wd_op_attention_tc_scratch_bytes(n_rows)) return WD_ERR_WORKSPACE_TOO_SMALL;
    int32_t* status = wd_op_status_ptr();
    if (!status) return WD_ERR_CUDA;
    cudaStream_t stream = (cudaStream_t)stream_;
    int sm = 148, dev = 0;
    WD_CUDA_TRY(cudaGetDevice(&dev));
    WD_CUDA_TRY(cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev));
    CUtensorMap map_k, map_vt;
    wd_status s = wd_attn_tc_encode_cache(&map_k, &map_vt, kcache, vcache_t, 1, n_kv_heads, seq_len, seq_len, 128);
    if (s != WD_OK) return s;
    const int n_tiles = (n_rows + 127) / 128;
    int32_t* lists = (int32_t*)scratch;
    wd_launch_fill_qtiles(lists, n_rows, n_vis, stream);
    WD_CUDA_TRY(cudaGetLastError());
    return wd_attn_tc_launch(q, n_rows, n_tiles, lists, lists + n_tiles, lists + 2 * n_tiles, lists + 3 * n_tiles, &map_k,
                             &map_vt, out, nullptr, n_q_heads, n_kv_heads, 128, 0, max_vis, sm, status, stream,
                             std::min(n_rows, 128));
}

extern "C" size_t wd_op_lm_unmask_scratch_bytes(int32_t n, int32_t vocab) {
    if (n < 1 || vocab < 1) return 0;
    // one statistics entry per (row, CTA of the LM-head launch), at most 256 CTAs
    return (size_t)n * 256 * 16;
}

extern "C" wd_status wd_op_lm_unmask(const void* x, const void* w, const int32_t* positions, int32_t n, int32_t vocab,
                                     int32_t k_in, int32_t k, float* logits, int32_t* row_token, double* row_sumexp,
                                     float* row_conf, int32_t* sel_pos, int32_t* sel_token, float* sel_conf,
                                     int32_t* n_sel, void* scratch, size_t scratch_bytes, void* stream_) {
    if (!x || !w || !positions || !logits || !row_token || !row_sumexp || !row_conf || !sel_pos || !sel_token ||
        !sel_conf || !n_sel || !scratch)
        return WD_ERR_NULL;
    if (n < 1 || vocab < 1 || k < 0 || k_in < 8 || k_in % 8) return WD_ERR_BAD_PARAM;
    if (n > 1024) return WD_ERR_CAPACITY;
    if (scratch_bytes < wd_op_lm_unmask_scratch_bytes(n, vocab)) return WD_ERR_WORKSPACE_TOO_SMALL;
    if ((uintptr_t)scratch % 8 || ((uintptr_t)x | (uintptr_t)w) % 16) return WD_ERR_MISALIGNED;
    int32_t* status = wd_op_status_ptr();
    if (!status) return WD_ERR_CUDA;
    cudaStream_t stream = (cudaStream_t)stream_;
    int sm = 148, dev = 0;
    WD_CUDA_TRY(cudaGetDevice(&dev));
    WD_CUDA_TRY(cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev));
    if (sm % 4 || sm > 256) return WD_ERR_UNSUPPORTED_ARCH;     // the launch puts one CTA group on each of up to four token tiles
    double* ch_sum = (double*)scratch;
    float* ch_max = (float*)(ch_sum + (size_t)n * 256);
    int32_t* ch_idx = (int32_t*)(ch_max + (size_t)n * 256);
    CUtensorMap mw;
    wd_status s = wd_tc_encode_bf16(&mw, w, vocab, k_in, 128);
    if (s != WD_OK) return s;
    WdTcSeg seg = {w, vocab, &mw};
    WdTcX xm;
    xm.ptr = x; xm.K = k_in; xm.keep = false;
    WdTcFuse fl;
    fl.mode = WD_FUSE_LMSTATS;
    fl.st_max = ch_max; fl.st_idx = ch_idx; fl.st_sum = ch_sum;
    fl.write_logits = 1;
    int ns = 1;
    s = wd_tc_gemm(&xm, &seg, 1, n, k_in, logits, (size_t)n * vocab, sm, status, stream, &ns, /*single split*/ true, &fl);
    if (s != WD_OK) return s;
    wd_launch_select(ch_max, ch_idx, ch_sum, fl.n_chunks, row_token, row_sumexp, positions, nullptr, n, 1, k, nullptr, 0,
                     n_sel, sel_pos, sel_token, sel_conf, row_conf, nullptr, nullptr, nullptr, stream);
    WD_CUDA_TRY(cudaGetLastError());
    return WD_OK;
}

extern "C" size_t wd_op_unmask_scratch_bytes(int32_t n, int32_t vocab) {
    if (n < 1 || vocab < 1) return 0;
    return (size_t)n * wd_unmask_chunks(vocab) * 16;
}

extern "C" wd_status wd_op_unmask(const float* logits, const int32_t* positions, int32_t n, int32_t vocab, int32_t k,
                                  int32_t* row_token, double* row_sumexp, float* row_conf, int32_t* sel_pos,
                                  int32_t* sel_token, float* sel_conf, int32_t* n_sel, void* scratch,
                                  size_t scratch_bytes, void* stream) {
    if (!logits || !positions || !row_token || !row_sumexp || !row_conf || !sel_pos || !sel_token || !sel_conf ||
        !n_sel || !scratch)
        return WD_ERR_NULL;
    if (n < 1 || vocab < 1 || k < 0) return WD_ERR_BAD_PARAM;
    if (scratch_bytes < wd_op_unmask_scratch_bytes(n, vocab)) return WD_ERR_WORKSPACE_TOO_SMALL;
    if ((uintptr_t)scratch % 8) return WD_ERR_MISALIGNED;
    cudaStream_t st = (cudaStream_t)stream;
    const int nch = wd_unmask_chunks(vocab);
    double* ch_sum = (double*)scratch;
    float* ch_max = (float*)(ch_sum + (size_t)n * nch);
    int32_t* ch_idx = (int32_t*)(ch_max + (size_t)n * nch);
    wd_launch_rowstats(logits, n, vocab, ch_max, ch_idx, ch_sum, st);
    wd_launch_select(ch_max, ch_idx, ch_sum, nch, row_token, row_sumexp, positions, nullptr, n, 1, k, nullptr, 0, n_sel,
                     sel_pos, sel_token, sel_conf, row_conf, nullptr, nullptr, nullptr, st);
    WD_CUDA_TRY(cudaGetLastError());
    return WD_OK;
}

extern "C" wd_status wd_debug_wait_expire(void* stream) { return wd_launch_wait_expire((cudaStream_t)stream); }

extern "C" wd_status wd_op_status(void) {
    int32_t* p = wd_op_status_ptr();
    if (!p) return WD_ERR_CUDA;
    WD_CUDA_TRY(cudaDeviceSynchronize());
    int32_t v = 0;
    WD_CUDA_TRY(cudaMemcpy(&v, p, 4, cudaMemcpyDeviceToHost));
    if (v != 0) cudaMemset(p, 0, 4);
    return v;
}
