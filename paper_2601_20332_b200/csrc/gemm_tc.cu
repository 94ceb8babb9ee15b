// Weight-streaming GEMM on the 5th-generation tensor cores (sm_100a).
//
//   y[tok, n] = sum_k x[tok, k] * w[n, k]          x: [rows, K] bf16, w: [n, K] bf16, y fp32
//
// The window holds few tokens, so the GEMMs of a normal step are bound by reading
// the weights once from HBM.  The kernel therefore puts the WEIGHT rows on the MMA's
// M = 128 axis and the tokens on its N axis (16..256), so no tensor-core rows are
// wasted on padding, and splits K across CTAs so that every SM streams weights:
//
//   grid = (weight tiles of 128 rows, token tiles of BN, K slices)
//   warp 0   TMA producer: [128 x 64] weight boxes and [BN x 64] activation boxes into a
//            ring of shared-memory stages (128-byte swizzle), completion on mbarriers
//   warp 1   allocates TMEM, issues tcgen05.mma (kind::f16, bf16 in, fp32 accumulate in
//            TMEM), releases stages with tcgen05.commit
//   warps 2-5 epilogue: tcgen05.ld of the [128 x BN] accumulator, coalesced fp32 stores
//            of this K slice's partial sums
//
// Split-K partial sums are written side by side ([slice][tok][n]); the kernel that
// consumes the GEMM output adds them, which keeps the result deterministic.
// Every wait is bounded: on expiry the CTA records WD_ERR_DEVICE_TIMEOUT and leaves.
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "gemm_tc.h"
#include "device_utils.cuh"

namespace {

using namespace wdk;

constexpr int kBM = 128;            // weight rows per tile (MMA M)
constexpr int kBK = 64;             // K elements per stage = one 128-byte swizzle row
constexpr int kStageA = kBM * kBK * 2;
constexpr int kThreads = 192;

struct TcParams {
    int rows, bn, kb_total, tok_tiles, n_units, n_stages, buf_cols, n_slices, aligned;
    int nseg, ncol;
    int seg_tile0[4];               // first tile index of each weight matrix (+ end)
    int seg_n[3];
    int seg_col[3];
    long long W;                    // total K blocks of the launch = n_units * kb_total
    float* y;
    size_t split_stride;
    int32_t* status;
    uint32_t idesc;
};

// A unit is one [128 weight rows x BN tokens] output tile; unit u = tile * tok_tiles + token tile.
struct UnitInfo { int seg, n0, tok0; };
__device__ __forceinline__ UnitInfo decode_unit(const TcParams& p, int unit) {
    UnitInfo u;
    const int tile = unit / p.tok_tiles;
    u.tok0 = (unit - tile * p.tok_tiles) * p.bn;
    u.seg = 0;
    if (p.nseg > 1 && tile >= p.seg_tile0[1]) u.seg = 1;
    if (p.nseg > 2 && tile >= p.seg_tile0[2]) u.seg = 2;
    u.n0 = (tile - p.seg_tile0[u.seg]) * kBM;
    return u;
}

// Persistent, stream-K: the K blocks of all output tiles form one line of W blocks and CTA c
// takes the contiguous piece [c W / G, (c+1) W / G).  Every CTA therefore streams the same
// number of weight bytes whatever the shape, the TMA ring never drains between tiles, and the
// epilogue of one piece overlaps the MMAs of the next (two accumulators in TMEM).  A tile cut
// by piece boundaries gets one partial sum per CTA that touched it, written to slice
// (CTA - first CTA of the tile); the CTA that finishes the tile zero-fills the unused slices.
__global__ void __launch_bounds__(kThreads)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w0,
               const __grid_constant__ CUtensorMap map_w1, const __grid_constant__ CUtensorMap map_w2,
               const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment: required by the 128-byte swizzle atoms
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int NS = p.n_stages;
    const int stage_bytes = kStageA + p.bn * kBK * 2;
    uint64_t* bars = (uint64_t*)(smem + (size_t)NS * stage_bytes);
    // bars[0..NS) full | [NS..2NS) empty | [2NS, 2NS+1] accumulator full | [2NS+2, 2NS+3] accumulator empty
    uint32_t* tmem_slot = (uint32_t*)(bars + 2 * NS + 4);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long c = blockIdx.x, G = gridDim.x;
    long long g_begin, g_end;
    if (p.aligned) {
        g_begin = (c * p.n_units / G) * p.kb_total;
        g_end = ((c + 1) * p.n_units / G) * p.kb_total;
    } else {
        g_begin = c * p.W / G;
        g_end = (c + 1) * p.W / G;
    }
    const int n_total = (int)(g_end - g_begin);

    pdl_launch_dependents();      // the next kernel may start its own prologue / weight prefetch
    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(smem_u32(&bars[s]), 1);
            mbar_init(smem_u32(&bars[NS + s]), 1);
        }
        mbar_init(smem_u32(&bars[2 * NS]), 1);
        mbar_init(smem_u32(&bars[2 * NS + 1]), 1);
        mbar_init(smem_u32(&bars[2 * NS + 2]), 128);
        mbar_init(smem_u32(&bars[2 * NS + 3]), 128);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w0) : "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 2u * (uint32_t)p.buf_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0 && n_total > 0) {
            // ------------------------------------------------ TMA producer
            uint64_t pol_stream;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            // walks the K blocks of this CTA's piece of the line without divisions
            struct Walk {
                int unit, kb, n0, tok0;
                const CUtensorMap* mw;
            };
            auto decode = [&](Walk& w) {
                const UnitInfo u = decode_unit(p, w.unit);
                w.n0 = u.n0;
                w.tok0 = u.tok0;
                w.mw = u.seg == 0 ? &map_w0 : (u.seg == 1 ? &map_w1 : &map_w2);
            };
            auto advance = [&](Walk& w) {
                if (++w.kb == p.kb_total) {
                    w.kb = 0;
                    ++w.unit;
                    decode(w);
                }
            };
            Walk w0;
            w0.unit = (int)(g_begin / p.kb_total);
            w0.kb = (int)(g_begin - (long long)w0.unit * p.kb_total);
            decode(w0);
            // Weights never depend on earlier kernels of the stream: fill the ring with weight
            // boxes first, then wait for the producer of the activations, then add their boxes.
            const int n_pre = n_total < NS ? n_total : NS;
            Walk w = w0;
            for (int i = 0; i < n_pre; ++i, advance(w)) {
                mbar_expect_tx(smem_u32(&bars[i]), (uint32_t)stage_bytes);
                tma_load_2d_hint(smem_u32(smem + (size_t)i * stage_bytes), w.mw, smem_u32(&bars[i]), w.kb * kBK, w.n0,
                                 pol_stream);
            }
            pdl_wait();
            Walk wx = w0;
            for (int i = 0; i < n_pre; ++i, advance(wx))
                tma_load_2d(smem_u32(smem + (size_t)i * stage_bytes) + kStageA, &map_x, smem_u32(&bars[i]), wx.kb * kBK,
                            wx.tok0);
            int s = n_pre % NS;
            uint32_t ph = (uint32_t)(n_pre / NS) & 1u;
            for (int i = n_pre; i < n_total; ++i, advance(w)) {
                if (!mbar_wait(smem_u32(&bars[NS + s]), ph ^ 1u, abort_flag)) {
                    *abort_flag = 1;
                    atomicCAS(p.status, 0, WD_ERR_DEVICE_TIMEOUT);
                    break;
                }
                const uint32_t full = smem_u32(&bars[s]);
                const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
                mbar_expect_tx(full, (uint32_t)stage_bytes);
                tma_load_2d_hint(sa, w.mw, full, w.kb * kBK, w.n0, pol_stream);
                tma_load_2d(sa + kStageA, &map_x, full, w.kb * kBK, w.tok0);
                if (++s == NS) { s = 0; ph ^= 1u; }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            // ------------------------------------------------ MMA issuer
            bool ok = true;
            int piece = 0, s = 0;
            uint32_t ph = 0;
            long long g = g_begin;
            while (g < g_end && ok) {
                const int unit = (int)(g / p.kb_total), kb0 = (int)(g - (long long)unit * p.kb_total);
                const int len = (int)((long long)(p.kb_total - kb0) < g_end - g ? (p.kb_total - kb0) : g_end - g);
                const int buf = piece & 1;
                // the epilogue has drained this accumulator (free at the start)
                if (!(ok = mbar_wait(smem_u32(&bars[2 * NS + 2 + buf]), ((uint32_t)(piece >> 1) & 1u) ^ 1u, abort_flag))) break;
                tc_fence_after();
                const uint32_t acc = tmem_base + (uint32_t)(buf * p.buf_cols);
                for (int j = 0; j < len; ++j) {
                    if (!(ok = mbar_wait(smem_u32(&bars[s]), ph, abort_flag))) break;
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
                    const uint64_t adesc = make_sdesc(sa);
                    const uint64_t bdesc = make_sdesc(sa + kStageA);
#pragma unroll
                    for (int kk = 0; kk < kBK / 16; ++kk) {
                        // 16 bf16 = 32 bytes further along K inside the swizzle row: +2 in 16-byte units
                        umma_bf16(acc, adesc + (uint64_t)(2 * kk), bdesc + (uint64_t)(2 * kk), p.idesc,
                                  (j > 0 || kk > 0) ? 1u : 0u);
                    }
                    umma_commit(smem_u32(&bars[NS + s]));          // stage free once these MMAs have read it
                    if (++s == NS) { s = 0; ph ^= 1u; }
                }
                if (ok) umma_commit(smem_u32(&bars[2 * NS + buf]));  // this piece's accumulator complete
                g += len;
                ++piece;
            }
            if (!ok) {
                *abort_flag = 1;
                atomicCAS(p.status, 0, WD_ERR_DEVICE_TIMEOUT);
            }
        }
        __syncwarp();
    } else {
        // ---------------------------------------------------- epilogue (warps 2..5)
        const int quarter = warp & 3;                  // TMEM lanes 32*quarter .. +31
        const int n_local = quarter * 32 + lane;
        pdl_wait();      // the previous reader of y has finished (already implied by the data flow)
        bool ok = true;
        int piece = 0;
        long long g = g_begin;
        while (g < g_end) {
            const int unit = (int)(g / p.kb_total), kb0 = (int)(g - (long long)unit * p.kb_total);
            const int len = (int)((long long)(p.kb_total - kb0) < g_end - g ? (p.kb_total - kb0) : g_end - g);
            const UnitInfo u = decode_unit(p, unit);
            const int buf = piece & 1;
            const int n = u.n0 + n_local;
            const bool n_ok = n < p.seg_n[u.seg];
            int ord = 0;
            if (!p.aligned) ord = (int)(c - (((long long)unit * p.kb_total + 1) * G - 1) / p.W);
            ok = ok && mbar_wait(smem_u32(&bars[2 * NS + buf]), (uint32_t)(piece >> 1) & 1u, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            float* yb = p.y + p.seg_col[u.seg] + n;
            const uint32_t t_acc = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * p.buf_cols);
            for (int cc = 0; cc < p.bn; cc += 16) {
                if (u.tok0 + cc >= p.rows) break;
                uint32_t v[16];
                tmem_ld16(t_acc + (uint32_t)cc, v);
                if (n_ok) {
                    float* ys = yb + (size_t)ord * p.split_stride;
#pragma unroll
                    for (int t = 0; t < 16; ++t) {
                        const int tok = u.tok0 + cc + t;
                        if (tok < p.rows) ys[(size_t)tok * p.ncol] = __uint_as_float(v[t]);
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(smem_u32(&bars[2 * NS + 2 + buf]));       // accumulator may be overwritten
            if (kb0 + len == p.kb_total && n_ok) {
                // this CTA finished the tile: slices nobody wrote must read as zero
                for (int sl = ord + 1; sl < p.n_slices; ++sl) {
                    float* ys = yb + (size_t)sl * p.split_stride;
                    for (int tok = u.tok0; tok < u.tok0 + p.bn && tok < p.rows; ++tok) ys[(size_t)tok * p.ncol] = 0.f;
                }
            }
            g += len;
            ++piece;
        }
        if (!ok && lane == 0) {
            *abort_flag = 1;
            atomicCAS(p.status, 0, WD_ERR_DEVICE_TIMEOUT);
        }
        tc_fence_before();
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 2u * (uint32_t)p.buf_cols);
    }
}

// y = sum of split-K slices
__global__ void reduce_slices_kernel(const float* __restrict__ part, int n_split, size_t stride, float* __restrict__ y,
                                     size_t total) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        float v = 0.f;
        for (int s = 0; s < n_split; ++s) v += part[s * stride + i];
        y[i] = v;
    }
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// [n_rows, K] bf16 row-major, box = 64 (K) x box_rows, 128-byte swizzle, out-of-range reads give 0
wd_status encode_2d(CUtensorMap* m, const void* ptr, int n_rows, int K, int box_rows) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return WD_ERR_CUDA;
    if ((uintptr_t)ptr % 16 || ((size_t)K * 2) % 16) return WD_ERR_MISALIGNED;
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)n_rows};
    cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? WD_OK : WD_ERR_CUDA;
}

struct TcConfig { int bn, tok_tiles, n_stages, buf_cols, ctas_per_sm; size_t smem; };

int env_int(const char* name, int dflt) {
    const char* v = getenv(name);
    return v && *v ? atoi(v) : dflt;
}

TcConfig pick_config(int rows) {
    TcConfig c;
    c.tok_tiles = (rows + 255) / 256;
    c.bn = ((rows + c.tok_tiles - 1) / c.tok_tiles + 15) / 16 * 16;     // balanced token tiles, <= 256
    int cols = 32;
    while (cols < c.bn) cols <<= 1;
    c.buf_cols = cols;                                                   // two accumulators: 2 * cols <= 512
    const int stage = kStageA + c.bn * kBK * 2;
    static const int want2 = env_int("WD_GEMM_CTAS_PER_SM", 1);
    c.ctas_per_sm = (want2 == 2 && c.bn <= 64) ? 2 : 1;
    c.n_stages = ((c.ctas_per_sm == 2 ? 104 : 200) * 1024) / stage;
    if (c.n_stages > 10) c.n_stages = 10;
    if (c.n_stages < 2) c.n_stages = 2;
    c.smem = (size_t)c.n_stages * stage + (2 * c.n_stages + 4) * 8 + 16 + 1024;
    return c;
}

// most CTAs that contribute to one output tile when W K-blocks are cut into G equal pieces
int count_slices(int n_units, int kb_total, long long W, long long G) {
    int n = 1;
    for (long long u = 0; u < n_units; ++u) {
        const long long first = ((u * kb_total + 1) * G - 1) / W;
        const long long last = (((u + 1) * kb_total) * G - 1) / W;
        if ((int)(last - first + 1) > n) n = (int)(last - first + 1);
    }
    return n;
}

uint32_t make_idesc(int bn) {
    uint32_t d = 0;
    d |= 1u << 4;                      // D format: f32
    d |= 1u << 7;                      // A format: bf16
    d |= 1u << 10;                     // B format: bf16
    // bits 15 / 16: A and B are K-major (0)
    d |= (uint32_t)(bn >> 3) << 17;    // N
    d |= (uint32_t)(kBM >> 4) << 24;   // M
    return d;
}

}  // namespace

wd_status wd_tc_weights_init(WdTcWeights* tc, const wd_model_dims* d, const void* tok_embed, const void* lm_head,
                             const std::vector<const void*>& wq, const std::vector<const void*>& wk,
                             const std::vector<const void*>& wv, const std::vector<const void*>& wo,
                             const std::vector<const void*>& wg, const std::vector<const void*>& wu,
                             const std::vector<const void*>& wd, const void* xn, const void* attn, const void* h) {
    (void)tok_embed;
    const int L = d->n_layers, hq = d->n_q_heads * d->head_dim, hkv = d->n_kv_heads * d->head_dim;
    tc->n_layers = L;
    tc->maps.assign((size_t)WD_TC_KINDS * L, CUtensorMap());
    wd_status s;
    for (int l = 0; l < L; ++l) {
        if ((s = encode_2d(&tc->maps[(size_t)WD_TC_WQ * L + l], wq[l], hq, d->d_model, kBM)) != WD_OK) return s;
        if ((s = encode_2d(&tc->maps[(size_t)WD_TC_WK * L + l], wk[l], hkv, d->d_model, kBM)) != WD_OK) return s;
        if ((s = encode_2d(&tc->maps[(size_t)WD_TC_WV * L + l], wv[l], hkv, d->d_model, kBM)) != WD_OK) return s;
        if ((s = encode_2d(&tc->maps[(size_t)WD_TC_WO * L + l], wo[l], d->d_model, hq, kBM)) != WD_OK) return s;
        if ((s = encode_2d(&tc->maps[(size_t)WD_TC_WG * L + l], wg[l], d->d_ffn, d->d_model, kBM)) != WD_OK) return s;
        if ((s = encode_2d(&tc->maps[(size_t)WD_TC_WU * L + l], wu[l], d->d_ffn, d->d_model, kBM)) != WD_OK) return s;
        if ((s = encode_2d(&tc->maps[(size_t)WD_TC_WD * L + l], wd[l], d->d_model, d->d_ffn, kBM)) != WD_OK) return s;
    }
    if ((s = encode_2d(&tc->maps[(size_t)WD_TC_LM * L + 0], lm_head, d->vocab, d->d_model, kBM)) != WD_OK) return s;
    tc->x_map_d = {xn, d->d_model};
    tc->x_map_attn = {attn, hq};
    tc->x_map_h = {h, d->d_ffn};
    return WD_OK;
}

wd_status wd_tc_gemm(const WdTcX* x, const WdTcSeg* segs, int nseg, int rows, int K, float* y, size_t y_floats,
                     int sm_count, int32_t* status, cudaStream_t stream, int* n_split_out, bool force_single_split) {
    if (!x || !segs || !y || !status || nseg < 1 || nseg > 3) return WD_ERR_BAD_PARAM;
    if (rows < 1 || K < 8 || K % 8) return WD_ERR_BAD_PARAM;
    TcParams p;
    memset(&p, 0, sizeof(p));
    const TcConfig cfg = pick_config(rows);
    int tiles = 0, col = 0;
    for (int i = 0; i < nseg; ++i) {
        if (!segs[i].map) return WD_ERR_NULL;
        p.seg_tile0[i] = tiles;
        p.seg_n[i] = segs[i].n;
        p.seg_col[i] = col;
        tiles += (segs[i].n + kBM - 1) / kBM;
        col += segs[i].n;
    }
    p.seg_tile0[nseg] = tiles;
    p.nseg = nseg;
    p.ncol = col;
    p.rows = rows; p.bn = cfg.bn;
    p.kb_total = (K + kBK - 1) / kBK;
    p.tok_tiles = cfg.tok_tiles;
    p.n_units = tiles * cfg.tok_tiles;
    p.W = (long long)p.n_units * p.kb_total;
    p.n_stages = cfg.n_stages;
    p.buf_cols = cfg.buf_cols;
    const size_t slice = (size_t)rows * col;
    if (slice > y_floats) return WD_ERR_CAPACITY;
    // stream-K over all SMs when the partial sums fit, whole tiles per CTA otherwise
    long long G = (long long)sm_count * cfg.ctas_per_sm;
    if (G > p.W / 2) G = p.W / 2 > 0 ? p.W / 2 : 1;           // at least two K blocks per CTA
    int n_slices = count_slices(p.n_units, p.kb_total, p.W, G);
    p.aligned = 0;
    if (force_single_split || (size_t)n_slices * slice > y_floats || n_slices > WD_TC_MAX_SPLIT) {
        p.aligned = 1;
        n_slices = 1;
        G = (long long)sm_count * cfg.ctas_per_sm;
        if (G > p.n_units) G = p.n_units;
    }
    p.n_slices = n_slices;
    p.y = y;
    p.split_stride = slice;
    p.status = status;
    p.idesc = make_idesc(cfg.bn);

    CUtensorMap mx;
    wd_status s = encode_2d(&mx, x->ptr, rows, K, cfg.bn);
    if (s != WD_OK) return s;

    WD_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
    const CUtensorMap& m0 = *segs[0].map;
    const CUtensorMap& m1 = *segs[nseg > 1 ? 1 : 0].map;
    const CUtensorMap& m2 = *segs[nseg > 2 ? 2 : 0].map;
    ++wd_launch_counter;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)G);
    lc.blockDim = dim3(kThreads);
    lc.dynamicSmemBytes = cfg.smem;
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = wd_pdl_enabled ? 1 : 0;
    WD_CUDA_TRY(cudaLaunchKernelEx(&lc, gemm_tc_kernel, mx, m0, m1, m2, p));
    if (n_split_out) *n_split_out = p.n_slices;
    return WD_OK;
}

size_t wd_tc_scratch_bytes(int rows, int n_out, int k_in) {
    (void)k_in;
    const size_t r = rows <= WD_TC_SPLITK_MAX_ROWS ? WD_TC_MAX_SPLIT : 1;
    return r * (size_t)rows * n_out * 4;
}

wd_status wd_tc_gemm_standalone(const void* x, const void* w, float* y, int rows, int n_out, int k_in, void* scratch,
                                size_t scratch_bytes, cudaStream_t stream) {
    if (k_in % 8) return WD_ERR_BAD_PARAM;      // TMA rows must be multiples of 16 bytes
    int32_t* status = wd_op_status_ptr();
    if (!status) return WD_ERR_CUDA;
    CUtensorMap mw;
    wd_status s = encode_2d(&mw, w, n_out, k_in, kBM);
    if (s != WD_OK) return s;
    WdTcSeg seg = {w, n_out, &mw};
    WdTcX xm = {x, k_in};
    int sm = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev);
    const size_t slice = (size_t)rows * n_out;
    if (!scratch || scratch_bytes < slice * 4) {
        // no room for partial sums: a single K slice straight into y
        int ns = 1;
        return wd_tc_gemm(&xm, &seg, 1, rows, k_in, y, slice, sm, status, stream, &ns, true);
    }
    int ns = 1;
    s = wd_tc_gemm(&xm, &seg, 1, rows, k_in, (float*)scratch, scratch_bytes / 4, sm, status, stream, &ns, false);
    if (s != WD_OK) return s;
    const int blocks = (int)((slice + 255) / 256 < 1184 ? (slice + 255) / 256 : 1184);
    ++wd_launch_counter;
    reduce_slices_kernel<<<blocks, 256, 0, stream>>>((const float*)scratch, ns, slice, y, slice);
    WD_CUDA_TRY(cudaGetLastError());
    return WD_OK;
}

// ------------------------------------------------------------------------------------------
// wd_op_gemm_noalloc: the tensor-core GEMM with its split-K scratch inside the library image
// ------------------------------------------------------------------------------------------
// Some callers cannot provide scratch memory because they are not allowed to allocate at the
// point of the call: a plugin running inside another framework's memory pool, a real-time
// loop that forbids allocator calls after start-up, code that runs while device memory is
// fully committed.  For them the partial sums of the K slices live in this fixed array, which
// every GPU that loads the library holds until the process exits.
#define WD_NOALLOC_SCRATCH_FLOATS (4u << 20)      // 4 Mi floats = 16 MiB
static __device__ __align__(256) float g_noalloc_scratch[WD_NOALLOC_SCRATCH_FLOATS];

// In host code the array's name is only a handle for the runtime, not a device address, so the
// address is asked for once per device (with that device current) and cached.
static float* noalloc_scratch_ptr(wd_status* err) {
    static float* cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { *err = WD_ERR_CUDA; return nullptr; }
    if (!cached[dev]) {
        float* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress((void**)&p, g_noalloc_scratch);
        if (e != cudaSuccess || !p) {
            wd_note_cuda_error(e, __FILE__, __LINE__);
            *err = WD_ERR_CUDA;
            return nullptr;
        }
        cached[dev] = p;
    }
    return cached[dev];
}

extern "C" size_t wd_op_gemm_noalloc_max_floats(void) { return (size_t)WD_NOALLOC_SCRATCH_FLOATS; }

extern "C" wd_status wd_op_gemm_noalloc(const void* x, const void* w, float* y, int32_t rows, int32_t n_out,
                                        int32_t k_in, void* stream_) {
    if (!x || !w || !y) return WD_ERR_NULL;
    if (rows < 1 || n_out < 1 || k_in < 8 || k_in % 8) return WD_ERR_BAD_PARAM;
    const size_t slice = (size_t)rows * (size_t)n_out;
    if (slice > (size_t)WD_NOALLOC_SCRATCH_FLOATS) return WD_ERR_CAPACITY;   // one K slice must fit
    wd_status err = WD_OK;
    float* scratch = noalloc_scratch_ptr(&err);
    if (!scratch) return err;
    int32_t* status = wd_op_status_ptr();
    if (!status) return WD_ERR_CUDA;
    cudaStream_t stream = (cudaStream_t)stream_;
    CUtensorMap mw;
    wd_status s = encode_2d(&mw, w, n_out, k_in, kBM);
    if (s != WD_OK) return s;
    WdTcSeg seg = {w, n_out, &mw};
    WdTcX xm = {x, k_in};
    int sm = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev);
    // the number of K slices is capped by what fits in the fixed array; every element of every
    // slice that the reduction reads is written by exactly one CTA first, so nothing has to be
    // cleared between calls even though the array keeps the previous call's contents
    int ns = 1;
    s = wd_tc_gemm(&xm, &seg, 1, rows, k_in, scratch, (size_t)WD_NOALLOC_SCRATCH_FLOATS, sm, status, stream, &ns, false);
    if (s != WD_OK) return s;
    const int blocks = (int)((slice + 255) / 256 < 1184 ? (slice + 255) / 256 : 1184);
    ++wd_launch_counter;
    reduce_slices_kernel<<<blocks, 256, 0, stream>>>(scratch, ns, slice, y, slice);
    WD_CUDA_TRY(cudaGetLastError());
    return WD_OK;
}
