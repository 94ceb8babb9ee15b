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
    int rows, K, bn, n_split, kb_total, n_stages, tmem_cols;
    int nseg, ncol;
    int seg_tile0[4];               // first tile index of each segment (+ end)
    int seg_n[3];
    int seg_col[3];
    float* y;
    size_t split_stride;
    int32_t* status;
    uint32_t idesc;
};

__global__ void __launch_bounds__(kThreads)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w0,
               const __grid_constant__ CUtensorMap map_w1, const __grid_constant__ CUtensorMap map_w2,
               const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment: required by the 128-byte swizzle atoms
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int stage_b = p.bn * kBK * 2;
    const int stage_bytes = kStageA + stage_b;
    uint64_t* bars = (uint64_t*)(smem + (size_t)p.n_stages * stage_bytes);
    // bars[0..NS) full, bars[NS..2NS) empty, bars[2NS] accumulator ready
    uint32_t* tmem_slot = (uint32_t*)(bars + 2 * p.n_stages + 1);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // token tile fastest: CTAs that share a weight tile run together and share it through L2
    const int tile = blockIdx.y, tok0 = blockIdx.x * p.bn, z = blockIdx.z;

    // which weight matrix does this tile belong to
    int seg = 0;
    if (p.nseg > 1 && tile >= p.seg_tile0[1]) seg = 1;
    if (p.nseg > 2 && tile >= p.seg_tile0[2]) seg = 2;
    const CUtensorMap* map_w = seg == 0 ? &map_w0 : (seg == 1 ? &map_w1 : &map_w2);
    const int n0 = (tile - p.seg_tile0[seg]) * kBM;           // first weight row of the tile
    const int kb_begin = (int)(((long long)z * p.kb_total) / p.n_split);
    const int kb_end = (int)(((long long)(z + 1) * p.kb_total) / p.n_split);
    const int n_kb = kb_end - kb_begin;

    pdl_launch_dependents();      // the next kernel may start its own prologue / weight prefetch
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.n_stages; ++s) {
            mbar_init(smem_u32(&bars[s]), 1);
            mbar_init(smem_u32(&bars[p.n_stages + s]), 1);
        }
        mbar_init(smem_u32(&bars[2 * p.n_stages]), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(map_w) : "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"((uint32_t)p.tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            // ------------------------------------------------ TMA producer
            uint64_t pol_stream, pol_keep;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
            // Weights never depend on earlier kernels of the stream: fill the ring with weight
            // boxes first, then wait for the producer of the activations, then add their boxes.
            const int n_pre = n_kb < p.n_stages ? n_kb : p.n_stages;
            for (int i = 0; i < n_pre; ++i) {
                const uint32_t full = smem_u32(&bars[i]);
                mbar_expect_tx(full, (uint32_t)stage_bytes);
                tma_load_2d_hint(smem_u32(smem + (size_t)i * stage_bytes), map_w, full, (kb_begin + i) * kBK, n0, pol_stream);
            }
            pdl_wait();
            for (int i = 0; i < n_pre; ++i)
                tma_load_2d_hint(smem_u32(smem + (size_t)i * stage_bytes) + kStageA, &map_x, smem_u32(&bars[i]),
                                 (kb_begin + i) * kBK, tok0, pol_keep);
            for (int i = n_pre; i < n_kb; ++i) {
                const int s = i % p.n_stages;
                const uint32_t ph = (uint32_t)(i / p.n_stages) & 1u;
                if (!mbar_wait(smem_u32(&bars[p.n_stages + s]), ph ^ 1u, abort_flag)) {
                    *abort_flag = 1;
                    atomicCAS(p.status, 0, WD_ERR_DEVICE_TIMEOUT);
                    break;
                }
                const uint32_t full = smem_u32(&bars[s]);
                const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
                mbar_expect_tx(full, (uint32_t)stage_bytes);
                const int kc = (kb_begin + i) * kBK;
                tma_load_2d_hint(sa, map_w, full, kc, n0, pol_stream);
                tma_load_2d_hint(sa + kStageA, &map_x, full, kc, tok0, pol_keep);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            // ------------------------------------------------ MMA issuer
            bool ok = true;
            for (int i = 0; i < n_kb && ok; ++i) {
                const int s = i % p.n_stages;
                const uint32_t ph = (uint32_t)(i / p.n_stages) & 1u;
                if (!mbar_wait(smem_u32(&bars[s]), ph, abort_flag)) {
                    *abort_flag = 1;
                    atomicCAS(p.status, 0, WD_ERR_DEVICE_TIMEOUT);
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
                const uint64_t adesc = make_sdesc(sa);
                const uint64_t bdesc = make_sdesc(sa + kStageA);
#pragma unroll
                for (int kk = 0; kk < kBK / 16; ++kk) {
                    // 16 bf16 = 32 bytes further along K inside the swizzle row: +2 in 16-byte units
                    umma_bf16(tmem_base, adesc + (uint64_t)(2 * kk), bdesc + (uint64_t)(2 * kk), p.idesc,
                              (i > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(smem_u32(&bars[p.n_stages + s]));     // stage free once these MMAs have read it
            }
            if (ok) umma_commit(smem_u32(&bars[2 * p.n_stages]));  // accumulator complete
        }
        __syncwarp();
    } else {
        // ---------------------------------------------------- epilogue (warps 2..5)
        const int quarter = warp & 3;                  // TMEM lanes 32*quarter .. +31
        const int n_local = quarter * 32 + lane;
        const int n = n0 + n_local;
        const bool n_ok = n < p.seg_n[seg];
        bool ok = n_kb > 0;
        if (ok) ok = mbar_wait(smem_u32(&bars[2 * p.n_stages]), 0, abort_flag);
        if (!ok && n_kb > 0 && lane == 0) {
            *abort_flag = 1;
            atomicCAS(p.status, 0, WD_ERR_DEVICE_TIMEOUT);
        }
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after();
        pdl_wait();      // the previous consumer of y has finished (already implied by the data flow)
        float* yb = p.y + (size_t)z * p.split_stride + p.seg_col[seg] + n;
        for (int c = 0; c < p.bn; c += 16) {
            if (tok0 + c >= p.rows) break;
            uint32_t v[16];
            if (ok) {
                tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c, v);
            } else {
#pragma unroll
                for (int t = 0; t < 16; ++t) v[t] = 0u;
            }
            if (n_ok) {
#pragma unroll
                for (int t = 0; t < 16; ++t) {
                    const int tok = tok0 + c + t;
                    if (tok < p.rows) yb[(size_t)tok * p.ncol] = __uint_as_float(v[t]);
                }
            }
        }
        tc_fence_before();
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols)
                     : "memory");
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

struct TcConfig { int bn, tok_tiles, n_stages, tmem_cols, ctas_per_sm; size_t smem; };

TcConfig pick_config(int rows) {
    TcConfig c;
    c.tok_tiles = (rows + 255) / 256;
    c.bn = ((rows + c.tok_tiles - 1) / c.tok_tiles + 15) / 16 * 16;     // balanced token tiles, <= 256
    int cols = 32;
    while (cols < c.bn) cols <<= 1;
    c.tmem_cols = cols;
    const int stage = kStageA + c.bn * kBK * 2;
    // two CTAs per SM while the token tile is narrow, so one CTA's epilogue overlaps the
    // other's streaming; one CTA with a deeper ring otherwise
    c.ctas_per_sm = c.bn <= 96 ? 2 : 1;
    const int budget = c.ctas_per_sm == 2 ? 108 * 1024 : 208 * 1024;
    c.n_stages = budget / stage;
    if (c.n_stages > 8) c.n_stages = 8;
    if (c.n_stages < 2) c.n_stages = 2;
    c.smem = (size_t)c.n_stages * stage + (2 * c.n_stages + 1) * 8 + 16 + 1024;
    return c;
}

int pick_split(int tiles, int kb_total, int slots, int rows, bool force_single, size_t y_floats, size_t slice_floats) {
    if (force_single || rows > WD_TC_SPLITK_MAX_ROWS) return 1;
    int best = 1;
    double best_eff = 0.0;
    for (int s = 1; s <= WD_TC_MAX_SPLIT; ++s) {
        if (s > 1 && kb_total / s < 4) break;                 // keep at least 4 K blocks per CTA
        if ((size_t)s * slice_floats > y_floats) break;
        const long long ctas = (long long)tiles * s;
        const long long waves = (ctas + slots - 1) / slots;
        const double eff = (double)ctas / (double)(waves * slots);
        if (eff > best_eff + 0.02) { best_eff = eff; best = s; }
    }
    return best;
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
    p.rows = rows; p.K = K; p.bn = cfg.bn;
    p.kb_total = (K + kBK - 1) / kBK;
    p.n_stages = cfg.n_stages;
    p.tmem_cols = cfg.tmem_cols;
    const size_t slice = (size_t)rows * col;
    if (slice > y_floats) return WD_ERR_CAPACITY;
    p.n_split = pick_split(tiles * cfg.tok_tiles, p.kb_total, sm_count * cfg.ctas_per_sm, rows, force_single_split,
                           y_floats, slice);
    p.y = y;
    p.split_stride = slice;
    p.status = status;
    p.idesc = make_idesc(cfg.bn);

    CUtensorMap mx;
    wd_status s = encode_2d(&mx, x->ptr, rows, K, cfg.bn);
    if (s != WD_OK) return s;

    WD_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
    dim3 grid(cfg.tok_tiles, tiles, p.n_split);
    const CUtensorMap& m0 = *segs[0].map;
    const CUtensorMap& m1 = *segs[nseg > 1 ? 1 : 0].map;
    const CUtensorMap& m2 = *segs[nseg > 2 ? 2 : 0].map;
    ++wd_launch_counter;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = grid;
    lc.blockDim = dim3(kThreads);
    lc.dynamicSmemBytes = cfg.smem;
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = wd_pdl_enabled ? 1 : 0;
    WD_CUDA_TRY(cudaLaunchKernelEx(&lc, gemm_tc_kernel, mx, m0, m1, m2, p));
    WD_CUDA_TRY(cudaGetLastError());
    if (n_split_out) *n_split_out = p.n_split;
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
