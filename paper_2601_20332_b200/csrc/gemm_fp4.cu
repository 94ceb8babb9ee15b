// NVFP4 weight-streaming GEMM on the block-scaled tensor-core path (sm_100a), an option outside the paper
// (which calls quantisation orthogonal to its method).
//
//   y[tok, n] = gx[tok] * gw[n] * sum_blocks (sx[tok, b] * sw[n, b]) * sum_{i in block b} qx[tok, i] * qw[n, i]
//
// Operands: 4-bit e2m1 codes packed two per byte (element 2j in the low nibble), one unsigned e4m3 scale
// per block of 16 elements along K, one float scale per row.  tcgen05.mma kind::mxf4nvf4 multiplies the
// codes and applies the block scales in hardware (fp32 accumulation in tensor memory); the row scales are
// applied in the epilogue.
//
// A stage of the ring holds one K block of 256 elements: [128 weight rows x 128 bytes] and [BN tokens x 128
// bytes] of codes in the 128-byte swizzled layout, plus their block scales [rows x 16 bytes].  The hardware
// reads block scales from tensor memory: for row r of an operand the four scales of one K = 64 instruction
// sit in lane r mod 32 (of every 32-lane quarter), 32-bit column r / 32, one scale per byte.  Four warps
// copy each stage's scales from shared memory into that layout (tcgen05.st, every warp its own quarter)
// before the MMA thread issues the stage's four instructions; two scale slots alternate.
//   warp 0      TMA producer (weights, which never depend on earlier kernels, before the dependency wait)
//   warp 1      MMA issuer
//   warps 2-5   epilogue: tcgen05.ld, row scales, coalesced fp32 stores of this K slice's partial sums
//   warps 6-9   block scales: shared memory -> tensor memory
// Work units are (weight tile, token tile, K slice), dealt round-robin to one CTA per SM; K slices are
// written side by side ([slice][tok][n]) and added by the consumer, as in the bf16 kernel.
// Every wait is bounded; on expiry the CTA records WD_ERR_DEVICE_TIMEOUT and leaves.
#include <cstdlib>
#include <cstring>

#include <cuda_fp8.h>

#include "gemm_tc.h"
#include "device_utils.cuh"

namespace {

using namespace wdk;

constexpr int kBM = 128;              // weight rows per tile
constexpr int kKB = 256;              // K elements per stage = 128 bytes of codes = one swizzle row
constexpr int kStageW = kBM * 128;    // 16 KB of weight codes
constexpr int kSfW = kBM * 16;        // 2 KB of weight block scales
constexpr int kThreads = 320;

struct Fp4Params {
    int rows, n_out, bn, kb_total, tok_tiles, n_tiles, n_slices, n_units, n_stages, buf_cols;
    int w_static;                     // the weights were written before the previous kernel started
    float* y;
    size_t split_stride;
    const float* gw;                  // [n_out] row scales of the weights
    const float* gx;                  // [rows] row scales of the activations
    int32_t* status;
    uint32_t idesc;
};

__device__ __forceinline__ void umma_fp4(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t sfa,
                                         uint32_t sfb, uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::mxf4nvf4.block_scale.block16 [%0], %1, %2, %3, [%5], [%6], p;\n}\n"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb) : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
gemm_fp4_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                const __grid_constant__ CUtensorMap map_sx, const __grid_constant__ CUtensorMap map_sw, const Fp4Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int NS = p.n_stages;
    const int x_bytes = p.bn * 128, sfx_bytes = p.bn * 16;
    // stage: weight codes | token codes | weight scales | token scales (rounded up to a multiple of 1024 bytes)
    const int stage_bytes = (kStageW + x_bytes + kSfW + sfx_bytes + 1023) & ~1023;
    uint64_t* bars = (uint64_t*)(smem + (size_t)NS * stage_bytes);
    // bars: [0, NS) full | [NS, 2NS) empty | 2NS.. accumulator full [2] | accumulator empty [2] | scales in tensor memory [2] |
    //       scale slot free [2]
    uint64_t* acc_full = bars + 2 * NS;
    uint64_t* acc_empty = acc_full + 2;
    uint64_t* sf_full = acc_empty + 2;
    uint64_t* sf_free = sf_full + 2;
    uint32_t* tmem_slot = (uint32_t*)(sf_free + 2);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x, c = blockIdx.x;
    const int n_my = c < p.n_units ? (p.n_units - c + G - 1) / G : 0;
    // unit -> (tile, token tile, K slice); slices innermost, so neighbouring CTAs share a weight tile's rows
    auto decode = [&](int u, int& n0, int& tok0, int& sl, int& kb0, int& kbn) {
        const int unit = c + u * G;
        sl = unit % p.n_slices;
        const int rest = unit / p.n_slices;
        tok0 = (rest % p.tok_tiles) * p.bn;
        n0 = (rest / p.tok_tiles) * kBM;
        kb0 = sl * p.kb_total / p.n_slices;
        kbn = (sl + 1) * p.kb_total / p.n_slices - kb0;
    };
    int n_total = 0;
    for (int u = 0; u < n_my; ++u) {
        int n0, tok0, sl, kb0, kbn;
        decode(u, n0, tok0, sl, kb0, kbn);
        n_total += kbn;
    }
    const uint32_t tmem_cols = 2u * (uint32_t)p.buf_cols + 64u <= 128u ? 128u : (2u * (uint32_t)p.buf_cols + 64u <= 256u ? 256u : 512u);

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(smem_u32(&bars[s]), 1);
            mbar_init(smem_u32(&bars[NS + s]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&acc_full[i]), 1);
            mbar_init(smem_u32(&acc_empty[i]), 128);
            mbar_init(smem_u32(&sf_full[i]), 128);
            mbar_init(smem_u32(&sf_free[i]), 1);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_sf = tmem_base + 2u * (uint32_t)p.buf_cols;      // two slots of 32 columns: 16 for A, 16 for B

    if (warp == 0) {
        if (lane == 0 && n_total > 0) {
            // ------------------------------------------------ TMA producer
            uint64_t pol_stream;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            struct Walk { int u, left, kb, n0, tok0; };
            auto enter = [&](Walk& w) {
                int sl, kb0, kbn;
                decode(w.u, w.n0, w.tok0, sl, kb0, kbn);
                w.kb = kb0;
                w.left = kbn;
            };
            auto advance = [&](Walk& w) {
                ++w.kb;
                if (--w.left == 0 && ++w.u < n_my) enter(w);
            };
            auto load_w = [&](const Walk& w, int s) {
                const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes), full = smem_u32(&bars[s]);
                mbar_expect_tx(full, (uint32_t)(kStageW + x_bytes + kSfW + sfx_bytes));
                tma_load_2d_hint(sa, &map_w, full, w.kb * 128, w.n0, pol_stream);
                tma_load_2d(sa + kStageW + x_bytes, &map_sw, full, w.kb * 16, w.n0);
            };
            auto load_x = [&](const Walk& w, int s) {
                const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes), full = smem_u32(&bars[s]);
                tma_load_2d(sa + kStageW, &map_x, full, w.kb * 128, w.tok0);
                tma_load_2d(sa + kStageW + x_bytes + kSfW, &map_sx, full, w.kb * 16, w.tok0);
            };
            Walk w, wx;
            w.u = 0;
            enter(w);
            wx = w;
            const int n_pre = n_total < NS ? n_total : NS;
            if (!p.w_static) pdl_wait();
            for (int i = 0; i < n_pre; ++i, advance(w)) load_w(w, i);        // weights first when they depend on nothing
            if (p.w_static) pdl_wait();
            for (int i = 0; i < n_pre; ++i, advance(wx)) load_x(wx, i);
            int s = n_pre % NS;
            uint32_t ph = (uint32_t)(n_pre / NS) & 1u;
            for (int i = n_pre; i < n_total; ++i, advance(w)) {
                if (!mbar_wait(smem_u32(&bars[NS + s]), ph ^ 1u, abort_flag)) {
                    *abort_flag = 1;
                    atomicCAS(p.status, 0, WD_ERR_DEVICE_TIMEOUT);
                    break;
                }
                load_w(w, s);
                load_x(w, s);
                if (++s == NS) { s = 0; ph ^= 1u; }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            // ------------------------------------------------ MMA issuer
            bool ok = true;
            int s = 0, i = 0;
            uint32_t ph = 0;
            for (int u = 0; u < n_my && ok; ++u) {
                int n0, tok0, sl, kb0, kbn;
                decode(u, n0, tok0, sl, kb0, kbn);
                const int buf = u & 1;
                const uint32_t par = (uint32_t)(u >> 1) & 1u;
                if (!(ok = mbar_wait(smem_u32(&acc_empty[buf]), par ^ 1u, abort_flag))) break;
                tc_fence_after();
                const uint32_t acc = tmem_base + (uint32_t)(buf * p.buf_cols);
                for (int j = 0; j < kbn; ++j, ++i) {
                    const int slot = i & 1;
                    if (!(ok = mbar_wait(smem_u32(&bars[s]), ph, abort_flag))) break;                       // codes landed
                    if (!(ok = mbar_wait(smem_u32(&sf_full[slot]), (uint32_t)(i >> 1) & 1u, abort_flag))) break;   // scales in tensor memory
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
                    const uint64_t adesc = make_sdesc(sa), bdesc = make_sdesc(sa + kStageW);
                    const uint32_t sf = tmem_sf + (uint32_t)(slot * 32);
#pragma unroll
                    for (int kq = 0; kq < 4; ++kq)       // 64 elements = 32 bytes further along K: +2 in 16-byte units
                        umma_fp4(acc, adesc + (uint64_t)(2 * kq), bdesc + (uint64_t)(2 * kq), p.idesc, sf + (uint32_t)(4 * kq),
                                 sf + 16u + (uint32_t)(4 * kq), (j > 0 || kq > 0) ? 1u : 0u);
                    umma_commit(smem_u32(&bars[NS + s]));      // stage free once these MMAs have read it
                    umma_commit(smem_u32(&sf_free[slot]));     // ... and the scale slot
                    if (++s == NS) { s = 0; ph ^= 1u; }
                }
                if (ok) umma_commit(smem_u32(&acc_full[buf]));
            }
            if (!ok) {
                *abort_flag = 1;
                atomicCAS(p.status, 0, WD_ERR_DEVICE_TIMEOUT);
            }
        }
        __syncwarp();
    } else if (warp < 6) {
        // ---------------------------------------------------- epilogue (warps 2..5)
        const int quarter = warp & 3;
        const int n_local = quarter * 32 + lane;
        pdl_wait();
        bool ok = true;
        for (int u = 0; u < n_my; ++u) {
            int n0, tok0, sl, kb0, kbn;
            decode(u, n0, tok0, sl, kb0, kbn);
            const int buf = u & 1;
            const uint32_t par = (uint32_t)(u >> 1) & 1u;
            const int n = n0 + n_local;
            const bool n_ok = n < p.n_out;
            ok = ok && mbar_wait(smem_u32(&acc_full[buf]), par, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const float gwn = n_ok ? p.gw[n] : 0.f;
            float* ys = p.y + (size_t)sl * p.split_stride + n;
            const uint32_t t_acc = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * p.buf_cols);
            for (int cc = 0; cc < p.bn; cc += 16) {
                if (tok0 + cc >= p.rows) break;
                uint32_t v[16];
                tmem_ld16(t_acc + (uint32_t)cc, v);
                if (n_ok) {
#pragma unroll
                    for (int t = 0; t < 16; ++t) {
                        const int tok = tok0 + cc + t;
                        if (tok < p.rows) ys[(size_t)tok * p.n_out] = __uint_as_float(v[t]) * gwn * __ldg(p.gx + tok);
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(smem_u32(&acc_empty[buf]));
        }
        if (!ok && lane == 0) {
            *abort_flag = 1;
            atomicCAS(p.status, 0, WD_ERR_DEVICE_TIMEOUT);
        }
        tc_fence_before();
    } else {
        // ---------------------------------------------------- block scales: shared memory -> tensor memory (warps 6..9)
        const int quarter = warp & 3;
        bool ok = true;
        int s = 0;
        uint32_t ph = 0;
        for (int i = 0; i < n_total; ++i) {
            const int slot = i & 1;
            ok = ok && mbar_wait(smem_u32(&bars[s]), ph, abort_flag);                                    // the stage's scales landed
            ok = ok && mbar_wait(smem_u32(&sf_free[slot]), ((uint32_t)(i >> 1) & 1u) ^ 1u, abort_flag);  // the slot's last readers are done
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint8_t* st = smem + (size_t)s * stage_bytes;
            const uint4* wsf = reinterpret_cast<const uint4*>(st + kStageW + x_bytes);                   // [128 rows] x 16 scales
            const uint4* xsf = reinterpret_cast<const uint4*>(st + kStageW + x_bytes + kSfW);            // [bn rows] x 16 scales
            uint32_t v[32];
#pragma unroll
            for (int r1 = 0; r1 < 4; ++r1) {
                // row lane + 32 r1 of either operand: its 16 scales = four instructions x four scales
                const uint4 a = wsf[lane + 32 * r1];
                const int xr = lane + 32 * r1;
                const uint4 b = xr < p.bn ? xsf[xr] : make_uint4(0u, 0u, 0u, 0u);
                v[0 + r1] = a.x; v[4 + r1] = a.y; v[8 + r1] = a.z; v[12 + r1] = a.w;          // column 4 kq + r1 of A's scales
                v[16 + r1] = b.x; v[20 + r1] = b.y; v[24 + r1] = b.z; v[28 + r1] = b.w;       // ... of B's
            }
            tmem_st32(tmem_sf + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(slot * 32), v);
            tc_fence_before();
            mbar_arrive(smem_u32(&sf_full[slot]));
            if (++s == NS) { s = 0; ph ^= 1u; }
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
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

// ---------------------------------------------------------------- quantisation
template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return __bfloat162float(__float2bfloat16_rn(*p)); }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// One block per row: row scale g = max|row| / (6 * 448) (1 for a zero row); per 16-element block the scale
// s = e4m3((max|block| / 6) / g) and the codes e2m1(x / (s * g)).  The input is taken as bfloat16 (a float
// input is rounded first).  K is a multiple of 16.
template <typename T>
__global__ void quantize_nvfp4_kernel(const T* __restrict__ x, int K, uint8_t* __restrict__ codes, uint8_t* __restrict__ sf,
                                      float* __restrict__ g_out) {
    __shared__ float red[32];
    pdl_launch_dependents();
    pdl_wait();
    const size_t row = blockIdx.x;
    const T* xr = x + row * (size_t)K;
    float amax = 0.f;
    for (int i = threadIdx.x; i < K; i += blockDim.x) amax = fmaxf(amax, fabsf(ldf<T>(xr + i)));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
    __syncthreads();
    amax = 0.f;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) amax = fmaxf(amax, red[i]);
    const float g = amax > 0.f ? __fdiv_rn(amax, 6.0f * 448.0f) : 1.f;
    if (threadIdx.x == 0) g_out[row] = g;
    for (int b = threadIdx.x; b < K / 16; b += blockDim.x) {
        float v[16];
        float bmax = 0.f;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            v[i] = ldf<T>(xr + 16 * b + i);
            bmax = fmaxf(bmax, fabsf(v[i]));
        }
        const uint32_t sc = (uint32_t)__nv_cvt_float_to_fp8(__fdiv_rn(__fdiv_rn(bmax, 6.0f), g), __NV_SATFINITE, __NV_E4M3);
        const float d = __fmul_rn(e4m3_value(sc), g);
        sf[row * (size_t)(K / 16) + b] = (uint8_t)sc;
        uint32_t lo = 0, hi = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            lo |= (d > 0.f ? e2m1_code(__fdiv_rn(v[i], d)) : 0u) << (4 * i);
            hi |= (d > 0.f ? e2m1_code(__fdiv_rn(v[8 + i], d)) : 0u) << (4 * i);
        }
        *reinterpret_cast<uint2*>(codes + row * (size_t)(K / 2) + 8 * b) = make_uint2(lo, hi);
    }
}

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

// [n_rows][row_bytes] bytes, box = box_bytes x box_rows, swizzled (codes) or plain (scales); out-of-range reads give 0
wd_status encode_bytes(CUtensorMap* m, const void* ptr, int n_rows, int row_bytes, int box_bytes, int box_rows, bool swizzle) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return WD_ERR_CUDA;
    if ((uintptr_t)ptr % 16 || row_bytes % 16) return WD_ERR_MISALIGNED;
    cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)n_rows};
    cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
    cuuint32_t box[2] = {(cuuint32_t)box_bytes, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? WD_OK : WD_ERR_CUDA;
}

}  // namespace

size_t wd_fp4_operand_bytes(int n_rows, int K) {
    return wd_align_up((size_t)n_rows * (K / 2), 256) + wd_align_up((size_t)n_rows * (K / 16), 256) + wd_align_up((size_t)n_rows * 4, 256);
}

void wd_fp4_operand_split(void* mem, int n_rows, int K, WdFp4Operand* op) {
    char* p = (char*)mem;
    op->codes = (uint8_t*)p; p += wd_align_up((size_t)n_rows * (K / 2), 256);
    op->sf = (uint8_t*)p; p += wd_align_up((size_t)n_rows * (K / 16), 256);
    op->g = (float*)p;
    op->n_rows = n_rows;
    op->K = K;
}

void wd_launch_quantize_nvfp4(int dtype, const void* x, int n_rows, int K, const WdFp4Operand* op, cudaStream_t st) {
    if (n_rows <= 0) return;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)n_rows);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = wd_pdl_enabled ? 1 : 0;
    ++wd_launch_counter;
    if (dtype == WD_F32) cudaLaunchKernelEx(&cfg, quantize_nvfp4_kernel<float>, (const float*)x, K, op->codes, op->sf, op->g);
    else cudaLaunchKernelEx(&cfg, quantize_nvfp4_kernel<__nv_bfloat16>, (const __nv_bfloat16*)x, K, op->codes, op->sf, op->g);
}

wd_status wd_fp4_gemm(const WdFp4Operand* x, const WdFp4Operand* w, float* y, size_t y_floats, int sm_count, int32_t* status,
                      cudaStream_t stream, int* n_split_out, bool force_single_split, bool w_static) {
    if (!x || !w || !y || !status) return WD_ERR_NULL;
    const int rows = x->n_rows, n_out = w->n_rows, K = x->K;
    if (rows < 1 || n_out < 1 || K < kKB || K % kKB || w->K != K) return WD_ERR_BAD_PARAM;
    Fp4Params p;
    memset(&p, 0, sizeof(p));
    p.rows = rows;
    p.n_out = n_out;
    p.tok_tiles = (rows + 127) / 128;
    p.bn = ((rows + p.tok_tiles - 1) / p.tok_tiles + 15) / 16 * 16;        // balanced token tiles, <= 128
    p.kb_total = K / kKB;
    p.n_tiles = (n_out + kBM - 1) / kBM;
    const size_t slice = (size_t)rows * n_out;
    if (slice > y_floats) return WD_ERR_CAPACITY;
    // K slices while (weight tile, token tile) pairs alone would leave SMs idle and the partial sums fit
    // K slices: the split count that minimises (waves of units over the SMs) x (stages per unit) x (time one SM
    // needs to take in a stage, about 63 GB/s whatever the source) + the write and re-read of one more partial
    // result per slice at HBM speed
    int ns = 1;
    if (!force_single_split) {
        const double t_stage = (double)(kStageW + p.bn * 128 + kSfW + p.bn * 16) / 63e9;
        const double t_slice = (double)slice * 8.0 / 6.5e12;
        double best = 1e30;
        for (int c = 1; c <= WD_TC_MAX_SPLIT && c <= p.kb_total && (size_t)c * slice <= y_floats; ++c) {
            const int units = p.n_tiles * p.tok_tiles * c;
            const double t = (double)((units + sm_count - 1) / sm_count) * ((p.kb_total + c - 1) / c) * t_stage + c * t_slice;
            if (t < best * 0.999) { best = t; ns = c; }
        }
    }
    p.n_slices = ns;
    p.n_units = p.n_tiles * p.tok_tiles * ns;
    int cols = 32;
    while (cols < p.bn) cols <<= 1;
    p.buf_cols = cols;
    const int stage = (kStageW + p.bn * 128 + kSfW + p.bn * 16 + 1023) & ~1023;
    p.n_stages = (200 * 1024) / stage;
    if (p.n_stages > 10) p.n_stages = 10;
    const size_t smem = (size_t)p.n_stages * stage + (2 * p.n_stages + 8) * 8 + 64 + 1024;
    p.y = y;
    p.split_stride = slice;
    p.gw = w->g;
    p.gx = x->g;
    p.status = status;
    p.w_static = w_static ? 1 : 0;
    // instruction descriptor of the block-scaled form: A and B e2m1 (format 1) K-major, unsigned e4m3 scales,
    // N in bits 17-22 (units of 8), M in bits 24-28 (units of 16), dense, K = 64
    p.idesc = (1u << 7) | (1u << 10) | ((uint32_t)(p.bn >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);

    CUtensorMap mx, mw, msx, msw;
    wd_status s;
    if ((s = encode_bytes(&mx, x->codes, rows, K / 2, 128, p.bn, true)) != WD_OK) return s;
    if ((s = encode_bytes(&mw, w->codes, n_out, K / 2, 128, kBM, true)) != WD_OK) return s;
    if ((s = encode_bytes(&msx, x->sf, rows, K / 16, 16, p.bn, false)) != WD_OK) return s;
    if ((s = encode_bytes(&msw, w->sf, n_out, K / 16, 16, kBM, false)) != WD_OK) return s;
    static bool attr_done[64] = {};
    int dev = 0;
    WD_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return WD_ERR_CUDA;
    if (!attr_done[dev]) {
        WD_CUDA_TRY(cudaFuncSetAttribute(gemm_fp4_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
        attr_done[dev] = true;
    }
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)(p.n_units < sm_count ? p.n_units : sm_count));
    lc.blockDim = dim3(kThreads);
    lc.dynamicSmemBytes = smem;
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = wd_pdl_enabled ? 1 : 0;
    ++wd_launch_counter;
    WD_CUDA_TRY(cudaLaunchKernelEx(&lc, gemm_fp4_kernel, mx, mw, msx, msw, p));
    if (n_split_out) *n_split_out = ns;
    return WD_OK;
}
