// Element-wise, gather/scatter, reduction and CUDA-core kernels of the step.
//
// These are the bandwidth- and latency-bound pieces around the GEMMs (embedding
// gather, RMSNorm, RoPE + K/V scatter, SwiGLU, residual add, unmask reduction)
// plus CUDA-core versions of the GEMM and of attention that work for any dtype
// and any index list; the fp32 configuration runs on them entirely and the
// bf16 tensor-core kernels are cross-checked against them.
#include <cstdlib>
#include <cstring>
#include <utility>
#include <vector>

#include <cuda_fp8.h>

#include "wd_internal.h"
#include "device_utils.cuh"

bool wd_pdl_enabled = true;

namespace {

using wdk::pdl_launch_dependents;
using wdk::pdl_wait;

#ifdef WD_GEMM_TRACE
// development clock stamps of the small kernels: every block appends (kind, wait returned, exit) to a ring
__device__ unsigned long long g_small_trace[16384][4];
__device__ unsigned int g_small_idx;
struct SmallStamp {
    unsigned long long t0, tm;
    int kind;
    __device__ SmallStamp(int k) : t0(0), tm(0), kind(k) { if (threadIdx.x == 0) t0 = wdk::global_ns(); }
    __device__ void mid() { if (threadIdx.x == 0) tm = wdk::global_ns(); }
    __device__ ~SmallStamp() {
        if (threadIdx.x == 0) {
            const unsigned int i = atomicAdd(&g_small_idx, 1u) & 16383u;
            g_small_trace[i][0] = (unsigned long long)kind;
            g_small_trace[i][1] = t0;
            g_small_trace[i][2] = wdk::global_ns();
            g_small_trace[i][3] = tm;
        }
    }
};
#define S_STAMP(kind) SmallStamp small_stamp_(kind)
#define S_MID() small_stamp_.mid()
extern "C" __attribute__((visibility("default"))) int wd_debug_small_trace(unsigned long long* host /*[16384][4]*/, unsigned int* idx) {
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(idx, g_small_idx, sizeof(unsigned int));
    return (int)cudaMemcpyFromSymbol(host, g_small_trace, sizeof(unsigned long long) * 16384 * 4);
}
#else
#define S_STAMP(kind) do { } while (0)
#define S_MID() do { } while (0)
#endif

// Launch with programmatic stream serialization: the kernel may start while its predecessor
// is still draining; it calls pdl_wait() before touching anything the predecessor wrote.
// Every small kernel asks for the largest shared-memory carve-out although it uses next to none: an SM keeps its
// carve-out while blocks are resident, and the next GEMM's blocks (some 200 KB each, launched early under
// programmatic dependent launch so that they can fetch weights ahead of their dependency) become resident
// beside a small kernel's blocks only if the SM is already configured for that much shared memory.
static void prefer_max_shared(const void* kernel) {
    static std::vector<std::pair<const void*, int>> done;      // (kernel, device) pairs already configured
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return; }
    for (const auto& e : done) if (e.first == kernel && e.second == dev) return;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) != cudaSuccess)
        cudaGetLastError();
    done.emplace_back(kernel, dev);
}

template <typename... KArgs, typename... Args>
void launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    static const bool carve = !(getenv("WD_NO_CARVEOUT") && atoi(getenv("WD_NO_CARVEOUT")));
    if (carve) prefer_max_shared((const void*)kernel);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = wd_pdl_enabled ? 1 : 0;
    ++wd_launch_counter;
    cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// block-wide sum; `red` is shared float[32]; every thread gets the result
__device__ __forceinline__ float block_sum(float v, float* red) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) red[w] = v;
    __syncthreads();
    float t = (lane < nw) ? red[lane] : 0.f;
    return warp_sum(t);
}
__device__ __forceinline__ float block_max(float v, float* red) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_max(v);
    __syncthreads();
    if (lane == 0) red[w] = v;
    __syncthreads();
    float t = (lane < nw) ? red[lane] : -INFINITY;
    return warp_max(t);
}

// Sum of n_split partial-sum slices at one float4 position.  Slices are loaded eight at a time
// before the first add so that their L2 round trips overlap (the narrow GEMMs of a few-row step leave up
// to six); the adds keep slice order.
template <int kWidth = 8>
__device__ __forceinline__ float4 sum_slices4(const float* __restrict__ p, int n_split, size_t stride) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s0 = 0; s0 < n_split; s0 += kWidth) {
        float4 t[kWidth];
#pragma unroll
        for (int k = 0; k < kWidth; ++k)
            t[k] = s0 + k < n_split ? *reinterpret_cast<const float4*>(p + (size_t)(s0 + k) * stride)
                                    : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int k = 0; k < kWidth; ++k) { acc.x += t[k].x; acc.y += t[k].y; acc.z += t[k].z; acc.w += t[k].w; }
    }
    return acc;
}
// The same with the loads pinned in program order (volatile), so that up to eight of them are in flight before the
// first add whatever the compiler would rather do with its registers: for kernels that are one L2 round trip long.
__device__ __forceinline__ float4 ld_f4_pinned(const float* p) {
    float4 v;
    asm volatile("ld.global.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ float4 sum_slices4_pinned(const float* __restrict__ p, int n_split, size_t stride) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s0 = 0; s0 < n_split; s0 += 8) {
        float4 t[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            t[k] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (s0 + k < n_split) t[k] = ld_f4_pinned(p + (size_t)(s0 + k) * stride);
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) { acc.x += t[k].x; acc.y += t[k].y; acc.z += t[k].z; acc.w += t[k].w; }
    }
    return acc;
}
__device__ __forceinline__ float sum_slices1(const float* __restrict__ p, int n_split, size_t stride) {
    float acc = 0.f;
    for (int s0 = 0; s0 < n_split; s0 += 4) {
        float t[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) t[k] = s0 + k < n_split ? p[(size_t)(s0 + k) * stride] : 0.f;
#pragma unroll
        for (int k = 0; k < 4; ++k) acc += t[k];
    }
    return acc;
}

// ---------------------------------------------------------------- device-side planner
// One block per sequence builds the step's index lists from the device-resident state (decoded
// flags, decode steps, the external window of the phase), so that consecutive steps can be
// enqueued without a host round trip.  The host passes only counts (which do not depend on
// which tokens were unmasked).  Handles the states whose visible set is a prefix range.
//   refresh:  external window = the first n_wex undecoded positions (ordered compaction),
//             rows = visible positions = 0 .. n_vis-1, active = the first n_act of the window
//             (window-only variant: rows = the window and the positions decoded since the
//             previous phase began, by a second ordered compaction over the visible range)
//   normal:   one pass over the window: undecoded members in order are active (the first A) or
//             buffer, decoded members whose age is 1..T are the transient; rows = active and
//             transient in position order
struct PlanArgs {
    int32_t refresh[WD_PLAN_MAX_BATCH], done[WD_PLAN_MAX_BATCH], n_wex[WD_PLAN_MAX_BATCH], n_vis[WD_PLAN_MAX_BATCH];
    int32_t row_off[WD_PLAN_MAX_BATCH + 1], act_off[WD_PLAN_MAX_BATCH + 1], vis_off[WD_PLAN_MAX_BATCH + 1],
        qt_off[WD_PLAN_MAX_BATCH + 1];
    int32_t t[WD_PLAN_MAX_BATCH];
    int32_t window_refresh[WD_PLAN_MAX_BATCH], prev_phase_start[WD_PLAN_MAX_BATCH];
    int32_t S, A, T, batch;
    const uint8_t* decoded;
    const int32_t* dec_step;
    int32_t* wex;                 // [batch][S]
    int32_t *row_seq, *row_pos, *act_row, *act_pos, *act_off_dev, *vis_off_dev, *vis_idx, *qt_seq, *qt_row0, *qt_n, *nvis_dev,
        *tseq_dev;
    int32_t* status;
};

// exclusive prefix sum of one flag per thread over the block; returns this thread's offset and the total
__device__ __forceinline__ int block_scan_flag(int flag, int* total, int* warp_sums) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const unsigned bal = __ballot_sync(0xffffffffu, flag);
    const int in_warp = __popc(bal & ((1u << lane) - 1u));
    __syncthreads();
    if (lane == 0) warp_sums[w] = __popc(bal);
    __syncthreads();
    int off = 0, tot = 0;
    for (int i = 0; i < nw; ++i) {
        const int v = warp_sums[i];
        if (i < w) off += v;
        tot += v;
    }
    *total = tot;
    return off + in_warp;
}

__global__ void plan_kernel(const PlanArgs a) {
    __shared__ int warp_sums[32];
    pdl_launch_dependents();
    pdl_wait();
    const int b = blockIdx.x;
    if (threadIdx.x == 0) {
        a.act_off_dev[b] = a.act_off[b];
        a.vis_off_dev[b] = a.vis_off[b];
        a.nvis_dev[b] = a.done[b] ? 0 : a.n_vis[b];
        a.tseq_dev[b] = a.t[b];
        if (b == a.batch - 1) { a.act_off_dev[a.batch] = a.act_off[a.batch]; a.vis_off_dev[a.batch] = a.vis_off[a.batch]; }
    }
    if (a.done[b]) return;
    const int S = a.S, row0 = a.row_off[b], act0 = a.act_off[b];
    const uint8_t* dec = a.decoded + (size_t)b * S;
    const int32_t* dstep = a.dec_step + (size_t)b * S;
    int32_t* wex = a.wex + (size_t)b * S;
    const int n_wex = a.n_wex[b], n_vis = a.n_vis[b];
    const int n_rows = a.row_off[b + 1] - row0, n_act = a.act_off[b + 1] - act0;
    // visible range and query tiles follow from the counts alone
    for (int j = threadIdx.x; j < n_vis; j += blockDim.x) a.vis_idx[a.vis_off[b] + j] = j;
    for (int j = threadIdx.x; j < a.qt_off[b + 1] - a.qt_off[b]; j += blockDim.x) {
        a.qt_seq[a.qt_off[b] + j] = b;
        a.qt_row0[a.qt_off[b] + j] = row0 + 128 * j;
        a.qt_n[a.qt_off[b] + j] = min(128, n_rows - 128 * j);
    }
    if (a.refresh[b]) {
        // ordered compaction of the undecoded positions: the first n_wex form the window
        int base = 0;
        for (int i0 = 0; i0 < S && base < n_wex; i0 += blockDim.x) {
            const int i = i0 + threadIdx.x;
            const int und = (i < S && !dec[i]) ? 1 : 0;
            int tot;
            const int idx = base + block_scan_flag(und, &tot, warp_sums);
            if (und && idx < n_wex) {
                wex[idx] = i;
                if (idx < n_act) { a.act_pos[act0 + idx] = i; a.act_row[act0 + idx] = row0 + i; }
            }
            base += tot;
        }
        if (base < n_wex && threadIdx.x == 0) atomicCAS(a.status, 0, WD_ERR_BOUNDS);   // counts and state disagree
        if (!a.window_refresh[b]) {
            for (int j = threadIdx.x; j < n_rows; j += blockDim.x) { a.row_seq[row0 + j] = b; a.row_pos[row0 + j] = j; }
            return;
        }
        // window-only refresh: inside the visible range every undecoded position belongs to the
        // window; decoded positions are rows when they were unmasked during the phase that just ended
        int n_und = 0, n_row = 0;
        for (int i0 = 0; i0 < n_vis; i0 += blockDim.x) {
            const int i = i0 + threadIdx.x;
            const int und = (i < n_vis && !dec[i]) ? 1 : 0;
            const int prev = (i < n_vis && dec[i] && dstep[i] >= a.prev_phase_start[b]) ? 1 : 0;   // "never" is a large negative step
            int tot_u, tot_r;
            const int rank_u = n_und + block_scan_flag(und, &tot_u, warp_sums);
            const int rank_r = n_row + block_scan_flag(und | prev, &tot_r, warp_sums);
            if (und | prev) {
                if (rank_r < n_rows) { a.row_seq[row0 + rank_r] = b; a.row_pos[row0 + rank_r] = i; }
                else atomicCAS(a.status, 0, WD_ERR_BOUNDS);
            }
            if (und && rank_u < n_act) a.act_row[act0 + rank_u] = row0 + rank_r;
            n_und += tot_u;
            n_row += tot_r;
        }
        if (threadIdx.x == 0 && n_row != n_rows) atomicCAS(a.status, 0, WD_ERR_BOUNDS);
        return;
    }
    int n_und = 0, n_row = 0;
    for (int j0 = 0; j0 < n_wex; j0 += blockDim.x) {
        const int j = j0 + threadIdx.x;
        int und = 0, trans = 0, pos = 0;
        if (j < n_wex) {
            pos = wex[j];
            und = dec[pos] ? 0 : 1;
            const long long age = (long long)a.t[b] - (long long)dstep[pos];
            trans = (!und && age >= 1 && age <= a.T) ? 1 : 0;
        }
        int tot_u, tot_r;
        const int rank_u = n_und + block_scan_flag(und, &tot_u, warp_sums);
        const int act = und && rank_u < a.A;
        const int rank_r = n_row + block_scan_flag(act | trans, &tot_r, warp_sums);
        if (act | trans) {
            if (rank_r < n_rows) { a.row_seq[row0 + rank_r] = b; a.row_pos[row0 + rank_r] = pos; }
            else atomicCAS(a.status, 0, WD_ERR_BOUNDS);
        }
        if (act) {
            if (rank_u < n_act) { a.act_pos[act0 + rank_u] = pos; a.act_row[act0 + rank_u] = row0 + rank_r; }
            else atomicCAS(a.status, 0, WD_ERR_BOUNDS);
        }
        n_und += tot_u;
        n_row += tot_r;
    }
    if (threadIdx.x == 0 && n_row != n_rows) atomicCAS(a.status, 0, WD_ERR_BOUNDS);
}

// ---------------------------------------------------------------- embedding gather + RoPE table
// One block per computed row.  Also fills this step's rotary table: (cos, sin) of
// pos * theta^(-2j/dh) for j < dh/2, evaluated in double so that the angle of a late position
// is not limited by float rounding of the frequency.
template <typename T>
__global__ void embed_kernel(const T* __restrict__ embed, const int32_t* __restrict__ ids,
                             const int32_t* __restrict__ row_seq, const int32_t* __restrict__ row_pos,
                             float* __restrict__ x, float2* __restrict__ rope_tab, int d, int S, int vocab, int dh,
                             double log2_theta, int32_t* status) {
    // Wait first, trigger second: programmatic launch orders a kernel only against its immediate
    // predecessor's trigger, and every later kernel of the step triggers at its start.  With the
    // trigger here after the wait, no later kernel starts before the planner kernel (this kernel's
    // predecessor when the device plans the step) has finished, so they may all read the step's
    // index lists before their own wait.
    pdl_wait();
    pdl_launch_dependents();
    const int r = blockIdx.x;
    const int pos = row_pos[r];
    for (int j = threadIdx.x; j < dh / 2; j += blockDim.x) {
        const double ang = (double)pos * exp2(-2.0 * (double)j / (double)dh * log2_theta);
        double sn, cs;
        sincos(ang, &sn, &cs);
        rope_tab[(size_t)r * (dh / 2) + j] = make_float2((float)cs, (float)sn);
    }
    const int id = ids[(size_t)row_seq[r] * S + pos];
    if (id < 0 || id >= vocab) {           // checked, never dereferenced
        if (threadIdx.x == 0) atomicCAS(status, 0, WD_ERR_BOUNDS);
        for (int c = threadIdx.x; c < d; c += blockDim.x) x[(size_t)r * d + c] = 0.f;
        return;
    }
    const T* src = embed + (size_t)id * d;
    for (int c = threadIdx.x; c < d; c += blockDim.x) x[(size_t)r * d + c] = to_f(src[c]);
}

// Same gather for the fused pipeline: besides x it writes xg = bf16(x * gain) (the un-normalised
// GEMM input; the 1/rms factor is applied by the GEMM's consumer) and the per-row sums of
// squares of every 128-column block, sumsq[block][row].  Warp w owns blocks w, w+8, ...; the
// sum inside a block is a fixed shuffle tree, so the result is reproducible bit for bit.
__global__ void embed_fused_kernel(const __nv_bfloat16* __restrict__ embed, const int32_t* __restrict__ ids,
                                   const int32_t* __restrict__ row_seq, const int32_t* __restrict__ row_pos,
                                   float* __restrict__ x, __nv_bfloat16* __restrict__ xg, const float* __restrict__ gain,
                                   float* __restrict__ sumsq, float2* __restrict__ rope_tab, int n_rows, int d, int S,
                                   int vocab, int dh, double log2_theta, int32_t* status) {
    pdl_wait();                   // wait first, trigger second: see embed_kernel
    pdl_launch_dependents();
    const int r = blockIdx.x;
    const int pos = row_pos[r];
    for (int j = threadIdx.x; j < dh / 2; j += blockDim.x) {
        const double ang = (double)pos * exp2(-2.0 * (double)j / (double)dh * log2_theta);
        double sn, cs;
        sincos(ang, &sn, &cs);
        rope_tab[(size_t)r * (dh / 2) + j] = make_float2((float)cs, (float)sn);
    }
    int id = ids[(size_t)row_seq[r] * S + pos];
    const bool bad = id < 0 || id >= vocab;
    if (bad) {
        if (threadIdx.x == 0) atomicCAS(status, 0, WD_ERR_BOUNDS);
        id = 0;
    }
    const __nv_bfloat16* src = embed + (size_t)id * d;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    for (int blk = w; blk < d / 128; blk += nw) {
        float ss = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int c = blk * 128 + lane * 4 + i;
            const float v = bad ? 0.f : __bfloat162float(src[c]);
            x[(size_t)r * d + c] = v;
            xg[(size_t)r * d + c] = __float2bfloat16_rn(v * gain[c]);
            ss += v * v;
        }
        ss = warp_sum(ss);
        if (lane == 0) sumsq[(size_t)blk * n_rows + r] = ss;
    }
}

// ---------------------------------------------------------------- RMSNorm (+ partial-sum add)
// One block per row; columns in groups of four (float4 loads, all slices of a group in flight
// together).  d must be a multiple of 4.
template <typename T> struct Vec4;
template <> struct Vec4<float> {
    static __device__ __forceinline__ void store(float* p, float a, float b, float c, float d) {
        *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d);
    }
};
template <> struct Vec4<__nv_bfloat16> {
    static __device__ __forceinline__ void store(__nv_bfloat16* p, float a, float b, float c, float d) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
        uint2 u;
        u.x = *reinterpret_cast<uint32_t*>(&lo);
        u.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(p) = u;
    }
};

// four floats -> four e4m3 codes (round to nearest even, saturating), lowest byte first
__device__ __forceinline__ uint32_t pack_e4m3(float a, float b, float c, float d) {
    return (uint32_t)__nv_cvt_float_to_fp8(a, __NV_SATFINITE, __NV_E4M3) |
           ((uint32_t)__nv_cvt_float_to_fp8(b, __NV_SATFINITE, __NV_E4M3) << 8) |
           ((uint32_t)__nv_cvt_float_to_fp8(c, __NV_SATFINITE, __NV_E4M3) << 16) |
           ((uint32_t)__nv_cvt_float_to_fp8(d, __NV_SATFINITE, __NV_E4M3) << 24);
}

// The front of the RMSNorm kernels: x += sum of the partial slices (if any), v = the row's float4 of this
// thread, returns 1 / rms of the row.
template <int MAXV, bool kPinned = false>
__device__ __forceinline__ float rmsnorm_front(float* __restrict__ xr, const float* __restrict__ part, int n_split,
                                               size_t split_stride, size_t row_off, int nv, int d, float eps,
                                               const float* __restrict__ gain, float4 (&v)[MAXV], float4 (&gv)[MAXV],
                                               float* red) {
    float4 add[MAXV];
    float ss = 0.f;
#pragma unroll
    for (int u = 0; u < MAXV; ++u) {             // all loads first: x, the gains and every slice of every group
        const int c4 = threadIdx.x + u * blockDim.x;
        if (c4 < nv) {
            if (kPinned) {
                // few rows: row, gains and every slice in flight together
                v[u] = ld_f4_pinned(xr + 4 * c4);
                gv[u] = ld_f4_pinned(gain + 4 * c4);
                if (part) add[u] = sum_slices4_pinned(part + row_off + 4 * c4, n_split, split_stride);
            } else {
                v[u] = reinterpret_cast<const float4*>(xr)[c4];
                gv[u] = reinterpret_cast<const float4*>(gain)[c4];   // not needed before the reduction, but no round trip after it
                if (part) add[u] = sum_slices4(part + row_off + 4 * c4, n_split, split_stride);
            }
        }
    }
#pragma unroll
    for (int u = 0; u < MAXV; ++u) {
        const int c4 = threadIdx.x + u * blockDim.x;
        if (c4 < nv) {
            float4 a = v[u];
            if (part) {
                a.x += add[u].x; a.y += add[u].y; a.z += add[u].z; a.w += add[u].w;
                reinterpret_cast<float4*>(xr)[c4] = a;
            }
            v[u] = a;
            ss += a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
        }
    }
    ss = block_sum(ss, red);
    return rsqrtf(ss / (float)d + eps);
}

template <typename T, int MAXV>
__global__ void __launch_bounds__(1024) rmsnorm_kernel(float* __restrict__ x, const float* __restrict__ part, int n_split,
                               size_t split_stride, const float* __restrict__ gain, float eps,
                               T* __restrict__ xn, const int32_t* __restrict__ row_idx, int d,
                               uint8_t* __restrict__ xq, float* __restrict__ sx) {
    __shared__ float red[32];
    pdl_launch_dependents();
    pdl_wait();
    S_STAMP(1);
    const int i = blockIdx.x;
    const int r = row_idx ? row_idx[i] : i;
    const int nv = d >> 2;
    float4 v[MAXV], gv[MAXV];
    const float inv = rmsnorm_front<MAXV>(x + (size_t)r * d, part, n_split, split_stride, (size_t)r * d, nv, d, eps, gain, v, gv, red);
    S_MID();
    if (xq) {
        // FP8 output: e4m3 codes of (value / s) with s = max |value| / 448 of this row (1 for a zero row)
        float amax = 0.f;
#pragma unroll
        for (int u = 0; u < MAXV; ++u) {
            const int c4 = threadIdx.x + u * blockDim.x;
            if (c4 < nv) {
                const float4 g = gv[u];
                v[u] = make_float4(v[u].x * inv * g.x, v[u].y * inv * g.y, v[u].z * inv * g.z, v[u].w * inv * g.w);
                amax = fmaxf(fmaxf(fmaxf(amax, fabsf(v[u].x)), fmaxf(fabsf(v[u].y), fabsf(v[u].z))), fabsf(v[u].w));
            }
        }
        amax = block_max(amax, red);
        const float s = amax > 0.f ? amax / 448.f : 1.f;
        if (threadIdx.x == 0) sx[i] = s;
#pragma unroll
        for (int u = 0; u < MAXV; ++u) {
            const int c4 = threadIdx.x + u * blockDim.x;
            if (c4 < nv) reinterpret_cast<uint32_t*>(xq + (size_t)i * d)[c4] = pack_e4m3(v[u].x / s, v[u].y / s, v[u].z / s, v[u].w / s);
        }
        return;
    }
#pragma unroll
    for (int u = 0; u < MAXV; ++u) {
        const int c4 = threadIdx.x + u * blockDim.x;
        if (c4 < nv) {
            const float4 g = gv[u];
            Vec4<T>::store(xn + (size_t)i * d + 4 * c4, v[u].x * inv * g.x, v[u].y * inv * g.y, v[u].z * inv * g.z,
                           v[u].w * inv * g.w);
        }
    }
}

// Few rows (one block per row cannot fill the machine, so the kernel is as long as its loads): 512 threads with two
// float4 each and all their loads — row, gains, up to eight K slices — in flight at once, which takes 80 registers;
// capped at 88 so that such a block (45 K registers) and a CTA of the next GEMM (18 K), launched early to fetch its
// weights, fit an SM's register file together.  With 1024 threads that budget is 40 registers, too few for the loads.
template <typename T>
__global__ void __maxnreg__(88) rmsnorm_rows_kernel(float* __restrict__ x, const float* __restrict__ part, int n_split,
                                                    size_t split_stride, const float* __restrict__ gain, float eps,
                                                    T* __restrict__ xn, const int32_t* __restrict__ row_idx, int d) {
    __shared__ float red[32];
    pdl_launch_dependents();
    pdl_wait();
    S_STAMP(1);
    const int i = blockIdx.x;
    const int r = row_idx ? row_idx[i] : i;
    const int nv = d >> 2;
    float4 v[2], gv[2];
    const float inv = rmsnorm_front<2, true>(x + (size_t)r * d, part, n_split, split_stride, (size_t)r * d, nv, d, eps, gain, v, gv, red);
    S_MID();
#pragma unroll
    for (int u = 0; u < 2; ++u) {
        const int c4 = threadIdx.x + u * blockDim.x;
        if (c4 < nv) {
            const float4 g = gv[u];
            Vec4<T>::store(xn + (size_t)i * d + 4 * c4, v[u].x * inv * g.x, v[u].y * inv * g.y, v[u].z * inv * g.z,
                           v[u].w * inv * g.w);
        }
    }
}

// The same with NVFP4 output of the bfloat16 rounding of the normalised row (a kernel of its own, so that the
// bf16 path's kernel carries neither its arguments nor its code): row scale max / (6 * 448), then blocks of 16
// elements held by four neighbouring lanes.  d % 16 == 0.
template <int MAXV>
__global__ void __launch_bounds__(1024, 1) rmsnorm_fp4_kernel(float* __restrict__ x, const float* __restrict__ part, int n_split,
                                   size_t split_stride, const float* __restrict__ gain, float eps,
                                   const int32_t* __restrict__ row_idx, int d, WdFp4Operand x4) {
    __shared__ float red[32];
    pdl_launch_dependents();
    pdl_wait();
    const int i = blockIdx.x;
    const int r = row_idx ? row_idx[i] : i;
    const int nv = d >> 2;
    float4 v[MAXV], gv[MAXV];
    const float inv = rmsnorm_front<MAXV>(x + (size_t)r * d, part, n_split, split_stride, (size_t)r * d, nv, d, eps, gain, v, gv, red);
    float amax = 0.f;
#pragma unroll
    for (int u = 0; u < MAXV; ++u) {
        const int c4 = threadIdx.x + u * blockDim.x;
        if (c4 < nv) {
            const float4 g = gv[u];
            v[u] = make_float4(wdk::bf16_round_f(v[u].x * inv * g.x), wdk::bf16_round_f(v[u].y * inv * g.y),
                               wdk::bf16_round_f(v[u].z * inv * g.z), wdk::bf16_round_f(v[u].w * inv * g.w));
            amax = fmaxf(fmaxf(fmaxf(amax, fabsf(v[u].x)), fmaxf(fabsf(v[u].y), fabsf(v[u].z))), fabsf(v[u].w));
        } else {
            v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
    amax = block_max(amax, red);
    const float gr = amax > 0.f ? __fdiv_rn(amax, 6.0f * 448.0f) : 1.f;
    if (threadIdx.x == 0) x4.g[i] = gr;
#pragma unroll
    for (int u = 0; u < MAXV; ++u) {
        const int c4 = threadIdx.x + u * blockDim.x;
        wdk::nvfp4_emit4(v[u], gr, c4 < nv, x4.codes + (size_t)i * (d >> 1), x4.sf + (size_t)i * (d >> 4), c4);
    }
}

// ---------------------------------------------------------------- CUDA-core GEMM
// y[rows, n] = x[rows, k] * w[n, k]^T.  32 x 64 output tile per block, 2 x 4 per thread.
template <typename T>
__global__ void gemm_plain_kernel(const T* __restrict__ x, const T* __restrict__ w, float* __restrict__ y,
                                  int rows, int n, int k, int ldy) {
    __shared__ float xs[32][33];
    __shared__ float ws[64][33];
    pdl_launch_dependents();
    pdl_wait();
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;          // 16 x 16
    const int r0 = blockIdx.y * 32, n0 = blockIdx.x * 64;
    float acc[2][4] = {};
    for (int k0 = 0; k0 < k; k0 += 32) {
        for (int i = threadIdx.x; i < 32 * 32; i += 256) {
            const int rr = i >> 5, kk = i & 31;
            xs[rr][kk] = (r0 + rr < rows && k0 + kk < k) ? to_f(x[(size_t)(r0 + rr) * k + k0 + kk]) : 0.f;
        }
        for (int i = threadIdx.x; i < 64 * 32; i += 256) {
            const int nn = i >> 5, kk = i & 31;
            ws[nn][kk] = (n0 + nn < n && k0 + kk < k) ? to_f(w[(size_t)(n0 + nn) * k + k0 + kk]) : 0.f;
        }
        __syncthreads();
#pragma unroll 8
        for (int kk = 0; kk < 32; ++kk) {
            const float a0 = xs[ty][kk], a1 = xs[ty + 16][kk];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float b = ws[tx + 16 * j][kk];
                acc[0][j] += a0 * b;
                acc[1][j] += a1 * b;
            }
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int r = r0 + ty + 16 * i;
        if (r >= rows) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = n0 + tx + 16 * j;
            if (c < n) y[(size_t)r * ldy + c] = acc[i][j];
        }
    }
}

// ---------------------------------------------------------------- RoPE + K/V scatter
// Adds the split-K slices of the fused q/k/v projection, rotates q and k heads by the row's
// table, writes q and the K/V cache rows.  K cache [batch][Hkv][S][dh]; V cache transposed
// [batch][Hkv][dh][Sp] so that attention can read V tiles with the key position contiguous.
// One 1-D grid, two kinds of 256-thread blocks:
//   blocks [0, n_qk):  (row, group of q/k heads), four rotation pairs per thread (one pair and
//                      groups of 4 heads when head_dim / 2 is not a multiple of 4)
//   blocks [n_qk, ..): (v head, 32 head dims, 32 rows): slices summed with the dims contiguous,
//                      transposed through shared memory and written with the rows (normally
//                      consecutive positions) contiguous, so neighbouring lanes share sectors
template <typename T>
__global__ void __launch_bounds__(256, 4) rope_scatter_kernel(const float* __restrict__ part, int n_split, size_t split_stride,
                                    const int32_t* __restrict__ row_seq, const int32_t* __restrict__ row_pos,
                                    const float2* __restrict__ rope_tab, T* __restrict__ q, T* __restrict__ kcache,
                                    T* __restrict__ vcache, int n_rows, int Hq, int Hkv, int dh, int S, int Sp,
                                    int n_qk, int qk_groups, int n_qk_blocks, int batch, int32_t* __restrict__ status) {
    __shared__ float tile[32][33];
    pdl_launch_dependents();
    pdl_wait();
    S_STAMP(2);
    const int half = dh >> 1;
    const int ncol = (Hq + 2 * Hkv) * dh;
    if ((int)blockIdx.x < n_qk_blocks) {
        // a block walks (row, head group) items n_qk_blocks apart: with thousands of rows one item per block
        // would be all launch overhead
        for (int item = blockIdx.x; item < n_qk; item += n_qk_blocks) {
            const int r = item / qk_groups, grp = item - r * qk_groups;
            const int pos = row_pos[r], b = row_seq[r];
            // index check: a cache row outside the state is recorded and not written
            const bool in_range = (unsigned)pos < (unsigned)S && (unsigned)b < (unsigned)batch;
            if (!in_range && threadIdx.x == 0) atomicCAS(status, 0, WD_ERR_BOUNDS);
            const float* pr = part + (size_t)r * ncol;
            if ((half & 3) == 0) {
                // four rotation pairs per thread (float4 loads, 8-byte bf16 stores): half/4 threads per head
                const int tph = half >> 2, hpb = blockDim.x / tph;
                const int h = grp * hpb + (int)threadIdx.x / tph, j = ((int)threadIdx.x % tph) * 4;
                // (the loads do not wait for the index check: only the store of a cache row does)
                if ((int)threadIdx.x < hpb * tph && h < Hq + Hkv) {
                    float4 a, bb, c01, c23;
                    if (n_split <= 4) {
                        // few slices (the usual case): the table and both halves' slices in flight together
                        float4 ta[4], tb[4];
                        c01 = ld_f4_pinned(reinterpret_cast<const float*>(rope_tab + (size_t)r * half + j));   // (cos, sin) x 2
                        c23 = ld_f4_pinned(reinterpret_cast<const float*>(rope_tab + (size_t)r * half + j + 2));
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            ta[k] = tb[k] = make_float4(0.f, 0.f, 0.f, 0.f);
                            if (k < n_split) {
                                ta[k] = ld_f4_pinned(pr + h * dh + j + (size_t)k * split_stride);
                                tb[k] = ld_f4_pinned(pr + h * dh + half + j + (size_t)k * split_stride);
                            }
                        }
                        a = bb = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            a.x += ta[k].x; a.y += ta[k].y; a.z += ta[k].z; a.w += ta[k].w;
                            bb.x += tb[k].x; bb.y += tb[k].y; bb.z += tb[k].z; bb.w += tb[k].w;
                        }
                    } else {
                        a = sum_slices4(pr + h * dh + j, n_split, split_stride);
                        bb = sum_slices4(pr + h * dh + half + j, n_split, split_stride);
                        c01 = *reinterpret_cast<const float4*>(rope_tab + (size_t)r * half + j);
                        c23 = *reinterpret_cast<const float4*>(rope_tab + (size_t)r * half + j + 2);
                    }
                    if (h >= Hq && !in_range) continue;
                    T* dst = h < Hq ? q + ((size_t)r * Hq + h) * dh : kcache + (((size_t)b * Hkv + (h - Hq)) * S + pos) * dh;
                    Vec4<T>::store(dst + j, a.x * c01.x - bb.x * c01.y, a.y * c01.z - bb.y * c01.w, a.z * c23.x - bb.z * c23.y,
                                   a.w * c23.z - bb.w * c23.w);
                    Vec4<T>::store(dst + j + half, bb.x * c01.x + a.x * c01.y, bb.y * c01.z + a.y * c01.w,
                                   bb.z * c23.x + a.z * c23.y, bb.w * c23.z + a.w * c23.w);
                }
                continue;
            }
            const int h0 = grp * 4;
            for (int i = threadIdx.x; i < 4 * half; i += blockDim.x) {
                const int h = h0 + i / half, j = i % half;
                if (h >= Hq + Hkv) break;
                if (h >= Hq && !in_range) continue;
                const float a = sum_slices1(pr + h * dh + j, n_split, split_stride);
                const float bb = sum_slices1(pr + h * dh + j + half, n_split, split_stride);
                const float2 cs = rope_tab[(size_t)r * half + j];
                const float ra = a * cs.x - bb * cs.y, rb = bb * cs.x + a * cs.y;
                T* dst = h < Hq ? q + ((size_t)r * Hq + h) * dh : kcache + (((size_t)b * Hkv + (h - Hq)) * S + pos) * dh;
                dst[j] = from_f<T>(ra);
                dst[j + half] = from_f<T>(rb);
            }
        }
        return;
    }
    const int vb = blockIdx.x - n_qk_blocks;
    const int dchunks = (dh + 31) / 32, rchunks = (n_rows + 31) / 32;
    const int kh = vb / (dchunks * rchunks), rem = vb - kh * dchunks * rchunks;
    const int d0 = (rem / rchunks) * 32, r0 = (rem % rchunks) * 32;
    const int lx = threadIdx.x & 31, ly = threadIdx.x >> 5;
    const int vcol = (Hq + Hkv) * dh + kh * dh + d0;
    const int r_out = r0 + lx;                                   // the row this thread writes after the transpose
    const int pos_out = r_out < n_rows ? row_pos[r_out] : 0, b_out = r_out < n_rows ? row_seq[r_out] : 0;
    if ((dh & 3) == 0) {
        // one float4 (four head dims of one row) per thread
        const int rr = threadIdx.x >> 3, d4 = (threadIdx.x & 7) * 4, r = r0 + rr;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (r < n_rows && d0 + d4 < dh) v = sum_slices4(part + (size_t)r * ncol + vcol + d4, n_split, split_stride);
        tile[rr][d4] = v.x; tile[rr][d4 + 1] = v.y; tile[rr][d4 + 2] = v.z; tile[rr][d4 + 3] = v.w;
    } else {
        for (int rr = ly; rr < 32; rr += 8) {
            const int r = r0 + rr;
            tile[rr][lx] = (r < n_rows && d0 + lx < dh)
                ? sum_slices1(part + (size_t)r * ncol + vcol + lx, n_split, split_stride) : 0.f;
        }
    }
    __syncthreads();
    const int r = r_out;
    if (r < n_rows) {
        const int pos = pos_out, b = b_out;
        if ((unsigned)pos < (unsigned)S && (unsigned)b < (unsigned)batch) {
            T* dst = vcache + ((size_t)b * Hkv + kh) * dh * Sp + pos;
            for (int dd = ly; dd < 32 && d0 + dd < dh; dd += 8) dst[(size_t)(d0 + dd) * Sp] = from_f<T>(tile[lx][dd]);
        } else if (ly == 0) {
            atomicCAS(status, 0, WD_ERR_BOUNDS);
        }
    }
}

// ---------------------------------------------------------------- CUDA-core attention
// One block (128 threads) per (row, head).  Scores of all visible positions in shared
// memory, then softmax, then the weighted sum of V rows.
template <typename T>
__global__ void attention_plain_kernel(const T* __restrict__ q, const T* __restrict__ kcache,
                                       const T* __restrict__ vcache, const int32_t* __restrict__ row_seq,
                                       const int32_t* __restrict__ vis_idx, const int32_t* __restrict__ vis_off,
                                       T* __restrict__ out, float* __restrict__ tap, int nv_single, int Hq,
                                       int Hkv, int dh, int S, int Sp, int batch, int32_t* __restrict__ status) {
    extern __shared__ float sc[];                 // [n_vis] scores, then dh floats of q
    __shared__ float red[32];
    pdl_launch_dependents();
    pdl_wait();
    const int r = blockIdx.x, h = blockIdx.y;
    int b = row_seq ? row_seq[r] : 0;
    if ((unsigned)b >= (unsigned)batch) {              // index check: recorded, the row reads sequence 0 instead
        if (threadIdx.x == 0) atomicCAS(status, 0, WD_ERR_BOUNDS);
        b = 0;
    }
    const int v0 = vis_off ? vis_off[b] : 0;
    const int nv = vis_off ? vis_off[b + 1] - v0 : nv_single;
    const int kvh = h / (Hq / Hkv);
    const T* kb = kcache + ((size_t)b * Hkv + kvh) * S * dh;
    const T* vb = vcache + ((size_t)b * Hkv + kvh) * dh * Sp;     // [dh][Sp]
    float* qs = sc + nv;
    for (int c = threadIdx.x; c < dh; c += blockDim.x) qs[c] = to_f(q[((size_t)r * Hq + h) * dh + c]);
    __syncthreads();
    const float scale = rsqrtf((float)dh);
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
    float mx = -INFINITY;
    for (int j = wid; j < nv; j += nw) {
        const int vi = vis_idx[v0 + j];
        if ((unsigned)vi >= (unsigned)S) {             // index check: recorded, the position is left out (weight 0)
            if (lane == 0) { atomicCAS(status, 0, WD_ERR_BOUNDS); sc[j] = -INFINITY; }
            continue;
        }
        const T* kr = kb + (size_t)vi * dh;
        float a = 0.f;
        for (int c = lane; c < dh; c += 32) a += qs[c] * to_f(kr[c]);
        a = warp_sum(a) * scale;
        if (lane == 0) sc[j] = a;
        mx = fmaxf(mx, a);
    }
    mx = block_max(mx, red);
    __syncthreads();
    float sum = 0.f;
    for (int j = threadIdx.x; j < nv; j += blockDim.x) {
        const float e = __expf(sc[j] - mx);
        sc[j] = e;
        sum += e;
    }
    sum = block_sum(sum, red);
    __syncthreads();
    const float inv = 1.f / sum;
    // V is stored transposed ([dh][Sp]): each warp takes head dims c = wid, wid + nw, ... and its
    // lanes stride over the visible positions, so consecutive lanes read consecutive positions
    for (int c = wid; c < dh; c += nw) {
        const T* vr = vb + (size_t)c * Sp;
        float a = 0.f;
        for (int j = lane; j < nv; j += 32) {
            const int vi = vis_idx[v0 + j];
            if ((unsigned)vi < (unsigned)S) a += sc[j] * to_f(vr[vi]);
        }
        a = warp_sum(a) * inv;
        if (lane == 0) {
            const size_t o = ((size_t)r * Hq + h) * dh + c;
            out[o] = from_f<T>(a);
            if (tap) tap[o] = a;
        }
    }
}

// ---------------------------------------------------------------- SwiGLU
// four columns per thread; F must be a multiple of 4
// (Registers capped at 51: three of its blocks and a CTA of the down-projection GEMM, launched early to fetch
// its weights, then fit an SM's register file together; the gate/up launch leaves at most four K slices.)
template <typename T>
__global__ void __launch_bounds__(256, 5) swiglu_kernel(const float* __restrict__ part, int n_split, size_t split_stride,
                                                        T* __restrict__ h, int n_rows, int F) {
    pdl_launch_dependents();
    pdl_wait();
    S_STAMP(3);
    const int f4 = F >> 2;
    const size_t total = (size_t)n_rows * f4, stride = (size_t)gridDim.x * blockDim.x;
    // two positions per iteration so that four (or more) loads are in flight per thread
    for (size_t i0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i0 < total; i0 += 2 * stride) {
        const size_t i1 = i0 + stride;
        const bool has1 = i1 < total;
        const size_t ra = i0 / f4, ca = i0 - ra * f4, rb = has1 ? i1 / f4 : ra, cb = has1 ? i1 - rb * f4 : ca;
        const float* pa = part + ra * 2 * F + 4 * ca;
        const float* pb = part + rb * 2 * F + 4 * cb;
        float4 ga, ua, gb, ub;
        if (n_split == 1) {
            ga = *reinterpret_cast<const float4*>(pa);
            ua = *reinterpret_cast<const float4*>(pa + F);
            gb = *reinterpret_cast<const float4*>(pb);
            ub = *reinterpret_cast<const float4*>(pb + F);
        } else {
            ga = sum_slices4<4>(pa, n_split, split_stride);
            ua = sum_slices4<4>(pa + F, n_split, split_stride);
            gb = sum_slices4<4>(pb, n_split, split_stride);
            ub = sum_slices4<4>(pb + F, n_split, split_stride);
        }
        Vec4<T>::store(h + ra * F + 4 * ca, ga.x / (1.f + __expf(-ga.x)) * ua.x, ga.y / (1.f + __expf(-ga.y)) * ua.y,
                       ga.z / (1.f + __expf(-ga.z)) * ua.z, ga.w / (1.f + __expf(-ga.w)) * ua.w);
        if (has1)
            Vec4<T>::store(h + rb * F + 4 * cb, gb.x / (1.f + __expf(-gb.x)) * ub.x, gb.y / (1.f + __expf(-gb.y)) * ub.y,
                           gb.z / (1.f + __expf(-gb.z)) * ub.z, gb.w / (1.f + __expf(-gb.w)) * ub.w);
    }
}

// Few rows: one position per thread, 32-bit index arithmetic, all of a thread's loads (gate and up, up to four K
// slices each) in flight together; registers capped like the kernel above, for the same reason.
template <typename T>
__global__ void __launch_bounds__(256, 5) swiglu_rows_kernel(const float* __restrict__ part, int n_split, size_t split_stride,
                                                             T* __restrict__ h, int n_rows, int F) {
    pdl_launch_dependents();
    pdl_wait();
    S_STAMP(3);
    const int f4 = F >> 2;
    const int i = (int)(blockIdx.x * blockDim.x + threadIdx.x);
    if (i >= n_rows * f4) return;
    const int r = i / f4, c = i - r * f4;
    const float* pg = part + (size_t)r * 2 * F + 4 * c;
    float4 tg[4], tu[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        tg[k] = tu[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (k < n_split) {
            tg[k] = ld_f4_pinned(pg + (size_t)k * split_stride);
            tu[k] = ld_f4_pinned(pg + (size_t)k * split_stride + F);
        }
    }
    float4 g = make_float4(0.f, 0.f, 0.f, 0.f), u = g;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        g.x += tg[k].x; g.y += tg[k].y; g.z += tg[k].z; g.w += tg[k].w;
        u.x += tu[k].x; u.y += tu[k].y; u.z += tu[k].z; u.w += tu[k].w;
    }
    for (int s0 = 4; s0 < n_split; ++s0) {          // (more than four slices: not on this path's shapes, kept correct)
        const float4 a = *reinterpret_cast<const float4*>(pg + (size_t)s0 * split_stride);
        const float4 b = *reinterpret_cast<const float4*>(pg + (size_t)s0 * split_stride + F);
        g.x += a.x; g.y += a.y; g.z += a.z; g.w += a.w;
        u.x += b.x; u.y += b.y; u.z += b.z; u.w += b.w;
    }
    Vec4<T>::store(h + (size_t)r * F + 4 * c, g.x / (1.f + __expf(-g.x)) * u.x, g.y / (1.f + __expf(-g.y)) * u.y,
                   g.z / (1.f + __expf(-g.z)) * u.z, g.w / (1.f + __expf(-g.w)) * u.w);
}

// FP8 variant: a cluster of four 256-thread blocks per row (light blocks, so that they are resident
// and waiting while the GEMM still runs); each keeps its quarter of h = silu(gate) * up in registers
// (up to kMaxV float4 per thread), the four partial maxima meet through distributed shared memory,
// then every block writes the e4m3 codes of its quarter (and block 0 the row's scale).
// The front of the quantising SwiGLU kernels: this block's quarter of h = silu(gate) * up of row r in g[] (fp32,
// or rounded to bfloat16 when kRound), returns the row's maximum |h| (over the four blocks of the cluster).
template <int kMaxV, bool kRound>
__device__ __forceinline__ float swiglu_quarter(const float* __restrict__ part, int n_split, size_t split_stride, int F,
                                                int r, int c_lo, int c_hi, float4 (&g)[kMaxV], float* red, float* my_max) {
    const float* pr = part + (size_t)r * 2 * F;
    // slice by slice, all of this thread's positions at once: 2 * kMaxV loads in flight per round trip
    float4 up[kMaxV];
#pragma unroll
    for (int u = 0; u < kMaxV; ++u) g[u] = up[u] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int sl = 0; sl < n_split; ++sl) {
        const float* ps = pr + (size_t)sl * split_stride;
        float4 tg[kMaxV], tu[kMaxV];
#pragma unroll
        for (int u = 0; u < kMaxV; ++u) {
            const int c4 = c_lo + (int)threadIdx.x + u * (int)blockDim.x;
            tg[u] = tu[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (c4 < c_hi) {
                tg[u] = *reinterpret_cast<const float4*>(ps + 4 * c4);
                tu[u] = *reinterpret_cast<const float4*>(ps + F + 4 * c4);
            }
        }
#pragma unroll
        for (int u = 0; u < kMaxV; ++u) {
            g[u].x += tg[u].x; g[u].y += tg[u].y; g[u].z += tg[u].z; g[u].w += tg[u].w;
            up[u].x += tu[u].x; up[u].y += tu[u].y; up[u].z += tu[u].z; up[u].w += tu[u].w;
        }
    }
    float amax = 0.f;
#pragma unroll
    for (int u = 0; u < kMaxV; ++u) {
        g[u] = make_float4(g[u].x / (1.f + __expf(-g[u].x)) * up[u].x, g[u].y / (1.f + __expf(-g[u].y)) * up[u].y,
                           g[u].z / (1.f + __expf(-g[u].z)) * up[u].z, g[u].w / (1.f + __expf(-g[u].w)) * up[u].w);
        if (kRound)
            g[u] = make_float4(wdk::bf16_round_f(g[u].x), wdk::bf16_round_f(g[u].y), wdk::bf16_round_f(g[u].z), wdk::bf16_round_f(g[u].w));
        amax = fmaxf(fmaxf(fmaxf(amax, fabsf(g[u].x)), fmaxf(fabsf(g[u].y), fabsf(g[u].z))), fabsf(g[u].w));
    }
    amax = block_max(amax, red);
    if (threadIdx.x == 0) *my_max = amax;
    wdk::cluster_sync();                            // the four partial maxima are in place
    const uint32_t local = wdk::smem_u32(my_max);
    for (uint32_t k = 0; k < 4; ++k) {
        float v;
        asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(wdk::cluster_map(local, k)));
        amax = fmaxf(amax, v);
    }
    wdk::cluster_sync();                            // nobody leaves while its maximum may still be read
    return amax;
}

template <int kMaxV>
__global__ void swiglu_fp8_kernel(const float* __restrict__ part, int n_split, size_t split_stride,
                                  uint8_t* __restrict__ hq, float* __restrict__ sh, int F) {
    __shared__ float red[32];
    __shared__ float my_max;
    pdl_launch_dependents();
    pdl_wait();
    const int r = blockIdx.x >> 2, quarter = blockIdx.x & 3, f4 = F >> 2;
    const int q4 = (f4 + 3) >> 2, c_lo = quarter * q4, c_hi = min(f4, c_lo + q4);     // this block's float4 columns
    float4 g[kMaxV];
    const float amax = swiglu_quarter<kMaxV, false>(part, n_split, split_stride, F, r, c_lo, c_hi, g, red, &my_max);
    const float s = amax > 0.f ? amax / 448.f : 1.f;
    if (threadIdx.x == 0 && quarter == 0) sh[r] = s;
#pragma unroll
    for (int u = 0; u < kMaxV; ++u) {
        const int c4 = c_lo + (int)threadIdx.x + u * (int)blockDim.x;
        if (c4 < c_hi) reinterpret_cast<uint32_t*>(hq + (size_t)r * F)[c4] = pack_e4m3(g[u].x / s, g[u].y / s, g[u].z / s, g[u].w / s);
    }
}

// NVFP4 variant: the bfloat16 rounding of h as codes, block scales and row scale (F % 64 == 0, so that every
// block's quarter is a whole number of 16-element blocks held by four neighbouring lanes).
template <int kMaxV>
__global__ void swiglu_fp4_kernel(const float* __restrict__ part, int n_split, size_t split_stride, int F, WdFp4Operand h4) {
    __shared__ float red[32];
    __shared__ float my_max;
    pdl_launch_dependents();
    pdl_wait();
    const int r = blockIdx.x >> 2, quarter = blockIdx.x & 3, f4 = F >> 2;
    const int q4 = (f4 + 3) >> 2, c_lo = quarter * q4, c_hi = min(f4, c_lo + q4);
    float4 g[kMaxV];
    const float amax = swiglu_quarter<kMaxV, true>(part, n_split, split_stride, F, r, c_lo, c_hi, g, red, &my_max);
    const float gr = amax > 0.f ? __fdiv_rn(amax, 6.0f * 448.0f) : 1.f;
    if (threadIdx.x == 0 && quarter == 0) h4.g[r] = gr;
#pragma unroll
    for (int u = 0; u < kMaxV; ++u) {
        const int c4 = c_lo + (int)threadIdx.x + u * (int)blockDim.x;
        wdk::nvfp4_emit4(g[u], gr, c4 < c_hi, h4.codes + (size_t)r * (F >> 1), h4.sf + (size_t)r * (F >> 4), c4);
    }
}

// Per-row e4m3 quantisation of a [n_rows, K] matrix (weights once at set-up; K % 4 == 0): one block per row
template <typename T>
__global__ void quantize_rows_kernel(const T* __restrict__ w, int K, uint8_t* __restrict__ q, float* __restrict__ s_out) {
    __shared__ float red[32];
    const T* wr = w + (size_t)blockIdx.x * K;
    float amax = 0.f;
    for (int k = threadIdx.x; k < K; k += blockDim.x) amax = fmaxf(amax, fabsf(to_f(wr[k])));
    amax = block_max(amax, red);
    const float s = amax > 0.f ? amax / 448.f : 1.f;
    if (threadIdx.x == 0) s_out[blockIdx.x] = s;
    for (int k4 = threadIdx.x; k4 < (K >> 2); k4 += blockDim.x)
        reinterpret_cast<uint32_t*>(q + (size_t)blockIdx.x * K)[k4] =
            pack_e4m3(to_f(wr[4 * k4]) / s, to_f(wr[4 * k4 + 1]) / s, to_f(wr[4 * k4 + 2]) / s, to_f(wr[4 * k4 + 3]) / s);
}

// total is a multiple of 4 (d is)
__global__ void residual_add_kernel(float* __restrict__ x, const float* __restrict__ part, int n_split,
                                    size_t split_stride, float* __restrict__ tap, size_t total) {
    pdl_launch_dependents();
    pdl_wait();
    const size_t n4 = total >> 2, stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i0 < n4; i0 += 2 * stride) {
        const size_t i1 = i0 + stride < n4 ? i0 + stride : i0;
        float4 xa = reinterpret_cast<const float4*>(x)[i0], xb = reinterpret_cast<const float4*>(x)[i1];
        const float4 pa = sum_slices4(part + 4 * i0, n_split, split_stride);
        const float4 pb = sum_slices4(part + 4 * i1, n_split, split_stride);
        xa.x += pa.x; xa.y += pa.y; xa.z += pa.z; xa.w += pa.w;
        reinterpret_cast<float4*>(x)[i0] = xa;
        if (tap) reinterpret_cast<float4*>(tap)[i0] = xa;
        if (i1 != i0) {
            xb.x += pb.x; xb.y += pb.y; xb.z += pb.z; xb.w += pb.w;
            reinterpret_cast<float4*>(x)[i1] = xb;
            if (tap) reinterpret_cast<float4*>(tap)[i1] = xb;
        }
    }
}

// ---------------------------------------------------------------- unmask reduction
// Stage 1: grid (active row, vocabulary chunk).  Per chunk: maximum with the lowest index
// (thread-strided scan, warp-shuffle tree, 8 warp results in order) and the sum of
// exp(l - chunk max) in double.  Stage 2 (select_kernel) merges the chunks of a row in chunk
// order, which is the same fixed order for every row, so identical logit rows give identical
// bits.  The sums are in double because they decide which rows are unmasked: in double the
// ranking agrees with an exact evaluation of the same float logits down to 1e-13 gaps.
__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__global__ void rowstats_kernel(const float* __restrict__ logits, int V, int chunk, float* __restrict__ ch_max,
                                int32_t* __restrict__ ch_idx, double* __restrict__ ch_sum) {
    __shared__ float s_val[8];
    __shared__ int s_idx[8];
    __shared__ double s_sum[8];
    __shared__ float s_max;
    pdl_launch_dependents();
    pdl_wait();
    const int v0 = blockIdx.y * chunk, v1 = min(V, v0 + chunk);
    const float* lr = logits + (size_t)blockIdx.x * V;
    float best = -INFINITY;
    int bi = 0x7fffffff;
    for (int v = v0 + threadIdx.x; v < v1; v += 256) {
        const float l = lr[v];
        if (l > best) { best = l; bi = v; }       // strictly greater keeps the lowest index
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ob > best || (ob == best && oi < bi)) { best = ob; bi = oi; }
    }
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (lane == 0) { s_val[w] = best; s_idx[w] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        float b = s_val[0];
        int i = s_idx[0];
        for (int j = 1; j < 8; ++j)
            if (s_val[j] > b || (s_val[j] == b && s_idx[j] < i)) { b = s_val[j]; i = s_idx[j]; }
        s_max = b;
        ch_max[(size_t)blockIdx.x * gridDim.y + blockIdx.y] = b;
        ch_idx[(size_t)blockIdx.x * gridDim.y + blockIdx.y] = i;
    }
    __syncthreads();
    const double m = (double)s_max;
    double sum = 0.0;
    for (int v = v0 + threadIdx.x; v < v1; v += 256) sum += exp((double)lr[v] - m);
    sum = warp_sum_d(sum);
    if (lane == 0) s_sum[w] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int j = 0; j < 8; ++j) t += s_sum[j];
        ch_sum[(size_t)blockIdx.x * gridDim.y + blockIdx.y] = t;
    }
}

// One block per sequence.  A warp merges the chunk statistics of one active row at a time (lanes
// over chunks, then a fixed shuffle tree, so identical rows give identical bits); then
// rank(i) = #{j : s_j < s_i or (s_j == s_i and pos_j < pos_i)}; positions are ascending inside a
// sequence, so "pos_j < pos_i" is "j < i".
__global__ void __launch_bounds__(1024) select_kernel(const float* __restrict__ ch_max, const int32_t* __restrict__ ch_idx,
                              const double* __restrict__ ch_sum, int n_chunks, int32_t* __restrict__ row_token,
                              double* __restrict__ row_sumexp, const int32_t* __restrict__ act_pos,
                              const int32_t* __restrict__ act_off, int n_single, int k, int32_t* __restrict__ ids,
                              int S, int32_t* __restrict__ n_sel, int32_t* __restrict__ sel_pos,
                              int32_t* __restrict__ sel_token, float* __restrict__ sel_conf,
                              float* __restrict__ row_conf, uint8_t* __restrict__ decoded,
                              int32_t* __restrict__ dec_step, const int32_t* __restrict__ step_of_seq) {
    pdl_launch_dependents();
    pdl_wait();
    const int b = blockIdx.x;
    const int a0 = act_off ? act_off[b] : 0;
    const int n = act_off ? act_off[b + 1] - a0 : n_single;
    const int kk = min(k, n);
    if (threadIdx.x == 0) n_sel[b] = kk;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    for (int i = w; i < n; i += nw) {
        const size_t base = (size_t)(a0 + i) * n_chunks;
        // row maximum and its lowest index: chunks ascend in index, so on equal maxima the lower chunk wins
        float m = -INFINITY;
        int tok = 0x7fffffff;
        for (int c = lane; c < n_chunks; c += 32) {
            const float cm = ch_max[base + c];
            const int ci = ch_idx[base + c];
            if (cm > m || (cm == m && ci < tok)) { m = cm; tok = ci; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float om = __shfl_xor_sync(0xffffffffu, m, o);
            const int oi = __shfl_xor_sync(0xffffffffu, tok, o);
            if (om > m || (om == m && oi < tok)) { m = om; tok = oi; }
        }
        double s = 0.0;
        for (int c = lane; c < n_chunks; c += 32) s += ch_sum[base + c] * exp((double)ch_max[base + c] - (double)m);
        s = warp_sum_d(s);
        if (lane == 0) {
            row_token[a0 + i] = tok;
            row_sumexp[a0 + i] = s;
            if (row_conf) row_conf[a0 + i] = (float)(1.0 / s);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const double si = row_sumexp[a0 + i];
        int rank = 0;
        for (int j = 0; j < n; ++j) {
            const double sj = row_sumexp[a0 + j];
            rank += (sj < si || (sj == si && j < i)) ? 1 : 0;
        }
        if (rank < kk) {
            const int pos = act_pos[a0 + i], tok = row_token[a0 + i];
            sel_pos[b * k + rank] = pos;
            sel_token[b * k + rank] = tok;
            sel_conf[b * k + rank] = (float)(1.0 / si);
            if (ids) ids[(size_t)b * S + pos] = tok;
            if (decoded) {                                  // device-resident planner state
                decoded[(size_t)b * S + pos] = 1;
                dec_step[(size_t)b * S + pos] = step_of_seq[b];
            }
        }
    }
}

__device__ int32_t g_op_status;

}  // namespace

thread_local long long wd_launch_counter = 0;

// ---------------------------------------------------------------- launchers

#define WD_DISPATCH(dtype, ...)                                   \
    do {                                                          \
        if ((dtype) == WD_F32) { using T = float; __VA_ARGS__; }  \
        else { using T = __nv_bfloat16; __VA_ARGS__; }            \
    } while (0)

void wd_launch_embed(int dtype, const void* embed, const int32_t* ids, const int32_t* row_seq,
                     const int32_t* row_pos, float* x, float2* rope_tab, int n_rows, int d, int S, int vocab, int dh,
                     float theta, int32_t* status, cudaStream_t st) {
    if (n_rows <= 0) return;
    const double l2 = log2((double)theta);
    WD_DISPATCH(dtype, launch_pdl(embed_kernel<T>, dim3(n_rows), dim3(256), 0, st, (const T*)embed, ids, row_seq,
                                  row_pos, x, rope_tab, d, S, vocab, dh, l2, status));
}

void wd_launch_embed_fused(const void* embed, const int32_t* ids, const int32_t* row_seq, const int32_t* row_pos,
                           float* x, void* xg, const float* gain, float* sumsq, float2* rope_tab, int n_rows, int d, int S,
                           int vocab, int dh, float theta, int32_t* status, cudaStream_t st) {
    if (n_rows <= 0) return;
    launch_pdl(embed_fused_kernel, dim3(n_rows), dim3(256), 0, st, (const __nv_bfloat16*)embed, ids, row_seq, row_pos, x,
               (__nv_bfloat16*)xg, gain, sumsq, rope_tab, n_rows, d, S, vocab, dh, log2((double)theta), status);
}

void wd_launch_rmsnorm(int dtype, float* x, const float* part, int n_split, size_t split_stride,
                       const float* gain, float eps, void* xn, const int32_t* row_idx, int n_rows,
                       int d, cudaStream_t st, uint8_t* xq, float* sx, const WdFp4Operand* x4p) {
    if (n_rows <= 0) return;
    // one float4 per thread where the row allows it: the kernel is a chain of dependent L2 round
    // trips, so short per-thread work matters more than occupancy
    const int nv = d >> 2;
    if (x4p) {
        const WdFp4Operand x4 = *x4p;
        if (n_rows >= 512 && nv >= 256 && nv <= 4096)
            launch_pdl(rmsnorm_fp4_kernel<4>, dim3(n_rows), dim3(((nv + 3) / 4 + 31) / 32 * 32), 0, st, x, part, n_split,
                       split_stride, gain, eps, row_idx, d, x4);
        else if (nv <= 1024)
            launch_pdl(rmsnorm_fp4_kernel<1>, dim3(n_rows), dim3((nv + 31) / 32 * 32), 0, st, x, part, n_split, split_stride,
                       gain, eps, row_idx, d, x4);
        else if (nv <= 2048)
            launch_pdl(rmsnorm_fp4_kernel<2>, dim3(n_rows), dim3(1024), 0, st, x, part, n_split, split_stride, gain, eps,
                       row_idx, d, x4);
        else
            launch_pdl(rmsnorm_fp4_kernel<8>, dim3(n_rows), dim3(1024), 0, st, x, part, n_split, split_stride, gain, eps,
                       row_idx, d, x4);
        return;
    }
    static const int rms_rows = getenv("WD_RMS_ROWS") ? atoi(getenv("WD_RMS_ROWS")) : 1;
    static const int rms_rows_max = getenv("WD_RMS_ROWS_MAX") ? atoi(getenv("WD_RMS_ROWS_MAX")) : 128;
    if (rms_rows && !xq && n_rows <= rms_rows_max && nv >= 512 && nv <= 1024 && nv % 2 == 0) {
        WD_DISPATCH(dtype, launch_pdl(rmsnorm_rows_kernel<T>, dim3(n_rows), dim3((nv / 2 + 31) / 32 * 32), 0, st, x, part, n_split,
                                      split_stride, gain, eps, (T*)xn, row_idx, d));
        return;
    }
    if (n_rows >= 512 && nv >= 256 && nv <= 4096) {
        // many rows: bandwidth matters, so more (smaller) blocks per SM with four float4 in flight per thread
        const int threads = ((nv + 3) / 4 + 31) / 32 * 32;
        WD_DISPATCH(dtype, launch_pdl(rmsnorm_kernel<T, 4>, dim3(n_rows), dim3(threads), 0, st, x, part, n_split,
                                      split_stride, gain, eps, (T*)xn, row_idx, d, xq, sx));
    } else if (nv <= 1024) {
        const int threads = (nv + 31) / 32 * 32;
        WD_DISPATCH(dtype, launch_pdl(rmsnorm_kernel<T, 1>, dim3(n_rows), dim3(threads), 0, st, x, part, n_split,
                                      split_stride, gain, eps, (T*)xn, row_idx, d, xq, sx));
    } else if (nv <= 2048) {
        WD_DISPATCH(dtype, launch_pdl(rmsnorm_kernel<T, 2>, dim3(n_rows), dim3(1024), 0, st, x, part, n_split,
                                      split_stride, gain, eps, (T*)xn, row_idx, d, xq, sx));
    } else {
        WD_DISPATCH(dtype, launch_pdl(rmsnorm_kernel<T, 8>, dim3(n_rows), dim3(1024), 0, st, x, part, n_split,
                                      split_stride, gain, eps, (T*)xn, row_idx, d, xq, sx));
    }
}

void wd_launch_gemm_plain(int dtype, const void* x, const void* w, float* y, int rows, int n, int k,
                          int ldy, cudaStream_t st) {
    if (rows <= 0 || n <= 0) return;
    dim3 grid(wd_ceil_div(n, 64), wd_ceil_div(rows, 32));
    WD_DISPATCH(dtype, launch_pdl(gemm_plain_kernel<T>, grid, dim3(256), 0, st, (const T*)x, (const T*)w, y, rows, n,
                                  k, ldy));
}

void wd_launch_rope_scatter(int dtype, const float* part, int n_split, size_t split_stride,
                            const int32_t* row_seq, const int32_t* row_pos, const float2* rope_tab, void* q,
                            void* kcache, void* vcache, int n_rows, int Hq, int Hkv, int dh, int S, int Sp,
                            int batch, int32_t* status, cudaStream_t st) {
    if (n_rows <= 0) return;
    const int half = dh >> 1;
    const int qk_groups = (half & 3) == 0 ? wd_ceil_div(Hq + Hkv, std::max(1, 256 / (half >> 2))) : wd_ceil_div(Hq + Hkv, 4);
    const int n_qk = n_rows * qk_groups;
    const int n_v = Hkv * wd_ceil_div(dh, 32) * wd_ceil_div(n_rows, 32);
    const int n_qk_blocks = std::min(n_qk, 148 * 8);
    WD_DISPATCH(dtype, launch_pdl(rope_scatter_kernel<T>, dim3(n_qk_blocks + n_v), dim3(256), 0, st, part, n_split,
                                  split_stride, row_seq, row_pos, rope_tab, (T*)q, (T*)kcache, (T*)vcache, n_rows, Hq,
                                  Hkv, dh, S, Sp, n_qk, qk_groups, n_qk_blocks, batch, status));
}

void wd_launch_attention_plain(int dtype, const void* q, const void* kcache, const void* vcache,
                               const int32_t* row_seq, const int32_t* vis_idx, const int32_t* vis_off,
                               void* out, float* tap, int n_rows, int max_vis, int Hq, int Hkv, int dh,
                               int S, int Sp, int batch, int32_t* status, cudaStream_t st) {
    if (n_rows <= 0) return;
    const size_t smem = (size_t)(max_vis + dh) * sizeof(float);
    dim3 grid(n_rows, Hq);
    if (dtype == WD_F32) {
        if (smem > 48 * 1024)
            cudaFuncSetAttribute(attention_plain_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        launch_pdl(attention_plain_kernel<float>, grid, dim3(128), smem, st, (const float*)q, (const float*)kcache,
                   (const float*)vcache, row_seq, vis_idx, vis_off, (float*)out, tap, max_vis, Hq, Hkv, dh, S, Sp, batch, status);
    } else {
        using T = __nv_bfloat16;
        if (smem > 48 * 1024)
            cudaFuncSetAttribute(attention_plain_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        launch_pdl(attention_plain_kernel<T>, grid, dim3(128), smem, st, (const T*)q, (const T*)kcache,
                   (const T*)vcache, row_seq, vis_idx, vis_off, (T*)out, tap, max_vis, Hq, Hkv, dh, S, Sp, batch, status);
    }
}

void wd_launch_swiglu(int dtype, const float* part, int n_split, size_t split_stride, void* h,
                      int n_rows, int F, cudaStream_t st) {
    if (n_rows <= 0) return;
    const size_t total = (size_t)n_rows * (F >> 2);
    static const int sw_rows = getenv("WD_SWIGLU_ROWS") ? atoi(getenv("WD_SWIGLU_ROWS")) : 1;
    // up to about a hundred rows (measured: -1.4 % on a 68-row step, +1 % at 352 rows, where two positions per thread pay)
    static const int sw_rows_max = getenv("WD_SWIGLU_ROWS_MAX") ? atoi(getenv("WD_SWIGLU_ROWS_MAX")) : 148 * 8 * 256;
    if (sw_rows && total <= (size_t)sw_rows_max) {
        WD_DISPATCH(dtype, launch_pdl(swiglu_rows_kernel<T>, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, st, part, n_split,
                                      split_stride, (T*)h, n_rows, F));
        return;
    }
    const int blocks = (int)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
    WD_DISPATCH(dtype, launch_pdl(swiglu_kernel<T>, dim3(blocks), dim3(256), 0, st, part, n_split, split_stride,
                                  (T*)h, n_rows, F));
}

static wd_status launch_swiglu_quant(const float* part, int n_split, size_t split_stride, uint8_t* hq, float* sh,
                                     const WdFp4Operand* h4p, int n_rows, int F, cudaStream_t st) {
    if (n_rows <= 0) return WD_OK;
    const int f4 = F >> 2;
    if (F % 4 || f4 > 8 * 1024 || (h4p && F % 64)) return WD_ERR_BAD_PARAM;
    const WdFp4Operand h4 = h4p ? *h4p : WdFp4Operand();
    ++wd_launch_counter;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(4 * n_rows);
    lc.blockDim = dim3(256);
    lc.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 4;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = wd_pdl_enabled ? 2 : 1;
    const int per_thread = ((f4 + 3) / 4 + 255) / 256;          // float4 per thread
    cudaError_t e;
    {
        static const bool carve = !(getenv("WD_NO_CARVEOUT") && atoi(getenv("WD_NO_CARVEOUT")));
        if (carve) {
            prefer_max_shared((const void*)swiglu_fp4_kernel<3>); prefer_max_shared((const void*)swiglu_fp4_kernel<5>);
            prefer_max_shared((const void*)swiglu_fp4_kernel<8>); prefer_max_shared((const void*)swiglu_fp8_kernel<3>);
            prefer_max_shared((const void*)swiglu_fp8_kernel<5>); prefer_max_shared((const void*)swiglu_fp8_kernel<8>);
        }
    }
    if (h4p) {
        if (per_thread <= 3) e = cudaLaunchKernelEx(&lc, swiglu_fp4_kernel<3>, part, n_split, split_stride, F, h4);
        else if (per_thread <= 5) e = cudaLaunchKernelEx(&lc, swiglu_fp4_kernel<5>, part, n_split, split_stride, F, h4);
        else e = cudaLaunchKernelEx(&lc, swiglu_fp4_kernel<8>, part, n_split, split_stride, F, h4);
    } else {
        if (per_thread <= 3) e = cudaLaunchKernelEx(&lc, swiglu_fp8_kernel<3>, part, n_split, split_stride, hq, sh, F);
        else if (per_thread <= 5) e = cudaLaunchKernelEx(&lc, swiglu_fp8_kernel<5>, part, n_split, split_stride, hq, sh, F);
        else e = cudaLaunchKernelEx(&lc, swiglu_fp8_kernel<8>, part, n_split, split_stride, hq, sh, F);
    }
    if (e != cudaSuccess) { wd_note_cuda_error(e, __FILE__, __LINE__); return WD_ERR_CUDA; }
    return WD_OK;
}

wd_status wd_launch_swiglu_fp8(const float* part, int n_split, size_t split_stride, uint8_t* hq, float* sh, int n_rows,
                               int F, cudaStream_t st) {
    return launch_swiglu_quant(part, n_split, split_stride, hq, sh, nullptr, n_rows, F, st);
}

wd_status wd_launch_swiglu_fp4(const float* part, int n_split, size_t split_stride, const WdFp4Operand* h4, int n_rows,
                               int F, cudaStream_t st) {
    if (!h4) return WD_ERR_NULL;
    return launch_swiglu_quant(part, n_split, split_stride, nullptr, nullptr, h4, n_rows, F, st);
}

void wd_launch_quantize_rows(int dtype, const void* w, int n_rows, int K, uint8_t* q, float* s, cudaStream_t st) {
    if (n_rows <= 0) return;
    WD_DISPATCH(dtype, (quantize_rows_kernel<T><<<n_rows, 256, 0, st>>>((const T*)w, K, q, s)));
    ++wd_launch_counter;
}

void wd_launch_residual_add(float* x, const float* part, int n_split, size_t split_stride,
                            float* tap, int n_rows, int d, cudaStream_t st) {
    if (n_rows <= 0) return;
    const size_t total = (size_t)n_rows * d, n4 = total >> 2;
    const int blocks = (int)((n4 + 255) / 256 < 148 * 8 ? (n4 + 255) / 256 : 148 * 8);
    launch_pdl(residual_add_kernel, dim3(blocks), dim3(256), 0, st, x, part, n_split, split_stride, tap, total);
}

int wd_unmask_chunks(int V) {
    int n = (V + 4095) / 4096;            // about 4096 logits per block
    if (n < 1) n = 1;
    if (n > WD_UNMASK_MAX_CHUNKS) n = WD_UNMASK_MAX_CHUNKS;
    return n;
}

void wd_launch_rowstats(const float* logits, int n, int V, float* ch_max, int32_t* ch_idx, double* ch_sum,
                        cudaStream_t st) {
    if (n <= 0) return;
    const int nch = wd_unmask_chunks(V);
    const int chunk = (V + nch - 1) / nch;
    launch_pdl(rowstats_kernel, dim3(n, nch), dim3(256), 0, st, logits, V, chunk, ch_max, ch_idx, ch_sum);
}

void wd_launch_select(const float* ch_max, const int32_t* ch_idx, const double* ch_sum, int n_chunks,
                      int32_t* row_token, double* row_sumexp, const int32_t* act_pos, const int32_t* act_off,
                      int n_single, int batch, int k, int32_t* ids, int S, int32_t* n_sel, int32_t* sel_pos,
                      int32_t* sel_token, float* sel_conf, float* row_conf, uint8_t* decoded, int32_t* dec_step,
                      const int32_t* step_of_seq, cudaStream_t st) {
    if (batch <= 0) return;
    // one warp per active row where the block allows it (a row is two dependent passes over its chunk statistics)
    launch_pdl(select_kernel, dim3(batch), dim3(1024), 0, st, ch_max, ch_idx, ch_sum, n_chunks, row_token, row_sumexp,
               act_pos, act_off, n_single, k, ids, S, n_sel, sel_pos, sel_token, sel_conf, row_conf, decoded, dec_step,
               step_of_seq);
}

void wd_launch_plan(const WdPlanLaunch& h, cudaStream_t st) {
    PlanArgs a;
    memset(&a, 0, sizeof(a));
    for (int b = 0; b < h.batch; ++b) {
        a.refresh[b] = h.refresh[b]; a.done[b] = h.done[b]; a.n_wex[b] = h.n_wex[b]; a.n_vis[b] = h.n_vis[b];
        a.t[b] = h.t[b];
        a.window_refresh[b] = h.window_refresh[b]; a.prev_phase_start[b] = h.prev_phase_start[b];
    }
    for (int b = 0; b <= h.batch; ++b) {
        a.row_off[b] = h.row_off[b]; a.act_off[b] = h.act_off[b]; a.vis_off[b] = h.vis_off[b]; a.qt_off[b] = h.qt_off[b];
    }
    a.S = h.S; a.A = h.A; a.T = h.T; a.batch = h.batch;
    a.decoded = h.decoded; a.dec_step = h.dec_step; a.wex = h.wex;
    a.row_seq = h.row_seq; a.row_pos = h.row_pos; a.act_row = h.act_row; a.act_pos = h.act_pos;
    a.act_off_dev = h.act_off_dev; a.vis_off_dev = h.vis_off_dev; a.vis_idx = h.vis_idx;
    a.qt_seq = h.qt_seq; a.qt_row0 = h.qt_row0; a.qt_n = h.qt_n; a.nvis_dev = h.nvis_dev; a.tseq_dev = h.tseq_dev;
    a.status = h.status;
    launch_pdl(plan_kernel, dim3(h.batch), dim3(256), 0, st, a);
}

// A bounded wait that is never satisfied: the barrier expects one arrival and nobody arrives.
__global__ void wait_expire_kernel(int32_t* status) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        wdk::mbar_init(wdk::smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!wdk::mbar_wait(wdk::smem_u32(&bar), 0, &abort_flag)) atomicCAS(status, 0, WD_ERR_DEVICE_TIMEOUT);
    }
}

wd_status wd_launch_wait_expire(cudaStream_t st) {
    int32_t* status = wd_op_status_ptr();
    if (!status) return WD_ERR_CUDA;
    wait_expire_kernel<<<1, 32, 0, st>>>(status);
    ++wd_launch_counter;
    return cudaGetLastError() == cudaSuccess ? WD_OK : WD_ERR_CUDA;
}

// In host code the symbol's name is a handle, not a device address: looked up once per device
// (with that device current) and remembered.
int32_t* wd_op_status_ptr() {
    static int32_t* cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!cached[dev]) {
        int32_t* p = nullptr;
        if (cudaGetSymbolAddress((void**)&p, g_op_status) != cudaSuccess) return nullptr;
        cached[dev] = p;
    }
    return cached[dev];
}

// Query-tile lists of ONE sequence whose n_rows rows all see positions [0, n_vis): tile t covers
// rows [128 t, 128 t + n).  Layout of `lists`: seq[n_tiles] | row0[n_tiles] | n[n_tiles] | n_vis[1].
__global__ void fill_qtiles_kernel(int32_t* lists, int n_rows, int n_vis) {
    const int n_tiles = (n_rows + 127) / 128;
    for (int t = threadIdx.x; t < n_tiles; t += blockDim.x) {
        lists[t] = 0;
        lists[n_tiles + t] = 128 * t;
        lists[2 * n_tiles + t] = min(128, n_rows - 128 * t);
    }
    if (threadIdx.x == 0) lists[3 * n_tiles] = n_vis;
}

void wd_launch_fill_qtiles(int32_t* lists, int n_rows, int n_vis, cudaStream_t st) {
    fill_qtiles_kernel<<<1, 128, 0, st>>>(lists, n_rows, n_vis);
    ++wd_launch_counter;
}
