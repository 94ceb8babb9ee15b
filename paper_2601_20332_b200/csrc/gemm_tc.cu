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
constexpr int kThreads = 192;         // TMA warp, MMA warp, 4 epilogue warps
constexpr int kThreadsWide = 320;     // ... 8 epilogue warps when a CTA carries two weight halves
constexpr int kThreadsPair = 320;     // two-CTA kernel: 8 epilogue warps, two per quarter of the accumulator rows

struct TcParams {
    int rows, bn, kb_total, tok_tiles, n_units, n_stages, buf_cols, n_slices, aligned;
    int trace_slot;                  // -DWD_GEMM_TRACE builds: which trace table this launch stamps
    int wide;                       // 1: a tile is 256 weight rows = two MMA halves sharing each activation box
    int tile_rows;                  // 128, or 256 when wide
    // > 1: the grid is tok_split groups of CTAs, group t working on token tile t only; the K-block
    // line then holds the weight tiles once (n_units, W count weight tiles), and the groups walk it
    // in step, so that a weight block fetched for one token tile is still in L2 for the others
    int tok_split;
    // pair kernel only, 1: a unit is [256 weight rows x 2*bn tokens] = two accumulators fed from the same
    // weight stage (each CTA holds bn token rows per K block: half of either accumulator's tokens)
    // 2: the two accumulators are the gate tile and the up tile of the same 256 FFN columns against one
    // token tile (both weight blocks in every stage); the epilogue writes h = silu(gate) * up as bf16
    int dual;
    // pair kernel, whole-tile schedule: > 0 = units are ordered (token group of tok_grp tiles, weight tile,
    // token tile in the group) and dealt to the pairs round-robin, so that the pairs running at the same
    // time share a few weight tiles and one group of token tiles (working set well inside the L2)
    int tok_grp;
    __nv_bfloat16* swiglu_h;        // dual == 2: [rows, ncol] with ncol = FFN width
    // FP8 operands: K blocks of 128 elements, outputs scaled by sw[segment][n] * sx[token]
    int fp8;
    const float* sw[3];
    const float* sx;
    int nseg, ncol;
    int seg_tile0[4];               // first tile index of each weight matrix (+ end)
    int seg_n[3];
    int seg_col[3];
    long long W;                    // total K blocks of the launch = n_units * kb_total
    float* y;
    size_t split_stride;
    int32_t* status;
    uint32_t idesc;
    WdTcFuse f;
};

// A unit is one [128 weight rows x BN tokens] output tile; unit u = tile * tok_tiles + token tile.
struct UnitInfo { int seg, n0, tok0; };
__device__ __forceinline__ UnitInfo decode_unit(const TcParams& p, int unit, int tok_group = 0) {
    UnitInfo u;
    int tile, tokt;
    if (p.tok_grp > 0) {
        const int per = p.seg_tile0[p.nseg] * p.tok_grp;            // units of a full token group
        const int n_grp = (p.tok_tiles + p.tok_grp - 1) / p.tok_grp;
        int grp = unit / per;
        if (grp >= n_grp) grp = n_grp - 1;                          // the last group may be smaller
        const int rem = unit - grp * per;
        const int gsz = min(p.tok_grp, p.tok_tiles - grp * p.tok_grp);
        tile = rem / gsz;
        tokt = grp * p.tok_grp + rem % gsz;
    } else {
        tile = p.tok_split > 1 ? unit : unit / p.tok_tiles;
        tokt = p.tok_split > 1 ? tok_group : unit - tile * p.tok_tiles;
    }
    u.tok0 = tokt * p.bn * (p.dual == 1 ? 2 : 1);
    u.seg = 0;
    if (p.nseg > 1 && tile >= p.seg_tile0[1]) u.seg = 1;
    if (p.nseg > 2 && tile >= p.seg_tile0[2]) u.seg = 2;
    u.n0 = (tile - p.seg_tile0[u.seg]) * p.tile_rows;
    return u;
}

// The pieces of one CTA's share [g_begin, g_end) of the K-block line, in the order they are
// processed: first the partial tile at the front of the share, then the partial tile at its
// back, then the whole tiles in between.  Partial tiles are the ones other CTAs also work on;
// doing them first lets those tiles complete (and their fused epilogue run) in the middle of the
// kernel instead of all at its end.
struct Sched {
    long long g_begin, g_end;
    int kb_total, head_len, tail_len, n_full, n_pieces;
    long long full_begin;
    long long stride = 0;           // > 0: whole units first, first + stride, ... (K blocks on the line)
    // whole units c, c + G, c + 2G, ... of n_units
    __device__ void init_strided(long long c, long long G, int n_units, int kb) {
        kb_total = kb;
        head_len = tail_len = 0;
        n_full = n_pieces = c < n_units ? (int)((n_units - c + G - 1) / G) : 0;
        g_begin = full_begin = c * kb;
        stride = G * kb;
        g_end = g_begin;
    }
    __device__ void init(long long gb, long long ge, int kb) {
        g_begin = gb; g_end = ge; kb_total = kb;
        const long long total = ge - gb;
        const int off = (int)(gb % kb);
        head_len = off ? (int)((long long)(kb - off) < total ? (kb - off) : total) : 0;
        const long long rest_begin = gb + head_len;
        const long long rest = ge - rest_begin;
        n_full = (int)(rest / kb);
        tail_len = (int)(rest - (long long)n_full * kb);
        full_begin = rest_begin;
        n_pieces = (head_len ? 1 : 0) + (tail_len ? 1 : 0) + n_full;
    }
    // piece i -> first K block on the line and length
    __device__ void piece(int i, long long& g, int& len) const {
        if (stride > 0) { g = full_begin + (long long)i * stride; len = kb_total; return; }
        if (head_len) { if (i == 0) { g = g_begin; len = head_len; return; } --i; }
        if (tail_len) { if (i == 0) { g = g_end - tail_len; len = tail_len; return; } --i; }
        g = full_begin + (long long)i * kb_total;
        len = kb_total;
    }
};

// number of CTAs whose piece of the line touches unit u
__device__ __forceinline__ int n_contrib(const TcParams& p, long long G, int unit) {
    if (p.aligned) return 1;
    const long long first = ((long long)unit * p.kb_total + 1) * G - 1;
    const long long last = ((long long)(unit + 1) * p.kb_total) * G - 1;
    return (int)(last / p.W - first / p.W) + 1;
}

__device__ __forceinline__ float4 ldcg4(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ void add4(float4& a, const float4 b) { a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; }
__device__ __forceinline__ void store_bf16x4(__nv_bfloat16* p, float a, float b, float c, float d) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    uint2 u;
    u.x = *reinterpret_cast<uint32_t*>(&lo);
    u.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(p) = u;
}
__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Adds slices [0, nc) of UN rows into acc, MS slices at a time: all loads of a group are issued
// before the first add, so their L2 round trips overlap; the adds keep slice order.
template <int UN, int MS>
__device__ __forceinline__ void add_slices(float4 (&acc)[UN], const float* const (&base)[UN], const bool (&valid)[UN],
                                           int nc, size_t stride) {
    for (int s0 = 0; s0 < nc; s0 += MS) {
        float4 tmp[UN][MS];
#pragma unroll
        for (int i = 0; i < UN; ++i)
#pragma unroll
            for (int k = 0; k < MS; ++k)
                tmp[i][k] = (valid[i] && s0 + k < nc) ? ldcg4(base[i] + (size_t)(s0 + k) * stride) : make_float4(0, 0, 0, 0);
#pragma unroll
        for (int i = 0; i < UN; ++i)
#pragma unroll
            for (int k = 0; k < MS; ++k) add4(acc[i], tmp[i][k]);
    }
}

// this lane's share of row r's sum of squares (the previous GEMM's per-block partial sums)
__device__ __forceinline__ float sumsq_lane(const TcParams& p, int r, int lane) {
    float ss = 0.f;
    for (int i = lane; i < p.f.n_prev_tiles; i += 32) ss += __ldcg(p.f.sumsq_in + (size_t)i * p.f.rows_total + r);
    return ss;
}

// Run by the 128 epilogue threads of the CTA that completed `unit` (e = 0..127).  Every
// partial slice of the tile is in y; sums are taken in slice order, so the result does not
// depend on which CTA arrived last.  A warp handles one token at a time, its lanes the tile's
// 128 columns as float4; the loads of several tokens and slices are issued together so that
// their L2 round trips overlap, and only then reduced.
__device__ void finalize_unit(const TcParams& p, long long G, int unit, int e) {
    const UnitInfo u = decode_unit(p, unit);
    const int nt = min(p.bn, p.rows - u.tok0);
    const int lane = e & 31, wq = e >> 5;
    if (p.f.mode == WD_FUSE_RESID) {
        // x += tile; xg = bf16(x * gain); per-row sum of squares over this tile's 128 columns
        constexpr int UN = 3;
        const int nc = n_contrib(p, G, unit);
        const int col = u.n0 + 4 * lane, d = p.ncol;
        const float4 g = p.f.gain_next ? *reinterpret_cast<const float4*>(p.f.gain_next + col) : make_float4(0, 0, 0, 0);
        for (int t0 = wq; t0 < nt; t0 += 4 * UN) {
            float4 v[UN];
            const float* base[UN];
            bool valid[UN];
#pragma unroll
            for (int i = 0; i < UN; ++i) {
                const int t = t0 + 4 * i;
                valid[i] = t < nt;
                const size_t o = (size_t)(u.tok0 + (valid[i] ? t : 0)) * d + col;
                base[i] = p.y + o;
                v[i] = valid[i] ? *reinterpret_cast<const float4*>(p.f.x + o) : make_float4(0, 0, 0, 0);
            }
            add_slices<UN, 3>(v, base, valid, nc, p.split_stride);
#pragma unroll
            for (int i = 0; i < UN; ++i) {
                const int t = t0 + 4 * i;
                if (valid[i]) {
                    const size_t o = (size_t)(u.tok0 + t) * d + col;
                    *reinterpret_cast<float4*>(p.f.x + o) = v[i];
                    if (p.f.gain_next) store_bf16x4(p.f.xg + o, v[i].x * g.x, v[i].y * g.y, v[i].z * g.z, v[i].w * g.w);
                    if (p.f.tap) *reinterpret_cast<float4*>(p.f.tap + o) = v[i];
                    const float ss = warp_sum_f(v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w);
                    if (lane == 0) p.f.sumsq_out[(size_t)(u.n0 >> 7) * p.f.rows_total + u.tok0 + t] = ss;
                }
            }
        }
    } else if (p.f.mode == WD_FUSE_QKV) {
        // one tile = one head (head_dim 128): scale by 1/rms, rotate q and k, write q / K / V^T.
        // Half a warp per token: lane quad q4 holds columns 4*q4.. and their rotation partners +64.
        constexpr int UN = 2;
        const int nc = n_contrib(p, G, unit);
        const int head = (p.seg_col[u.seg] + u.n0) >> 7;            // index among q | k | v heads
        const int q4 = lane & 15, tsel = lane >> 4;
        const size_t col = (size_t)p.seg_col[u.seg] + u.n0 + 4 * q4;
        for (int t0 = 2 * wq; t0 < nt; t0 += 8 * UN) {
            float4 a[UN], b[UN];
            const float* base_a[UN];
            const float* base_b[UN];
            bool valid[UN];
            float ss0[UN], ss1[UN];
#pragma unroll
            for (int i = 0; i < UN; ++i) {
                const int tb = t0 + 8 * i;                          // this warp's token pair: tb, tb + 1
                const int t = tb + tsel;
                valid[i] = t < nt;
                a[i] = b[i] = make_float4(0, 0, 0, 0);
                base_a[i] = p.y + (size_t)(u.tok0 + (valid[i] ? t : 0)) * p.ncol + col;
                base_b[i] = base_a[i] + 64;
                // every lane loads its share of both rows' sums of squares (full-warp reductions below)
                ss0[i] = tb < nt ? sumsq_lane(p, u.tok0 + tb, lane) : 0.f;
                ss1[i] = tb + 1 < nt ? sumsq_lane(p, u.tok0 + tb + 1, lane) : 0.f;
            }
            add_slices<UN, 3>(a, base_a, valid, nc, p.split_stride);
            add_slices<UN, 3>(b, base_b, valid, nc, p.split_stride);
#pragma unroll
            for (int i = 0; i < UN; ++i) {
                const float s0 = warp_sum_f(ss0[i]), s1 = warp_sum_f(ss1[i]);
                const int t = t0 + 8 * i + tsel;
                if (!valid[i]) continue;
                const float inv = rsqrtf((tsel ? s1 : s0) * p.f.inv_d + p.f.eps);
                const int r = u.tok0 + t;
                const float av[4] = {a[i].x * inv, a[i].y * inv, a[i].z * inv, a[i].w * inv};
                const float bv[4] = {b[i].x * inv, b[i].y * inv, b[i].z * inv, b[i].w * inv};
                const int pos = p.f.row_pos[r], sq = p.f.row_seq[r];
                if (head < p.f.Hq + p.f.Hkv) {
                    const float4 c01 = *reinterpret_cast<const float4*>(p.f.rope_tab + (size_t)r * 64 + 4 * q4);
                    const float4 c23 = *reinterpret_cast<const float4*>(p.f.rope_tab + (size_t)r * 64 + 4 * q4 + 2);
                    const float cs[4] = {c01.x, c01.z, c23.x, c23.z}, sn[4] = {c01.y, c01.w, c23.y, c23.w};
                    float ra[4], rb[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        ra[k] = av[k] * cs[k] - bv[k] * sn[k];
                        rb[k] = bv[k] * cs[k] + av[k] * sn[k];
                    }
                    __nv_bfloat16* dst = head < p.f.Hq
                        ? p.f.q + ((size_t)r * p.f.Hq + head) * 128
                        : p.f.kcache + (((size_t)sq * p.f.Hkv + (head - p.f.Hq)) * p.f.S + pos) * 128;
                    store_bf16x4(dst + 4 * q4, ra[0], ra[1], ra[2], ra[3]);
                    store_bf16x4(dst + 64 + 4 * q4, rb[0], rb[1], rb[2], rb[3]);
                } else {
                    __nv_bfloat16* dst = p.f.vcache + ((size_t)sq * p.f.Hkv + (head - p.f.Hq - p.f.Hkv)) * 128 * p.f.Sp + pos;
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        dst[(size_t)(4 * q4 + k) * p.f.Sp] = __float2bfloat16_rn(av[k]);
                        dst[(size_t)(64 + 4 * q4 + k) * p.f.Sp] = __float2bfloat16_rn(bv[k]);
                    }
                }
            }
        }
    } else if (p.f.mode == WD_FUSE_SWIGLU) {
        // gate tile t and up tile t (same columns of the two matrices): h = silu(g) * u
        constexpr int UN = 3;
        const int tile = unit / p.tok_tiles, tokt = unit - tile * p.tok_tiles;
        const int t_in = tile - p.seg_tile0[u.seg];
        const int ug = (p.seg_tile0[0] + t_in) * p.tok_tiles + tokt, uu = (p.seg_tile0[1] + t_in) * p.tok_tiles + tokt;
        const int ncg = n_contrib(p, G, ug), ncu = n_contrib(p, G, uu);
        const int col = u.n0 + 4 * lane;
        for (int t0 = wq; t0 < nt; t0 += 4 * UN) {
            float4 gv[UN], uv[UN];
            const float* base_g[UN];
            const float* base_u[UN];
            bool valid[UN];
            float ss[UN];
#pragma unroll
            for (int i = 0; i < UN; ++i) {
                const int t = t0 + 4 * i;
                valid[i] = t < nt;
                gv[i] = uv[i] = make_float4(0, 0, 0, 0);
                base_g[i] = p.y + (size_t)(u.tok0 + (valid[i] ? t : 0)) * p.ncol + col;
                base_u[i] = base_g[i] + p.f.F;
                ss[i] = valid[i] ? sumsq_lane(p, u.tok0 + t, lane) : 0.f;
            }
            add_slices<UN, 2>(gv, base_g, valid, ncg, p.split_stride);
            add_slices<UN, 2>(uv, base_u, valid, ncu, p.split_stride);
#pragma unroll
            for (int i = 0; i < UN; ++i) {
                const int t = t0 + 4 * i;
                if (valid[i]) {            // uniform across the warp
                    const float inv = rsqrtf(warp_sum_f(ss[i]) * p.f.inv_d + p.f.eps);
                    const float g0 = gv[i].x * inv, g1 = gv[i].y * inv, g2 = gv[i].z * inv, g3 = gv[i].w * inv;
                    store_bf16x4(p.f.h + (size_t)(u.tok0 + t) * p.f.F + col,
                                 g0 / (1.f + __expf(-g0)) * (uv[i].x * inv), g1 / (1.f + __expf(-g1)) * (uv[i].y * inv),
                                 g2 / (1.f + __expf(-g2)) * (uv[i].z * inv), g3 / (1.f + __expf(-g3)) * (uv[i].w * inv));
                }
            }
        }
    }
}

// Persistent, stream-K: the K blocks of all output tiles form one line of W blocks and CTA c
// takes the contiguous piece [c W / G, (c+1) W / G).  Every CTA therefore streams the same
// number of weight bytes whatever the shape, the TMA ring never drains between tiles, and the
// epilogue of one piece overlaps the MMAs of the next (two accumulators in TMEM).  A tile cut
// by piece boundaries gets one partial sum per CTA that touched it, written to slice
// (CTA - first CTA of the tile); the CTA that finishes the tile zero-fills the unused slices.
// kWide: two weight halves per CTA (many tokens).  kLmStats: the LM-head epilogue that reduces
// the logits to per-row statistics.  Separate instantiations keep the plain weight-streaming
// kernel free of the other variants' code (its issue loops are sensitive to it).
#ifdef WD_GEMM_TRACE
// clock stamps of the last launch per slot (q/k/v, o, gate/up, down, other): [slot][CTA][event]
__device__ unsigned long long g_gemm_trace[8][160][8];
#define G_STAMP(k) do { g_gemm_trace[p.trace_slot & 7][blockIdx.x < 160 ? blockIdx.x : 159][k] = global_ns(); } while (0)
#else
#define G_STAMP(k) do { } while (0)
#endif

template <bool kWide, bool kLmStats, bool kFp8 = false>
__global__ void __launch_bounds__(kWide ? kThreadsWide : kThreads)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w0,
               const __grid_constant__ CUtensorMap map_w1, const __grid_constant__ CUtensorMap map_w2,
               const TcParams p) {
    constexpr int kKE = kFp8 ? 128 : kBK;                 // K elements per block: one 128-byte swizzle row
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment: required by the 128-byte swizzle atoms
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int NS = p.n_stages;
    const int stage_a = p.tile_rows * kBK * 2;            // 16 KB, or 32 KB when wide
    const int stage_bytes = stage_a + p.bn * kBK * 2;
    uint64_t* bars = (uint64_t*)(smem + (size_t)NS * stage_bytes);
    // bars[0..NS) full | [NS..2NS) empty | [2NS, 2NS+1] accumulator full | [2NS+2, 2NS+3] accumulator empty
    uint32_t* tmem_slot = (uint32_t*)(bars + 2 * NS + 4);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
    int* last_flag = (int*)(tmem_slot + 2);
    float* lm_scratch = (float*)(tmem_slot + 4);           // 23 KB for the LM-head statistics

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long G = gridDim.x / (p.tok_split > 1 ? p.tok_split : 1), c = blockIdx.x % G;
    const int tok_group = (int)(blockIdx.x / G);
    long long g_begin, g_end;
    if (p.aligned) {
        g_begin = (c * p.n_units / G) * p.kb_total;
        g_end = ((c + 1) * p.n_units / G) * p.kb_total;
    } else {
        g_begin = c * p.W / G;
        g_end = (c + 1) * p.W / G;
    }
    const int n_total = (int)(g_end - g_begin);
    Sched sch;
    sch.init(g_begin, g_end, p.kb_total);

    pdl_launch_dependents();      // the next kernel may start its own prologue / weight prefetch
    if (threadIdx.x == 0) {
        G_STAMP(0);
        for (int s = 0; s < NS; ++s) {
            mbar_init(smem_u32(&bars[s]), 1);
            mbar_init(smem_u32(&bars[NS + s]), 1);
        }
        mbar_init(smem_u32(&bars[2 * NS]), 1);
        mbar_init(smem_u32(&bars[2 * NS + 1]), 1);
        mbar_init(smem_u32(&bars[2 * NS + 2]), kWide ? 256 : 128);
        mbar_init(smem_u32(&bars[2 * NS + 3]), kWide ? 256 : 128);
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
            // walks the K blocks of this CTA's pieces in schedule order without per-block divisions
            struct Walk {
                int piece, left, kb, n0, tok0;
                const CUtensorMap* mw;
            };
            auto enter = [&](Walk& w) {                    // position on the first block of piece w.piece
                long long g;
                int len;
                sch.piece(w.piece, g, len);
                const int unit = (int)(g / p.kb_total);
                w.kb = (int)(g - (long long)unit * p.kb_total);
                w.left = len;
                const UnitInfo u = decode_unit(p, unit, tok_group);
                w.n0 = u.n0;
                w.tok0 = u.tok0;
                w.mw = u.seg == 0 ? &map_w0 : (u.seg == 1 ? &map_w1 : &map_w2);
            };
            auto advance = [&](Walk& w) {
                ++w.kb;
                if (--w.left == 0 && ++w.piece < sch.n_pieces) enter(w);
            };
            Walk w0;
            w0.piece = 0;
            enter(w0);
            // Weights never depend on earlier kernels of the stream: fill the ring with weight
            // boxes first, then wait for the producer of the activations, then add their boxes.
            const int n_pre = n_total < NS ? n_total : NS;
            Walk w = w0;
            for (int i = 0; i < n_pre; ++i, advance(w)) {
                mbar_expect_tx(smem_u32(&bars[i]), (uint32_t)stage_bytes);
                tma_load_2d_hint(smem_u32(smem + (size_t)i * stage_bytes), w.mw, smem_u32(&bars[i]), w.kb * kKE, w.n0,
                                 pol_stream);
                if (kWide)
                    tma_load_2d_hint(smem_u32(smem + (size_t)i * stage_bytes) + kStageA, w.mw, smem_u32(&bars[i]),
                                     w.kb * kKE, w.n0 + kBM, pol_stream);
            }
            G_STAMP(1);
            pdl_wait();
            G_STAMP(2);
            Walk wx = w0;
            for (int i = 0; i < n_pre; ++i, advance(wx))
                tma_load_2d(smem_u32(smem + (size_t)i * stage_bytes) + stage_a, &map_x, smem_u32(&bars[i]), wx.kb * kKE,
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
                tma_load_2d_hint(sa, w.mw, full, w.kb * kKE, w.n0, pol_stream);
                if (kWide) tma_load_2d_hint(sa + kStageA, w.mw, full, w.kb * kKE, w.n0 + kBM, pol_stream);
                tma_load_2d(sa + stage_a, &map_x, full, w.kb * kKE, w.tok0);
                if (++s == NS) { s = 0; ph ^= 1u; }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            // ------------------------------------------------ MMA issuer
            bool ok = true;
            int s = 0;
            uint32_t ph = 0;
            for (int piece = 0; piece < sch.n_pieces && ok; ++piece) {
                long long g;
                int len;
                sch.piece(piece, g, len);
                // normal: two accumulators used alternately; wide: one accumulator pair (both weight halves)
                const int buf = kWide ? 0 : (piece & 1);
                const uint32_t par = kWide ? ((uint32_t)piece & 1u) : ((uint32_t)(piece >> 1) & 1u);
                // the epilogue has drained this accumulator (free at the start)
                if (!(ok = mbar_wait(smem_u32(&bars[2 * NS + 2 + buf]), par ^ 1u, abort_flag))) break;
                tc_fence_after();
                const uint32_t acc = tmem_base + (uint32_t)(buf * p.buf_cols);
                for (int j = 0; j < len; ++j) {
                    if (!(ok = mbar_wait(smem_u32(&bars[s]), ph, abort_flag))) break;
                    tc_fence_after();
                    if (piece == 0 && j == 0) G_STAMP(3);
                    const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
                    const uint64_t adesc = make_sdesc(sa);
                    const uint64_t bdesc = make_sdesc(sa + stage_a);
                    const uint64_t adesc1 = make_sdesc(sa + kStageA);   // second weight half (wide)
#pragma unroll
                    for (int kk = 0; kk < kBK / 16; ++kk) {
                        // 16 bf16 = 32 bytes further along K inside the swizzle row: +2 in 16-byte units
                        if (kFp8)
                            umma_f8(acc, adesc + (uint64_t)(2 * kk), bdesc + (uint64_t)(2 * kk), p.idesc,
                                    (j > 0 || kk > 0) ? 1u : 0u);
                        else
                            umma_bf16(acc, adesc + (uint64_t)(2 * kk), bdesc + (uint64_t)(2 * kk), p.idesc,
                                      (j > 0 || kk > 0) ? 1u : 0u);
                        if (kWide)
                            umma_bf16(acc + (uint32_t)p.buf_cols, adesc1 + (uint64_t)(2 * kk), bdesc + (uint64_t)(2 * kk),
                                      p.idesc, (j > 0 || kk > 0) ? 1u : 0u);
                    }
                    umma_commit(smem_u32(&bars[NS + s]));          // stage free once these MMAs have read it
                    if (++s == NS) { s = 0; ph ^= 1u; }
                }
                if (ok) umma_commit(smem_u32(&bars[2 * NS + buf]));  // this piece's accumulator complete
            }
            G_STAMP(4);
            if (!ok) {
                *abort_flag = 1;
                atomicCAS(p.status, 0, WD_ERR_DEVICE_TIMEOUT);
            }
        }
        __syncwarp();
    } else {
        // ---------------------------------------------------- epilogue (warps 2..5; wide: 2..9)
        const int quarter = warp & 3;                  // TMEM lanes 32*quarter .. +31
        const int half_sel = (warp - 2) >> 2;          // wide: which weight half this warp drains
        const int n_local = half_sel * kBM + quarter * 32 + lane;
        pdl_wait();      // the previous reader of y has finished (already implied by the data flow)
        bool ok = true;
        for (int piece = 0; piece < sch.n_pieces; ++piece) {
            long long g;
            int len;
            sch.piece(piece, g, len);
            const int unit = (int)(g / p.kb_total), kb0 = (int)(g - (long long)unit * p.kb_total);
            const UnitInfo u = decode_unit(p, unit, tok_group);
            const int buf = kWide ? 0 : (piece & 1);
            const uint32_t par = kWide ? ((uint32_t)piece & 1u) : ((uint32_t)(piece >> 1) & 1u);
            const int n = u.n0 + n_local;
            const bool n_ok = n < p.seg_n[u.seg];
            int ord = 0;
            if (!p.aligned) ord = (int)(c - (((long long)unit * p.kb_total + 1) * G - 1) / p.W);
            // FP8: the row scales of this token tile go to shared memory while the MMAs still run
            float* sx_s = lm_scratch + (kLmStats ? 5664 : 0);
            if (kFp8) {
                epi_sync();                                        // the previous piece's readers are done
                for (int i = (int)threadIdx.x - 64; i < ((p.bn + 31) & ~31); i += 128)
                    sx_s[i] = (i < p.bn && u.tok0 + i < p.rows) ? p.sx[u.tok0 + i] : 0.f;
                epi_sync();
            }
            ok = ok && mbar_wait(smem_u32(&bars[2 * NS + buf]), par, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            if (threadIdx.x == 64 && piece == sch.n_pieces - 1) G_STAMP(5);
            float* yb = p.y + p.seg_col[u.seg] + n;
            const float sw_n = (kFp8 && n_ok) ? p.sw[u.seg][n] : 1.f;      // FP8: scale of this weight row
            const uint32_t t_acc = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)((buf + half_sel) * p.buf_cols);
            if constexpr (!kLmStats) {
                for (int cc = 0; cc < p.bn; cc += 16) {
                    if (u.tok0 + cc >= p.rows) break;
                    uint32_t v[16];
                    tmem_ld16(t_acc + (uint32_t)cc, v);
                    if (n_ok) {
                        float* ys = yb + (size_t)ord * p.split_stride;
#pragma unroll
                        for (int t = 0; t < 16; ++t) {
                            const int tok = u.tok0 + cc + t;
                            if (tok < p.rows)
                                ys[(size_t)tok * p.ncol] = kFp8 ? __uint_as_float(v[t]) * sw_n * sx_s[cc + t] : __uint_as_float(v[t]);
                        }
                    }
                }
            } else {
                // LM head: per token maximum / lowest argmax / sum exp over this tile's 128 logits, folded
                // into the CTA's running statistics.  A thread holds one vocabulary entry for 32 tokens;
                // the chunk is transposed through shared memory so that a thread then owns one token and
                // a quarter of the tile's vocabulary entries, and the four quarters are merged per token.
                float* run_m = lm_scratch;                          // [256] running statistics of this CTA
                int* run_i = (int*)(lm_scratch + 256);
                double* run_s = (double*)(lm_scratch + 512);
                float* g_m = lm_scratch + 1024;                     // [4 quarters][32 tokens]
                int* g_i = (int*)(lm_scratch + 1152);
                double* g_s = (double*)(lm_scratch + 1280);
                float* tr = lm_scratch + 1536;                      // [32 tokens][129]: padded against bank conflicts
                const int e = (int)threadIdx.x - 64, tt = e & 31, gq = e >> 5;
                for (int cc = 0; cc < p.bn; cc += 32) {
                    if (u.tok0 + cc >= p.rows) break;
                    uint32_t v[32];
                    tmem_ld32(t_acc + (uint32_t)cc, v);
                    if (kFp8) {
#pragma unroll
                        for (int t = 0; t < 32; ++t)
                            v[t] = __float_as_uint(__uint_as_float(v[t]) * sw_n * sx_s[cc + t]);
                    }
                    if (n_ok && p.f.write_logits) {
#pragma unroll
                        for (int t = 0; t < 32; ++t)
                            if (u.tok0 + cc + t < p.rows) yb[(size_t)(u.tok0 + cc + t) * p.ncol] = __uint_as_float(v[t]);
                    }
#pragma unroll
                    for (int t = 0; t < 32; ++t) tr[t * 129 + n_local] = n_ok ? __uint_as_float(v[t]) : -INFINITY;
                    epi_sync();
                    float x[32];
                    float bm = -INFINITY;
                    int bj = 0;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        x[j] = tr[tt * 129 + 32 * gq + j];
                        if (x[j] > bm) { bm = x[j]; bj = j; }       // strict: the lowest index stays on ties
                    }
                    // single-precision exp (1 ulp) of each term, double accumulation: sums good to ~1e-9
                    double sm = 0.0;
                    if (bm > -INFINITY) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) sm += (double)expf(x[j] - bm);
                    }
                    g_m[gq * 32 + tt] = bm;
                    g_i[gq * 32 + tt] = u.n0 + 32 * gq + bj;
                    g_s[gq * 32 + tt] = sm;
                    epi_sync();
                    if (e < 32 && u.tok0 + cc + e < p.rows) {
                        // quarters ascend in vocabulary index, and so do the tiles of a CTA: on equal
                        // maxima the earlier index stays
                        float tm = g_m[e];
                        int ti = g_i[e];
                        for (int w = 1; w < 4; ++w)
                            if (g_m[w * 32 + e] > tm) { tm = g_m[w * 32 + e]; ti = g_i[w * 32 + e]; }
                        double ts = 0.0;
                        for (int w = 0; w < 4; ++w)
                            if (g_m[w * 32 + e] > -INFINITY) ts += g_s[w * 32 + e] * exp((double)g_m[w * 32 + e] - (double)tm);
                        const int tl = cc + e;
                        if (piece == 0) {
                            run_m[tl] = tm; run_i[tl] = ti; run_s[tl] = ts;
                        } else if (tm > run_m[tl]) {
                            run_s[tl] = run_s[tl] * exp((double)run_m[tl] - (double)tm) + ts;
                            run_m[tl] = tm; run_i[tl] = ti;
                        } else {
                            run_s[tl] += ts * exp((double)tm - (double)run_m[tl]);
                        }
                    }
                    // the next chunk's writes to the transpose tile and to the quarter statistics come
                    // after its own barrier, which every thread reaches only after the reads above
                }
            }
            tc_fence_before();
            mbar_arrive(smem_u32(&bars[2 * NS + 2 + buf]));       // accumulator may be overwritten
            if (p.f.mode != WD_FUSE_NONE && p.f.mode != WD_FUSE_LMSTATS) {
                // count this piece's arrival at its tile; the CTA that arrives last finishes the tile
                const int e = (int)threadIdx.x - 64;
                __threadfence();
                epi_sync();
                if (e == 0) {
                    int idx = unit, expected;
                    if (p.f.mode == WD_FUSE_SWIGLU) {
                        const int tile = unit / p.tok_tiles, tokt = unit - tile * p.tok_tiles;
                        const int t_in = tile - p.seg_tile0[u.seg];
                        idx = t_in * p.tok_tiles + tokt;
                        expected = n_contrib(p, G, (p.seg_tile0[0] + t_in) * p.tok_tiles + tokt) +
                                   n_contrib(p, G, (p.seg_tile0[1] + t_in) * p.tok_tiles + tokt);
                    } else {
                        expected = n_contrib(p, G, unit);
                    }
                    const int old = atomicAdd(p.f.counters + idx, 1);
                    const int last = (old + 1 == expected) ? 1 : 0;
                    if (last) p.f.counters[idx] = 0;               // ready for the next launch
                    *last_flag = last;
                    __threadfence();
                }
                epi_sync();
                if (*last_flag) finalize_unit(p, G, unit, e);
                epi_sync();
            } else if (kb0 + len == p.kb_total && n_ok && p.f.mode == WD_FUSE_NONE) {
                // this CTA finished the tile: slices nobody wrote must read as zero
                for (int sl = ord + 1; sl < p.n_slices; ++sl) {
                    float* ys = yb + (size_t)sl * p.split_stride;
                    for (int tok = u.tok0; tok < u.tok0 + p.bn && tok < p.rows; ++tok) ys[(size_t)tok * p.ncol] = 0.f;
                }
            }
        }
        if (threadIdx.x == 64) G_STAMP(6);
        if (!ok && lane == 0) {
            *abort_flag = 1;
            atomicCAS(p.status, 0, WD_ERR_DEVICE_TIMEOUT);
        }
        if (kLmStats && sch.n_pieces > 0) {
            // one (max, argmax, sum exp) per token for all the vocabulary tiles this CTA covered
            float* run_m = lm_scratch;
            int* run_i = (int*)(lm_scratch + 256);
            double* run_s = (double*)(lm_scratch + 512);
            epi_sync();
            // this CTA's token tile: rows tok_group * bn .. ; entry c of the row's G statistics
            for (int t = (int)threadIdx.x - 64; t < p.bn && tok_group * p.bn + t < p.rows; t += 128) {
                const size_t si = (size_t)(tok_group * p.bn + t) * G + c;
                p.f.st_max[si] = run_m[t];
                p.f.st_idx[si] = run_i[t];
                p.f.st_sum[si] = run_s[t];
            }
        }
        tc_fence_before();
    }
    __syncthreads();
    if (threadIdx.x == 0) G_STAMP(7);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 2u * (uint32_t)p.buf_cols);
    }
}

#ifdef WD_GEMM_TRACE
extern "C" __attribute__((visibility("default"))) int wd_debug_gemm_trace(unsigned long long* host /*[8][160][8]*/) {
    cudaDeviceSynchronize();
    return (int)cudaMemcpyFromSymbol(host, g_gemm_trace, sizeof(unsigned long long) * 8 * 160 * 8);
}
#endif

// ------------------------------------------------------------------------------------------
// Chain kernel: the projections between two attention calls as ONE persistent launch (few rows)
// ------------------------------------------------------------------------------------------
// A normal step of the windowed method computes a few dozen rows (Section 4.3), so a block is four
// weight streams (q/k/v, output projection, gate/up, down) separated by work that touches a few
// hundred KB: summing split-K partial tiles, the residual add, 1/rms, SwiGLU, RoPE and the cache
// write.  As separate launches every one of those boundaries idles the memory system for several
// microseconds (the last CTA's epilogue, the launch dependency, the first operand round trip),
// which is where a third of the step went.  Here up to four consecutive GEMMs run inside one
// launch of one CTA per SM, each with the persistent stream-K schedule of gemm_tc_kernel:
//   * the TMA warp streams the weight boxes of GEMM g+1 straight after those of GEMM g: weights
//     never depend on anything, so the ring keeps filling while GEMM g is still being finished;
//     only the small activation box of a stage waits until GEMM g+1's input exists;
//   * the CTA that completes an output tile of GEMM g finishes it (finalize_unit: the residual add
//     and the next GEMM's bf16 input, SwiGLU, or RoPE and the cache rows) and counts it on a device
//     counter; GEMM g+1's input exists when the counter has reached the number of tiles, which the
//     TMA thread polls (bounded, with back-off);
//   * the MMA warp and the epilogue warps run as in gemm_tc_kernel, on a stage and accumulator
//     sequence that simply continues across GEMMs.
// All CTAs are resident at the same time (one per SM, never more CTAs than SMs), so a CTA that
// waits for the counter waits for CTAs that are running.  Every wait is bounded as elsewhere.
constexpr int kChainMax = 4;

struct ChainParams {
    int n_gemm;
    TcParams g[kChainMax];
    int32_t* ready;                   // [kChainMax] tiles finished, counted up across launches (wraps)
    int32_t target[kChainMax];        // counter value at which this launch's GEMM i is completely finished
};
struct ChainMaps {
    CUtensorMap x[kChainMax];
    CUtensorMap w[kChainMax][3];
};

__device__ __forceinline__ int32_t ld_acquire_gpu(const int32_t* p) {
    int32_t v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// orders this thread's generic-proxy accesses to global memory with accesses through the async proxy (TMA)
__device__ __forceinline__ void fence_proxy_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }

#ifdef WD_CK_TRACE
// development aid (not compiled by default): globaltimer stamps of the last chain launch
__device__ unsigned long long g_chain_trace[160][64];
#define CH_STAMP(slot) do { if ((slot) < 64) g_chain_trace[blockIdx.x < 160 ? blockIdx.x : 159][(slot)] = global_ns(); } while (0)
#else
#define CH_STAMP(slot) do { } while (0)
#endif

__global__ void __launch_bounds__(kThreads)
gemm_chain_kernel(const __grid_constant__ ChainMaps maps, const __grid_constant__ ChainParams cp) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const TcParams& p0 = cp.g[0];                          // rows, bn, ring and accumulator shape are common to the chain
    const int NS = p0.n_stages;
    const int stage_a = kStageA;
    const int stage_bytes = stage_a + p0.bn * kBK * 2;
    uint64_t* bars = (uint64_t*)(smem + (size_t)NS * stage_bytes);
    // bars[0..NS) full | [NS..2NS) empty | [2NS, 2NS+1] accumulator full | [2NS+2, 2NS+3] accumulator empty
    uint32_t* tmem_slot = (uint32_t*)(bars + 2 * NS + 4);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
    int* last_flag = (int*)(tmem_slot + 2);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long G = gridDim.x, c = blockIdx.x;
    // this CTA's share of every GEMM's line of K blocks
    Sched sch[kChainMax];
    int n_tot[kChainMax];
    long long total = 0;
#pragma unroll
    for (int g = 0; g < kChainMax; ++g) {
        n_tot[g] = 0;
        if (g < cp.n_gemm) {
            const long long gb = c * cp.g[g].W / G, ge = (c + 1) * cp.g[g].W / G;
            sch[g].init(gb, ge, cp.g[g].kb_total);
            n_tot[g] = (int)(ge - gb);
            total += n_tot[g];
        }
    }

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        CH_STAMP(60);
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
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 2u * (uint32_t)p0.buf_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0 && total > 0) {
            // ------------------------------------------------ TMA producer: a weight cursor and an activation cursor
            uint64_t pol_stream;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            struct Cur {
                int g, piece, left, kb, n0, tok0;
                const CUtensorMap* mw;
                long long i;                               // stages issued so far
                int s;                                     // ring slot of stage i, kept by increments (no division in the loop)
                uint32_t ph;                               // (i / NS) & 1
            };
            auto enter = [&](Cur& w) {                     // first block of piece w.piece of GEMM w.g
                while (w.g < cp.n_gemm && w.piece >= sch[w.g].n_pieces) { ++w.g; w.piece = 0; }
                if (w.g >= cp.n_gemm) return;
                const TcParams& p = cp.g[w.g];
                long long gl;
                int len;
                sch[w.g].piece(w.piece, gl, len);
                const int unit = (int)(gl / p.kb_total);
                w.kb = (int)(gl - (long long)unit * p.kb_total);
                w.left = len;
                const UnitInfo u = decode_unit(p, unit, 0);
                w.n0 = u.n0;
                w.tok0 = u.tok0;
                w.mw = &maps.w[w.g][u.seg];
            };
            auto advance = [&](Cur& w) {
                ++w.i;
                if (++w.s == NS) { w.s = 0; w.ph ^= 1u; }
                ++w.kb;
                if (--w.left == 0) { ++w.piece; enter(w); }
            };
            Cur cw, cx;
            cw.g = 0; cw.piece = 0; cw.i = 0; cw.s = 0; cw.ph = 0;
            enter(cw);
            cx = cw;
            bool rdy[kChainMax] = {false, false, false, false};
            unsigned long long t_idle = 0;
            bool ok = true;
            auto issue_w = [&]() {
                const int s = cw.s;
                mbar_expect_tx(smem_u32(&bars[s]), (uint32_t)stage_bytes);
                tma_load_2d_hint(smem_u32(smem + (size_t)s * stage_bytes), cw.mw, smem_u32(&bars[s]), cw.kb * kBK, cw.n0, pol_stream);
                advance(cw);
            };
            while (cx.i < total && ok) {
                // 1. an activation box that can go goes first (its weight box is already on the way)
                if (cx.i < cw.i) {
                    const int g = cx.g;
                    if (!rdy[g] && g > 0 && (int32_t)(ld_acquire_gpu(cp.ready + (g - 1)) - cp.target[g - 1]) >= 0) {
                        fence_proxy_async_global();            // the finishers' plain stores -> this thread's TMA loads
                        rdy[g] = true;
                        CH_STAMP(g * 14);
                    }
                    if (rdy[g]) {
                        const int s = cx.s;
                        tma_load_2d(smem_u32(smem + (size_t)s * stage_bytes) + stage_a, &maps.x[g], smem_u32(&bars[s]), cx.kb * kBK,
                                    cx.tok0);
                        advance(cx);
                        t_idle = 0;
                        continue;
                    }
                }
                // 2. weights: as far ahead as the ring allows
                if (cw.i < total) {
                    const int s = cw.s;
                    const uint32_t ph = cw.ph;
                    if (cw.i < NS || mbar_try_wait(smem_u32(&bars[NS + s]), ph ^ 1u)) {
                        issue_w();
                        t_idle = 0;
                        continue;
                    }
                    if (cx.i == cw.i) {
                        // nothing else to do until this slot is free: the plain bounded wait
                        if (!mbar_wait(smem_u32(&bars[NS + s]), ph ^ 1u, abort_flag)) { ok = false; break; }
                        issue_w();
                        t_idle = 0;
                        continue;
                    }
                }
                // 3. the ring is full of weights whose activations do not exist yet
                if (!rdy[0]) {
                    pdl_wait();                                // sit out the previous kernel
                    rdy[0] = true;
                    CH_STAMP(0);
                    continue;
                }
                if (*abort_flag) ok = false;
                const unsigned long long now = global_ns();
                if (t_idle == 0) t_idle = now;
                else if (now - t_idle > kWaitNs) ok = false;
            }
            if (!ok) {
                *abort_flag = 1;
                atomicCAS(p0.status, 0, WD_ERR_DEVICE_TIMEOUT);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            // ------------------------------------------------ MMA issuer
            bool ok = true;
            int s = 0, pc = 0;
            uint32_t ph = 0;
            for (int g = 0; g < cp.n_gemm && ok; ++g) {
                const uint32_t idesc = cp.g[g].idesc;
                for (int piece = 0; piece < sch[g].n_pieces && ok; ++piece, ++pc) {
                    long long gl;
                    int len;
                    sch[g].piece(piece, gl, len);
                    const int buf = pc & 1;
                    const uint32_t par = (uint32_t)(pc >> 1) & 1u;
                    if (!(ok = mbar_wait(smem_u32(&bars[2 * NS + 2 + buf]), par ^ 1u, abort_flag))) break;
                    tc_fence_after();
                    const uint32_t acc = tmem_base + (uint32_t)(buf * p0.buf_cols);
                    for (int j = 0; j < len; ++j) {
                        if (!(ok = mbar_wait(smem_u32(&bars[s]), ph, abort_flag))) break;
                        if (piece == 0 && j == 0) CH_STAMP(g * 14 + 1);
                        tc_fence_after();
                        const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
                        const uint64_t adesc = make_sdesc(sa), bdesc = make_sdesc(sa + stage_a);
#pragma unroll
                        for (int kk = 0; kk < kBK / 16; ++kk)
                            umma_bf16(acc, adesc + (uint64_t)(2 * kk), bdesc + (uint64_t)(2 * kk), idesc, (j > 0 || kk > 0) ? 1u : 0u);
                        umma_commit(smem_u32(&bars[NS + s]));
                        if (++s == NS) { s = 0; ph ^= 1u; }
                    }
                    if (ok) umma_commit(smem_u32(&bars[2 * NS + buf]));
                    CH_STAMP(g * 14 + 2);
                }
            }
            if (!ok) {
                *abort_flag = 1;
                atomicCAS(p0.status, 0, WD_ERR_DEVICE_TIMEOUT);
            }
        }
        __syncwarp();
    } else {
        // ---------------------------------------------------- epilogue (warps 2..5)
        const int quarter = warp & 3;
        const int n_local = quarter * 32 + lane;
        const int e = (int)threadIdx.x - 64;
        pdl_wait();
        bool ok = true;
        int pc = 0;
        for (int g = 0; g < cp.n_gemm && ok; ++g) {
            const TcParams& p = cp.g[g];
            for (int piece = 0; piece < sch[g].n_pieces; ++piece, ++pc) {
                long long gl;
                int len;
                sch[g].piece(piece, gl, len);
                const int unit = (int)(gl / p.kb_total);
                const UnitInfo u = decode_unit(p, unit, 0);
                const int buf = pc & 1;
                const uint32_t par = (uint32_t)(pc >> 1) & 1u;
                const int n = u.n0 + n_local;
                const int ord = (int)(c - (((long long)unit * p.kb_total + 1) * G - 1) / p.W);
                ok = ok && mbar_wait(smem_u32(&bars[2 * NS + buf]), par, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                float* ys = p.y + p.seg_col[u.seg] + n + (size_t)ord * p.split_stride;
                const uint32_t t_acc = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * p0.buf_cols);
                for (int cc = 0; cc < p.bn; cc += 16) {
                    if (u.tok0 + cc >= p.rows) break;
                    uint32_t v[16];
                    tmem_ld16(t_acc + (uint32_t)cc, v);
#pragma unroll
                    for (int t = 0; t < 16; ++t) {
                        const int tok = u.tok0 + cc + t;
                        if (tok < p.rows) ys[(size_t)tok * p.ncol] = __uint_as_float(v[t]);
                    }
                }
                tc_fence_before();
                mbar_arrive(smem_u32(&bars[2 * NS + 2 + buf]));       // accumulator may be overwritten
                if (e == 0 && piece < 3) CH_STAMP(g * 14 + 3 + 3 * piece);
                // count this piece's arrival at its tile; the CTA that arrives last finishes the tile
                __threadfence();
                epi_sync();
                if (e == 0) {
                    int idx = unit, expected;
                    if (p.f.mode == WD_FUSE_SWIGLU) {
                        const int tile = unit / p.tok_tiles, tokt = unit - tile * p.tok_tiles;
                        const int t_in = tile - p.seg_tile0[u.seg];
                        idx = t_in * p.tok_tiles + tokt;
                        expected = n_contrib(p, G, (p.seg_tile0[0] + t_in) * p.tok_tiles + tokt) +
                                   n_contrib(p, G, (p.seg_tile0[1] + t_in) * p.tok_tiles + tokt);
                    } else {
                        expected = n_contrib(p, G, unit);
                    }
                    const int old = atomicAdd(p.f.counters + idx, 1);
                    const int last = (old + 1 == expected) ? 1 : 0;
                    if (last) p.f.counters[idx] = 0;               // ready for the next GEMM that uses this counter
                    *last_flag = last;
                    __threadfence();
                }
                epi_sync();
                if (e == 0 && piece < 3) CH_STAMP(g * 14 + 4 + 3 * piece);
                if (*last_flag) {
                    finalize_unit(p, G, unit, e);
                    // the finished tile is the next GEMM's input (read by TMA) and the next finisher's x
                    fence_proxy_async_global();
                    __threadfence();
                    epi_sync();
                    if (e == 0) atomicAdd(cp.ready + g, 1);
                    if (e == 0 && piece < 3) CH_STAMP(g * 14 + 5 + 3 * piece);
                } else {
                    epi_sync();
                }
            }
        }
        if (!ok && lane == 0) {
            *abort_flag = 1;
            atomicCAS(p0.status, 0, WD_ERR_DEVICE_TIMEOUT);
        }
        tc_fence_before();
    }
    __syncthreads();
    if (threadIdx.x == 0) CH_STAMP(61);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 2u * (uint32_t)p0.buf_cols);
    }
}

#ifdef WD_CK_TRACE
extern "C" __attribute__((visibility("default"))) int wd_debug_chain_trace(unsigned long long* host /*[160][64]*/) {
    cudaDeviceSynchronize();
    return (int)cudaMemcpyFromSymbol(host, g_chain_trace, sizeof(unsigned long long) * 160 * 64);
}
#endif

// Two-CTA variant for many tokens (compute-bound shapes).  The CTA pair of a cluster works on one
// [256 weight rows x BN tokens] tile with tcgen05.mma.cta_group::2: each CTA loads its own 128 weight
// rows and HALF of the token rows of every K block (the tensor cores of both SMs read both halves),
// so the operand traffic per flop into shared memory is two thirds of the one-CTA [128 x BN] tile's,
// while the ring keeps its depth and both accumulators stay double-buffered.  Same persistent
// stream-K schedule, same output layout; the pair is the scheduling unit (c = pair index).
//   even CTA: expects the bytes of both CTAs on its "full" barriers (the odd CTA's TMA loads count
//             on them through .cta_group::2), issues every MMA, releases the stages and publishes the
//             accumulators in BOTH CTAs (tcgen05.commit with a CTA mask)
//   both:     TMA producer for their own operand halves, epilogue for their own 128 weight rows;
//             epilogue warps of both CTAs arrive on the even CTA's "accumulator empty" barriers
// Two-accumulator modes (TcParams::dual): each weight stage feeds two MMA chains, either against two
// halves of a 2*BN-token super-tile (the weights enter shared memory once per 512 tokens) or with the
// gate and the up block of the same FFN columns against one token tile (the epilogue then writes
// silu(gate) * up as bf16).  With BN > 128 the two accumulators fill the tensor memory, so there is one
// accumulator set and the epilogue of a unit does not overlap the next unit's MMAs.
// Whole-tile schedule: units are dealt round-robin in (token group, weight tile, token tile) order so
// that the pairs running at one time share a few weight tiles and one token group in the L2.
template <bool kFp8>
__global__ void __launch_bounds__(kThreadsPair)
gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w0,
                    const __grid_constant__ CUtensorMap map_w1, const __grid_constant__ CUtensorMap map_w2,
                    const TcParams p) {
    constexpr int kKE = kFp8 ? 128 : kBK;                 // K elements per block
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int NS = p.n_stages;
    const int half_bn = p.bn >> 1;                        // token rows of one accumulator held by this CTA
    const int tok_rows = p.dual == 1 ? p.bn : half_bn;    // token rows this CTA loads per K block
    const bool gate_up = p.dual == 2;                     // two weight blocks (gate, up) per stage
    const int stage_a = gate_up ? 2 * kStageA : kStageA;  // this CTA's 128 weight rows (of gate and of up)
    const int stage_bytes = stage_a + tok_rows * kBK * 2;
    // accumulator sets of (dual ? 2 : 1) * buf_cols columns: two sets (MMA of one tile overlaps the
    // epilogue of the previous one) when they fit the 512 columns, else one
    const int set_cols = (p.dual ? 2 : 1) * p.buf_cols;
    const int n_sets = 2 * set_cols <= 512 ? 2 : 1;
    uint64_t* bars = (uint64_t*)(smem + (size_t)NS * stage_bytes);
    // bars[0..NS) full (used in the even CTA) | [NS..2NS) empty | [2NS, 2NS+1] accumulator full |
    // [2NS+2, 2NS+3] accumulator empty (used in the even CTA; every epilogue warp of both CTAs arrives once)
    uint32_t* tmem_slot = (uint32_t*)(bars + 2 * NS + 4);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();              // 0: issues the MMAs
    if (threadIdx.x == 0) G_STAMP(0);
    // pairs per token group, this pair's index in its group, its token group (see TcParams::tok_split)
    const long long G = (gridDim.x >> 1) / (p.tok_split > 1 ? p.tok_split : 1), c = (blockIdx.x >> 1) % G;
    const int tok_group = (int)((blockIdx.x >> 1) / G);
    Sched sch;
    int n_total;
    if (p.aligned && p.tok_grp > 0) {
        sch.init_strided(c, G, p.n_units, p.kb_total);
        n_total = sch.n_pieces * p.kb_total;
    } else {
        long long g_begin, g_end;
        if (p.aligned) {
            g_begin = (c * p.n_units / G) * p.kb_total;
            g_end = ((c + 1) * p.n_units / G) * p.kb_total;
        } else {
            g_begin = c * p.W / G;
            g_end = (c + 1) * p.W / G;
        }
        n_total = (int)(g_end - g_begin);
        sch.init(g_begin, g_end, p.kb_total);
    }

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(smem_u32(&bars[s]), 1);
            mbar_init(smem_u32(&bars[NS + s]), 1);
        }
        mbar_init(smem_u32(&bars[2 * NS]), 1);
        mbar_init(smem_u32(&bars[2 * NS + 1]), 1);
        mbar_init(smem_u32(&bars[2 * NS + 2]), 2 * (kThreadsPair / 32 - 2));
        mbar_init(smem_u32(&bars[2 * NS + 3]), 2 * (kThreadsPair / 32 - 2));
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w0) : "memory");
    }
    if (warp == 1) tmem2_alloc(smem_u32(tmem_slot), (uint32_t)(n_sets * set_cols));   // the same warp in both CTAs
    tc_fence_before();
    __syncthreads();
    cluster_sync();               // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0 && n_total > 0) {
            // ------------------------------------------------ TMA producer (both CTAs, own halves)
            // weights that one or two units use are streamed past the L2 (evict first); with more token
            // tiles the same weight block is wanted again by the units that follow: keep it (evict last)
            uint64_t pol_stream;
            if (p.tok_tiles > 2)
                asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_stream));
            else
                asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            struct Walk {
                int piece, left, kb, n0, tok0;
                const CUtensorMap* mw;
            };
            auto enter = [&](Walk& w) {
                long long g;
                int len;
                sch.piece(w.piece, g, len);
                const int unit = (int)(g / p.kb_total);
                w.kb = (int)(g - (long long)unit * p.kb_total);
                w.left = len;
                const UnitInfo u = decode_unit(p, unit, tok_group);
                w.n0 = u.n0 + (int)rank * kBM;
                w.tok0 = u.tok0 + (int)rank * tok_rows;
                w.mw = u.seg == 0 ? &map_w0 : (u.seg == 1 ? &map_w1 : &map_w2);
            };
            auto advance = [&](Walk& w) {
                ++w.kb;
                if (--w.left == 0 && ++w.piece < sch.n_pieces) enter(w);
            };
            Walk w0;
            w0.piece = 0;
            enter(w0);
            const int n_pre = n_total < NS ? n_total : NS;
            Walk w = w0;
            for (int i = 0; i < n_pre; ++i, advance(w)) {
                if (rank == 0) mbar_expect_tx(smem_u32(&bars[i]), 2u * (uint32_t)stage_bytes);
                tma2_load_2d_hint(smem_u32(smem + (size_t)i * stage_bytes), w.mw, cluster_map(smem_u32(&bars[i]), 0),
                                  w.kb * kKE, w.n0, pol_stream);
                if (gate_up)
                    tma2_load_2d_hint(smem_u32(smem + (size_t)i * stage_bytes) + kStageA, &map_w1,
                                      cluster_map(smem_u32(&bars[i]), 0), w.kb * kKE, w.n0, pol_stream);
            }
            G_STAMP(1);
            pdl_wait();
            G_STAMP(2);
            Walk wx = w0;
            for (int i = 0; i < n_pre; ++i, advance(wx))
                tma2_load_2d(smem_u32(smem + (size_t)i * stage_bytes) + stage_a, &map_x,
                             cluster_map(smem_u32(&bars[i]), 0), wx.kb * kKE, wx.tok0);
            int s = n_pre % NS;
            uint32_t ph = (uint32_t)(n_pre / NS) & 1u;
            for (int i = n_pre; i < n_total; ++i, advance(w)) {
                if (!mbar_wait(smem_u32(&bars[NS + s]), ph ^ 1u, abort_flag)) {
                    *abort_flag = 1;
                    atomicCAS(p.status, 0, WD_ERR_DEVICE_TIMEOUT);
                    break;
                }
                const uint32_t full = cluster_map(smem_u32(&bars[s]), 0);
                const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
                if (rank == 0) mbar_expect_tx(smem_u32(&bars[s]), 2u * (uint32_t)stage_bytes);
                tma2_load_2d_hint(sa, w.mw, full, w.kb * kKE, w.n0, pol_stream);
                if (gate_up) tma2_load_2d_hint(sa + kStageA, &map_w1, full, w.kb * kKE, w.n0, pol_stream);
                tma2_load_2d(sa + stage_a, &map_x, full, w.kb * kKE, w.tok0);
                if (++s == NS) { s = 0; ph ^= 1u; }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            // ------------------------------------------------ MMA issuer (even CTA only)
            bool ok = true;
            int s = 0;
            uint32_t ph = 0;
            for (int piece = 0; piece < sch.n_pieces && ok; ++piece) {
                long long g;
                int len;
                sch.piece(piece, g, len);
                const int buf = n_sets == 2 ? piece & 1 : 0;
                const uint32_t par = (uint32_t)(n_sets == 2 ? piece >> 1 : piece) & 1u;
                // the epilogues of both CTAs have drained this accumulator set (free at the start)
                if (!(ok = mbar_wait(smem_u32(&bars[2 * NS + 2 + buf]), par ^ 1u, abort_flag))) break;
                tc_fence_after();
                const uint32_t acc = tmem_base + (uint32_t)(buf * set_cols);
                for (int j = 0; j < len; ++j) {
                    if (!(ok = mbar_wait(smem_u32(&bars[s]), ph, abort_flag))) break;
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
                    const uint64_t adesc = make_sdesc(sa);
                    const uint64_t bdesc = make_sdesc(sa + stage_a);
#pragma unroll
                    for (int kk = 0; kk < kBK / 16; ++kk) {
                        if (kFp8)
                            umma2_f8(acc, adesc + (uint64_t)(2 * kk), bdesc + (uint64_t)(2 * kk), p.idesc,
                                     (j > 0 || kk > 0) ? 1u : 0u);
                        else
                            umma2_bf16(acc, adesc + (uint64_t)(2 * kk), bdesc + (uint64_t)(2 * kk), p.idesc,
                                       (j > 0 || kk > 0) ? 1u : 0u);
                    }
                    if (p.dual) {
                        // second accumulator: the same weight rows against the other half of the token rows
                        // (offset of half_bn rows of 128 bytes, in 16-byte units), or the up weights against
                        // the same token rows
                        const uint64_t adesc1 = gate_up ? adesc + (uint64_t)(kStageA >> 4) : adesc;
                        const uint64_t bdesc1 = gate_up ? bdesc : bdesc + (uint64_t)(half_bn * 8);
                        const uint32_t acc1 = acc + (uint32_t)p.buf_cols;
#pragma unroll
                        for (int kk = 0; kk < kBK / 16; ++kk) {
                            if (kFp8)
                                umma2_f8(acc1, adesc1 + (uint64_t)(2 * kk), bdesc1 + (uint64_t)(2 * kk), p.idesc,
                                         (j > 0 || kk > 0) ? 1u : 0u);
                            else
                                umma2_bf16(acc1, adesc1 + (uint64_t)(2 * kk), bdesc1 + (uint64_t)(2 * kk), p.idesc,
                                           (j > 0 || kk > 0) ? 1u : 0u);
                        }
                    }
                    umma2_commit_mc(smem_u32(&bars[NS + s]), 3);          // stage free in both CTAs
                    if (++s == NS) { s = 0; ph ^= 1u; }
                }
                if (ok) umma2_commit_mc(smem_u32(&bars[2 * NS + buf]), 3);  // accumulator complete in both CTAs
            }
            if (!ok) {
                *abort_flag = 1;
                atomicCAS(p.status, 0, WD_ERR_DEVICE_TIMEOUT);
            }
        }
        __syncwarp();
    } else {
        // ---------------------------------------------------- epilogue (warps 2..9 of both CTAs)
        // Warp w reads the accumulator rows (TMEM lanes) of quarter w % 4; the two warps of a quarter
        // take alternate 16-column chunks.  (Plain loops on purpose: a version that kept the next
        // chunk's tcgen05.ld in flight behind lambdas compiled to twice the instructions per chunk.)
        const int quarter = warp & 3;
        const int hf = (warp - 2) >> 2;
        constexpr int n_hf = 2;
        const int n_local = (int)rank * kBM + quarter * 32 + lane;
        pdl_wait();
        bool ok = true;
        for (int piece = 0; piece < sch.n_pieces; ++piece) {
            long long g;
            int len;
            sch.piece(piece, g, len);
            const int unit = (int)(g / p.kb_total), kb0 = (int)(g - (long long)unit * p.kb_total);
            const UnitInfo u = decode_unit(p, unit, tok_group);
            const int buf = n_sets == 2 ? piece & 1 : 0;
            const uint32_t par = (uint32_t)(n_sets == 2 ? piece >> 1 : piece) & 1u;
            const int n = u.n0 + n_local;
            const bool n_ok = n < p.seg_n[u.seg];
            int ord = 0;
            if (!p.aligned) ord = (int)(c - (((long long)unit * p.kb_total + 1) * G - 1) / p.W);
            ok = ok && mbar_wait(smem_u32(&bars[2 * NS + buf]), par, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            float* yb = p.y + p.seg_col[u.seg] + n;
            const float sw_n = (kFp8 && n_ok) ? p.sw[u.seg][n] : 1.f;
            const uint32_t t_acc = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * set_cols);
            float* ys = yb + (size_t)ord * p.split_stride;
            // Accumulator a, column col: columns [0, half_bn) are the token rows the even CTA holds,
            // the rest the odd CTA's.  One accumulator (or gate/up): token tok0 + col.  Two token
            // halves: the even CTA holds tokens [tok0, tok0 + bn), the odd one [tok0 + bn, tok0 + 2 bn),
            // accumulator a the a-th half of each.
            const int col_step = 16 * n_hf;
            if (gate_up) {
                // h = silu(gate) * up
                __nv_bfloat16* hb = p.swiglu_h + n;
                for (int cc = 16 * hf; cc < p.bn; cc += col_step) {
                    if (u.tok0 + cc >= p.rows) break;
                    uint32_t vg[16], vu[16];
                    tmem_ld16_issue(t_acc + (uint32_t)cc, vg);
                    tmem_ld16(t_acc + (uint32_t)(p.buf_cols + cc), vu);
                    tmem_ld16_wait(vg);
                    if (n_ok) {
#pragma unroll
                        for (int t = 0; t < 16; ++t) {
                            const int tok = u.tok0 + cc + t;
                            const float gv = __uint_as_float(vg[t]);
                            if (tok < p.rows)
                                hb[(size_t)tok * p.ncol] = __float2bfloat16(__fdividef(gv, 1.f + __expf(-gv)) * __uint_as_float(vu[t]));
                        }
                    }
                }
            }
            for (int a = 0; a < (gate_up ? 0 : p.dual ? 2 : 1); ++a) {
                for (int cc = 16 * hf; cc < p.bn; cc += col_step) {
                    int tk[16];
#pragma unroll
                    for (int t = 0; t < 16; ++t) {
                        const int col = cc + t;
                        tk[t] = p.dual != 1 ? u.tok0 + col
                                            : (col < half_bn ? u.tok0 + a * half_bn + col : u.tok0 + p.bn + a * half_bn + col - half_bn);
                    }
                    if (tk[0] >= p.rows) continue;           // tk[0] is the chunk's smallest token (same for the whole warp)
                    uint32_t v[16];
                    tmem_ld16(t_acc + (uint32_t)(a * p.buf_cols + cc), v);
                    if (n_ok) {
#pragma unroll
                        for (int t = 0; t < 16; ++t) {
                            const int tok = tk[t];
                            if (tok < p.rows)
                                ys[(size_t)tok * p.ncol] = kFp8 ? __uint_as_float(v[t]) * sw_n * p.sx[tok] : __uint_as_float(v[t]);
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(cluster_map(smem_u32(&bars[2 * NS + 2 + buf]), 0));   // accumulator may be overwritten
            if (kb0 + len == p.kb_total && n_ok) {
                // this pair finished the tile: slices nobody wrote must read as zero
                for (int sl = ord + 1; sl < p.n_slices; ++sl) {
                    float* ys = yb + (size_t)sl * p.split_stride;
                    for (int tok = u.tok0 + hf; tok < u.tok0 + (p.dual == 1 ? 2 : 1) * p.bn && tok < p.rows; tok += n_hf)
                        ys[(size_t)tok * p.ncol] = 0.f;
                }
            }
        }
        if (!ok && lane == 0) {
            *abort_flag = 1;
            atomicCAS(p.status, 0, WD_ERR_DEVICE_TIMEOUT);
        }
        tc_fence_before();
    }
    __syncthreads();
    cluster_sync();               // neither CTA frees tensor memory or leaves while the other may still signal it
    if (threadIdx.x == 0) G_STAMP(7);
    if (warp == 1) {
        tc_fence_after();
        tmem2_dealloc(tmem_base, (uint32_t)(n_sets * set_cols));
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

// [n_rows, K] bytes (e4m3 codes) row-major, box = 128 (K) x box_rows, 128-byte swizzle
wd_status encode_2d8(CUtensorMap* m, const void* ptr, int n_rows, int K, int box_rows) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return WD_ERR_CUDA;
    if ((uintptr_t)ptr % 16 || K % 16) return WD_ERR_MISALIGNED;
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)n_rows};
    cuuint64_t strides[1] = {(cuuint64_t)K};
    cuuint32_t box[2] = {128u, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? WD_OK : WD_ERR_CUDA;
}

struct TcConfig { int bn, tok_tiles, n_stages, buf_cols, ctas_per_sm, wide, tile_rows; size_t smem; };

int env_int(const char* name, int dflt) {
    const char* v = getenv(name);
    return v && *v ? atoi(v) : dflt;
}

TcConfig pick_config(int rows, bool allow_wide, bool lm_stats) {
    TcConfig c;
    // Many tokens: the GEMM is bound by operand traffic from L2 into shared memory, so a CTA
    // carries two 128-row weight halves that share every activation box ([256 x BN] per CTA).
    static const int wide_from = env_int("WD_GEMM_WIDE_FROM", 512);   // measured: pays from a few hundred rows when every CTA gets whole tiles
    c.wide = (allow_wide && rows >= wide_from) ? 1 : 0;
    c.tile_rows = c.wide ? 2 * kBM : kBM;
    static const int bn_max = env_int("WD_GEMM_BN_MAX", 256);      // tuning knob (multiple of 16, <= 256)
    c.tok_tiles = (rows + bn_max - 1) / bn_max;
    if (lm_stats && c.tok_tiles == 3) c.tok_tiles = 4;             // the LM head takes one CTA group per token tile
    c.bn = ((rows + c.tok_tiles - 1) / c.tok_tiles + 15) / 16 * 16;     // balanced token tiles, <= 256
    int cols = 32;
    while (cols < c.bn) cols <<= 1;
    c.buf_cols = cols;                                                   // two accumulators: 2 * cols <= 512
    const int stage = c.tile_rows * kBK * 2 + c.bn * kBK * 2;
    static const int want2 = env_int("WD_GEMM_CTAS_PER_SM", 1);
    c.ctas_per_sm = (want2 == 2 && c.bn <= 64 && !c.wide) ? 2 : 1;
    c.n_stages = ((c.ctas_per_sm == 2 ? 96 : 192) * 1024) / stage;
    if (c.n_stages > 10) c.n_stages = 10;
    if (c.n_stages < 2) c.n_stages = 2;
    c.smem = (size_t)c.n_stages * stage + (2 * c.n_stages + 4) * 8 + 16 + (lm_stats ? 24576 : 8192) + 1024;
    return c;
}

// index of the current device, or -1 (beyond the 64 the per-device tables hold, or on an error)
int current_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return -1;
    return dev;
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

uint32_t make_idesc(int bn, int m = kBM, bool fp8 = false) {
    uint32_t d = 0;
    d |= 1u << 4;                      // D format: f32
    if (!fp8) {
        d |= 1u << 7;                  // A format: bf16 (kind::f8f6f4: 0 = e4m3)
        d |= 1u << 10;                 // B format: bf16
    }
    // bits 15 / 16: A and B are K-major (0)
    d |= (uint32_t)(bn >> 3) << 17;    // N
    d |= (uint32_t)(m >> 4) << 24;     // M (256: the two-CTA form)
    return d;
}

// launch of gemm_tc_pair_kernel: same contract as wd_tc_gemm
wd_status tc_gemm_pair(const WdTcX* x, const WdTcSeg* segs, int nseg, int rows, int K, float* y, size_t y_floats,
                       int sm_count, int32_t* status, cudaStream_t stream, int* n_split_out, bool force_single_split,
                       const WdTcFp8* fp8, const WdTcSwiglu* sg) {
    TcParams p;
    memset(&p, 0, sizeof(p));
    if (fp8) {
        p.fp8 = 1;
        for (int i = 0; i < 3; ++i) p.sw[i] = fp8->sw[i < nseg ? i : 0];
        p.sx = fp8->sx;
    }
    const int kke = fp8 ? 128 : kBK;
    p.tile_rows = 2 * kBM;
    // Two accumulators per weight stage (token super-tiles of 2*bn rows): the weights enter shared memory
    // once for up to 512 tokens, but the accumulators fill the tensor memory, so the epilogue no longer
    // overlaps the next tile.  Measured: pays for the widest weight matrices (gate/up) once every pair
    // gets at least two whole units, costs 10-25 % on the narrow ones.  0 = never, 1 = that rule, 2 = always.
    static const int dual_mode = env_int("WD_GEMM_DUAL", 1);
    {
        int tiles_all = 0, ncol_all = 0;
        for (int i = 0; i < nseg; ++i) {
            tiles_all += (segs[i].n + p.tile_rows - 1) / p.tile_rows;
            ncol_all += segs[i].n;
        }
        // whole units pay when every pair gets two or more, or when the one or two rounds are nearly full
        const long long pairs = sm_count / 2;
        auto full_rounds = [&](long long units) {
            return units >= 2 * pairs || (units >= pairs && 10 * units >= 9 * pairs * ((units + pairs - 1) / pairs));
        };
        const long long dual_units = (long long)tiles_all * ((rows + 511) / 512);
        p.dual = (dual_mode == 2 || (dual_mode == 1 && ncol_all >= 16384 && dual_units >= 2 * pairs)) ? 1 : 0;
        // gate and up against the same tokens, h = silu(gate) * up written by the epilogue: needs whole
        // tiles per pair (no partial sums)
        static const int swiglu_fused = env_int("WD_GEMM_SWIGLU", 1);
        if (sg && sg->h && swiglu_fused && !fp8 && nseg == 2 && segs[0].n == segs[1].n && dual_mode != 0) {
            const long long gu_units = (long long)((segs[0].n + p.tile_rows - 1) / p.tile_rows) * ((rows + 255) / 256);
            if (full_rounds(gu_units)) p.dual = 2;
        }
    }
    if (p.dual == 1) {
        p.tok_tiles = (rows + 511) / 512;                                   // super-tiles
        p.bn = ((rows + 2 * p.tok_tiles - 1) / (2 * p.tok_tiles) + 15) / 16 * 16;   // balanced, <= 256
    } else {
        p.tok_tiles = (rows + 255) / 256;
        p.bn = ((rows + p.tok_tiles - 1) / p.tok_tiles + 15) / 16 * 16;    // balanced token tiles, <= 256
    }
    int cols = 32;
    while (cols < p.bn) cols <<= 1;
    p.buf_cols = cols;
    const int half_bn = p.bn / 2;
    const int tok_rows = p.dual == 1 ? p.bn : half_bn;                      // token rows per CTA and K block
    const int stage = (p.dual == 2 ? 2 : 1) * kStageA + tok_rows * kBK * 2;
    p.n_stages = (192 * 1024) / stage;
    if (p.n_stages > 10) p.n_stages = 10;
    const size_t smem = (size_t)p.n_stages * stage + (2 * p.n_stages + 4) * 8 + 16 + 256 + 1024;
    int tiles = 0, col = 0;
    for (int i = 0; i < nseg; ++i)
        if (!segs[i].map) return WD_ERR_NULL;
    if (p.dual == 2) {
        // one line of (gate tile, up tile) pairs; the output has the FFN width
        nseg = 1;
        p.seg_tile0[0] = 0;
        p.seg_n[0] = segs[0].n;
        p.seg_col[0] = 0;
        tiles = (segs[0].n + p.tile_rows - 1) / p.tile_rows;
        col = segs[0].n;
        p.swiglu_h = sg->h;
        force_single_split = true;
    } else {
        for (int i = 0; i < nseg; ++i) {
            p.seg_tile0[i] = tiles;
            p.seg_n[i] = segs[i].n;
            p.seg_col[i] = col;
            tiles += (segs[i].n + p.tile_rows - 1) / p.tile_rows;
            col += segs[i].n;
        }
    }
    p.seg_tile0[nseg] = tiles;
    p.nseg = nseg;
    p.ncol = col;
    p.rows = rows;
    p.kb_total = (K + kke - 1) / kke;
    // two token tiles: one group of pairs per token tile, walking the weight K blocks in step
    const int ts = (!p.dual && p.tok_tiles == 2 && (sm_count / 2) % 2 == 0) ? 2 : 1;
    p.tok_split = ts;
    p.n_units = ts > 1 ? tiles : tiles * p.tok_tiles;
    p.W = (long long)p.n_units * p.kb_total;
    const size_t slice = (size_t)rows * col;
    if (p.dual != 2 && slice > y_floats) return WD_ERR_CAPACITY;
    long long G = sm_count / 2 / ts;                                       // CTA pairs (per token group)
    if (G > p.W / 2) G = p.W / 2 > 0 ? p.W / 2 : 1;
    int n_slices = count_slices(p.n_units, p.kb_total, p.W, G);
    p.aligned = 0;
    // With several whole tiles per pair the imbalance of whole-tile scheduling is small, and one
    // slice instead of two or three saves the consumers (and the zero fill) most of their traffic.
    static const int aligned_from = env_int("WD_GEMM_ALIGNED_UNITS", 2);
    if (force_single_split || (size_t)n_slices * slice > y_floats || n_slices > WD_TC_MAX_SPLIT ||
        p.n_units >= aligned_from * G) {
        p.aligned = 1;
        n_slices = 1;
        G = sm_count / 2 / ts;
        if (G > p.n_units) G = p.n_units;
    }
    static const int tok_grp = env_int("WD_GEMM_TOK_GROUP", 16);          // 0 = contiguous units per pair
    p.tok_grp = (p.aligned && ts == 1) ? tok_grp : 0;
    p.n_slices = n_slices;
    p.y = y;
    p.split_stride = slice;
    p.status = status;
    p.trace_slot = nseg == 3 ? 0 : ((nseg == 2 || p.dual == 2) ? 2 : (K == col ? 1 : (K > col ? 3 : 4)));
    p.idesc = make_idesc(p.bn, 2 * kBM, fp8 != nullptr);

    CUtensorMap mx;
    bool hit = false;
    for (const WdTcX::Entry& e : x->cache)
        if (e.rows == rows && e.bn == tok_rows) { mx = e.map; hit = true; break; }
    if (!hit) {
        wd_status s = fp8 ? encode_2d8(&mx, x->ptr, rows, K, tok_rows) : encode_2d(&mx, x->ptr, rows, K, tok_rows);
        if (s != WD_OK) return s;
        if (x->keep) {
            if (x->cache.size() >= 16) x->cache.erase(x->cache.begin());
            x->cache.push_back({rows, tok_rows, mx});
        }
    }
    static bool attr_done[64] = {};     // the attribute belongs to the function on ONE device: set once per device
    const int dev = current_device();
    if (dev < 0) return WD_ERR_CUDA;
    if (!attr_done[dev]) {
        WD_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
        WD_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
        attr_done[dev] = true;
    }
    const CUtensorMap& m0 = *segs[0].map;
    const CUtensorMap& m1 = *segs[(nseg > 1 || p.dual == 2) ? 1 : 0].map;
    const CUtensorMap& m2 = *segs[nseg > 2 ? 2 : 0].map;
    if (sg) sg->done = p.dual == 2;
    ++wd_launch_counter;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)(2 * G * ts));
    lc.blockDim = dim3(kThreadsPair);
    lc.dynamicSmemBytes = smem;
    lc.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = wd_pdl_enabled ? 2 : 1;
    if (fp8) WD_CUDA_TRY(cudaLaunchKernelEx(&lc, gemm_tc_pair_kernel<true>, mx, m0, m1, m2, p));
    else WD_CUDA_TRY(cudaLaunchKernelEx(&lc, gemm_tc_pair_kernel<false>, mx, m0, m1, m2, p));
    if (n_split_out) *n_split_out = p.n_slices;
    return WD_OK;
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
                     int sm_count, int32_t* status, cudaStream_t stream, int* n_split_out, bool force_single_split,
                     const WdTcFuse* fuse, const WdTcFp8* fp8, const WdTcSwiglu* sg) {
    if (!x || !segs || !y || !status || nseg < 1 || nseg > 3) return WD_ERR_BAD_PARAM;
    if (sg) sg->done = false;
    if (rows < 1 || K < 8 || K % 8) return WD_ERR_BAD_PARAM;
    TcParams p;
    memset(&p, 0, sizeof(p));
    const bool fused = fuse && fuse->mode != WD_FUSE_NONE;
    if (fp8) {
        if (K % 16 || !fp8->sx || (fused && fuse->mode != WD_FUSE_LMSTATS)) return WD_ERR_BAD_PARAM;
        p.fp8 = 1;
        for (int i = 0; i < 3; ++i) {
            p.sw[i] = fp8->sw[i < nseg ? i : 0];
            if (!p.sw[i]) return WD_ERR_NULL;
        }
        p.sx = fp8->sx;
    }
    const int kke = fp8 ? 128 : kBK;
    // Many tokens: CTA pairs on [256 x BN] tiles (tcgen05 cta_group::2)
    static const int pair_from = env_int("WD_GEMM_PAIR_FROM", 256);        // rows from which pairs are used; 0 = never
    if (!fused && pair_from > 0 && rows > pair_from && sm_count >= 2)
        return tc_gemm_pair(x, segs, nseg, rows, K, y, y_floats, sm_count, status, stream, n_split_out, force_single_split,
                            fp8, sg);
    // The wide tile halves the operand traffic per flop but has a shallower ring and an epilogue
    // that does not overlap the next tile: it pays once every CTA gets at least one whole tile.
    long long wide_units = 0;
    for (int i = 0; i < nseg; ++i) wide_units += (segs[i].n + 2 * kBM - 1) / (2 * kBM);
    wide_units *= (rows + 255) / 256;
    static const int wide_min_units = env_int("WD_GEMM_WIDE_MIN_UNITS", 0);     // tuning knob; 0 = one unit per SM
    TcConfig cfg = pick_config(rows, !fused && !fp8 && wide_units >= (wide_min_units > 0 ? wide_min_units : sm_count),
                               fuse && fuse->mode == WD_FUSE_LMSTATS);
    if (x->smem_cap > 0 && cfg.smem > (size_t)x->smem_cap) {
        // a shorter ring, so that the CTA fits beside the producer kernel's (see WdTcX::smem_cap); the plain
        // bf16 form does not use the epilogue scratch either
        if (!fused && !fp8) cfg.smem -= 7168;
        const size_t per_stage = (size_t)cfg.tile_rows * kBK * 2 + (size_t)cfg.bn * kBK * 2 + 16;
        while (cfg.n_stages > 3 && cfg.smem > (size_t)x->smem_cap) {
            --cfg.n_stages;
            cfg.smem -= per_stage;
        }
    }
    p.wide = cfg.wide;
    p.tile_rows = cfg.tile_rows;
    int tiles = 0, col = 0;
    for (int i = 0; i < nseg; ++i) {
        if (!segs[i].map) return WD_ERR_NULL;
        p.seg_tile0[i] = tiles;
        p.seg_n[i] = segs[i].n;
        p.seg_col[i] = col;
        tiles += (segs[i].n + cfg.tile_rows - 1) / cfg.tile_rows;
        col += segs[i].n;
    }
    p.seg_tile0[nseg] = tiles;
    p.nseg = nseg;
    p.ncol = col;
    p.rows = rows; p.bn = cfg.bn;
    p.kb_total = (K + kke - 1) / kke;
    p.tok_tiles = cfg.tok_tiles;
    // Two or four token tiles: one group of CTAs per token tile, all groups walking the same line of
    // weight K blocks in step, so a weight block comes from HBM once and from L2 for the other groups
    // (with one line over (weight tile, token tile) units the second visit came a whole pass later,
    // after the block had left the L2: DRAM traffic was twice the weight bytes)
    const int slots = sm_count * cfg.ctas_per_sm;
    const bool lm = fuse && fuse->mode == WD_FUSE_LMSTATS;
    const int ts = ((!fused || lm) && !cfg.wide && (cfg.tok_tiles == 2 || cfg.tok_tiles == 4) && slots % cfg.tok_tiles == 0)
                       ? cfg.tok_tiles : 1;
    p.tok_split = ts;
    p.n_units = ts > 1 ? tiles : tiles * cfg.tok_tiles;
    p.W = (long long)p.n_units * p.kb_total;
    p.n_stages = cfg.n_stages;
    p.buf_cols = cfg.buf_cols;
    // (trace builds) q/k/v, o, gate/up, down of a block by their shape; everything else in slot 4
    p.trace_slot = nseg == 3 ? 0 : (nseg == 2 ? 2 : (lm ? 4 : (K == col ? 1 : (K > col ? 3 : 4))));
    const size_t slice = (size_t)rows * col;
    if (slice > y_floats) return WD_ERR_CAPACITY;
    // stream-K over all SMs when the partial sums fit, whole tiles per CTA otherwise
    // (G = CTAs per token group)
    long long G = (long long)slots / ts;
    if (G > p.W / 2) G = p.W / 2 > 0 ? p.W / 2 : 1;           // at least two K blocks per CTA
    int n_slices = count_slices(p.n_units, p.kb_total, p.W, G);
    p.aligned = 0;
    if (force_single_split || (size_t)n_slices * slice > y_floats || n_slices > WD_TC_MAX_SPLIT) {
        p.aligned = 1;
        n_slices = 1;
        G = (long long)slots / ts;
        if (G > p.n_units) G = p.n_units;
    }
    p.n_slices = n_slices;
    p.y = y;
    p.split_stride = slice;
    p.status = status;
    p.idesc = make_idesc(cfg.bn, kBM, fp8 != nullptr);
    if (fuse) {
        p.f = *fuse;
        if (fuse->mode != WD_FUSE_NONE && fuse->mode != WD_FUSE_LMSTATS && !fuse->counters) return WD_ERR_NULL;
        if (fuse->mode == WD_FUSE_LMSTATS && (!p.aligned || cfg.wide || cfg.tok_tiles != ts || nseg != 1 || !fuse->st_max ||
                                              !fuse->st_idx || !fuse->st_sum))
            return WD_ERR_BAD_PARAM;
        fuse->n_chunks = (int)G;          // one statistics entry per (row, CTA)
        if (fuse->mode == WD_FUSE_SWIGLU && (nseg != 2 || segs[0].n != segs[1].n)) return WD_ERR_BAD_PARAM;
        if (fuse->mode != WD_FUSE_NONE && fuse->mode != WD_FUSE_LMSTATS && col % kBM) return WD_ERR_BAD_PARAM;   // whole tiles only
    }

    CUtensorMap mx;
    bool hit = false;
    for (const WdTcX::Entry& e : x->cache)
        if (e.rows == rows && e.bn == cfg.bn) { mx = e.map; hit = true; break; }
    if (!hit) {
        wd_status s = fp8 ? encode_2d8(&mx, x->ptr, rows, K, cfg.bn) : encode_2d(&mx, x->ptr, rows, K, cfg.bn);
        if (s != WD_OK) return s;
        if (x->keep) {
            if (x->cache.size() >= 16) x->cache.erase(x->cache.begin());
            x->cache.push_back({rows, cfg.bn, mx});
        }
    }
    static bool attr_done[64] = {};     // set once per device
    const int dev = current_device();
    if (dev < 0) return WD_ERR_CUDA;
    if (!attr_done[dev]) {
        WD_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
        WD_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
        WD_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
        WD_CUDA_TRY(cudaFuncSetAttribute((gemm_tc_kernel<false, false, true>), cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
        WD_CUDA_TRY(cudaFuncSetAttribute((gemm_tc_kernel<false, true, true>), cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
        attr_done[dev] = true;
    }
    const CUtensorMap& m0 = *segs[0].map;
    const CUtensorMap& m1 = *segs[nseg > 1 ? 1 : 0].map;
    const CUtensorMap& m2 = *segs[nseg > 2 ? 2 : 0].map;
    ++wd_launch_counter;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)(G * ts));
    lc.blockDim = dim3(cfg.wide ? kThreadsWide : kThreads);
    lc.dynamicSmemBytes = cfg.smem;
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = wd_pdl_enabled ? 1 : 0;
    if (fp8 && p.f.mode == WD_FUSE_LMSTATS) WD_CUDA_TRY(cudaLaunchKernelEx(&lc, (gemm_tc_kernel<false, true, true>), mx, m0, m1, m2, p));
    else if (fp8) WD_CUDA_TRY(cudaLaunchKernelEx(&lc, (gemm_tc_kernel<false, false, true>), mx, m0, m1, m2, p));
    else if (cfg.wide) WD_CUDA_TRY(cudaLaunchKernelEx(&lc, gemm_tc_kernel<true, false>, mx, m0, m1, m2, p));
    else if (p.f.mode == WD_FUSE_LMSTATS) WD_CUDA_TRY(cudaLaunchKernelEx(&lc, gemm_tc_kernel<false, true>, mx, m0, m1, m2, p));
    else WD_CUDA_TRY(cudaLaunchKernelEx(&lc, gemm_tc_kernel<false, false>, mx, m0, m1, m2, p));
    if (n_split_out) *n_split_out = p.n_slices;
    return WD_OK;
}

// ---- chain launch -------------------------------------------------------------------------
bool wd_tc_chain_rows_ok(int rows) { return rows >= 1 && rows <= 256; }

wd_status wd_tc_chain(const WdTcChainItem* items, int n, int rows, float* y, size_t y_floats, int sm_count,
                      int32_t* status, WdTcChainState* cs, cudaStream_t stream) {
    if (!items || !y || !status || !cs || !cs->ready_dev) return WD_ERR_NULL;
    if (n < 1 || n > kChainMax || !wd_tc_chain_rows_ok(rows)) return WD_ERR_BAD_PARAM;
    const TcConfig cfg = pick_config(rows, false, false);
    if (cfg.tok_tiles != 1 || cfg.ctas_per_sm != 1) return WD_ERR_BAD_PARAM;
    static ChainParams cp;              // large: kept off the stack (host threads do not step one context concurrently)
    static ChainMaps maps;
    memset(&cp, 0, sizeof(cp));
    cp.n_gemm = n;
    cp.ready = cs->ready_dev;
    const long long G = sm_count;
    int32_t add[kChainMax] = {0, 0, 0, 0};
    for (int g = 0; g < n; ++g) {
        const WdTcChainItem& it = items[g];
        if (!it.x || !it.segs || it.nseg < 1 || it.nseg > 3 || it.K < 8 || it.K % 8) return WD_ERR_BAD_PARAM;
        const int mode = it.fuse.mode;
        if (mode != WD_FUSE_QKV && mode != WD_FUSE_RESID && mode != WD_FUSE_SWIGLU) return WD_ERR_BAD_PARAM;
        if (!it.fuse.counters) return WD_ERR_NULL;
        TcParams& p = cp.g[g];
        p.tile_rows = kBM;
        int tiles = 0, col = 0;
        for (int i = 0; i < it.nseg; ++i) {
            if (!it.segs[i].map || it.segs[i].n % kBM) return WD_ERR_BAD_PARAM;      // whole tiles only
            p.seg_tile0[i] = tiles;
            p.seg_n[i] = it.segs[i].n;
            p.seg_col[i] = col;
            tiles += it.segs[i].n / kBM;
            col += it.segs[i].n;
            maps.w[g][i] = *it.segs[i].map;
        }
        for (int i = it.nseg; i < 3; ++i) maps.w[g][i] = *it.segs[0].map;
        if (mode == WD_FUSE_SWIGLU && (it.nseg != 2 || it.segs[0].n != it.segs[1].n)) return WD_ERR_BAD_PARAM;
        p.seg_tile0[it.nseg] = tiles;
        p.nseg = it.nseg;
        p.ncol = col;
        p.rows = rows;
        p.bn = cfg.bn;
        p.kb_total = (it.K + kBK - 1) / kBK;
        p.tok_tiles = 1;
        p.tok_split = 1;
        p.n_units = tiles;
        p.W = (long long)tiles * p.kb_total;
        p.n_stages = cfg.n_stages;
        p.buf_cols = cfg.buf_cols;
        if (G > p.W / 2) return WD_ERR_BAD_PARAM;                  // at least two K blocks per CTA and GEMM
        const size_t slice = (size_t)rows * col;
        const int n_slices = count_slices(p.n_units, p.kb_total, p.W, G);
        if ((size_t)n_slices * slice > y_floats || n_slices > WD_TC_MAX_SPLIT) return WD_ERR_CAPACITY;
        p.n_slices = n_slices;
        p.y = y;
        p.split_stride = slice;
        p.status = status;
        p.idesc = make_idesc(cfg.bn, kBM, false);
        p.f = it.fuse;
        // one count per finished tile (gate and up tile of the same columns finish together)
        add[g] = mode == WD_FUSE_SWIGLU ? p.seg_tile0[1] : tiles;
        bool hit = false;
        for (const WdTcX::Entry& e : it.x->cache)
            if (e.rows == rows && e.bn == cfg.bn) { maps.x[g] = e.map; hit = true; break; }
        if (!hit) {
            wd_status s = encode_2d(&maps.x[g], it.x->ptr, rows, it.K, cfg.bn);
            if (s != WD_OK) return s;
            if (it.x->keep) {
                if (it.x->cache.size() >= 16) it.x->cache.erase(it.x->cache.begin());
                it.x->cache.push_back({rows, cfg.bn, maps.x[g]});
            }
        }
    }
    for (int g = n; g < kChainMax; ++g) {
        maps.x[g] = maps.x[0];
        for (int i = 0; i < 3; ++i) maps.w[g][i] = maps.w[0][0];
    }
    for (int g = 0; g < n; ++g) {
        cs->ready_host[g] = (int32_t)((uint32_t)cs->ready_host[g] + (uint32_t)add[g]);     // wraps; the kernel compares differences
        cp.target[g] = cs->ready_host[g];
    }
    static bool attr_done[64] = {};
    const int dev = current_device();
    if (dev < 0) return WD_ERR_CUDA;
    if (!attr_done[dev]) {
        WD_CUDA_TRY(cudaFuncSetAttribute(gemm_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
        attr_done[dev] = true;
    }
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
    WD_CUDA_TRY(cudaLaunchKernelEx(&lc, gemm_chain_kernel, maps, cp));
    return WD_OK;
}

void wd_launch_reduce_slices(const float* part, int n_split, size_t stride, float* y, size_t total, cudaStream_t st) {
    const int blocks = (int)((total + 255) / 256 < 1184 ? (total + 255) / 256 : 1184);
    ++wd_launch_counter;
    reduce_slices_kernel<<<blocks, 256, 0, st>>>(part, n_split, stride, y, total);
}

wd_status wd_tc_encode_fp8(CUtensorMap* m, const void* ptr, int n_rows, int K, int box_rows) {
    return encode_2d8(m, ptr, n_rows, K, box_rows);
}

wd_status wd_tc_encode_bf16(CUtensorMap* m, const void* ptr, int n_rows, int K, int box_rows) {
    return encode_2d(m, ptr, n_rows, K, box_rows);
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
    WdTcX xm;
    xm.ptr = x; xm.K = k_in; xm.keep = false;
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

// FP8 single operation: operands already quantised (codes + row scales); slices: room for the partial sums
wd_status wd_tc_gemm_standalone_fp8(const uint8_t* xq, const float* sx, const uint8_t* wq, const float* sw, float* y,
                                    int rows, int n_out, int k_in, float* slices, size_t slice_floats, cudaStream_t stream) {
    if (k_in % 16) return WD_ERR_BAD_PARAM;
    int32_t* status = wd_op_status_ptr();
    if (!status) return WD_ERR_CUDA;
    CUtensorMap mw;
    wd_status s = encode_2d8(&mw, wq, n_out, k_in, kBM);
    if (s != WD_OK) return s;
    WdTcSeg seg = {wq, n_out, &mw};
    WdTcX xm;
    xm.ptr = xq; xm.K = k_in; xm.fp8 = 1; xm.keep = false;
    WdTcFp8 f8;
    f8.sw[0] = sw; f8.sx = sx;
    int sm = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev);
    const size_t slice = (size_t)rows * n_out;
    if (slice_floats < slice) return WD_ERR_WORKSPACE_TOO_SMALL;
    int ns = 1;
    s = wd_tc_gemm(&xm, &seg, 1, rows, k_in, slices, slice_floats, sm, status, stream, &ns, false, nullptr, &f8);
    if (s != WD_OK) return s;
    const int blocks = (int)((slice + 255) / 256 < 1184 ? (slice + 255) / 256 : 1184);
    ++wd_launch_counter;
    reduce_slices_kernel<<<blocks, 256, 0, stream>>>(slices, ns, slice, y, slice);
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
    WdTcX xm;                       // one-off operand: its descriptor is encoded on the stack (no host allocation)
    xm.ptr = x; xm.K = k_in; xm.keep = false;
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
