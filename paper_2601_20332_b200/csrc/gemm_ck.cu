// Few-token weight-streaming GEMM whose epilogue does the consumer's work (sm_100a).
//
//   y[tok, n] = sum_k x[tok, k] * w[n, k]        x: [rows <= 128, K] bf16, w: [n, K] bf16
//
// In a normal step of the windowed method only the active tokens and a few recently decoded ones
// are computed (Section 4.3 of the paper), so every projection is bound by reading its weights
// once, and what follows a projection (RoPE and the K/V cache write of Section 4.3's cache-write
// equation, the residual add, SwiGLU) touches a few hundred KB.  As separate kernels those
// consumers cost more than the bytes they move: each sits on the dependency chain between two
// weight streams.  Here the split-K partial tiles never leave the chip:
//
//   * a thread-block cluster of 4 CTAs owns one [128 weight rows x BN tokens] output tile at a time;
//     CTA r of the cluster streams the r-th quarter of the tile's K blocks (TMA ring, tcgen05.mma,
//     accumulator in tensor memory), so all SMs stream weights whatever the number of tiles;
//   * each CTA then sends every token column of its partial tile to the CTA that owns that token
//     (token t belongs to CTA t mod 4) with plain stores into the owner's shared memory
//     (distributed shared memory), and tells the owners with a remote mbarrier arrive;
//   * the owner adds the four partial columns in a fixed order (deterministic) and finishes them:
//       QKV     scale by 1/rms (the GEMM input is bf16(x * gain), not yet normalised), rotate q and k
//               at the row's absolute position, write q and the K / transposed-V cache rows;
//       RESID   x += tile; xg = bf16(x * next gain) for the next GEMM; per-row sum of squares of the
//               tile's 128 columns (the next GEMM's owners turn the sums into 1/rms);
//       SWIGLU  gate tile j and up tile j go to the same cluster one after the other; the owners keep the
//               gate sums in registers and write h = silu(g) * u as bf16 when the up tile arrives.
//   Clusters take tiles round-robin; accumulators are double-buffered so the MMAs of the next tile
//   run while this one is being sent and reduced.
//   * An SM takes in about 32 bytes per clock (63 GB/s) whatever the source, and with few tokens the
//     activation tile of a K block is a quarter of the weight tile's bytes.  A CTA's K range is the same
//     for all of its tiles, so when its activation slice fits (tokens x K / 4 x 2 bytes <= 96 KB) it is
//     loaded once and stays in shared memory; the ring then carries weights only.
//
// Every wait is bounded (two seconds); on expiry the CTA records WD_ERR_DEVICE_TIMEOUT, stops working
// and goes to the closing cluster barrier, which every thread reaches on every path.
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "gemm_tc.h"
#include "device_utils.cuh"

namespace {

using namespace wdk;

constexpr int kBM = 128;              // weight rows per tile (MMA M)
constexpr int kBK = 64;               // K elements per stage: one 128-byte swizzle row
constexpr int kStageW = kBM * kBK * 2;
constexpr int kCS = 4;                // CTAs per cluster = K slices per tile
constexpr int kThreads = 192;         // TMA warp, MMA warp, 4 epilogue warps
constexpr int kMaxGrp = 8;            // most groups of 4 token slots per owner: 128 tokens / 16

struct CkParams {
    int rows, bn, kb_total, n_units, n_stages, acc_cols, nsub, pitch;
    int xres;                         // 1: the CTA's activation slice stays in shared memory (loaded once)
    int nseg;
    int seg_tile0[4];                 // first unit of each weight matrix (+ end)
    int seg_col[3];                   // first output column of each weight matrix
    int batch;
    uint32_t idesc;
    int32_t* status;
    WdTcFuse f;
};

__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// 16 bytes into another CTA's shared memory; the store counts its bytes on the mbarrier `bar` of that same CTA
// (both shared::cluster addresses), so the receiver needs no fence and no separate arrival from the sender
__device__ __forceinline__ void st_async_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
                 ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d), "r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster_relaxed(uint32_t cluster_bar) {
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
// bounded wait whose success makes the other CTAs' stores (released at cluster scope) visible
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    unsigned long long t0 = 0;
    for (uint32_t it = 0; it < kWaitLimit; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n.reg .pred p;\n"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n"
            "selp.u32 %0, 1, 0, p;\n}\n"
            : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
        if (it >= 128) {
            __nanosleep(64);
            if ((it & 255) == 0) {
                if (*abort_flag) return false;
                const unsigned long long now = global_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > kWaitNs) return false;
            }
        }
    }
    return false;
}
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
// unit -> weight matrix and first weight row.  SWIGLU: units alternate gate tile j (matrix 0), up tile j (matrix 1).
template <int kMode>
__device__ __forceinline__ void decode_unit(const CkParams& p, int unit, int& seg, int& n0) {
    if (kMode == WD_FUSE_SWIGLU) {
        seg = unit & 1;
        n0 = (unit >> 1) * kBM;
        return;
    }
    seg = 0;
    if (p.nseg > 1 && unit >= p.seg_tile0[1]) seg = 1;
    if (p.nseg > 2 && unit >= p.seg_tile0[2]) seg = 2;
    n0 = (unit - p.seg_tile0[seg]) * kBM;
}

#ifdef WD_CK_TRACE
// development aid (not compiled by default): globaltimer stamps of the last launch of every mode
__device__ unsigned long long g_ck_trace[4][160][32];
#define CK_STAMP(slot) do { if ((slot) < 32) g_ck_trace[kMode][blockIdx.x < 160 ? blockIdx.x : 159][(slot)] = global_ns(); } while (0)
#else
#define CK_STAMP(slot) do { } while (0)
#endif

template <int kMode>
__global__ void __launch_bounds__(kThreads, 1)
gemm_ck_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w0,
               const __grid_constant__ CUtensorMap map_w1, const __grid_constant__ CUtensorMap map_w2, const CkParams p) {
    extern __shared__ uint8_t smem_raw[];
    // the same offsets in every CTA of the cluster (the dynamic window starts at the same address)
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int NS = p.n_stages;
    const int x_bytes = p.bn * kBK * 2;                           // activation tile of one K block
    const int stage_bytes = kStageW + (p.xres ? 0 : x_bytes);
    const int pitch = p.pitch;                                    // token slots per owner (bn / 4), padded so that pitch / 4 is odd
    const int kb_max = (p.kb_total + kCS - 1) / kCS;              // most K blocks of a CTA
    uint8_t* xres = smem + (size_t)NS * stage_bytes;              // [kb_max][bn x 64] resident activation slice (xres only)
    float* red = (float*)(xres + (p.xres ? (size_t)kb_max * x_bytes : 0));   // [source CTA][128 columns][pitch]
    uint64_t* bars = (uint64_t*)(red + (size_t)kCS * kBM * pitch);
    // bars: [0, NS) full | [NS, 2NS) empty | 2NS, 2NS+1 accumulator full | 2NS+2, 2NS+3 accumulator empty |
    //       2NS+4 partial tiles of all four CTAs are in this CTA's buffer | 2NS+5 all four owners have read what this CTA sent |
    //       [2NS+6, 2NS+6+kb_max) resident activation tile of a K block has landed (xres only)
    uint64_t* red_full = bars + 2 * NS + 4;
    uint64_t* red_empty = bars + 2 * NS + 5;
    uint64_t* x_full = bars + 2 * NS + 6;
    uint32_t* tmem_slot = (uint32_t*)(x_full + (p.xres ? kb_max : 0));
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
    float* inv_s = (float*)(tmem_slot + 2);                       // [32] 1/rms of the owned tokens
    int* pos_s = (int*)(inv_s + 32);                              // [32] their positions
    int* seq_s = pos_s + 32;                                      // [32] their sequences
    float* ss_s = (float*)(seq_s + 32);                           // [4 warps][32] partial sums of squares

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int cluster_id = blockIdx.x / kCS, n_clusters = gridDim.x / kCS;
    // units come in groups of nsub (SWIGLU: gate tile, up tile) that stay together; groups are dealt round-robin
    const int n_groups = p.n_units / p.nsub;
    const int n_my = (cluster_id < n_groups ? (n_groups - cluster_id + n_clusters - 1) / n_clusters : 0) * p.nsub;
    const int kb_begin = (int)rank * p.kb_total / kCS, kb_len = ((int)rank + 1) * p.kb_total / kCS - kb_begin;
    const int n_total = n_my * kb_len;                            // stages this CTA streams
    // local unit u -> global unit
    auto unit_of = [&](int u) { return (cluster_id + (u / p.nsub) * n_clusters) * p.nsub + u % p.nsub; };

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        CK_STAMP(0);
        for (int s = 0; s < NS; ++s) {
            mbar_init(smem_u32(&bars[s]), 1);
            mbar_init(smem_u32(&bars[NS + s]), 1);
        }
        mbar_init(smem_u32(&bars[2 * NS]), 1);
        mbar_init(smem_u32(&bars[2 * NS + 1]), 1);
        mbar_init(smem_u32(&bars[2 * NS + 2]), 128);
        mbar_init(smem_u32(&bars[2 * NS + 3]), 128);
        mbar_init(smem_u32(red_full), 1);              // the owner's own expect_tx arrival; the data counts as bytes
        mbar_init(smem_u32(red_empty), kCS);           // one arrival per owner
        if (p.xres)
            for (int j = 0; j < kb_max; ++j) mbar_init(smem_u32(&x_full[j]), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w0) : "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 2u * (uint32_t)p.acc_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // Nobody may arrive on, or store into, another CTA before that CTA's barriers exist: arrive now,
    // wait where the first remote operation (or the end of the kernel) comes.
    cluster_arrive();

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        struct Walk { int u, left, kb, n0; const CUtensorMap* mw; };
        auto enter = [&](Walk& w) {                       // first K block of local unit w.u
            int seg, n0;
            decode_unit<kMode>(p, unit_of(w.u), seg, n0);
            w.n0 = n0;
            w.kb = kb_begin;
            w.left = kb_len;
            w.mw = seg == 0 ? &map_w0 : (seg == 1 ? &map_w1 : &map_w2);
        };
        auto advance = [&](Walk& w) {
            ++w.kb;
            if (--w.left == 0 && ++w.u < n_my) enter(w);
        };
        Walk w, wx;
        const int n_pre = n_total < NS ? n_total : NS;
        uint64_t pol_stream = 0;
        if (lane == 0 && n_total > 0) {
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            w.u = 0;
            enter(w);
            wx = w;
            // weights never depend on earlier kernels of the stream: fill the ring with them first
            for (int i = 0; i < n_pre; ++i, advance(w)) {
                mbar_expect_tx(smem_u32(&bars[i]), (uint32_t)stage_bytes);
                tma_load_2d_hint(smem_u32(smem + (size_t)i * stage_bytes), w.mw, smem_u32(&bars[i]), w.kb * kBK, w.n0, pol_stream);
            }
        }
        if (lane == 0) CK_STAMP(1);
        __syncwarp();
        cluster_wait();
        if (lane == 0) CK_STAMP(2);
        if (lane == 0 && n_total > 0) {
            pdl_wait();                                   // the activations come from the previous kernel
            CK_STAMP(3);
            if (p.xres) {
                // the whole slice, in the order the MMAs need it; every tile has its own barrier
                for (int j = 0; j < kb_len; ++j) {
                    mbar_expect_tx(smem_u32(&x_full[j]), (uint32_t)x_bytes);
                    tma_load_2d(smem_u32(xres + (size_t)j * x_bytes), &map_x, smem_u32(&x_full[j]), (kb_begin + j) * kBK, 0);
                }
            } else {
                for (int i = 0; i < n_pre; ++i, advance(wx))
                    tma_load_2d(smem_u32(smem + (size_t)i * stage_bytes) + kStageW, &map_x, smem_u32(&bars[i]), wx.kb * kBK, 0);
            }
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
                if (!p.xres) tma_load_2d(sa + kStageW, &map_x, full, w.kb * kBK, 0);
                if (++s == NS) { s = 0; ph ^= 1u; }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        cluster_wait();
        if (lane == 0) {
            bool ok = true;
            int s = 0;
            uint32_t ph = 0;
            for (int u = 0; u < n_my && ok; ++u) {
                const int buf = u & 1;
                const uint32_t par = (uint32_t)(u >> 1) & 1u;
                if (!(ok = mbar_wait(smem_u32(&bars[2 * NS + 2 + buf]), par ^ 1u, abort_flag))) break;   // accumulators drained
                tc_fence_after();
                const uint32_t acc = tmem_base + (uint32_t)(buf * p.acc_cols);
                for (int j = 0; j < kb_len; ++j) {
                    if (!(ok = mbar_wait(smem_u32(&bars[s]), ph, abort_flag))) break;
                    // resident activations: tile j landed during the first unit (the wait returns at once afterwards)
                    if (p.xres && !(ok = mbar_wait(smem_u32(&x_full[j]), 0u, abort_flag))) break;
                    if (u == 0 && j == 0) CK_STAMP(4);
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
                    const uint64_t adesc = make_sdesc(sa);
                    const uint64_t bdesc = make_sdesc(p.xres ? smem_u32(xres + (size_t)j * x_bytes) : sa + kStageW);
#pragma unroll
                    for (int kk = 0; kk < kBK / 16; ++kk)
                        umma_bf16(acc, adesc + (uint64_t)(2 * kk), bdesc + (uint64_t)(2 * kk), p.idesc, (j > 0 || kk > 0) ? 1u : 0u);
                    umma_commit(smem_u32(&bars[NS + s]));              // stage free once these MMAs have read it
                    if (++s == NS) { s = 0; ph ^= 1u; }
                }
                if (ok) umma_commit(smem_u32(&bars[2 * NS + buf]));     // this unit's accumulators complete
                CK_STAMP(5 + u * 4);
            }
            if (!ok) {
                *abort_flag = 1;
                atomicCAS(p.status, 0, WD_ERR_DEVICE_TIMEOUT);
            }
        }
        __syncwarp();
    } else {
        // ---------------------------------------------------------------- epilogue (warps 2..5)
        const int quarter = warp & 3;                      // TMEM lanes 32 * quarter .. + 31
        const int n_local = quarter * 32 + lane;           // source side: the weight row (output column) this thread drains
        const int e = (int)threadIdx.x - 64;               // owner side: see the modes below
        const int n_chunks = (p.rows + 15) >> 4;           // 16-token chunks that hold a valid token
        const int n_grp = n_chunks;                        // groups of 4 token slots per owner (one per chunk)
        // bytes every owner receives per unit: 4 sources x 128 columns x 4 slots per chunk x 4 bytes
        const uint32_t tx_bytes = (uint32_t)(kCS * kBM * 4 * n_chunks * 4);
        cluster_wait();
        pdl_wait();                                        // x, sums of squares, index lists: previous kernels
        if (e == 0 && n_my > 0) mbar_expect_tx(smem_u32(red_full), tx_bytes);     // unit 0's partial tiles
        uint32_t red_remote[kCS], full_remote[kCS];
#pragma unroll
        for (int o = 0; o < kCS; ++o) {
            red_remote[o] = cluster_map(smem_u32(red), (uint32_t)o);
            full_remote[o] = cluster_map(smem_u32(red_full), (uint32_t)o);
        }
        // per owned token slot tl (token tl * 4 + rank), the same for every unit: 1 / rms, position, sequence
        for (int tl = warp - 2; tl < 4 * n_grp; tl += 4) {
            const int tok = tl * kCS + (int)rank;
            if (kMode != WD_FUSE_RESID) {
                float ss = 0.f;
                if (tok < p.rows)
                    for (int j = lane; j < p.f.n_prev_tiles; j += 32) ss += __ldcg(p.f.sumsq_in + (size_t)j * p.f.rows_total + tok);
                ss = warp_sum_f(ss);
                if (lane == 0) inv_s[tl] = tok < p.rows ? rsqrtf(ss * p.f.inv_d + p.f.eps) : 0.f;
            }
            if (kMode == WD_FUSE_QKV && lane == 0) {
                pos_s[tl] = tok < p.rows ? p.f.row_pos[tok] : -1;
                seq_s[tl] = tok < p.rows ? p.f.row_seq[tok] : -1;
            }
        }
        // QKV: thread = (column pair (n, n + 64), half of the token groups); its rotation factors for every token it handles
        const int qn = e & 63, qh = e >> 6;
        float2 cs[kMaxGrp / 2][4];
        if (kMode == WD_FUSE_QKV) {
#pragma unroll
            for (int gi = 0; gi < kMaxGrp / 2; ++gi)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int g = qh + 2 * gi, tok = (4 * g + j) * kCS + (int)rank;
                    cs[gi][j] = (g < n_grp && tok < p.rows) ? p.f.rope_tab[(size_t)tok * 64 + qn] : make_float2(1.f, 0.f);
                }
        }
        epi_sync();
        float gate[kMaxGrp][4];                            // SWIGLU: the gate tile's sums, until the up tile arrives
#pragma unroll
        for (int g = 0; g < kMaxGrp; ++g)
#pragma unroll
            for (int j = 0; j < 4; ++j) gate[g][j] = 0.f;
        bool ok = true;
        for (int u = 0; u < n_my; ++u) {
            int seg, n0;
            decode_unit<kMode>(p, unit_of(u), seg, n0);
            const int buf = u & 1;
            const uint32_t par = (uint32_t)(u >> 1) & 1u;
            // RESID: this unit's x values (thread = column e), asked for before the waits
            float xv[kMaxGrp][4];
            float gain = 0.f;
            if (kMode == WD_FUSE_RESID) {
#pragma unroll
                for (int g = 0; g < kMaxGrp; ++g)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int tok = (4 * g + j) * kCS + (int)rank;
                        xv[g][j] = (g < n_grp && tok < p.rows) ? p.f.x[(size_t)tok * p.f.F + n0 + e] : 0.f;
                    }
                if (p.f.gain_next) gain = p.f.gain_next[n0 + e];
            }
            // every owner has read what this CTA sent for the previous unit
            if (u > 0) ok = ok && mbar_wait_cluster(smem_u32(red_empty), (uint32_t)(u - 1) & 1u, abort_flag);
            ok = ok && mbar_wait(smem_u32(&bars[2 * NS + buf]), par, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (threadIdx.x == 64) CK_STAMP(5 + u * 4 + 1);
            tc_fence_after();
            // ---- send: of the 16 tokens of a chunk, tokens o, o + 4, o + 8, o + 12 go to CTA o as one 16-byte
            // store into its buffer [source][column][slot]; the store itself counts on the owner's barrier
            {
                const uint32_t t_acc = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * p.acc_cols);
                const uint32_t off = (uint32_t)((((int)rank) * kBM + n_local) * pitch) * 4u;
                for (int c = 0; c < n_chunks; ++c) {
                    uint32_t v[16];
                    tmem_ld16(t_acc + (uint32_t)(16 * c), v);
#pragma unroll
                    for (int o = 0; o < kCS; ++o)
                        st_async_v4(red_remote[o] + off + (uint32_t)(16 * c), v[o], v[o + 4], v[o + 8], v[o + 12], full_remote[o]);
                }
            }
            tc_fence_before();
            mbar_arrive(smem_u32(&bars[2 * NS + 2 + buf]));           // accumulators may be overwritten
            if (threadIdx.x == 64) CK_STAMP(5 + u * 4 + 2);
            // ---- own: the four partial columns of this CTA's tokens are here
            ok = mbar_wait_cluster(smem_u32(red_full), (uint32_t)u & 1u, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (threadIdx.x == 64 && u == 0) CK_STAMP(23);
            if (kMode == WD_FUSE_QKV) {
                const int head = (p.seg_col[seg] + n0) >> 7;            // among the q | k | v heads
#pragma unroll
                for (int gi = 0; gi < kMaxGrp / 2; ++gi) {
                    const int g = qh + 2 * gi;
                    if (g >= n_grp) break;
                    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
#pragma unroll
                    for (int src = 0; src < kCS; ++src) {
                        const float4 pa = *reinterpret_cast<const float4*>(red + (size_t)(src * kBM + qn) * pitch + 4 * g);
                        const float4 pb = *reinterpret_cast<const float4*>(red + (size_t)(src * kBM + qn + 64) * pitch + 4 * g);
                        a.x += pa.x; a.y += pa.y; a.z += pa.z; a.w += pa.w;
                        b.x += pb.x; b.y += pb.y; b.z += pb.z; b.w += pb.w;
                    }
                    const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int tl = 4 * g + j, tok = tl * kCS + (int)rank;
                        if (tok >= p.rows) break;
                        const float inv = inv_s[tl];
                        const float x0 = av[j] * inv, x1 = bv[j] * inv;
                        const int pos = pos_s[tl], sq = seq_s[tl];
                        if (head >= p.f.Hq && !((unsigned)pos < (unsigned)p.f.S && (unsigned)sq < (unsigned)p.batch)) {
                            if (qn == 0) atomicCAS(p.status, 0, WD_ERR_BOUNDS);      // index check: recorded, no cache row written
                            continue;
                        }
                        if (head < p.f.Hq + p.f.Hkv) {
                            const float2 c2 = cs[gi][j];
                            __nv_bfloat16* dst = head < p.f.Hq
                                ? p.f.q + ((size_t)tok * p.f.Hq + head) * 128
                                : p.f.kcache + (((size_t)sq * p.f.Hkv + (head - p.f.Hq)) * p.f.S + pos) * 128;
                            dst[qn] = __float2bfloat16_rn(x0 * c2.x - x1 * c2.y);
                            dst[qn + 64] = __float2bfloat16_rn(x1 * c2.x + x0 * c2.y);
                        } else {
                            __nv_bfloat16* dst = p.f.vcache + ((size_t)sq * p.f.Hkv + (head - p.f.Hq - p.f.Hkv)) * 128 * p.f.Sp + pos;
                            dst[(size_t)qn * p.f.Sp] = __float2bfloat16_rn(x0);
                            dst[(size_t)(qn + 64) * p.f.Sp] = __float2bfloat16_rn(x1);
                        }
                    }
                }
            } else if (kMode == WD_FUSE_RESID) {
                // thread = column e; per token the sum of squares over the tile's 128 columns goes through shared memory
#pragma unroll
                for (int g = 0; g < kMaxGrp; ++g) {
                    if (g >= n_grp) break;
                    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int src = 0; src < kCS; ++src) {
                        const float4 pa = *reinterpret_cast<const float4*>(red + (size_t)(src * kBM + e) * pitch + 4 * g);
                        a.x += pa.x; a.y += pa.y; a.z += pa.z; a.w += pa.w;
                    }
                    const float av[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int tl = 4 * g + j, tok = tl * kCS + (int)rank;
                        float sq = 0.f;
                        if (tok < p.rows) {
                            const float v = xv[g][j] + av[j];
                            const size_t o = (size_t)tok * p.f.F + n0 + e;
                            p.f.x[o] = v;
                            if (p.f.gain_next) p.f.xg[o] = __float2bfloat16_rn(v * gain);
                            if (p.f.tap) p.f.tap[o] = v;
                            sq = v * v;
                        }
                        sq = warp_sum_f(sq);
                        if (lane == 0) ss_s[(warp - 2) * 32 + tl] = sq;
                    }
                }
                epi_sync();
                if (e < 4 * n_grp) {
                    const int tok = e * kCS + (int)rank;
                    if (tok < p.rows)
                        p.f.sumsq_out[(size_t)(n0 >> 7) * p.f.rows_total + tok] = (ss_s[e] + ss_s[32 + e]) + (ss_s[64 + e] + ss_s[96 + e]);
                }
            } else {
                // thread = column e.  Gate tile (seg 0): keep silu-ready sums; up tile (seg 1): h = silu(g) * u
#pragma unroll
                for (int g = 0; g < kMaxGrp; ++g) {
                    if (g >= n_grp) break;
                    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int src = 0; src < kCS; ++src) {
                        const float4 pa = *reinterpret_cast<const float4*>(red + (size_t)(src * kBM + e) * pitch + 4 * g);
                        a.x += pa.x; a.y += pa.y; a.z += pa.z; a.w += pa.w;
                    }
                    const float av[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int tl = 4 * g + j, tok = tl * kCS + (int)rank;
                        const float v = av[j] * inv_s[tl];
                        if (seg == 0) gate[g][j] = v;
                        else if (tok < p.rows) {
                            const float gt = gate[g][j];
                            p.f.h[(size_t)tok * p.f.F + n0 + e] = __float2bfloat16_rn(gt / (1.f + __expf(-gt)) * v);
                        }
                    }
                }
            }
            if (threadIdx.x == 64 && u == 0) CK_STAMP(24);
            // ---- the buffer has been read: the sources may send the next unit (nobody waits after the last one)
            if (u + 1 < n_my) {
                epi_sync();                                          // every thread of this CTA has read its part
                if (e == 0) {
                    mbar_expect_tx(smem_u32(red_full), tx_bytes);    // the next unit's partial tiles
                    asm volatile("fence.acq_rel.cluster;" ::: "memory");
#pragma unroll
                    for (int o = 0; o < kCS; ++o) mbar_arrive_cluster_relaxed(cluster_map(smem_u32(red_empty), (uint32_t)o));
                }
            }
            if (threadIdx.x == 64) CK_STAMP(5 + u * 4 + 3);
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
        tmem_dealloc(tmem_base, 2u * (uint32_t)p.acc_cols);
    }
    // no CTA leaves while another may still store into it or arrive on its barriers
    if (threadIdx.x == 0) CK_STAMP(30);
    cluster_arrive();
    cluster_wait();
    if (threadIdx.x == 0) CK_STAMP(31);
}

int env_int(const char* name, int dflt) {
    const char* v = getenv(name);
    return v && *v ? atoi(v) : dflt;
}

uint32_t make_idesc(int bn) {
    uint32_t d = 0;
    d |= 1u << 4;                      // D format: f32
    d |= 1u << 7;                      // A format: bf16
    d |= 1u << 10;                     // B format: bf16
    d |= (uint32_t)(bn >> 3) << 17;    // N
    d |= (uint32_t)(kBM >> 4) << 24;   // M
    return d;
}

// slots per owner and column in the partial-tile buffer: bn / 4, padded so that 16-byte accesses of eight
// neighbouring columns fall into different banks (pitch / 4 odd)
int ck_pitch(int bn) {
    const int tl = bn / kCS;
    return (tl / 4) % 2 ? tl : tl + 4;
}
constexpr int kMinStages = 4;          // a shallower ring does not keep an SM's memory port busy
constexpr int kXresMax = 96 * 1024;    // largest resident activation slice

struct CkLayout { int bn, pitch, xres, kb_max, n_stages; size_t smem; };

// multi: the CTAs get several tiles each (only then does a resident activation slice save anything)
CkLayout ck_layout(int rows, int K, bool multi) {
    CkLayout l;
    l.bn = (rows + 15) / 16 * 16;
    l.pitch = ck_pitch(l.bn);
    l.kb_max = (K / kBK + kCS - 1) / kCS;
    const size_t x_bytes = (size_t)l.bn * kBK * 2;
    static const int xres_on = env_int("WD_CK_XRES", 1);
    l.xres = (xres_on && multi && l.kb_max * x_bytes <= (size_t)kXresMax) ? 1 : 0;
    const size_t fixed = 1024 + (l.xres ? l.kb_max * x_bytes : 0) + (size_t)kCS * kBM * l.pitch * 4 + 2048 + (size_t)l.kb_max * 8;
    const size_t stage = kStageW + (l.xres ? 0 : x_bytes);
    int ns = (int)((227 * 1024 - fixed) / stage);
    if (ns > 12) ns = 12;
    static const int ns_cap = env_int("WD_CK_STAGES", 0);            // tuning knob: fewer ring stages
    if (ns_cap >= 2 && ns_cap < ns) ns = ns_cap;
    l.n_stages = ns;
    l.smem = fixed + (size_t)(ns > 0 ? ns : 0) * stage;
    return l;
}

template <int kMode>
wd_status launch(const CUtensorMap& mx, const CUtensorMap& m0, const CUtensorMap& m1, const CUtensorMap& m2,
                 const CkParams& p, size_t smem, int sm_count, cudaStream_t stream) {
    static bool attr_done[64] = {};
    static int max_clusters[64] = {};
    int dev = 0;
    WD_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return WD_ERR_CUDA;
    cudaLaunchConfig_t lc = {};
    lc.blockDim = dim3(kThreads);
    lc.dynamicSmemBytes = smem;
    lc.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kCS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    if (!attr_done[dev]) {
        WD_CUDA_TRY(cudaFuncSetAttribute(gemm_ck_kernel<kMode>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        // how many clusters of 4 the device holds at one time with one CTA per SM (fewer than SMs / 4
        // when the SM count of a GPC is not a multiple of 4)
        lc.gridDim = dim3((unsigned)(sm_count / kCS * kCS));
        lc.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, gemm_ck_kernel<kMode>, &lc) != cudaSuccess || n < 1) {
            cudaGetLastError();
            n = sm_count / kCS * 3 / 4;
        }
        max_clusters[dev] = n < sm_count / kCS ? n : sm_count / kCS;
        if (getenv("WD_CK_DEBUG")) fprintf(stderr, "gemm_ck mode %d: %d clusters of %d fit (smem %zu, stages %d, resident x %d)\n", kMode, n, kCS, smem, p.n_stages, p.xres);
        attr_done[dev] = true;
    }
    static const int cap = env_int("WD_CK_CLUSTERS", 0);               // tuning knob: 0 = what the device holds
    int n_clusters = max_clusters[dev];
    if (cap > 0 && cap < n_clusters) n_clusters = cap;
    if (n_clusters > p.n_units / p.nsub) n_clusters = p.n_units / p.nsub;
    lc.gridDim = dim3((unsigned)(n_clusters * kCS));
    lc.numAttrs = wd_pdl_enabled ? 2 : 1;
    ++wd_launch_counter;
    WD_CUDA_TRY(cudaLaunchKernelEx(&lc, gemm_ck_kernel<kMode>, mx, m0, m1, m2, p));
    return WD_OK;
}

}  // namespace

int wd_ck_max_rows() {
    int r = 128;
    while (r > 16 && ck_layout(r, 16384, false).n_stages < kMinStages) r -= 16;
    return r;
}

bool wd_ck_usable(int rows, int K, const WdTcSeg* segs, int nseg, const WdTcFuse* fuse) {
    if (!fuse) return false;
    if (fuse->mode != WD_FUSE_QKV && fuse->mode != WD_FUSE_RESID && fuse->mode != WD_FUSE_SWIGLU) return false;
    if (rows < 1 || rows > 128 || K % kBK || K / kBK < kCS) return false;
    for (int i = 0; i < nseg; ++i)
        if (segs[i].n % kBM || !segs[i].map) return false;
    if (fuse->mode == WD_FUSE_SWIGLU && (nseg != 2 || segs[0].n != segs[1].n)) return false;
    if (fuse->mode == WD_FUSE_RESID && nseg != 1) return false;
    if (ck_layout(rows, K, true).n_stages < kMinStages || ck_layout(rows, K, false).n_stages < kMinStages) return false;
    return true;
}

wd_status wd_ck_gemm(const WdTcX* x, const WdTcSeg* segs, int nseg, int rows, int K, int sm_count, int32_t* status,
                     cudaStream_t stream, const WdTcFuse* fuse) {
    if (!x || !segs || !status || !fuse) return WD_ERR_NULL;
    if (!wd_ck_usable(rows, K, segs, nseg, fuse)) return WD_ERR_BAD_PARAM;
    CkParams p;
    memset(&p, 0, sizeof(p));
    p.rows = rows;
    p.bn = (rows + 15) / 16 * 16;
    p.kb_total = K / kBK;
    p.nsub = fuse->mode == WD_FUSE_SWIGLU ? 2 : 1;
    int cols = 32;
    while (cols < p.bn) cols <<= 1;
    p.acc_cols = cols;                                     // two accumulators: 2 * cols <= 256
    int units = 0, col = 0;
    for (int i = 0; i < nseg; ++i) {
        p.seg_tile0[i] = units;
        p.seg_col[i] = col;
        units += segs[i].n / kBM;
        col += segs[i].n;
    }
    p.seg_tile0[nseg] = units;
    p.nseg = nseg;
    p.n_units = units;                                     // SWIGLU: gate and up tiles alternate (see decode_unit)
    p.batch = fuse->batch;
    p.idesc = make_idesc(p.bn);
    p.status = status;
    p.f = *fuse;
    if (fuse->mode == WD_FUSE_RESID) p.f.F = col;          // row pitch of x, xg and the tap
    int dev = 0;
    WD_CUDA_TRY(cudaGetDevice(&dev));
    const int groups = units / p.nsub;
    // several tiles per CTA (then the activation slice is kept resident if it fits)?  Decided on the nominal
    // cluster count; the launch may find that the device holds fewer clusters, which only adds rounds.
    const CkLayout lay = ck_layout(rows, K, groups * p.nsub > sm_count / kCS);
    if (lay.n_stages < kMinStages) return WD_ERR_CAPACITY;
    p.pitch = lay.pitch;
    p.xres = lay.xres;
    p.n_stages = lay.n_stages;
    const size_t smem = lay.smem;

    CUtensorMap mx;
    bool hit = false;
    for (const WdTcX::Entry& e : x->cache)
        if (e.rows == rows && e.bn == p.bn) { mx = e.map; hit = true; break; }
    if (!hit) {
        wd_status s = wd_tc_encode_bf16(&mx, x->ptr, rows, K, p.bn);
        if (s != WD_OK) return s;
        if (x->keep) {
            if (x->cache.size() >= 16) x->cache.erase(x->cache.begin());
            x->cache.push_back({rows, p.bn, mx});
        }
    }
    const CUtensorMap& m0 = *segs[0].map;
    const CUtensorMap& m1 = *segs[nseg > 1 ? 1 : 0].map;
    const CUtensorMap& m2 = *segs[nseg > 2 ? 2 : 0].map;
    if (fuse->mode == WD_FUSE_QKV) return launch<WD_FUSE_QKV>(mx, m0, m1, m2, p, smem, sm_count, stream);
    if (fuse->mode == WD_FUSE_RESID) return launch<WD_FUSE_RESID>(mx, m0, m1, m2, p, smem, sm_count, stream);
    return launch<WD_FUSE_SWIGLU>(mx, m0, m1, m2, p, smem, sm_count, stream);
}

#ifdef WD_CK_TRACE
extern "C" __attribute__((visibility("default"))) int wd_debug_ck_trace(unsigned long long* host /*[4][160][32]*/) {
    cudaDeviceSynchronize();
    return (int)cudaMemcpyFromSymbol(host, g_ck_trace, sizeof(unsigned long long) * 4 * 160 * 32);
}
#endif
