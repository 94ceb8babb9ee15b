// Windowed bidirectional attention on the tensor cores (sm_100a), head_dim 128, bf16.
//
//   out[r, h, :] = softmax_j( q[r,h,:] . K[kvh, j, :] / sqrt(dh) ) V[kvh, j, :],   j in [0, n_vis)
//
// for the rows computed this step.  With a decoded prompt prefix the visible set of a sequence
// is always a range [0, n_vis) (decoded prefix | external window), so K and V tiles are plain
// TMA boxes of the cache; arbitrary index lists go through the CUDA-core kernel instead.
//
// One CTA per (128-row query tile of one sequence, query head):
//   warp 0    TMA: the Q tile once, then [128 keys x 128] K boxes and [128 x 128 keys] boxes of
//             the transposed V cache into a two-stage ring
//   warp 1    tcgen05.mma: S = Q K^T into TMEM, then O_tile = P V into TMEM; software-pipelined:
//             S and O_tile are double-buffered, Q K^T of the next key tile is issued before P V
//             of the current one, so the tensor core works while the softmax threads are busy
//   warps 2-9 two threads per query row (each takes 64 of the tile's 128 columns): tcgen05.ld of
//             its half of the S row, online softmax in fp32 (exp2 with the scale folded in; the
//             two halves exchange their row maxima through shared memory), P as bf16 into shared
//             memory in the 128-byte swizzled operand layout, then tcgen05.ld of its half of the
//             O_tile row accumulated in registers with the running rescale; final O / l as bf16
// Query rows beyond the tile's valid rows are computed on whatever the box holds and discarded
// (rows are independent).  Keys at or beyond n_vis are masked by selection, and their V
// columns are zeroed in shared memory, so stale or poisoned cache rows cannot leak in.
// When there are few (tile, head) pairs, as in a normal step, the keys are also split across
// the CTAs of a thread-block cluster (grid.z = cluster size <= 8) so that the machine is filled:
// each CTA leaves its running maximum, sum and unnormalised output in its own shared memory, and
// after a cluster barrier every CTA merges a share of the rows, reading the other parts through
// distributed shared memory in a fixed order (no global round trip, no atomics).
// Every wait is bounded; on expiry the CTA records WD_ERR_DEVICE_TIMEOUT and leaves.
#include <cstring>

#include <cstdlib>

#include "attention_tc.h"
#include "device_utils.cuh"

namespace {

using namespace wdk;

constexpr int kTile = 128;                 // query rows per CTA = keys per step = head_dim
constexpr int kAtom = kTile * 64 * 2;      // one [128 x 64] bf16 swizzle-atom column: 16 KB
constexpr int kOperand = 2 * kAtom;        // a [128 x 128] bf16 operand: 32 KB
constexpr int kThreads = 320;            // TMA warp, MMA warp, 8 softmax warps
constexpr int kTmemCols = 512;             // S0, S1: columns 0..255; O_tile0, O_tile1: columns 256..511
constexpr int kBars = 21;
constexpr int kMaxCluster = 8;             // portable cluster size

struct AttnParams {
    const int32_t* qtile_seq;    // [n_tiles] sequence of the tile
    const int32_t* qtile_row0;   // [n_tiles] first row (index into the step's row list)
    const int32_t* qtile_n;      // [n_tiles] valid rows
    const int32_t* seq_nvis;     // [batch] visible positions [0, n_vis)
    __nv_bfloat16* out;          // [rows][Hq*dh]
    float* tap;                  // optional fp32 copy
    int Hq, Hkv, layer;
    float scale_log2e;           // log2(e) / sqrt(dh)
    int32_t* status;
    uint32_t idesc;
    // split over the keys: CTA z of (tile, head) takes key tiles [z * tiles_per_split, ...); the
    // max_parts CTAs of a (tile, head) pair form one cluster
    int tiles_per_split, max_parts;
    // head packing (grouped-query attention with few rows): a 128-row query tile holds `pack` slots of `slot`
    // rows, one query head of the same KV head each (slot >= the tile's valid rows); grid.y = Hkv * tiles_per_kv
    int pack, slot, slot_shift, tiles_per_kv;      // slot = 128 / pack = 1 << slot_shift
};

__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t dsmem_addr(uint32_t local, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
    return r;
}
__device__ __forceinline__ float4 dsmem_ld4(uint32_t a) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ float2 dsmem_ld2(uint32_t a) {
    float2 v;
    asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(a));
    return v;
}

// 2^x by the special-function unit alone (x <= 0 here: results in [0, 1], denormals flushed)
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
}

// barrier indices
constexpr int kQFull = 0, kKFull = 1, kKEmpty = 4, kVFull = 7, kVEmpty = 10, kSFull = 13, kPFull = 15, kOFull = 17,
              kOEmpty = 19;
constexpr int kStages = 3;                 // K stages and V stages

// kSingle: every CTA has at most one key tile (few keys, or keys split finely over the cluster): one K and one
// V stage, one S and one O buffer (256 tensor-memory columns), no running rescale — 97 KB of shared memory
// instead of 225 KB and fewer registers, so that the CTAs of the next kernel (the output projection, with a
// ring cut to fit) can be resident beside it and fetch their weights while the attention runs.
#ifdef WD_GEMM_TRACE
__device__ unsigned long long g_attn_end[64];       // latest CTA exit per layer
__device__ unsigned long long g_attn_trace[160][8]; // per CTA (last launch): entry, wait returned, S ready, P written, O ready, part written, merged, exit
#define A_STAMP(k) do { const unsigned int b_ = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z); g_attn_trace[b_ < 160 ? b_ : 159][k] = global_ns(); } while (0)
#else
#define A_STAMP(k) do { } while (0)
#endif

template <bool kSingle>
__device__ __forceinline__ void attention_tc_body(const CUtensorMap& map_q, const CUtensorMap& map_k, const CUtensorMap& map_vt,
                                                  const AttnParams& p) {
    constexpr int NS = kSingle ? 1 : kStages;
    constexpr uint32_t kCols = kSingle ? 256u : (uint32_t)kTmemCols;
    constexpr uint32_t kOBase = kSingle ? (uint32_t)kTile : (uint32_t)(2 * kTile);     // first column of the O buffers
    extern __shared__ uint8_t smem_raw[];
    // the same offset in every CTA of the cluster (the dynamic window starts at the same address)
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sQ = smem;                          // 32 KB
    uint8_t* sK = smem + kOperand;               // 3 stages x 32 KB
    uint8_t* sV = sK + NS * kOperand;       // 3 stages x 32 KB (transposed V tiles)
    uint64_t* bars = (uint64_t*)(sV + NS * kOperand);
    // q_full | k_full[3] | k_empty[3] | v_full[3] | v_empty[3] | s_full[2] | p_full[2] | o_full[2] | o_empty[2].
    // p_full and o_empty count the 256 softmax threads.  p_full is one barrier per S buffer, not one for all
    // tiles: the softmax threads can finish P(i+1) before the MMA thread has looked at P(i)'s barrier (it waits
    // for V(i) first), and a single barrier would then have gone through two phases unseen; P(i+2) on the
    // other hand needs S(i+2), which is issued only after the MMA thread has seen P(i).  P never touches shared memory: the softmax
    // threads write it as bf16 over the S buffer they have just read (tcgen05.st) and P V takes its A
    // operand from tensor memory.  No "S empty" / "P empty" barriers are needed: the tensor core runs the
    // MMAs in issue order (Q K^T(i+1), P V(i), Q K^T(i+2), ...), so S buffer i & 1 is rewritten by
    // Q K^T(i+2) only after P V(i) has read P(i) from it, and P V(i) was issued after P(i) was complete.
    // K and V stages are released separately: a K stage as soon as Q K^T has read it, a V stage after P V.
    uint32_t* tmem_slot = (uint32_t*)(bars + kBars + 1);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
    // after the last P V the K/V ring is free: this CTA's part of a split lives there
    float* part_o = (float*)sK;                            // [128 rows][128], 16-byte chunks XOR-swizzled by row
    // [128 rows][2] running maximum, sum: behind the part's 64 KB; with one stage each that is the end of the
    // ring, so it goes where Q was (every Q K^T has completed by then)
    float* part_ml = kSingle ? (float*)sQ : (float*)(sK + 2 * kOperand);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tile = blockIdx.x;
    const int b = p.qtile_seq[tile], row0 = p.qtile_row0[tile], n_valid = p.qtile_n[tile];
    const int group = p.Hq / p.Hkv;
    const int kvh = (int)blockIdx.y / p.tiles_per_kv, hg = (int)blockIdx.y % p.tiles_per_kv;
    const int h = kvh * group + hg * p.pack;              // query head of slot 0; slot j holds head h + j
    const int n_slots = min(p.pack, group - hg * p.pack);  // slots of this tile that hold a head

    pdl_launch_dependents();
    // The index lists are complete before this kernel can start: a host-planned step copies them in
    // front of its first kernel, and a device-planned step's embedding kernel (the planner kernel's
    // successor) triggers its dependents only after its own wait, i.e. after the planner has finished.
    const int n_vis = p.seq_nvis[b];
    const int n_kt_all = (n_vis + kTile - 1) / kTile;
    const int n_parts = (n_kt_all + p.tiles_per_split - 1) / p.tiles_per_split;
    const int kt_begin = (int)blockIdx.z * p.tiles_per_split;
    // a CTA without key tiles still takes part in the cluster barriers below
    const bool has_work = kt_begin < n_kt_all;
    const int n_kt = has_work ? min(p.tiles_per_split, n_kt_all - kt_begin) : 0;
    uint32_t tmem_base = 0;
    if (has_work) {
        if (threadIdx.x == 0) {
            for (int i = 0; i < kBars; ++i)
                mbar_init(smem_u32(&bars[i]), (i == kPFull || i == kPFull + 1 || i == kOEmpty || i == kOEmpty + 1) ? 256u : 1u);
            *abort_flag = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kCols);
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        tmem_base = *tmem_slot;
    }
    if (threadIdx.x == 64) A_STAMP(0);
    pdl_wait();                                   // q and the cache rows come from the previous kernel
    if (threadIdx.x == 64) A_STAMP(1);

    if (!has_work) {
        // nothing to compute
    } else if (warp == 0) {
        if (lane == 0) {
            // ---------------------------------------------------- TMA producer
            const uint32_t qf = smem_u32(&bars[kQFull]);
            // slot j: rows [row0, row0 + slot) of head h + j at tile rows [j * slot, ...); slots without a head
            // stay unwritten (their rows of S and O are never read)
            mbar_expect_tx(qf, (uint32_t)(n_slots * p.slot * 256));
            for (int j = 0; j < n_slots; ++j) {
                const uint32_t dst = smem_u32(sQ) + (uint32_t)(j * p.slot * 128);
                tma_load_2d(dst, &map_q, qf, (h + j) * kTile, row0);
                tma_load_2d(dst + kAtom, &map_q, qf, (h + j) * kTile + 64, row0);
            }
            const int bh = b * p.Hkv + kvh;
            auto load_k = [&](int j) -> bool {
                const int ks = j % NS;
                const uint32_t ph = (uint32_t)(j / NS) & 1u;
                const uint32_t kfull = smem_u32(&bars[kKFull + ks]);
                if (!mbar_wait(smem_u32(&bars[kKEmpty + ks]), ph ^ 1u, abort_flag)) return false;   // stage free
                const uint32_t sk = smem_u32(sK + (size_t)ks * kOperand);
                const int kv0 = (kt_begin + j) * kTile;
                mbar_expect_tx(kfull, kOperand);
                tma_load_4d(sk, &map_k, kfull, 0, kv0, bh, p.layer);            // keys kv0.., dims 0..63
                tma_load_4d(sk + kAtom, &map_k, kfull, 64, kv0, bh, p.layer);   // dims 64..127
                return true;
            };
            // order of need: K(0), K(1), V(0), K(2), V(1), ...
            bool ok = load_k(0);
            for (int i = 0; i < n_kt && ok; ++i) {
                if (i + 1 < n_kt && !(ok = load_k(i + 1))) break;
                const int vs = i % NS;
                const uint32_t ph = (uint32_t)(i / NS) & 1u;
                const uint32_t vfull = smem_u32(&bars[kVFull + vs]);
                const uint32_t sv = smem_u32(sV + (size_t)vs * kOperand);
                const int kv0 = (kt_begin + i) * kTile;
                if (!(ok = mbar_wait(smem_u32(&bars[kVEmpty + vs]), ph ^ 1u, abort_flag))) break;   // stage free
                mbar_expect_tx(vfull, kOperand);
                tma_load_4d(sv, &map_vt, vfull, kv0, 0, bh, p.layer);           // all dims, keys kv0..kv0+63
                tma_load_4d(sv + kAtom, &map_vt, vfull, kv0 + 64, 0, bh, p.layer);
            }
            if (!ok) {
                *abort_flag = 1;
                atomicCAS(p.status, 0, WD_ERR_DEVICE_TIMEOUT);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------------------------------------------- MMA issuer
            // tile i uses K/V stage i % 3, S buffer i & 1, O_tile buffer i & 1
            bool ok = mbar_wait(smem_u32(&bars[kQFull]), 0, abort_flag);
            const uint64_t qd0 = make_sdesc(smem_u32(sQ)), qd1 = make_sdesc(smem_u32(sQ) + kAtom);
            auto issue_qk = [&](int j) -> bool {           // S[j&1] = Q K(j)^T
                const int s = j & 1, ks = j % NS;
                if (!mbar_wait(smem_u32(&bars[kKFull + ks]), (uint32_t)(j / NS) & 1u, abort_flag)) return false;   // K(j) landed
                tc_fence_after();
                const uint32_t sk = smem_u32(sK + (size_t)ks * kOperand);
                const uint64_t kd0 = make_sdesc(sk), kd1 = make_sdesc(sk + kAtom);
                const uint32_t acc = tmem_base + (uint32_t)(s * kTile);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) umma_bf16(acc, qd0 + 2 * kk, kd0 + 2 * kk, p.idesc, kk > 0);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) umma_bf16(acc, qd1 + 2 * kk, kd1 + 2 * kk, p.idesc, 1u);
                umma_commit(smem_u32(&bars[kKEmpty + ks]));    // K stage free once these MMAs have read it
                umma_commit(smem_u32(&bars[kSFull + s]));
                return true;
            };
            ok = ok && issue_qk(0);
            for (int i = 0; i < n_kt && ok; ++i) {
                const int s = i & 1, vs = i % NS;
                const uint32_t ph = (uint32_t)(i >> 1) & 1u;
                if (i + 1 < n_kt && !(ok = issue_qk(i + 1))) break;                           // runs ahead of the softmax
                if (!(ok = mbar_wait(smem_u32(&bars[kVFull + vs]), (uint32_t)(i / NS) & 1u, abort_flag))) break;   // V(i) landed
                if (!(ok = mbar_wait(smem_u32(&bars[kPFull + s]), ph, abort_flag))) break;              // P(i) written
                if (!(ok = mbar_wait(smem_u32(&bars[kOEmpty + s]), ph ^ 1u, abort_flag))) break;        // O_tile(i-2) folded
                tc_fence_after();
                const uint32_t sv = smem_u32(sV + (size_t)vs * kOperand);
                const uint64_t vd0 = make_sdesc(sv), vd1 = make_sdesc(sv + kAtom);
                const uint32_t acc = tmem_base + kOBase + (uint32_t)(s * kTile);
                const uint32_t pa = tmem_base + (uint32_t)(s * kTile);       // P(i): 64 columns over S(i)
                // O_tile = P V: reduction over the 128 keys of the tile, 16 keys = 8 columns of P per MMA
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) umma_bf16_ta(acc, pa + 8 * kk, vd0 + 2 * kk, p.idesc, kk > 0);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) umma_bf16_ta(acc, pa + 32 + 8 * kk, vd1 + 2 * kk, p.idesc, 1u);
                umma_commit(smem_u32(&bars[kVEmpty + vs]));    // V stage free
                umma_commit(smem_u32(&bars[kOFull + s]));      // O_tile(i) ready
            }
            if (!ok) {
                *abort_flag = 1;
                atomicCAS(p.status, 0, WD_ERR_DEVICE_TIMEOUT);
            }
        }
        __syncwarp();
    } else {
        // -------------------------------------------------------- softmax + accumulate (two threads per row)
        const int quarter = warp & 3;                      // TMEM lanes 32*quarter .. +31
        const int hf = (warp - 2) >> 2;                    // which 64 columns of a 128-wide tile
        const int r = quarter * 32 + lane;                 // query row of the tile = TMEM lane
        // warps whose 32 rows are all beyond the valid ones only keep the barrier counts right.
        // The test is per warp, not per row: tcgen05.ld is warp-collective and must not diverge.
        const int sj = r >> p.slot_shift, rr_ = r & (p.slot - 1);       // slot (head h + sj) and row within the slot
        const bool live = ((quarter * 32) >> p.slot_shift) < n_slots && ((quarter * 32) & (p.slot - 1)) < n_valid;
        const bool valid = sj < n_slots && rr_ < n_valid;
        const int c_off = 64 * hf;
        const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16);
        float* xch = (float*)(tmem_slot + 4);              // [2][128] exchange between the two halves (row sums)
        uint16_t* xm = (uint16_t*)xch;                     // the same 1 KB as [2 parities][2][128] bf16 row maxima
        float o[64];
#pragma unroll
        for (int c = 0; c < 64; ++c) o[c] = 0.f;
        float m = -INFINITY, l = 0.f, alpha_prev = 0.f;
        bool ok = true;
        // o += O_tile(j) with tile j's rescale factor; done one tile late so that P V(j) has had
        // time to finish while this thread was busy with the next tile's softmax
        auto fold = [&](int j, float alpha) {
            const int s = j & 1;
            if (!mbar_wait(smem_u32(&bars[kOFull + s]), (uint32_t)(j >> 1) & 1u, abort_flag)) { *abort_flag = 1; ok = false; }
            tc_fence_after();
            if (live) {
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(t_row + kOBase + (uint32_t)(s * kTile + c_off + c0), v);
#pragma unroll
                    for (int c = 0; c < 32; ++c) o[c0 + c] = kSingle ? __uint_as_float(v[c]) : o[c0 + c] * alpha + __uint_as_float(v[c]);
                }
            }
            tc_fence_before();
            mbar_arrive(smem_u32(&bars[kOEmpty + s]));     // O_tile buffer may be overwritten
        };
        for (int i = 0; i < n_kt; ++i) {
            const int s = i & 1;
            // A failed wait must not leave the loop before the named barrier below (the other
            // warps would wait there for ever): it raises the CTA's abort flag, every thread still
            // reaches the barrier, and all of them leave together right after it.
            if (!mbar_wait(smem_u32(&bars[kSFull + s]), (uint32_t)(i >> 1) & 1u, abort_flag)) *abort_flag = 1;
            tc_fence_after();
            if (threadIdx.x == 64 && i == 0) A_STAMP(2);
            const int n_keys = min(kTile, n_vis - (kt_begin + i) * kTile);   // valid keys in this tile
            // keys past n_vis may hold anything: zero their V columns so that 0 * garbage stays 0.
            // Thread (r, hf) owns row r (a head dim) of atom hf (keys 64*hf..) of the transposed V tile.
            if (n_keys < c_off + 64) {
                if (!mbar_wait(smem_u32(&bars[kVFull + i % NS]), (uint32_t)(i / NS) & 1u, abort_flag)) *abort_flag = 1;   // V landed
                uint8_t* vt = sV + (size_t)(i % NS) * kOperand + hf * kAtom + r * 128;
                for (int kv = max(n_keys - c_off, 0); kv < 64; ++kv)
                    *reinterpret_cast<uint16_t*>(vt + (((kv >> 3) ^ (r & 7)) << 4) + (kv & 7) * 2) = 0;
            }
            // This thread's 64 raw scores stay in registers for both passes.  The softmax warps are
            // bound by instruction issue, so the passes are kept to one FMNMX, then one FFMA + one MUFU
            // + one FADD (+ half a pack) per score: the scale is folded into the exponent's FFMA
            // (exp2(s * c - m * c)), and only the last, ragged key tile pays for the masking.
            float sc[64];
            float mx = -INFINITY;
            if (live) {
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(t_row + (uint32_t)(s * kTile + c_off + c0), v);
                    if (n_keys >= kTile) {
#pragma unroll
                        for (int c = 0; c < 32; ++c) {
                            sc[c0 + c] = __uint_as_float(v[c]);
                            mx = fmaxf(mx, sc[c0 + c]);
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < 32; ++c) {
                            sc[c0 + c] = (c_off + c0 + c < n_keys) ? __uint_as_float(v[c]) : -INFINITY;
                            mx = fmaxf(mx, sc[c0 + c]);
                        }
                    }
                }
                mx *= p.scale_log2e;                       // the scale is positive; -inf stays -inf
            }
            // The two halves of a row must use the same reference value, and any upper bound of the scores
            // serves (softmax does not depend on it): each half rounds its maximum up to bf16 and both take
            // the larger.  Sixteen bits per value leave room for one buffer per tile parity, so a thread
            // that is already a tile ahead cannot overwrite what its partner has yet to read.
            {
                uint32_t mb = __float_as_uint(mx);
                mb = (mb & 0x80000000u) ? (mb & 0xffff0000u) : ((mb + 0xffffu) & 0xffff0000u);
                mx = __uint_as_float(mb);
                xm[((i & 1) * 2 + hf) * kTile + r] = (uint16_t)(mb >> 16);
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (*abort_flag) { ok = false; break; }
            float alpha = 0.f;
            if (live) {
                mx = fmaxf(fmaxf(mx, __uint_as_float((uint32_t)xm[((i & 1) * 2 + (hf ^ 1)) * kTile + r] << 16)), m);
                alpha = ex2_approx(m - mx);                // m = -inf on the first tile gives 0
                m = mx;
                l *= alpha;
            }
            // P(i) as bf16 pairs over the S buffer: both threads of the row hold their scores in registers
            // (the barrier above), and the tensor core is done with whatever these columns held before
            if (live) {
                uint32_t pw[32];
                const float neg_mx = -mx;
                float l0 = 0.f, l1 = 0.f;
#pragma unroll
                for (int g = 0; g < 32; ++g) {
                    // masked keys: fma(-inf, c, -m) = -inf, exp2(-inf) = 0
                    const float p0 = ex2_approx(fmaf(sc[2 * g], p.scale_log2e, neg_mx));
                    const float p1 = ex2_approx(fmaf(sc[2 * g + 1], p.scale_log2e, neg_mx));
                    l0 += p0;
                    l1 += p1;
                    pw[g] = pack_bf16(p0, p1);
                }
                l += l0 + l1;
                tmem_st32(t_row + (uint32_t)(s * kTile + 32 * hf), pw);
            }
            fence_proxy_async_smem();                      // the zeroed V columns -> visible to the MMA
            tc_fence_before();
            mbar_arrive(smem_u32(&bars[kPFull + s]));
            if (threadIdx.x == 64 && i == n_kt - 1) A_STAMP(3);
            if (!kSingle && i > 0) fold(i - 1, alpha_prev);
            alpha_prev = alpha;
        }
        if (ok && n_kt > 0) fold(n_kt - 1, alpha_prev);
        if (threadIdx.x == 64) A_STAMP(4);
        // row sum = sum of the two halves (same running maximum on both sides)
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (*abort_flag) {
            ok = false;
            if (threadIdx.x == 64) atomicCAS(p.status, 0, WD_ERR_DEVICE_TIMEOUT);
        }
        xch[hf * kTile + r] = l;
        asm volatile("bar.sync 1, 256;" ::: "memory");
        l += xch[(hf ^ 1) * kTile + r];
        if (n_parts == 1) {
            if (ok && valid) {
                const float inv = 1.f / l;
                const size_t base = ((size_t)(row0 + rr_) * p.Hq + h + sj) * kTile + c_off;
                uint4* dst = reinterpret_cast<uint4*>(p.out + base);
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    uint4 u;
                    u.x = pack_bf16(o[8 * g + 0] * inv, o[8 * g + 1] * inv);
                    u.y = pack_bf16(o[8 * g + 2] * inv, o[8 * g + 3] * inv);
                    u.z = pack_bf16(o[8 * g + 4] * inv, o[8 * g + 5] * inv);
                    u.w = pack_bf16(o[8 * g + 6] * inv, o[8 * g + 7] * inv);
                    dst[g] = u;
                }
                if (p.tap) {
#pragma unroll
                    for (int c = 0; c < 64; ++c) p.tap[base + c] = o[c] * inv;
                }
            }
        } else if (valid) {
            // this CTA's part: every tensor-core read of the K/V ring has completed (the last fold
            // waited for the last P V), so the ring is reused.  Chunk c of row r sits at c ^ (r & 31).
            float4* dst = reinterpret_cast<float4*>(part_o + (size_t)r * kTile);
#pragma unroll
            for (int g = 0; g < 16; ++g)
                dst[(hf * 16 + g) ^ (r & 31)] = make_float4(o[4 * g], o[4 * g + 1], o[4 * g + 2], o[4 * g + 3]);
            if (hf == 0) *reinterpret_cast<float2*>(part_ml + r * 2) = make_float2(m, l);
        }
    }
    if (p.max_parts > 1) {
        // ------------------------------------------------------------ merge across the cluster
        if (threadIdx.x == 64) A_STAMP(5);
        cluster_sync_all();                                // every part is in place and visible
        if (has_work && n_parts > 1 && warp >= 2) {
            // CTA z merges rows [z * per, (z + 1) * per).  An item = (row, group of 4 columns); a
            // thread takes items t, t + 256, ... and keeps kItems x kParts remote loads in flight.
            constexpr int kItems = 2, kParts = 4;
            // (rows are counted over the valid rows of all slots: index q = slot * n_valid + row within the slot)
            const int n_tot = n_slots * n_valid;
            const int per = (n_tot + n_parts - 1) / n_parts;
            const int r_lo = min((int)blockIdx.z * per, n_tot), r_hi = min(r_lo + per, n_tot);
            const int t = (int)threadIdx.x - 64, n_items = (r_hi - r_lo) * 32;
            const uint32_t lo = smem_u32(part_o), lml = smem_u32(part_ml);
            for (int it0 = t; it0 < n_items; it0 += 256 * kItems) {
                float mxx[kItems], lsum[kItems];
                float4 acc[kItems];
#pragma unroll
                for (int u = 0; u < kItems; ++u) {
                    mxx[u] = -INFINITY;
                    lsum[u] = 0.f;
                    acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
                for (int z0 = 0; z0 < n_parts; z0 += kParts) {       // parts in order of z
                    float2 ml[kItems][kParts];
                    float4 v[kItems][kParts];
#pragma unroll
                    for (int u = 0; u < kItems; ++u) {
                        const int item = it0 + u * 256, qq = r_lo + (item >> 5), cg = item & 31;
                        const int rr = (qq / n_valid) * p.slot + qq % n_valid;         // tile row
#pragma unroll
                        for (int zz = 0; zz < kParts; ++zz) {
                            ml[u][zz] = make_float2(-INFINITY, 0.f);
                            v[u][zz] = make_float4(0.f, 0.f, 0.f, 0.f);
                            if (item < n_items && z0 + zz < n_parts) {
                                ml[u][zz] = dsmem_ld2(dsmem_addr(lml + (uint32_t)rr * 8u, (uint32_t)(z0 + zz)));
                                v[u][zz] = dsmem_ld4(dsmem_addr(lo + (uint32_t)rr * 512u + (uint32_t)((cg ^ (rr & 31)) << 4),
                                                                (uint32_t)(z0 + zz)));
                            }
                        }
                    }
#pragma unroll
                    for (int u = 0; u < kItems; ++u) {
                        if (it0 + u * 256 >= n_items) continue;
                        float mnew = mxx[u];
#pragma unroll
                        for (int zz = 0; zz < kParts; ++zz) mnew = fmaxf(mnew, ml[u][zz].x);
                        const float keep = exp2f(mxx[u] - mnew);       // -inf on the first chunk gives 0
                        mxx[u] = mnew;
                        lsum[u] *= keep;
                        acc[u].x *= keep; acc[u].y *= keep; acc[u].z *= keep; acc[u].w *= keep;
#pragma unroll
                        for (int zz = 0; zz < kParts; ++zz) {
                            const float wgt = exp2f(ml[u][zz].x - mnew);   // absent parts: exp2(-inf) = 0
                            lsum[u] += ml[u][zz].y * wgt;
                            acc[u].x += v[u][zz].x * wgt; acc[u].y += v[u][zz].y * wgt;
                            acc[u].z += v[u][zz].z * wgt; acc[u].w += v[u][zz].w * wgt;
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < kItems; ++u) {
                    const int item = it0 + u * 256, qq = r_lo + (item >> 5), cg = item & 31;
                    if (item >= n_items) continue;
                    const float inv = 1.f / lsum[u];
                    const size_t base = ((size_t)(row0 + qq % n_valid) * p.Hq + h + qq / n_valid) * kTile + 4 * cg;
                    uint2 w2;
                    w2.x = pack_bf16(acc[u].x * inv, acc[u].y * inv);
                    w2.y = pack_bf16(acc[u].z * inv, acc[u].w * inv);
                    *reinterpret_cast<uint2*>(p.out + base) = w2;
                    if (p.tap)
                        *reinterpret_cast<float4*>(p.tap + base) =
                            make_float4(acc[u].x * inv, acc[u].y * inv, acc[u].z * inv, acc[u].w * inv);
                }
            }
        }
        if (threadIdx.x == 64) A_STAMP(6);
        cluster_sync_all();                                // no CTA leaves while its part may still be read
    }
    if (has_work) {
        tc_fence_before();
        __syncthreads();
        if (warp == 1) {
            tc_fence_after();
            tmem_dealloc(tmem_base, kCols);
        }
    }
#ifdef WD_GEMM_TRACE
    if (threadIdx.x == 0) atomicMax(&g_attn_end[p.layer & 63], global_ns());
    if (threadIdx.x == 64) A_STAMP(7);
#endif
}

__global__ void __launch_bounds__(kThreads, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                    const __grid_constant__ CUtensorMap map_vt, const AttnParams p) {
    attention_tc_body<false>(map_q, map_k, map_vt, p);
}

// (128 registers: 320 threads of this kernel and the 192 of a GEMM CTA fit the register file together)
__global__ void __maxnreg__(128)
attention_tc_single_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                           const __grid_constant__ CUtensorMap map_vt, const AttnParams p) {
    attention_tc_body<true>(map_q, map_k, map_vt, p);
}

#ifdef WD_GEMM_TRACE
extern "C" __attribute__((visibility("default"))) int wd_debug_attn_stamps(unsigned long long* host /*[160][8]*/) {
    cudaDeviceSynchronize();
    return (int)cudaMemcpyFromSymbol(host, g_attn_trace, sizeof(unsigned long long) * 160 * 8);
}
extern "C" __attribute__((visibility("default"))) int wd_debug_attn_trace(unsigned long long* host /*[64]*/) {
    cudaDeviceSynchronize();
    return (int)cudaMemcpyFromSymbol(host, g_attn_end, sizeof(unsigned long long) * 64);
}
#endif

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

}  // namespace

// K cache [L][BH][S][dh] -> dims (dh, S, BH, L), box (64, 128, 1, 1);
// transposed V cache [L][BH][dh][Sp] -> dims (Sp, dh, BH, L), box (64, 128, 1, 1)
wd_status wd_attn_tc_encode_cache(CUtensorMap* map_k, CUtensorMap* map_vt, const void* kcache, const void* vcache,
                                  int L, int BH, int S, int Sp, int dh) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return WD_ERR_CUDA;
    if (dh != kTile) return WD_ERR_BAD_PARAM;
    {
        cuuint64_t dims[4] = {(cuuint64_t)dh, (cuuint64_t)S, (cuuint64_t)BH, (cuuint64_t)L};
        cuuint64_t strides[3] = {(cuuint64_t)dh * 2, (cuuint64_t)S * dh * 2, (cuuint64_t)BH * S * dh * 2};
        cuuint32_t box[4] = {64, 128, 1, 1}, estr[4] = {1, 1, 1, 1};
        if (enc(map_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(kcache), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return WD_ERR_CUDA;
    }
    {
        cuuint64_t dims[4] = {(cuuint64_t)Sp, (cuuint64_t)dh, (cuuint64_t)BH, (cuuint64_t)L};
        cuuint64_t strides[3] = {(cuuint64_t)Sp * 2, (cuuint64_t)dh * Sp * 2, (cuuint64_t)BH * dh * Sp * 2};
        cuuint32_t box[4] = {64, 128, 1, 1}, estr[4] = {1, 1, 1, 1};
        if (enc(map_vt, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(vcache), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return WD_ERR_CUDA;
    }
    return WD_OK;
}

wd_status wd_attn_tc_launch(const void* q, int n_rows, int n_tiles, const int32_t* qtile_seq, const int32_t* qtile_row0,
                            const int32_t* qtile_n, const int32_t* seq_nvis, const CUtensorMap* map_k,
                            const CUtensorMap* map_vt, void* out, float* tap, int Hq, int Hkv, int dh, int layer,
                            int max_vis, int sm_count, int32_t* status, cudaStream_t stream, int max_tile_rows,
                            size_t* smem_used) {
    if (dh != kTile) return WD_ERR_BAD_PARAM;
    if (n_tiles <= 0) return WD_OK;
    EncodeTiledFn enc = get_encode();
    if (!enc) return WD_ERR_CUDA;
    // the query descriptor depends only on (buffer, rows, heads): the same for every layer of a step
    static CUtensorMap mq;
    static const void* mq_ptr = nullptr;
    static int mq_rows = -1, mq_hq = -1, mq_dev = -1, mq_slot = -1;
    int dev = 0;
    WD_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return WD_ERR_CUDA;
    // Grouped-query attention with few rows per tile: 2 or 4 query heads of one KV head share a 128-row tile
    // (slots of 64 or 32 rows), so their K/V tiles are loaded once and the grid shrinks by that factor
    const int group = Hq / Hkv;
    static const int pack_max = getenv("WD_ATTN_PACK") ? atoi(getenv("WD_ATTN_PACK")) : 4;     // 1 switches packing off
    int pack = 1;
    if (max_tile_rows > 0 && group > 1) {
        if (max_tile_rows <= 32 && group >= 4) pack = 4;
        else if (max_tile_rows <= 64) pack = 2;
        if (pack > pack_max) pack = pack_max >= 2 ? 2 : 1;
        if (pack == 2 && max_tile_rows > 64) pack = 1;
    }
    const int slot = kTile / pack;
    if (mq_ptr != q || mq_rows != n_rows || mq_hq != Hq || mq_dev != dev || mq_slot != slot) {
        cuuint64_t dims[2] = {(cuuint64_t)Hq * dh, (cuuint64_t)n_rows};
        cuuint64_t strides[1] = {(cuuint64_t)Hq * dh * 2};
        cuuint32_t box[2] = {64, (cuuint32_t)slot}, estr[2] = {1, 1};
        if (enc(&mq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(q), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return WD_ERR_CUDA;
        mq_ptr = q; mq_rows = n_rows; mq_hq = Hq; mq_dev = dev; mq_slot = slot;
    }
    AttnParams p;
    memset(&p, 0, sizeof(p));
    p.qtile_seq = qtile_seq; p.qtile_row0 = qtile_row0; p.qtile_n = qtile_n; p.seq_nvis = seq_nvis;
    p.out = (__nv_bfloat16*)out; p.tap = tap;
    p.Hq = Hq; p.Hkv = Hkv; p.layer = layer;
    p.scale_log2e = 1.4426950408889634f / sqrtf((float)dh);
    p.status = status;
    p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTile >> 3) << 17) | ((uint32_t)(kTile >> 4) << 24);
    // split the keys across the CTAs of a cluster while (tile, head) pairs alone would leave SMs idle
    const int max_kt = (max_vis + kTile - 1) / kTile;
    p.pack = pack;
    p.slot = slot;
    p.slot_shift = pack == 1 ? 7 : (pack == 2 ? 6 : 5);
    p.tiles_per_kv = (group + pack - 1) / pack;
    const int grid_y = Hkv * p.tiles_per_kv;
    int want = sm_count / (n_tiles * grid_y);
    if (want < 1) want = 1;
    if (want > kMaxCluster) want = kMaxCluster;
    if (want > max_kt) want = max_kt;
    p.tiles_per_split = (max_kt + want - 1) / want;
    p.max_parts = (max_kt + p.tiles_per_split - 1) / p.tiles_per_split;
    static const int single_on = getenv("WD_ATTN_SINGLE") ? atoi(getenv("WD_ATTN_SINGLE")) : 1;
    const bool single = single_on && p.tiles_per_split == 1;
    const size_t smem_of[2] = {(1 + 2 * kStages) * (size_t)kOperand + (kBars + 1) * 8 + 16 + 2 * kTile * 4 + 1024,
                               (1 + 2) * (size_t)kOperand + (kBars + 1) * 8 + 16 + 2 * kTile * 4 + 1024};
    const size_t smem = smem_of[single ? 1 : 0];
    if (smem_used) *smem_used = smem;
    static bool attr_done[64] = {};     // the attribute is per device
    if (!attr_done[dev]) {
        WD_CUDA_TRY(cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_of[0]));
        WD_CUDA_TRY(cudaFuncSetAttribute(attention_tc_single_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_of[1]));
        // the whole SM's shared memory although the kernel takes less than half: the output projection's CTAs are
        // to be resident beside it, and an SM keeps its carve-out while blocks are resident
        if (!(getenv("WD_NO_CARVEOUT") && atoi(getenv("WD_NO_CARVEOUT"))))
            WD_CUDA_TRY(cudaFuncSetAttribute(attention_tc_single_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                             cudaSharedmemCarveoutMaxShared));
        attr_done[dev] = true;
    }
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(n_tiles, grid_y, p.max_parts);
    lc.blockDim = dim3(kThreads);
    lc.dynamicSmemBytes = smem;
    lc.stream = stream;
    cudaLaunchAttribute attr[2];
    int n_attr = 0;
    if (p.max_parts > 1) {
        attr[n_attr].id = cudaLaunchAttributeClusterDimension;
        attr[n_attr].val.clusterDim.x = 1;
        attr[n_attr].val.clusterDim.y = 1;
        attr[n_attr].val.clusterDim.z = (unsigned)p.max_parts;
        ++n_attr;
    }
    if (wd_pdl_enabled) {
        attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
        ++n_attr;
    }
    lc.attrs = attr;
    lc.numAttrs = n_attr;
    ++wd_launch_counter;
    if (single) WD_CUDA_TRY(cudaLaunchKernelEx(&lc, attention_tc_single_kernel, mq, *map_k, *map_vt, p));
    else WD_CUDA_TRY(cudaLaunchKernelEx(&lc, attention_tc_kernel, mq, *map_k, *map_vt, p));
    return WD_OK;
}
