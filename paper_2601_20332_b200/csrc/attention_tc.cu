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
// CTAs (grid.z) so that the machine is filled: each CTA leaves its running maximum, sum and
// unnormalised output in scratch and the last one to arrive merges them in a fixed order.
// Every wait is bounded; on expiry the CTA records WD_ERR_DEVICE_TIMEOUT and leaves.
#include <cstring>

#include "attention_tc.h"
#include "device_utils.cuh"

namespace {

using namespace wdk;

constexpr int kTile = 128;                 // query rows per CTA = keys per step = head_dim
constexpr int kAtom = kTile * 64 * 2;      // one [128 x 64] bf16 swizzle-atom column: 16 KB
constexpr int kOperand = 2 * kAtom;        // a [128 x 128] bf16 operand: 32 KB
constexpr int kThreads = 320;            // TMA warp, MMA warp, 8 softmax warps
constexpr int kTmemCols = 512;             // S0, S1: columns 0..255; O_tile0, O_tile1: columns 256..511
constexpr int kBars = 15;

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
    // split over the keys: CTA z of (tile, head) takes key tiles [z * tiles_per_split, ...) and, when a
    // sequence needs more than one CTA, leaves (m, l, unnormalised O) in scratch; the CTA that arrives
    // last merges the parts in order of z
    int tiles_per_split, max_parts;
    float* part_o;               // [(tile * Hq + h) * max_parts + z][128 rows][128]
    float* part_ml;              // [(tile * Hq + h) * max_parts + z][128 rows][2]
    int32_t* counters;           // [n_tiles * Hq], zero between launches
};

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
}

__global__ void __launch_bounds__(kThreads, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                    const __grid_constant__ CUtensorMap map_vt, const AttnParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sQ = smem;                          // 32 KB
    uint8_t* sP = smem + kOperand;               // 32 KB
    uint8_t* sKV = smem + 2 * kOperand;          // 2 stages x (K 32 KB + V^T 32 KB)
    uint64_t* bars = (uint64_t*)(smem + 2 * kOperand + 4 * kOperand);
    // 0 q_full | 1,2 kv_full | 3,4 kv_empty | 5,6 s_full | 7,8 s_empty | 9 p_full | 10 p_empty |
    // 11,12 o_full | 13,14 o_empty.  "empty" barriers that the softmax threads signal count 256.
    uint32_t* tmem_slot = (uint32_t*)(bars + kBars + 1);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tile = blockIdx.x, h = blockIdx.y;
    const int b = p.qtile_seq[tile], row0 = p.qtile_row0[tile], n_valid = p.qtile_n[tile];
    const int kvh = h / (p.Hq / p.Hkv);

    pdl_launch_dependents();
    // the index lists were copied before the first kernel of the step: safe to read right away
    const int n_vis = p.seq_nvis[b];
    const int n_kt_all = (n_vis + kTile - 1) / kTile;
    const int n_parts = (n_kt_all + p.tiles_per_split - 1) / p.tiles_per_split;
    const int kt_begin = (int)blockIdx.z * p.tiles_per_split;
    if (kt_begin >= n_kt_all) return;                       // nothing for this CTA (uniform exit)
    const int n_kt = min(p.tiles_per_split, n_kt_all - kt_begin);
    if (threadIdx.x == 0) {
        for (int i = 0; i < kBars; ++i)
            mbar_init(smem_u32(&bars[i]), (i == 7 || i == 8 || i == 9 || i == 13 || i == 14) ? 256u : 1u);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();                                   // q and the cache rows come from the previous kernel

    if (warp == 0) {
        if (lane == 0) {
            // ---------------------------------------------------- TMA producer
            const uint32_t qf = smem_u32(&bars[0]);
            mbar_expect_tx(qf, kOperand);
            tma_load_2d(smem_u32(sQ), &map_q, qf, h * kTile, row0);
            tma_load_2d(smem_u32(sQ) + kAtom, &map_q, qf, h * kTile + 64, row0);
            for (int i = 0; i < n_kt; ++i) {
                const int s = i & 1;
                const uint32_t ph = (uint32_t)(i >> 1) & 1u;
                if (!mbar_wait(smem_u32(&bars[3 + s]), ph ^ 1u, abort_flag)) {
                    *abort_flag = 1;
                    atomicCAS(p.status, 0, WD_ERR_DEVICE_TIMEOUT);
                    break;
                }
                const uint32_t full = smem_u32(&bars[1 + s]);
                const uint32_t sk = smem_u32(sKV + (size_t)s * 2 * kOperand), sv = sk + kOperand;
                mbar_expect_tx(full, 2 * kOperand);
                const int kv0 = (kt_begin + i) * kTile, bh = b * p.Hkv + kvh;
                tma_load_4d(sk, &map_k, full, 0, kv0, bh, p.layer);            // keys kv0.., dims 0..63
                tma_load_4d(sk + kAtom, &map_k, full, 64, kv0, bh, p.layer);   // dims 64..127
                tma_load_4d(sv, &map_vt, full, kv0, 0, bh, p.layer);           // all dims, keys kv0..kv0+63
                tma_load_4d(sv + kAtom, &map_vt, full, kv0 + 64, 0, bh, p.layer);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------------------------------------------- MMA issuer
            // tile i uses K/V stage i&1, S buffer i&1, O_tile buffer i&1; every barrier that is
            // completed once per two tiles has parity (i>>1)&1 for tile i
            bool ok = mbar_wait(smem_u32(&bars[0]), 0, abort_flag);
            const uint64_t qd0 = make_sdesc(smem_u32(sQ)), qd1 = make_sdesc(smem_u32(sQ) + kAtom);
            const uint64_t pd0 = make_sdesc(smem_u32(sP)), pd1 = make_sdesc(smem_u32(sP) + kAtom);
            auto issue_qk = [&](int j) -> bool {           // S[j&1] = Q K(j)^T
                const int s = j & 1;
                const uint32_t ph = (uint32_t)(j >> 1) & 1u;
                if (!mbar_wait(smem_u32(&bars[1 + s]), ph, abort_flag)) return false;        // K(j), V(j) landed
                if (!mbar_wait(smem_u32(&bars[7 + s]), ph ^ 1u, abort_flag)) return false;   // S(j-2) has been read
                tc_fence_after();
                const uint32_t sk = smem_u32(sKV + (size_t)s * 2 * kOperand);
                const uint64_t kd0 = make_sdesc(sk), kd1 = make_sdesc(sk + kAtom);
                const uint32_t acc = tmem_base + (uint32_t)(s * kTile);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) umma_bf16(acc, qd0 + 2 * kk, kd0 + 2 * kk, p.idesc, kk > 0);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) umma_bf16(acc, qd1 + 2 * kk, kd1 + 2 * kk, p.idesc, 1u);
                umma_commit(smem_u32(&bars[5 + s]));
                return true;
            };
            ok = ok && issue_qk(0);
            for (int i = 0; i < n_kt && ok; ++i) {
                const int s = i & 1;
                const uint32_t ph = (uint32_t)(i >> 1) & 1u;
                if (i + 1 < n_kt && !(ok = issue_qk(i + 1))) break;                           // runs ahead of the softmax
                if (!(ok = mbar_wait(smem_u32(&bars[9]), (uint32_t)i & 1u, abort_flag))) break;      // P(i) written
                if (!(ok = mbar_wait(smem_u32(&bars[13 + s]), ph ^ 1u, abort_flag))) break;         // O_tile(i-2) folded
                tc_fence_after();
                const uint32_t sv = smem_u32(sKV + (size_t)s * 2 * kOperand) + kOperand;
                const uint64_t vd0 = make_sdesc(sv), vd1 = make_sdesc(sv + kAtom);
                const uint32_t acc = tmem_base + (uint32_t)(2 * kTile + s * kTile);
                // O_tile = P V: reduction over the 128 keys of the tile
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) umma_bf16(acc, pd0 + 2 * kk, vd0 + 2 * kk, p.idesc, kk > 0);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) umma_bf16(acc, pd1 + 2 * kk, vd1 + 2 * kk, p.idesc, 1u);
                umma_commit(smem_u32(&bars[3 + s]));       // K/V stage free
                umma_commit(smem_u32(&bars[10]));          // P buffer free
                umma_commit(smem_u32(&bars[11 + s]));      // O_tile(i) ready
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
        const int c_off = 64 * hf;
        const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16);
        float* xch = (float*)(tmem_slot + 4);              // [2][128] exchange between the two halves
        float o[64];
#pragma unroll
        for (int c = 0; c < 64; ++c) o[c] = 0.f;
        float m = -INFINITY, l = 0.f, alpha_prev = 0.f;
        bool ok = true;
        // o += O_tile(j) with tile j's rescale factor; done one tile late so that P V(j) has had
        // time to finish while this thread was busy with the next tile's softmax
        auto fold = [&](int j, float alpha) {
            const int s = j & 1;
            if (!mbar_wait(smem_u32(&bars[11 + s]), (uint32_t)(j >> 1) & 1u, abort_flag)) { *abort_flag = 1; ok = false; }
            tc_fence_after();
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(t_row + (uint32_t)(2 * kTile + s * kTile + c_off + c0), v);
#pragma unroll
                for (int c = 0; c < 32; ++c) o[c0 + c] = o[c0 + c] * alpha + __uint_as_float(v[c]);
            }
            tc_fence_before();
            mbar_arrive(smem_u32(&bars[13 + s]));          // O_tile buffer may be overwritten
        };
        for (int i = 0; i < n_kt; ++i) {
            const int s = i & 1;
            // A failed wait must not leave the loop before the named barrier below (the other
            // warps would wait there for ever): it raises the CTA's abort flag, every thread still
            // reaches the barrier, and all of them leave together right after it.
            if (!mbar_wait(smem_u32(&bars[5 + s]), (uint32_t)(i >> 1) & 1u, abort_flag)) *abort_flag = 1;
            tc_fence_after();
            const int n_keys = min(kTile, n_vis - (kt_begin + i) * kTile);   // valid keys in this tile
            // keys past n_vis may hold anything: zero their V columns so that 0 * garbage stays 0.
            // Thread (r, hf) owns row r (a head dim) of atom hf (keys 64*hf..) of the transposed V tile.
            if (n_keys < c_off + 64) {
                uint8_t* vt = sKV + (size_t)s * 2 * kOperand + kOperand + hf * kAtom + r * 128;
                for (int kv = max(n_keys - c_off, 0); kv < 64; ++kv)
                    *reinterpret_cast<uint16_t*>(vt + (((kv >> 3) ^ (r & 7)) << 4) + (kv & 7) * 2) = 0;
            }
            // scaled scores of this thread's 64 keys, kept in registers for both passes
            float sc[64];
            float mx = -INFINITY;
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(t_row + (uint32_t)(s * kTile + c_off + c0), v);
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    sc[c0 + c] = (c_off + c0 + c < n_keys) ? __uint_as_float(v[c]) * p.scale_log2e : -INFINITY;
                    mx = fmaxf(mx, sc[c0 + c]);
                }
            }
            tc_fence_before();
            mbar_arrive(smem_u32(&bars[7 + s]));           // S buffer may be overwritten
            xch[hf * kTile + r] = mx;
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (*abort_flag) { ok = false; break; }
            mx = fmaxf(fmaxf(mx, xch[(hf ^ 1) * kTile + r]), m);
            const float alpha = exp2f(m - mx);             // m = -inf on the first tile gives 0
            m = mx;
            l *= alpha;
            // P V of the previous tile must have finished reading the P buffer
            if (!mbar_wait(smem_u32(&bars[10]), ((uint32_t)i & 1u) ^ 1u, abort_flag)) { *abort_flag = 1; ok = false; }
            uint8_t* prow = sP + hf * kAtom + r * 128;
#pragma unroll
            for (int g = 0; g < 8; ++g) {                  // eight 16-byte chunks of 8 keys
                float pr[8];
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    pr[c] = exp2f(sc[8 * g + c] - mx);     // masked keys: exp2(-inf) = 0
                    l += pr[c];
                }
                uint4 u;
                u.x = pack_bf16(pr[0], pr[1]);
                u.y = pack_bf16(pr[2], pr[3]);
                u.z = pack_bf16(pr[4], pr[5]);
                u.w = pack_bf16(pr[6], pr[7]);
                *reinterpret_cast<uint4*>(prow + ((g ^ (r & 7)) << 4)) = u;
            }
            fence_proxy_async_smem();                      // P and the zeroed V columns -> visible to the MMA
            mbar_arrive(smem_u32(&bars[9]));
            if (i > 0) fold(i - 1, alpha_prev);
            alpha_prev = alpha;
        }
        if (ok && n_kt > 0) fold(n_kt - 1, alpha_prev);
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
            if (ok && r < n_valid) {
                const float inv = 1.f / l;
                const size_t base = ((size_t)(row0 + r) * p.Hq + h) * kTile + c_off;
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
        } else {
            // leave this CTA's part in scratch, count the arrival, the last CTA merges
            const size_t slot = ((size_t)tile * p.Hq + h) * p.max_parts;
            if (ok && r < n_valid) {
                float4* dst = reinterpret_cast<float4*>(p.part_o + ((slot + blockIdx.z) * kTile + r) * kTile + c_off);
#pragma unroll
                for (int g = 0; g < 16; ++g) dst[g] = make_float4(o[4 * g], o[4 * g + 1], o[4 * g + 2], o[4 * g + 3]);
                if (hf == 0)
                    *reinterpret_cast<float2*>(p.part_ml + ((slot + blockIdx.z) * kTile + r) * 2) = make_float2(m, l);
            }
            // one fence after the barrier publishes every thread's part (fences are cumulative)
            asm volatile("bar.sync 1, 256;" ::: "memory");
            int* last_flag = (int*)(tmem_slot + 2);
            if (threadIdx.x == 64) {
                __threadfence();
                const int old = atomicAdd(p.counters + tile * p.Hq + h, 1);
                const int last = old + 1 == n_parts ? 1 : 0;
                if (last) p.counters[tile * p.Hq + h] = 0;
                *last_flag = last;
                __threadfence();
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (*last_flag) {
                // warp w merges rows w, w + 8, ...; lanes hold 4 columns each
                for (int rr = warp - 2; rr < n_valid; rr += 8) {
                    float mxx = -INFINITY;
                    for (int z = 0; z < n_parts; ++z) mxx = fmaxf(mxx, __ldcg(p.part_ml + ((slot + z) * kTile + rr) * 2));
                    float lsum = 0.f;
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (int z = 0; z < n_parts; ++z) {
                        const float2 ml = __ldcg(reinterpret_cast<const float2*>(p.part_ml + ((slot + z) * kTile + rr) * 2));
                        const float wgt = exp2f(ml.x - mxx);
                        const float4 v = __ldcg(reinterpret_cast<const float4*>(p.part_o + ((slot + z) * kTile + rr) * kTile) + lane);
                        lsum += ml.y * wgt;
                        acc.x += v.x * wgt; acc.y += v.y * wgt; acc.z += v.z * wgt; acc.w += v.w * wgt;
                    }
                    const float inv = 1.f / lsum;
                    const size_t base = ((size_t)(row0 + rr) * p.Hq + h) * kTile + 4 * lane;
                    uint2 u;
                    u.x = pack_bf16(acc.x * inv, acc.y * inv);
                    u.y = pack_bf16(acc.z * inv, acc.w * inv);
                    *reinterpret_cast<uint2*>(p.out + base) = u;
                    if (p.tap) *reinterpret_cast<float4*>(p.tap + base) = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
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
                            int max_vis, int sm_count, float* scratch, int32_t* counters, int32_t* status,
                            cudaStream_t stream) {
    if (dh != kTile) return WD_ERR_BAD_PARAM;
    if (n_tiles <= 0) return WD_OK;
    EncodeTiledFn enc = get_encode();
    if (!enc) return WD_ERR_CUDA;
    // the query descriptor depends only on (buffer, rows, heads): the same for every layer of a step
    static CUtensorMap mq;
    static const void* mq_ptr = nullptr;
    static int mq_rows = -1, mq_hq = -1;
    if (mq_ptr != q || mq_rows != n_rows || mq_hq != Hq) {
        cuuint64_t dims[2] = {(cuuint64_t)Hq * dh, (cuuint64_t)n_rows};
        cuuint64_t strides[1] = {(cuuint64_t)Hq * dh * 2};
        cuuint32_t box[2] = {64, 128}, estr[2] = {1, 1};
        if (enc(&mq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(q), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return WD_ERR_CUDA;
        mq_ptr = q; mq_rows = n_rows; mq_hq = Hq;
    }
    AttnParams p;
    memset(&p, 0, sizeof(p));
    p.qtile_seq = qtile_seq; p.qtile_row0 = qtile_row0; p.qtile_n = qtile_n; p.seq_nvis = seq_nvis;
    p.out = (__nv_bfloat16*)out; p.tap = tap;
    p.Hq = Hq; p.Hkv = Hkv; p.layer = layer;
    p.scale_log2e = 1.4426950408889634f / sqrtf((float)dh);
    p.status = status;
    p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTile >> 3) << 17) | ((uint32_t)(kTile >> 4) << 24);
    // split the keys across CTAs while (tile, head) pairs alone would leave SMs idle
    const int max_kt = (max_vis + kTile - 1) / kTile;
    int want = sm_count / (n_tiles * Hq);
    if (want < 1 || !scratch || !counters || n_tiles * Hq > WD_ATTN_SPLIT_SLOTS / 2) want = 1;
    if (want > max_kt) want = max_kt;
    p.tiles_per_split = (max_kt + want - 1) / want;
    p.max_parts = (max_kt + p.tiles_per_split - 1) / p.tiles_per_split;
    if ((long long)n_tiles * Hq * p.max_parts > WD_ATTN_SPLIT_SLOTS) { p.tiles_per_split = max_kt; p.max_parts = 1; }
    p.part_o = scratch;
    p.part_ml = scratch ? scratch + (size_t)WD_ATTN_SPLIT_SLOTS * kTile * kTile : nullptr;
    p.counters = counters;
    const size_t smem = 6 * (size_t)kOperand + (kBars + 1) * 8 + 16 + 2 * kTile * 4 + 1024;
    static bool attr_done = false;      // one device per process
    if (!attr_done) {
        WD_CUDA_TRY(cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attr_done = true;
    }
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(n_tiles, Hq, p.max_parts);
    lc.blockDim = dim3(kThreads);
    lc.dynamicSmemBytes = smem;
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = wd_pdl_enabled ? 1 : 0;
    ++wd_launch_counter;
    WD_CUDA_TRY(cudaLaunchKernelEx(&lc, attention_tc_kernel, mq, *map_k, *map_vt, p));
    return WD_OK;
}
