// Element-wise, gather/scatter, reduction and CUDA-core kernels of the step.
//
// These are the bandwidth- and latency-bound pieces around the GEMMs (embedding
// gather, RMSNorm, RoPE + K/V scatter, SwiGLU, residual add, unmask reduction)
// plus CUDA-core versions of the GEMM and of attention that work for any dtype
// and any index list; the fp32 configuration runs on them entirely and the
// bf16 tensor-core kernels are cross-checked against them.
#include "wd_internal.h"

namespace {

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

// ---------------------------------------------------------------- embedding gather
template <typename T>
__global__ void embed_kernel(const T* __restrict__ embed, const int32_t* __restrict__ ids,
                             const int32_t* __restrict__ row_seq, const int32_t* __restrict__ row_pos,
                             float* __restrict__ x, int d, int S, int vocab, int32_t* status) {
    const int r = blockIdx.x;
    const int id = ids[(size_t)row_seq[r] * S + row_pos[r]];
    if (id < 0 || id >= vocab) {           // checked, never dereferenced
        if (threadIdx.x == 0) atomicCAS(status, 0, WD_ERR_BOUNDS);
        for (int c = threadIdx.x; c < d; c += blockDim.x) x[(size_t)r * d + c] = 0.f;
        return;
    }
    const T* src = embed + (size_t)id * d;
    for (int c = threadIdx.x; c < d; c += blockDim.x) x[(size_t)r * d + c] = to_f(src[c]);
}

// ---------------------------------------------------------------- RMSNorm (+ partial-sum add)
template <typename T>
__global__ void rmsnorm_kernel(float* __restrict__ x, const float* __restrict__ part, int n_split,
                               size_t split_stride, const float* __restrict__ gain, float eps,
                               T* __restrict__ xn, const int32_t* __restrict__ row_idx, int d) {
    __shared__ float red[32];
    const int i = blockIdx.x;
    const int r = row_idx ? row_idx[i] : i;
    float* xr = x + (size_t)r * d;
    float ss = 0.f;
    for (int c = threadIdx.x; c < d; c += blockDim.x) {
        float v = xr[c];
        if (part) {
            for (int s = 0; s < n_split; ++s) v += part[s * split_stride + (size_t)r * d + c];
            xr[c] = v;
        }
        ss += v * v;
    }
    ss = block_sum(ss, red);
    const float inv = rsqrtf(ss / (float)d + eps);
    for (int c = threadIdx.x; c < d; c += blockDim.x)
        xn[(size_t)i * d + c] = from_f<T>(xr[c] * inv * gain[c]);
}

// ---------------------------------------------------------------- CUDA-core GEMM
// y[rows, n] = x[rows, k] * w[n, k]^T.  32 x 64 output tile per block, 2 x 4 per thread.
template <typename T>
__global__ void gemm_plain_kernel(const T* __restrict__ x, const T* __restrict__ w, float* __restrict__ y,
                                  int rows, int n, int k, int ldy) {
    __shared__ float xs[32][33];
    __shared__ float ws[64][33];
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
// One block per row.  Rotation pairs (j, j + dh/2) by pos * theta^(-2j/dh), fp32 math.
template <typename T>
__global__ void rope_scatter_kernel(const float* __restrict__ part, int n_split, size_t split_stride,
                                    const int32_t* __restrict__ row_seq, const int32_t* __restrict__ row_pos,
                                    T* __restrict__ q, T* __restrict__ kcache, T* __restrict__ vcache,
                                    int Hq, int Hkv, int dh, int S, float log2_theta) {
    const int r = blockIdx.x;
    const int pos = row_pos[r], b = row_seq[r];
    const int half = dh >> 1;
    const int ncol = (Hq + 2 * Hkv) * dh;
    const float* pr = part + (size_t)r * ncol;
    auto col = [&](int c) {
        float v = 0.f;
        for (int s = 0; s < n_split; ++s) v += pr[s * split_stride + c];
        return v;
    };
    // q and k heads: (Hq + Hkv) * half pairs
    const int n_pairs = (Hq + Hkv) * half;
    for (int i = threadIdx.x; i < n_pairs; i += blockDim.x) {
        const int h = i / half, j = i - h * half;
        const float inv_freq = exp2f(-2.f * (float)j / (float)dh * log2_theta);
        float sn, cs;
        sincosf((float)pos * inv_freq, &sn, &cs);
        const float a = col(h * dh + j), bb = col(h * dh + j + half);
        const float ra = a * cs - bb * sn, rb = bb * cs + a * sn;
        if (h < Hq) {
            T* dst = q + ((size_t)r * Hq + h) * dh;
            dst[j] = from_f<T>(ra);
            dst[j + half] = from_f<T>(rb);
        } else {
            const int kh = h - Hq;
            T* dst = kcache + (((size_t)b * Hkv + kh) * S + pos) * dh;
            dst[j] = from_f<T>(ra);
            dst[j + half] = from_f<T>(rb);
        }
    }
    const int v0 = (Hq + Hkv) * dh;
    for (int i = threadIdx.x; i < Hkv * dh; i += blockDim.x) {
        const int kh = i / dh, c = i - kh * dh;
        vcache[(((size_t)b * Hkv + kh) * S + pos) * dh + c] = from_f<T>(col(v0 + i));
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
                                       int Hkv, int dh, int S) {
    extern __shared__ float sc[];                 // [n_vis] scores, then dh floats of q
    __shared__ float red[32];
    const int r = blockIdx.x, h = blockIdx.y;
    const int b = row_seq ? row_seq[r] : 0;
    const int v0 = vis_off ? vis_off[b] : 0;
    const int nv = vis_off ? vis_off[b + 1] - v0 : nv_single;
    const int kvh = h / (Hq / Hkv);
    const T* kb = kcache + ((size_t)b * Hkv + kvh) * S * dh;
    const T* vb = vcache + ((size_t)b * Hkv + kvh) * S * dh;
    float* qs = sc + nv;
    for (int c = threadIdx.x; c < dh; c += blockDim.x) qs[c] = to_f(q[((size_t)r * Hq + h) * dh + c]);
    __syncthreads();
    const float scale = rsqrtf((float)dh);
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
    float mx = -INFINITY;
    for (int j = wid; j < nv; j += nw) {
        const T* kr = kb + (size_t)vis_idx[v0 + j] * dh;
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
    for (int c = threadIdx.x; c < dh; c += blockDim.x) {
        float a = 0.f;
        for (int j = 0; j < nv; ++j) a += sc[j] * to_f(vb[(size_t)vis_idx[v0 + j] * dh + c]);
        a *= inv;
        const size_t o = ((size_t)r * Hq + h) * dh + c;
        out[o] = from_f<T>(a);
        if (tap) tap[o] = a;
    }
}

// ---------------------------------------------------------------- SwiGLU
template <typename T>
__global__ void swiglu_kernel(const float* __restrict__ part, int n_split, size_t split_stride,
                              T* __restrict__ h, int n_rows, int F) {
    const size_t total = (size_t)n_rows * F;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (size_t)gridDim.x * blockDim.x) {
        const size_t r = i / F, c = i - r * F;
        float g = 0.f, u = 0.f;
        for (int s = 0; s < n_split; ++s) {
            const float* p = part + s * split_stride + r * 2 * F;
            g += p[c];
            u += p[F + c];
        }
        h[i] = from_f<T>(g / (1.f + __expf(-g)) * u);
    }
}

__global__ void residual_add_kernel(float* __restrict__ x, const float* __restrict__ part, int n_split,
                                    size_t split_stride, float* __restrict__ tap, size_t total) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (size_t)gridDim.x * blockDim.x) {
        float v = x[i];
        for (int s = 0; s < n_split; ++s) v += part[s * split_stride + i];
        x[i] = v;
        if (tap) tap[i] = v;
    }
}

// ---------------------------------------------------------------- unmask reduction
// One block of 256 threads per active row, the same reduction order for every row:
// thread-strided scan, warp-shuffle tree, then the 8 warp results in lane order.
// The sum of exponentials is taken in double precision: it decides which rows are unmasked,
// and in double the ranking agrees with an exact evaluation of the same float logits except
// for gaps at the 1e-13 level (the work is a few million exps per step).
__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__global__ void rowstats_kernel(const float* __restrict__ logits, int V, int32_t* __restrict__ row_token,
                                double* __restrict__ row_sumexp) {
    __shared__ float s_val[8];
    __shared__ int s_idx[8];
    __shared__ double s_sum[8];
    __shared__ float s_max;
    const float* lr = logits + (size_t)blockIdx.x * V;
    float best = -INFINITY;
    int bi = 0x7fffffff;
    for (int v = threadIdx.x; v < V; v += 256) {
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
        row_token[blockIdx.x] = i;
    }
    __syncthreads();
    const double m = (double)s_max;
    double sum = 0.0;
    for (int v = threadIdx.x; v < V; v += 256) sum += exp((double)lr[v] - m);
    sum = warp_sum_d(sum);
    if (lane == 0) s_sum[w] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int j = 0; j < 8; ++j) t += s_sum[j];
        row_sumexp[blockIdx.x] = t;
    }
}

// One block per sequence.  rank(i) = #{j : s_j < s_i or (s_j == s_i and pos_j < pos_i)}; positions
// are ascending inside a sequence, so "pos_j < pos_i" is "j < i".
__global__ void select_kernel(const int32_t* __restrict__ row_token, const double* __restrict__ row_sumexp,
                              const int32_t* __restrict__ act_pos, const int32_t* __restrict__ act_off,
                              int n_single, int k, int32_t* __restrict__ ids, int S, int32_t* __restrict__ n_sel,
                              int32_t* __restrict__ sel_pos, int32_t* __restrict__ sel_token,
                              float* __restrict__ sel_conf, float* __restrict__ row_conf) {
    const int b = blockIdx.x;
    const int a0 = act_off ? act_off[b] : 0;
    const int n = act_off ? act_off[b + 1] - a0 : n_single;
    const int kk = min(k, n);
    if (threadIdx.x == 0) n_sel[b] = kk;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const double si = row_sumexp[a0 + i];
        const float conf = (float)(1.0 / si);
        if (row_conf) row_conf[a0 + i] = conf;
        int rank = 0;
        for (int j = 0; j < n; ++j) {
            const double sj = row_sumexp[a0 + j];
            rank += (sj < si || (sj == si && j < i)) ? 1 : 0;
        }
        if (rank < kk) {
            const int pos = act_pos[a0 + i], tok = row_token[a0 + i];
            sel_pos[b * k + rank] = pos;
            sel_token[b * k + rank] = tok;
            sel_conf[b * k + rank] = conf;
            if (ids) ids[(size_t)b * S + pos] = tok;
        }
    }
}

__device__ int32_t g_op_status;

}  // namespace

// ---------------------------------------------------------------- launchers

#define WD_DISPATCH(dtype, ...)                                   \
    do {                                                          \
        ++wd_launch_counter;                                      \
        if ((dtype) == WD_F32) { using T = float; __VA_ARGS__; }  \
        else { using T = __nv_bfloat16; __VA_ARGS__; }            \
    } while (0)

thread_local long long wd_launch_counter = 0;

void wd_launch_embed(int dtype, const void* embed, const int32_t* ids, const int32_t* row_seq,
                     const int32_t* row_pos, float* x, int n_rows, int d, int S, int vocab,
                     int32_t* status, cudaStream_t st) {
    if (n_rows <= 0) return;
    WD_DISPATCH(dtype, embed_kernel<T><<<n_rows, 256, 0, st>>>((const T*)embed, ids, row_seq, row_pos, x, d,
                                                               S, vocab, status));
}

void wd_launch_rmsnorm(int dtype, float* x, const float* part, int n_split, size_t split_stride,
                       const float* gain, float eps, void* xn, const int32_t* row_idx, int n_rows,
                       int d, cudaStream_t st) {
    if (n_rows <= 0) return;
    WD_DISPATCH(dtype, rmsnorm_kernel<T><<<n_rows, 256, 0, st>>>(x, part, n_split, split_stride, gain, eps,
                                                                 (T*)xn, row_idx, d));
}

void wd_launch_gemm_plain(int dtype, const void* x, const void* w, float* y, int rows, int n, int k,
                          int ldy, cudaStream_t st) {
    if (rows <= 0 || n <= 0) return;
    dim3 grid(wd_ceil_div(n, 64), wd_ceil_div(rows, 32));
    WD_DISPATCH(dtype, gemm_plain_kernel<T><<<grid, 256, 0, st>>>((const T*)x, (const T*)w, y, rows, n, k, ldy));
}

void wd_launch_rope_scatter(int dtype, const float* part, int n_split, size_t split_stride,
                            const int32_t* row_seq, const int32_t* row_pos, void* q, void* kcache,
                            void* vcache, int n_rows, int Hq, int Hkv, int dh, int S, float theta,
                            cudaStream_t st) {
    if (n_rows <= 0) return;
    const float l2 = log2f(theta);
    WD_DISPATCH(dtype, rope_scatter_kernel<T><<<n_rows, 256, 0, st>>>(part, n_split, split_stride, row_seq,
                                                                      row_pos, (T*)q, (T*)kcache, (T*)vcache,
                                                                      Hq, Hkv, dh, S, l2));
}

void wd_launch_attention_plain(int dtype, const void* q, const void* kcache, const void* vcache,
                               const int32_t* row_seq, const int32_t* vis_idx, const int32_t* vis_off,
                               void* out, float* tap, int n_rows, int max_vis, int Hq, int Hkv, int dh,
                               int S, cudaStream_t st) {
    if (n_rows <= 0) return;
    const size_t smem = (size_t)(max_vis + dh) * sizeof(float);
    dim3 grid(n_rows, Hq);
    ++wd_launch_counter;
    if (dtype == WD_F32) {
        if (smem > 48 * 1024)
            cudaFuncSetAttribute(attention_plain_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        attention_plain_kernel<float><<<grid, 128, smem, st>>>((const float*)q, (const float*)kcache,
                                                               (const float*)vcache, row_seq, vis_idx, vis_off,
                                                               (float*)out, tap, max_vis, Hq, Hkv, dh, S);
    } else {
        using T = __nv_bfloat16;
        if (smem > 48 * 1024)
            cudaFuncSetAttribute(attention_plain_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        attention_plain_kernel<T><<<grid, 128, smem, st>>>((const T*)q, (const T*)kcache, (const T*)vcache,
                                                           row_seq, vis_idx, vis_off, (T*)out, tap, max_vis, Hq, Hkv, dh,
                                                           S);
    }
}

void wd_launch_swiglu(int dtype, const float* part, int n_split, size_t split_stride, void* h,
                      int n_rows, int F, cudaStream_t st) {
    if (n_rows <= 0) return;
    const size_t total = (size_t)n_rows * F;
    const int blocks = (int)((total + 255) / 256 < 148 * 8 ? (total + 255) / 256 : 148 * 8);
    WD_DISPATCH(dtype, swiglu_kernel<T><<<blocks, 256, 0, st>>>(part, n_split, split_stride, (T*)h, n_rows, F));
}

void wd_launch_residual_add(float* x, const float* part, int n_split, size_t split_stride,
                            float* tap, int n_rows, int d, cudaStream_t st) {
    if (n_rows <= 0) return;
    const size_t total = (size_t)n_rows * d;
    const int blocks = (int)((total + 255) / 256 < 148 * 8 ? (total + 255) / 256 : 148 * 8);
    ++wd_launch_counter;
    residual_add_kernel<<<blocks, 256, 0, st>>>(x, part, n_split, split_stride, tap, total);
}

void wd_launch_rowstats(const float* logits, int n, int V, int32_t* row_token, double* row_sumexp,
                        cudaStream_t st) {
    if (n <= 0) return;
    ++wd_launch_counter;
    rowstats_kernel<<<n, 256, 0, st>>>(logits, V, row_token, row_sumexp);
}

void wd_launch_select(const int32_t* row_token, const double* row_sumexp, const int32_t* act_pos,
                      const int32_t* act_off, int n_single, int batch, int k, int32_t* ids, int S,
                      int32_t* n_sel, int32_t* sel_pos, int32_t* sel_token, float* sel_conf,
                      float* row_conf, cudaStream_t st) {
    if (batch <= 0) return;
    ++wd_launch_counter;
    select_kernel<<<batch, 256, 0, st>>>(row_token, row_sumexp, act_pos, act_off, n_single, k, ids, S, n_sel,
                                         sel_pos, sel_token, sel_conf, row_conf);
}

int32_t* wd_op_status_ptr() {
    int32_t* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_op_status) != cudaSuccess) return nullptr;
    return p;
}
