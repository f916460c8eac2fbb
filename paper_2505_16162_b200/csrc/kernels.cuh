// Device kernels of the KNN-SSD decode hot path (sm_100a).
//
// Conventions: activations, logits and every inter-kernel buffer are fp32; big
// weight matrices are bf16 (or fp32 for the small fp32 configuration), row-major
// [out][in]; K/V cache entries are stored in the weight dtype, rounded to nearest
// even when bf16.  Every reduction has a fixed order that does not depend on how
// many rows M a launch carries, so a row of a verification pass is computed
// exactly like the same row in a one-row pass.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace knnssd {

typedef unsigned short bf16_t;  // raw bf16 bit pattern

// Codes a kernel may leave in the device error word (besides the codes of bounded waits that gave up, all < 100).
enum { ERR_BAD_TOKEN = 101, ERR_BAD_LOGITS = 102 };

// Session scalars that live on the device so that a whole round can be enqueued
// without the host knowing the accepted count of the previous one.
struct DeviceState {
    int len;        // committed context length
    int produced;   // tokens emitted so far
    int last_accept;
    int last_next;
};

__device__ __forceinline__ float bf16_bits_to_float(unsigned int b) { return __uint_as_float(b << 16); }

// Round to nearest even on the bit pattern.  A NaN stays a NaN (the integer rounding alone would carry the all-ones
// NaN over into -0, and a non-finite activation would silently turn into zeros downstream).
__device__ __forceinline__ bf16_t float_to_bf16_rne(float f) {
    const unsigned int u = __float_as_uint(f);
    const unsigned int r = (u + 0x7FFFu + ((u >> 16) & 1u)) >> 16;
    return (bf16_t)((u & 0x7FFFFFFFu) > 0x7F800000u ? 0x7FC0u : r);
}

// 16-byte streaming load of weights: read-only path, do not keep in L1.
__device__ __forceinline__ uint4 ld_stream16(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

template <typename WT> struct WeightLoad;
template <> struct WeightLoad<bf16_t> {
    // eight consecutive weights starting at element index e (e % 8 == 0)
    static __device__ __forceinline__ void load8(const bf16_t *row, int e, float (&w)[8]) {
        const uint4 v = ld_stream16(row + e);
        w[0] = __uint_as_float(v.x << 16); w[1] = __uint_as_float(v.x & 0xFFFF0000u);
        w[2] = __uint_as_float(v.y << 16); w[3] = __uint_as_float(v.y & 0xFFFF0000u);
        w[4] = __uint_as_float(v.z << 16); w[5] = __uint_as_float(v.z & 0xFFFF0000u);
        w[6] = __uint_as_float(v.w << 16); w[7] = __uint_as_float(v.w & 0xFFFF0000u);
    }
    static __device__ __forceinline__ float load1(const bf16_t *p) { return bf16_bits_to_float(*p); }
    static __device__ __forceinline__ void store1(bf16_t *p, float f) { *p = float_to_bf16_rne(f); }
};
template <> struct WeightLoad<float> {
    static __device__ __forceinline__ void load8(const float *row, int e, float (&w)[8]) {
        const uint4 a = ld_stream16(row + e), b = ld_stream16(row + e + 4);
        w[0] = __uint_as_float(a.x); w[1] = __uint_as_float(a.y); w[2] = __uint_as_float(a.z); w[3] = __uint_as_float(a.w);
        w[4] = __uint_as_float(b.x); w[5] = __uint_as_float(b.y); w[6] = __uint_as_float(b.z); w[7] = __uint_as_float(b.w);
    }
    static __device__ __forceinline__ float load1(const float *p) { return *p; }
    static __device__ __forceinline__ void store1(float *p, float f) { *p = f; }
};

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

// ---------------------------------------------------------------------------------------------
// Embedding gather + rotary table.  x[m][:] = E[tok[m]][:];  cs[m][i] = (cos, sin)(pos_m * inv_freq[i]),
// pos_m = state->len + pos_off + m.  Angles in fp64 so that long contexts lose nothing.
// grid = M blocks.
// ---------------------------------------------------------------------------------------------
template <typename WT>
__global__ void embed_rope_kernel(const WT *__restrict__ E, const int *__restrict__ tok, int d, float *__restrict__ x,
                                  const DeviceState *__restrict__ st, int pos_off, const double *__restrict__ inv_freq,
                                  int half, float2 *__restrict__ cs, int vocab, int *__restrict__ err) {
    const int m = blockIdx.x;
    int t = tok[m];
    if (t < 0 || t >= vocab) {                 // never gather outside the table: report and read row 0 instead
        if (threadIdx.x == 0) atomicExch(err, ERR_BAD_TOKEN);
        t = 0;
    }
    const WT *row = E + (size_t)t * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) x[(size_t)m * d + i] = WeightLoad<WT>::load1(row + i);
    const int pos = st->len + pos_off + m;
    for (int i = threadIdx.x; i < half; i += blockDim.x) {
        double s, c;
        sincos((double)pos * inv_freq[i], &s, &c);
        cs[m * half + i] = make_float2((float)c, (float)s);
    }
}

// ---------------------------------------------------------------------------------------------
// Weight-streaming linear kernel:  for every output unit u and row m < M
//     acc = sum_i W[u][i] * (gain[i] * x[m][i]);   then an epilogue:
//   EPI_STORE : y[m][u]  = acc * rinv[m]                 (rinv = 1 if no gain: plain linear)
//   EPI_ADD   : y[m][u] += acc                           (residual update, output projection)
//   EPI_SWIGLU: y[m][u]  = silu(g) * v, g and v the results of rows u of W[0] (gate) and W[1] (up)
// rinv[m] = 1/sqrt(mean_i x[m][i]^2 + eps) is RMSNorm's scalar, applied after the dot product
// (the norm is linear in x up to that scalar), so the normalised activations never touch memory.
// Up to three stacked matrices (q, k, v) share one launch; unit u of the stack maps to a row of one of them.
// One warp owns a unit: lanes stride over the row in 16-byte pieces, fp32 FMAs, shuffle reduction.
// The FMA order of a given (u, m) depends only on n_in, never on M or on the grid.
// ---------------------------------------------------------------------------------------------
enum { EPI_STORE = 0, EPI_ADD = 1, EPI_SWIGLU = 2 };

struct LinearArgs {
    const void *W[3];
    int rows[3];        // rows of each stacked matrix (unused entries 0)
    int units;          // output units (for SWIGLU: d_ff; else the sum of rows)
    int n_in;
    const float *x;     // [M][n_in]
    const float *gain;  // [n_in] or nullptr
    float eps;
    float *y;           // [M][units]
    int epi;
    int M;
};

template <typename WT, int MT>
__global__ void __launch_bounds__(256) linear_kernel(const LinearArgs a) {
    __shared__ float s_red[8][MT];
    __shared__ float s_rinv[MT];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = a.n_in;
    const bool normed = a.gain != nullptr;

    if (normed) {
        float ss[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            const float *xr = a.x + (size_t)min(m, a.M - 1) * K;
            float s = 0.f;
            for (int i = tid * 4; i < K; i += 256 * 4) {
                const float4 v = __ldg(reinterpret_cast<const float4 *>(xr + i));
                s = fmaf(v.x, v.x, s); s = fmaf(v.y, v.y, s); s = fmaf(v.z, v.z, s); s = fmaf(v.w, v.w, s);
            }
            ss[m] = warp_sum(s);
        }
        if (lane == 0)
#pragma unroll
            for (int m = 0; m < MT; ++m) s_red[warp][m] = ss[m];
        __syncthreads();
        if (tid < MT) {
            float s = 0.f;
            for (int w = 0; w < 8; ++w) s += s_red[w][tid];
            s_rinv[tid] = 1.0f / sqrtf(s / (float)K + a.eps);
        }
        __syncthreads();
    }

    const int nwarps = gridDim.x * 8, gw = blockIdx.x * 8 + warp;
    const int u0 = (int)(((long long)gw * a.units) / nwarps), u1 = (int)(((long long)(gw + 1) * a.units) / nwarps);
    const bool swiglu = a.epi == EPI_SWIGLU;
    const int step = swiglu ? 1 : 2;
    const int nchunks = K >> 3;

    for (int u = u0; u < u1; u += step) {
        const WT *wrow[2];
        int nslots;
        if (swiglu) {
            wrow[0] = reinterpret_cast<const WT *>(a.W[0]) + (size_t)u * K;
            wrow[1] = reinterpret_cast<const WT *>(a.W[1]) + (size_t)u * K;
            nslots = 2;
        } else {
            nslots = min(2, u1 - u);
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                int uu = u + min(r, nslots - 1), which = 0;
                if (uu >= a.rows[0]) { uu -= a.rows[0]; which = 1; }
                if (which == 1 && uu >= a.rows[1]) { uu -= a.rows[1]; which = 2; }
                wrow[r] = reinterpret_cast<const WT *>(a.W[which]) + (size_t)uu * K;
            }
        }
        float acc[2][MT];
#pragma unroll
        for (int r = 0; r < 2; ++r)
#pragma unroll
            for (int m = 0; m < MT; ++m) acc[r][m] = 0.f;

        for (int c = lane; c < nchunks; c += 32) {
            const int e = c << 3;
            float w0[8], w1[8];
            WeightLoad<WT>::load8(wrow[0], e, w0);
            WeightLoad<WT>::load8(wrow[1], e, w1);
            if (normed) {
                const float4 g0 = __ldg(reinterpret_cast<const float4 *>(a.gain + e));
                const float4 g1 = __ldg(reinterpret_cast<const float4 *>(a.gain + e + 4));
                const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
                for (int j = 0; j < 8; ++j) { w0[j] *= g[j]; w1[j] *= g[j]; }
            }
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                const float *xr = a.x + (size_t)min(m, a.M - 1) * K + e;
                const float4 x0 = __ldg(reinterpret_cast<const float4 *>(xr));
                const float4 x1 = __ldg(reinterpret_cast<const float4 *>(xr + 4));
                const float xv[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    acc[0][m] = fmaf(w0[j], xv[j], acc[0][m]);
                    acc[1][m] = fmaf(w1[j], xv[j], acc[1][m]);
                }
            }
        }
#pragma unroll
        for (int r = 0; r < 2; ++r)
#pragma unroll
            for (int m = 0; m < MT; ++m) acc[r][m] = warp_sum(acc[r][m]);

        if (lane == 0) {
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                if (m >= a.M) break;
                const float ri = normed ? s_rinv[m] : 1.0f;
                float *yr = a.y + (size_t)m * a.units;
                if (swiglu) {
                    const float g = acc[0][m] * ri, v = acc[1][m] * ri;
                    yr[u] = g / (1.0f + expf(-g)) * v;
                } else {
                    for (int r = 0; r < nslots; ++r) {
                        const float val = acc[r][m] * ri;
                        if (a.epi == EPI_ADD) yr[u + r] += val; else yr[u + r] = val;
                    }
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// RoPE + KV append.  qkv[m] = [q (H heads) | k (Hkv heads) | v (Hkv heads)], head_dim hd each.
// q is rotated in place; k is rotated and written to the cache at position pos_m; v is written as is.
// Pairing (i, i + hd/2).  grid = (H + 2*Hkv, M), block = hd/2 threads.
// Cache layout: [kv_head][max_seq][hd] for this layer.
// ---------------------------------------------------------------------------------------------
template <typename WT>
__global__ void rope_kv_kernel(float *__restrict__ qkv, int H, int Hkv, int hd, const float2 *__restrict__ cs,
                               WT *__restrict__ kc, WT *__restrict__ vc, int max_seq,
                               const DeviceState *__restrict__ st, int pos_off) {
    const int head = blockIdx.x, m = blockIdx.y, i = threadIdx.x, half = hd >> 1;
    const int pos = st->len + pos_off + m;
    float *base = qkv + (size_t)m * (H + 2 * Hkv) * hd + (size_t)head * hd;
    if (head < H + Hkv) {
        const float2 c = cs[m * half + i];
        const float a = base[i], b = base[i + half];
        const float ra = a * c.x - b * c.y, rb = b * c.x + a * c.y;
        if (head < H) {
            base[i] = ra;
            base[i + half] = rb;
        } else {
            WT *dst = kc + ((size_t)(head - H) * max_seq + pos) * hd;
            WeightLoad<WT>::store1(dst + i, ra);
            WeightLoad<WT>::store1(dst + i + half, rb);
        }
    } else {
        WT *dst = vc + ((size_t)(head - H - Hkv) * max_seq + pos) * hd;
        WeightLoad<WT>::store1(dst + i, base[i]);
        WeightLoad<WT>::store1(dst + i + half, base[i + half]);
    }
}

// ---------------------------------------------------------------------------------------------
// Attention over the KV cache, split along the context at fixed absolute boundaries of ATT_CHUNK
// positions.  Row m (query at position pos_m) attends to positions [0, pos_m].  Each (head, m, split)
// block produces an un-normalised partial (max, sum, o[hd]); attn_merge_kernel combines the splits in
// index order.  grid = (H, M, n_splits), block = 128 threads.
// ---------------------------------------------------------------------------------------------
constexpr int ATT_CHUNK = 256;

template <typename WT, int HD>
__global__ void __launch_bounds__(128) attn_partial_kernel(const float *__restrict__ qkv, int H, int Hkv,
                                                            const WT *__restrict__ kc, const WT *__restrict__ vc,
                                                            int max_seq, const DeviceState *__restrict__ st, int pos_off,
                                                            float *__restrict__ part_o, float2 *__restrict__ part_ml,
                                                            int n_splits) {
    const int head = blockIdx.x, m = blockIdx.y, split = blockIdx.z;
    const int T = st->len + pos_off + m + 1;           // positions attended: [0, T)
    const int t0 = split * ATT_CHUNK;
    if (t0 >= T) return;
    const int t1 = min(T, t0 + ATT_CHUNK), nt = t1 - t0;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int kvh = head / (H / Hkv);
    __shared__ float s_q[HD];
    __shared__ float s_p[ATT_CHUNK];
    __shared__ float s_w[4];
    const float *q = qkv + (size_t)m * (H + 2 * Hkv) * HD + (size_t)head * HD;
    if (tid < HD) s_q[tid] = q[tid];
    __syncthreads();
    const WT *kbase = kc + ((size_t)kvh * max_seq + t0) * HD;
    const WT *vbase = vc + ((size_t)kvh * max_seq + t0) * HD;
    const float scale = 1.0f / sqrtf((float)HD);
    constexpr int EPL = HD / 32;             // elements per lane
    float qv[EPL];
#pragma unroll
    for (int j = 0; j < EPL; ++j) qv[j] = s_q[lane * EPL + j];
    for (int t = warp; t < nt; t += 4) {
        const WT *kr = kbase + (size_t)t * HD + lane * EPL;
        float s = 0.f;
#pragma unroll
        for (int j = 0; j < EPL; ++j) s = fmaf(qv[j], WeightLoad<WT>::load1(kr + j), s);
        s = warp_sum(s);
        if (lane == 0) s_p[t] = s * scale;
    }
    __syncthreads();
    float mx = -INFINITY;
    for (int t = tid; t < nt; t += 128) mx = fmaxf(mx, s_p[t]);
    mx = warp_max(mx);
    if (lane == 0) s_w[warp] = mx;
    __syncthreads();
    mx = fmaxf(fmaxf(s_w[0], s_w[1]), fmaxf(s_w[2], s_w[3]));
    __syncthreads();
    float sum = 0.f;
    for (int t = tid; t < nt; t += 128) {
        const float p = expf(s_p[t] - mx);
        s_p[t] = p;
        sum += p;
    }
    sum = warp_sum(sum);
    if (lane == 0) s_w[warp] = sum;
    __syncthreads();
    sum = (s_w[0] + s_w[1]) + (s_w[2] + s_w[3]);
    const size_t pidx = ((size_t)m * H + head) * n_splits + split;
    if (tid < HD) {
        float o = 0.f;
        for (int t = 0; t < nt; ++t) o = fmaf(s_p[t], WeightLoad<WT>::load1(vbase + (size_t)t * HD + tid), o);
        part_o[pidx * HD + tid] = o;
    }
    if (tid == 0) part_ml[pidx] = make_float2(mx, sum);
}

// grid = (H, M), block = HD threads.  out[m][head*HD + e] = sum_s o_s[e] e^{m_s - m*} / sum_s l_s e^{m_s - m*}
template <int HD>
__global__ void attn_merge_kernel(const float *__restrict__ part_o, const float2 *__restrict__ part_ml, int H,
                                  const DeviceState *__restrict__ st, int pos_off, int n_splits,
                                  float *__restrict__ out) {
    const int head = blockIdx.x, m = blockIdx.y, e = threadIdx.x;
    const int T = st->len + pos_off + m + 1;
    const int ns = min(n_splits, (T + ATT_CHUNK - 1) / ATT_CHUNK);
    const size_t base = ((size_t)m * H + head) * n_splits;
    float mx = -INFINITY;
    for (int s = 0; s < ns; ++s) mx = fmaxf(mx, part_ml[base + s].x);
    float l = 0.f, o = 0.f;
    for (int s = 0; s < ns; ++s) {
        const float2 ml = part_ml[base + s];
        const float w = expf(ml.x - mx);
        l = fmaf(ml.y, w, l);
        o = fmaf(part_o[(base + s) * HD + e], w, o);
    }
    out[(size_t)m * H * HD + (size_t)head * HD + e] = o / l;
}

// ---------------------------------------------------------------------------------------------
// RMSNorm of M rows written out (only where the normalised hidden state itself is an output:
// the pooled vector and the hidden-state parity output).  grid = M, block = 256.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) rmsnorm_rows_kernel(const float *__restrict__ x, const float *__restrict__ gain,
                                                           int d, float eps, float *__restrict__ h) {
    __shared__ float s_red[8];
    const int m = blockIdx.x, tid = threadIdx.x;
    const float *xr = x + (size_t)m * d;
    float s = 0.f;
    for (int i = tid * 4; i < d; i += 1024) {
        const float4 v = *reinterpret_cast<const float4 *>(xr + i);
        s = fmaf(v.x, v.x, s); s = fmaf(v.y, v.y, s); s = fmaf(v.z, v.z, s); s = fmaf(v.w, v.w, s);
    }
    s = warp_sum(s);
    if ((tid & 31) == 0) s_red[tid >> 5] = s;
    __syncthreads();
    float tot = 0.f;
    for (int w = 0; w < 8; ++w) tot += s_red[w];
    const float rinv = 1.0f / sqrtf(tot / (float)d + eps);
    for (int i = tid; i < d; i += 256) h[(size_t)m * d + i] = xr[i] * rinv * gain[i];
}

// Running fp64 sum of hidden rows in row order (the pooled vector's numerator).  grid = ceil(d/256).
__global__ void pool_accumulate_kernel(const float *__restrict__ h, int M, int d, double *__restrict__ sum, int overwrite) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= d) return;
    double s = overwrite ? 0.0 : sum[i];
    for (int m = 0; m < M; ++m) s += (double)h[(size_t)m * d + i];
    sum[i] = s;
}
__global__ void pool_finish_kernel(const double *__restrict__ sum, int d, double inv_count, float *__restrict__ v) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < d) v[i] = (float)(sum[i] * inv_count);
}

// ---------------------------------------------------------------------------------------------
// Greedy arg-max per row, lowest index on ties.  Stage 1: grid = (NB, M) blocks scan slices;
// stage 2: grid = M blocks of 32 threads fold the NB partials.
// ---------------------------------------------------------------------------------------------
// A NaN never wins a comparison, so it is passed over like -inf.  A row without any value above -inf (all NaN or
// -inf) leaves the index at its start value; argmax_checked turns that into token 0 and an error code.
__device__ __forceinline__ void argmax_fold(float &bv, int &bi, float v, int i) {
    if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
}
__device__ __forceinline__ int argmax_checked(int bi, int V, int *err) {
    if (bi < 0 || bi >= V) { atomicExch(err, ERR_BAD_LOGITS); return 0; }
    return bi;
}

__global__ void __launch_bounds__(256) argmax_partial_kernel(const float *__restrict__ logits, int V, int NB,
                                                             float *__restrict__ pv, int *__restrict__ pi) {
    __shared__ float s_v[8];
    __shared__ int s_i[8];
    const int b = blockIdx.x, m = blockIdx.y, tid = threadIdx.x;
    const int per = (V + NB - 1) / NB, i0 = b * per, i1 = min(V, i0 + per);
    const float *row = logits + (size_t)m * V;
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int i = i0 + tid; i < i1; i += 256) argmax_fold(bv, bi, row[i], i);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        argmax_fold(bv, bi, ov, oi);
    }
    if ((tid & 31) == 0) { s_v[tid >> 5] = bv; s_i[tid >> 5] = bi; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < 8; ++w) argmax_fold(bv, bi, s_v[w], s_i[w]);
        pv[m * NB + b] = bv;
        pi[m * NB + b] = bi;
    }
}

__global__ void argmax_final_kernel(const float *__restrict__ pv, const int *__restrict__ pi, int NB, int *__restrict__ out,
                                    int V, int *__restrict__ err) {
    const int m = blockIdx.x, lane = threadIdx.x;
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int b = lane; b < NB; b += 32) argmax_fold(bv, bi, pv[m * NB + b], pi[m * NB + b]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        argmax_fold(bv, bi, ov, oi);
    }
    if (lane == 0) out[m] = argmax_checked(bi, V, err);
}

// ---------------------------------------------------------------------------------------------
// Greedy acceptance and rollback (one thread).  chain[0] = pending token, chain[1..k] = drafted tokens,
// target[j] = the full model's greedy token after row j.  a = longest agreeing prefix; the emitted tokens
// d_0..d_{a-1}, target[a] are appended to out_tokens; target[a] becomes the pending token; the committed
// length grows by a + 1 (rows beyond it are dead).
// ---------------------------------------------------------------------------------------------
__global__ void accept_kernel(int *__restrict__ chain, const int *__restrict__ target, int k, DeviceState *__restrict__ st,
                              int *__restrict__ out_tokens, int out_cap, int *__restrict__ accept_log, int round_idx) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    int a = 0;
    while (a < k && target[a] == chain[a + 1]) ++a;
    const int next = target[a];
    int p = st->produced;
    for (int j = 0; j < a && p < out_cap; ++j) out_tokens[p++] = chain[j + 1];
    if (p < out_cap) out_tokens[p++] = next;
    st->produced = p;
    st->len += a + 1;
    st->last_accept = a;
    st->last_next = next;
    chain[0] = next;
    if (accept_log) accept_log[round_idx] = a;
}

// ---------------------------------------------------------------------------------------------
// Cosine top-1 over the anchors.  One warp per anchor: dot(v, a) / (|v| |a|) with the anchor's
// inverse norm precomputed (or computed here when inv_norm == nullptr).  Then one block folds the
// n cosines to the arg-max, lowest index on ties.  A zero / non-finite norm sets *flag.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) cosine_scores_kernel(const float *__restrict__ v, const float *__restrict__ anchors,
                                                            const float *__restrict__ inv_norm, int n, int d,
                                                            float *__restrict__ cosines, int *__restrict__ flag) {
    const int lane = threadIdx.x & 31, a = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (a >= n) return;
    const float *ar = anchors + (size_t)a * d;
    float dot = 0.f, vv = 0.f, aa = 0.f;
    for (int i = lane; i < d; i += 32) {
        const float x = v[i], y = ar[i];
        dot = fmaf(x, y, dot);
        vv = fmaf(x, x, vv);
        aa = fmaf(y, y, aa);
    }
    dot = warp_sum(dot); vv = warp_sum(vv); aa = warp_sum(aa);
    if (lane == 0) {
        const bool bad = !(vv > 0.f) || !isfinite(vv) || !(aa > 0.f) || !isfinite(aa);
        if (bad) { *flag = 1; cosines[a] = -INFINITY; return; }
        const float ia = inv_norm ? inv_norm[a] : 1.0f / sqrtf(aa);
        cosines[a] = dot * (1.0f / sqrtf(vv)) * ia;
    }
}

// out[0] = best flat index (as int bits), out[1] = cosine bits.
__global__ void cosine_argmax_kernel(const float *__restrict__ cosines, int n, int *__restrict__ out) {
    __shared__ float s_v[8];
    __shared__ int s_i[8];
    const int tid = threadIdx.x;
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int i = tid; i < n; i += 256) argmax_fold(bv, bi, cosines[i], i);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        argmax_fold(bv, bi, ov, oi);
    }
    if ((tid & 31) == 0) { s_v[tid >> 5] = bv; s_i[tid >> 5] = bi; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < 8; ++w) argmax_fold(bv, bi, s_v[w], s_i[w]);
        out[0] = bi;
        out[1] = __float_as_int(bv);
    }
}

__global__ void anchor_inv_norm_kernel(const float *__restrict__ anchors, int n, int d, float *__restrict__ inv_norm,
                                       int *__restrict__ flag) {
    const int lane = threadIdx.x & 31, a = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (a >= n) return;
    float aa = 0.f;
    for (int i = lane; i < d; i += 32) { const float y = anchors[(size_t)a * d + i]; aa = fmaf(y, y, aa); }
    aa = warp_sum(aa);
    if (lane == 0) {
        if (!(aa > 0.f) || !isfinite(aa)) { *flag = 1; inv_norm[a] = 0.f; }
        else inv_norm[a] = 1.0f / sqrtf(aa);
    }
}

__global__ void set_state_kernel(DeviceState *st, int len, int produced) {
    st->len = len; st->produced = produced; st->last_accept = 0; st->last_next = -1;
}
__global__ void emit_first_token_kernel(const int *chain, DeviceState *st, int *out_tokens, int len) {
    out_tokens[0] = chain[0]; st->produced = 1; st->len = len;
}

}  // namespace knnssd
