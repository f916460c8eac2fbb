// Stochastic speculative sampling on the logits of the draft and verification passes (sm_100a).
//
// The paper's set-up lists temperature 0.2 and top-p 0.85 (App. C.1) and the method is to leave the distribution of
// the generated tokens unchanged (Sec. 1, Sec. 3.1); it prints no acceptance rule for the sampled case.  The rule
// used is the one of speculative sampling with that property: p and q are the full and the draft model's next-token
// distributions after temperature and nucleus filtering; a draft d ~ q is kept with probability min(1, p(d) / q(d));
// at the first rejection the token is drawn from the normalised positive part of p - q; if every draft is kept one
// more token is drawn from p.  Random numbers are inputs (one uniform per draw), consumed through the inverse CDF in
// token-id order, so that the choices are reproducible.
//
// All three kernels run one block of 1024 threads per row: the work is a few passes over <= 152 k floats that sit in
// L2, far below the cost of the pass that produced the logits.  Every sum has a fixed order.
#pragma once
#include "kernels.cuh"

namespace knnssd {
namespace sampling {

constexpr int NT = 1024;

// Sum over the block in a fixed order (thread partials -> warp trees -> warps in order); every thread gets the result.
__device__ __forceinline__ float block_sum(float v, float *sh) {
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) t += sh[w];
    return t;
}
__device__ __forceinline__ float block_max(float v, float *sh) {
    v = warp_max(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = sh[0];
#pragma unroll
    for (int w = 1; w < NT / 32; ++w) t = fmaxf(t, sh[w]);
    return t;
}
__device__ __forceinline__ int block_count(int v, int *sh) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    int t = 0;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) t += sh[w];
    return t;
}

// probs[row] = nucleus-filtered softmax(logits[row] / temperature), renormalised.  A token is kept iff the probability
// mass of the tokens ranked before it (higher probability first, lower id first among equals) is below top_p.
// The mass above a value is a decreasing step function of the value, so the smallest kept probability x0 is found by
// bisection over the bit patterns of positive floats; tokens whose probability equals x0 are ranked by id.
// grid = rows, NT threads.  probs doubles as scratch for the unfiltered probabilities.
__global__ void __launch_bounds__(NT) filtered_probs_kernel(const float *__restrict__ logits, int V, float inv_temperature, float top_p,
                                                            float *__restrict__ probs) {
    __shared__ float shf[NT / 32];
    __shared__ int shi[NT / 32];
    const float *l = logits + (size_t)blockIdx.x * V;
    float *p = probs + (size_t)blockIdx.x * V;
    const int tid = threadIdx.x;
    float m = -INFINITY;
    for (int i = tid; i < V; i += NT) m = fmaxf(m, l[i]);
    m = block_max(m, shf);
    float s = 0.f;
    for (int i = tid; i < V; i += NT) {
        const float e = expf((l[i] - m) * inv_temperature);
        p[i] = e;
        s += e;
    }
    s = block_sum(s, shf);
    float pmax = 0.f;
    for (int i = tid; i < V; i += NT) {
        const float v = p[i] / s;
        p[i] = v;
        pmax = fmaxf(pmax, v);
    }
    pmax = block_max(pmax, shf);
    auto mass_above = [&](float x) {
        float a = 0.f;
        for (int i = tid; i < V; i += NT) { const float v = p[i]; a += v > x ? v : 0.f; }
        return block_sum(a, shf);
    };
    // smallest x (as a bit pattern) with mass_above(x) < top_p; mass_above(pmax) = 0
    unsigned lo = 0u, hi = __float_as_uint(pmax);
    if (mass_above(0.f) < top_p) hi = 0u;
    while (hi > lo + 1u) {
        const unsigned mid = lo + (hi - lo) / 2u;
        if (mass_above(__uint_as_float(mid)) < top_p) hi = mid; else lo = mid;
    }
    const float x0 = __uint_as_float(hi);
    // tokens at exactly x0: the n-th of them by id (n = 0, 1, ..) is kept iff mass_above(x0) + n x0 < top_p
    const float a0 = mass_above(x0);
    int c = 0;
    for (int i = tid; i < V; i += NT) c += p[i] == x0 ? 1 : 0;
    c = block_count(c, shi);
    int nk = 0;
    for (int n = tid; n < c; n += NT) nk += (a0 + (float)n * x0 < top_p) ? 1 : 0;
    nk = block_count(nk, shi);
    if (nk < 1) nk = 1;                       // the first token at x0 is kept by the definition of x0
    int id_cut = V;                           // tokens at x0 with id < id_cut are kept
    if (nk < c) {
        int jl = 0, jh = V;                   // smallest J with #{j < J : p_j == x0} >= nk
        while (jh > jl + 1) {
            const int jm = jl + (jh - jl) / 2;
            int g = 0;
            for (int i = tid; i < jm; i += NT) g += p[i] == x0 ? 1 : 0;
            g = block_count(g, shi);
            if (g >= nk) jh = jm; else jl = jm;
        }
        id_cut = jh;
    }
    float z = 0.f;
    for (int i = tid; i < V; i += NT) {
        const float v = p[i];
        z += (v > x0 || (v == x0 && i < id_cut)) ? v : 0.f;
    }
    z = block_sum(z, shf);
    for (int i = tid; i < V; i += NT) {
        const float v = p[i];
        p[i] = (v > x0 || (v == x0 && i < id_cut)) ? v / z : 0.f;
    }
}

// Inverse CDF in token-id order: the smallest id x with w_0 + .. + w_x > u * sum(w); w_i = a_i (b == nullptr) or
// max(a_i - b_i, 0), falling back to a if that is zero everywhere.  Thread t owns the ids [t C, (t + 1) C).
// Called by all NT threads of a block; every thread returns the token.
__device__ __forceinline__ int block_sample(const float *__restrict__ a, const float *__restrict__ b, int V, float u, float *shf, int *shi) {
    __shared__ float part[NT];
    __shared__ int s_tok, s_last;
    const int tid = threadIdx.x, C = (V + NT - 1) / NT, i0 = tid * C, i1 = min(V, i0 + C);
    bool use_b = b != nullptr;
    for (int attempt = 0; attempt < 2; ++attempt) {
        float s = 0.f;
        int last = -1;
        for (int i = i0; i < i1; ++i) {
            const float w = use_b ? fmaxf(a[i] - b[i], 0.f) : a[i];
            if (w > 0.f) last = i;
            s += w;
        }
        part[tid] = s;
        // last id with weight, over the block
        int lm = last;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) lm = max(lm, __shfl_xor_sync(0xffffffffu, lm, o));
        __syncthreads();
        if ((tid & 31) == 0) shi[tid >> 5] = lm;
        __syncthreads();
        if (tid == 0) {
            int t = -1;
            for (int w = 0; w < NT / 32; ++w) t = max(t, shi[w]);
            s_last = t;
            // exclusive scan of the thread sums in thread order
            float run = 0.f;
            for (int k = 0; k < NT; ++k) { const float v = part[k]; part[k] = run; run += v; }
            shf[0] = run;
            s_tok = -1;
        }
        __syncthreads();
        const float total = shf[0];
        if (use_b && !(total > 0.f)) { use_b = false; __syncthreads(); continue; }
        const float target = u * total;
        const float excl = part[tid], incl = tid + 1 < NT ? part[tid + 1] : total;
        // the chunk in which the running sum first exceeds the target
        if (excl <= target && incl > target && i0 < i1) {
            float acc = excl;
            int tok = -1;
            for (int i = i0; i < i1; ++i) {
                acc += use_b ? fmaxf(a[i] - b[i], 0.f) : a[i];
                if (acc > target) { tok = i; break; }
            }
            if (tok >= 0) atomicMax(&s_tok, tok);       // at most one chunk qualifies; atomic only for safety
        }
        __syncthreads();
        const int tok = s_tok >= 0 ? s_tok : s_last;     // target rounded up to the total: the last id with weight
        __syncthreads();
        return tok;
    }
    return 0;
}

// token <- draw from weights w[V] with the uniform *u_ptr (u_val if u_ptr is null).  One block.
__global__ void __launch_bounds__(NT) sample_kernel(const float *__restrict__ w, int V, const float *__restrict__ u_ptr, float u_val,
                                                    int *__restrict__ token) {
    __shared__ float shf[NT / 32];
    __shared__ int shi[NT / 32];
    const int tok = block_sample(w, nullptr, V, u_ptr ? *u_ptr : u_val, shf, shi);
    if (threadIdx.x == 0) *token = tok < 0 ? 0 : tok;
}

// One verification round of speculative sampling.  p [k+1][V], q [k][V] filtered distributions, drafts [k] (device),
// u_accept [k] (device), u_final (*u_final_ptr if given).  out[0] = number of drafts kept, out[1] = the token emitted
// after them.  One block.
__global__ void __launch_bounds__(NT) spec_accept_kernel(const float *__restrict__ p, const float *__restrict__ q, const int *__restrict__ drafts,
                                                         int k, int V, const float *__restrict__ u_accept,
                                                         const float *__restrict__ u_final_ptr, float u_final, int *__restrict__ out) {
    if (u_final_ptr) u_final = *u_final_ptr;
    __shared__ float shf[NT / 32];
    __shared__ int shi[NT / 32];
    __shared__ int s_rej;
    if (threadIdx.x == 0) {
        int j = 0;
        for (; j < k; ++j) {
            int d = drafts[j];
            if (d < 0 || d >= V) break;                          // a token outside the vocabulary is never kept
            if (!(u_accept[j] * q[(size_t)j * V + d] < p[(size_t)j * V + d])) break;
        }
        s_rej = j;
    }
    __syncthreads();
    const int j = s_rej;
    const int tok = j < k ? block_sample(p + (size_t)j * V, q + (size_t)j * V, V, u_final, shf, shi)
                          : block_sample(p + (size_t)k * V, nullptr, V, u_final, shf, shi);
    if (threadIdx.x == 0) { out[0] = j; out[1] = tok < 0 ? 0 : tok; }
}

// The round's result into the session (one thread): res[0] = drafts kept, res[1] = the token after them; chain[1 .. k]
// the drafts.  Same bookkeeping as the greedy accept step.
__global__ void commit_sampled_kernel(int *__restrict__ chain, const int *__restrict__ res, DeviceState *__restrict__ st,
                                      int *__restrict__ out_tokens, int out_cap, int *__restrict__ accept_log, int round_idx) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    const int a = res[0], next = res[1];
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

}  // namespace sampling
}  // namespace knnssd
