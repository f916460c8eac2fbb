// One decoder pass as ONE persistent kernel (sm_100a): one CTA per SM, launched cooperatively.
//
// The pass is a list of operations (embedding, the linear maps of the retained sublayers, KV-cache attention,
// LM head, arg-max) that every CTA walks in the same order.  Inside a CTA the producer warp walks the list on
// its own and streams the weights of every linear map into the shared-memory ring as fast as stages free up:
// weights do not depend on activations, so it runs ahead across operation boundaries.  The eight consumer
// warps execute the operations; between operations that depend on each other they meet all other CTAs at a
// grid-wide barrier (a monotonic counter in global memory).  While consumers wait there - or work through an
// attention operation, which reads the KV cache with plain loads - the ring keeps filling with the next linear
// map's weights, so the HBM stream does not stop at operation boundaries.
//
// Sublayers the skip mask leaves out are simply absent from the list: none of their weights is ever touched.
//
// Every wait is bounded.  A barrier or ring wait that gives up raises a device-wide abort word; every CTA then
// falls through the rest of the list without waiting or touching memory, and the host reports a timeout.
#pragma once
#include "linear_stream.cuh"

namespace knnssd {
namespace pass {

using stream::LinPhase;
using stream::Ring;
using stream::NCW;

constexpr int MAXM = 8;            // rows per pass this kernel handles
constexpr int SEGP = 64;           // attention: positions per segment (fixed absolute boundaries)
constexpr unsigned BAR_SPIN_LIMIT = 4000000u;

enum { OP_EMBED = 0, OP_LINEAR = 1, OP_ATTN = 2, OP_HIDDEN = 3, OP_ARGMAX = 4 };

struct Op {
    int type;
    int barrier_after;   // 1: all CTAs meet before the next operation starts
    int is_head;         // OP_LINEAR: the LM head (runs on rows head_row0.. only)
    int layer;
    LinPhase lin;        // OP_LINEAR
    bf16_t *kc, *vc;     // OP_ATTN: this layer's cache [n_kv_heads][max_seq][head_dim]
};

struct Model {           // what does not change from pass to pass
    const bf16_t *tok_embed;
    const float *final_norm;
    float rms_eps;
    int d_model, H, Hkv, hd, vocab, max_seq, n_seg_max;
    const double *inv_freq;    // [hd/2]
    float *x, *qkv, *attn, *logits, *hfinal;
    float2 *rope_cs;           // [MAXM][hd/2]
    float *part_o;             // [MAXM][H][n_seg_max][hd]
    float2 *part_ml;           // [MAXM][H][n_seg_max]
    int *attn_cnt;             // [MAXM][H], zero between passes
    float *amax_v;             // [MAXM][grid]
    int *amax_i;
    int *amax_cnt;             // [1], zero between passes
    const DeviceState *state;
    unsigned long long *bar;   // grid barrier counter (monotonic)
    int *gabort;               // device-wide abort word
    int *err;
    unsigned long long *trace; // optional [n_ops][2] nanosecond stamps of CTA 0 (work done, barrier passed); nullptr = off
};

struct Params {
    const Op *ops;
    int n_ops;
    int M;                     // rows of this pass (1..MAXM)
    const int *tok;            // [M] token ids (device)
    int pos_off;               // first row sits at position state->len + pos_off
    int head_row0;             // rows >= head_row0 get logits and an arg-max (== M: none)
    int *argmax_out;           // [M - head_row0]
    int want_hidden;
    unsigned long long bar_base;   // value of *bar when this launch starts
};

__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// ---- grid-wide barrier among the consumer warps of all CTAs -----------------------------------------------
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long *p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

// Called by all 256 consumer threads.  Returns false once the pass has been aborted.
__device__ __forceinline__ bool grid_barrier(const Model &md, const Ring &r, unsigned long long target, int tid, bool alive) {
    __threadfence();
    asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
    if (tid == 0 && alive) {
        atomicAdd(md.bar, 1ULL);
        unsigned spins = 0;
        while (ld_acquire_u64(md.bar) < target) {
            if (*r.abort_flag || *reinterpret_cast<volatile int *>(md.gabort)) { *r.abort_flag = 1; break; }
            if (++spins > BAR_SPIN_LIMIT) {
                *r.abort_flag = 1;
                atomicExch(md.gabort, 1);
                atomicExch(md.err, 7);
                break;
            }
            __nanosleep(32);
        }
        __threadfence();
    }
    asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
    return alive && !*r.abort_flag;
}

// ---- embedding gather + rotary table ----------------------------------------------------------------------
__device__ __forceinline__ void embed_phase(const Model &md, const Params &pr, int cta, int tid) {
    const int d = md.d_model, half = md.hd >> 1;
    if (cta < pr.M) {
        const int m = cta;
        const bf16_t *row = md.tok_embed + (size_t)pr.tok[m] * d;
        for (int i = tid; i < d; i += NCW * 32) __stcg(md.x + (size_t)m * d + i, bf16_bits_to_float(row[i]));
    }
    if (cta == (pr.M < (int)gridDim.x ? pr.M : 0)) {       // one more CTA fills the (cos, sin) table of all rows
        const int p0 = md.state->len + pr.pos_off;
        for (int idx = tid; idx < pr.M * half; idx += NCW * 32) {
            const int m = idx / half, i = idx % half;
            double s, c;
            sincos((double)(p0 + m) * md.inv_freq[i], &s, &c);
            __stcg(md.rope_cs + idx, make_float2((float)c, (float)s));
        }
    }
}

// ---- RMSNorm of the rows written out (hidden-state output) -------------------------------------------------
__device__ __forceinline__ void hidden_phase(const Model &md, const Params &pr, const Ring &r, int cta, int tid) {
    if (cta >= pr.M) return;          // whole CTAs only: the named barrier below is CTA-local
    const int d = md.d_model, m = cta, lane = tid & 31, warp = tid >> 5;
    const float *xr = md.x + (size_t)m * d;
    float s = 0.f;
    for (int i = tid; i < d; i += NCW * 32) { const float v = __ldcg(xr + i); s = fmaf(v, v, s); }
    s = warp_sum(s);
    if (lane == 0) r.red_ss[warp] = s;
    asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
    float tot = 0.f;
    for (int w = 0; w < NCW; ++w) tot += r.red_ss[w];
    const float rinv = 1.0f / sqrtf(tot / (float)d + md.rms_eps);
    for (int i = tid; i < d; i += NCW * 32) __stcg(md.hfinal + (size_t)m * d + i, __ldcg(xr + i) * rinv * md.final_norm[i]);
    asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
}

// ---- greedy arg-max: every CTA scans a slice of each row, the last one to finish folds the partials --------
__device__ __forceinline__ void argmax_phase(const Model &md, const Params &pr, const Ring &r, int cta, int n_cta, int tid) {
    const int V = md.vocab, lane = tid & 31, warp = tid >> 5;
    const int per = (V + n_cta - 1) / n_cta, i0 = cta * per, i1 = min(V, i0 + per);
    float *s_v = r.red;
    int *s_i = reinterpret_cast<int *>(r.red + 64);
    int *s_last = reinterpret_cast<int *>(r.red + 128);
    const int rows = pr.M - pr.head_row0;
    for (int m = 0; m < rows; ++m) {
        const float *row = md.logits + (size_t)(pr.head_row0 + m) * V;
        float bv = -INFINITY;
        int bi = 0x7fffffff;
        for (int i = i0 + tid; i < i1; i += NCW * 32) argmax_fold(bv, bi, __ldcg(row + i), i);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            argmax_fold(bv, bi, ov, oi);
        }
        if (lane == 0) { s_v[warp] = bv; s_i[warp] = bi; }
        asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
        if (tid == 0) {
            for (int w = 1; w < NCW; ++w) argmax_fold(bv, bi, s_v[w], s_i[w]);
            __stcg(md.amax_v + m * n_cta + cta, bv);
            __stcg(md.amax_i + m * n_cta + cta, bi);
        }
        asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
    }
    __threadfence();
    asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
    if (tid == 0) *s_last = (atomicAdd(md.amax_cnt, 1) == n_cta - 1);
    asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
    if (*s_last) {
        __threadfence();
        if (warp < rows && warp < NCW) {
            for (int m = warp; m < rows; m += NCW) {
                float bv = -INFINITY;
                int bi = 0x7fffffff;
                for (int b = lane; b < n_cta; b += 32) argmax_fold(bv, bi, __ldcg(md.amax_v + m * n_cta + b), __ldcg(md.amax_i + m * n_cta + b));
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                    argmax_fold(bv, bi, ov, oi);
                }
                if (lane == 0) pr.argmax_out[m] = bi;
            }
        }
        if (tid == 0) *md.amax_cnt = 0;
    }
    asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
}

// ---- attention over the KV cache ------------------------------------------------------------------------------
// Rows m = 0..M-1 sit at positions P0 + m; row m attends to positions [0, P0 + m].  The context is cut at fixed
// absolute boundaries into segments of SEGP positions; one warp handles one (query head, segment) for all rows:
// it reads each K and V row of the segment once (8 bytes per lane, a whole 256-byte row per warp access), in
// register batches of 16 positions with the next batch always in flight, takes the 16 dot products of a batch with
// a transposed butterfly, keeps an online softmax per row over 32-position chunks and writes an un-normalised
// partial (max, sum, o).  The warp that completes the last segment of a (row, head) merges the partials in segment
// order.  K/V of the M new positions come from the projection buffer (rotated, rounded to bf16 exactly as they are
// stored); the warp of the first query head of each KV group also writes them to the cache.  Loops over batches stay
// rolled on purpose: the unrolled form of this code does not fit the instruction cache.
template <int HD> struct KVVec;
template <> struct KVVec<128> { typedef uint2 T; };
template <> struct KVVec<64> { typedef uint32_t T; };

template <int HD> __device__ __forceinline__ void kv_unpack(const typename KVVec<HD>::T &v, float (&f)[HD / 32]);
template <> __device__ __forceinline__ void kv_unpack<128>(const uint2 &v, float (&f)[4]) {
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xFFFF0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xFFFF0000u);
}
template <> __device__ __forceinline__ void kv_unpack<64>(const uint32_t &v, float (&f)[2]) {
    f[0] = __uint_as_float(v << 16); f[1] = __uint_as_float(v & 0xFFFF0000u);
}
template <int HD> __device__ __forceinline__ typename KVVec<HD>::T kv_pack(const float (&f)[HD / 32]);
template <> __device__ __forceinline__ uint2 kv_pack<128>(const float (&f)[4]) {
    return make_uint2((uint32_t)float_to_bf16_rne(f[0]) | ((uint32_t)float_to_bf16_rne(f[1]) << 16),
                      (uint32_t)float_to_bf16_rne(f[2]) | ((uint32_t)float_to_bf16_rne(f[3]) << 16));
}
template <> __device__ __forceinline__ uint32_t kv_pack<64>(const float (&f)[2]) {
    return (uint32_t)float_to_bf16_rne(f[0]) | ((uint32_t)float_to_bf16_rne(f[1]) << 16);
}
template <int HD> __device__ __forceinline__ typename KVVec<HD>::T kv_zero();
template <> __device__ __forceinline__ uint2 kv_zero<128>() { return make_uint2(0u, 0u); }
template <> __device__ __forceinline__ uint32_t kv_zero<64>() { return 0u; }

// Sum over lanes of v[i], delivered to every lane whose (lane & 15) == i (i = 0..15): 16 shuffles for 16 sums.
__device__ __forceinline__ float transposed_sum16(float (&v)[16], int lane) {
#pragma unroll
    for (int step = 8; step >= 1; step >>= 1) {
        const bool up = (lane & step) != 0;
#pragma unroll
        for (int i = 0; i < step; ++i) {
            const float send = up ? v[i] : v[i + step];
            const float keep = up ? v[i + step] : v[i];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, step);
        }
    }
    return v[0] + __shfl_xor_sync(0xffffffffu, v[0], 16);
}

constexpr int ATT_B = 16;          // positions per register batch (one batch is always in flight ahead of the math)

// MR = rows the code is unrolled for (1: draft steps, 8: verification); rows >= M are skipped at run time.
template <int HD, int MR>
__device__ __forceinline__ void attn_phase(const Model &md, const Op &op, const Params &pr, const Ring &r, int cta, int n_cta,
                                           int warp, int lane) {
    constexpr int DPL = HD / 32, HALF = HD / 2;
    typedef typename KVVec<HD>::T VT;
    const int M = pr.M, H = md.H, Hkv = md.Hkv, G = H / Hkv;
    const int P0 = md.state->len + pr.pos_off, Ttot = P0 + M;
    const int n_seg = (Ttot + SEGP - 1) / SEGP, n_tasks = H * n_seg;
    const int qstride = (H + 2 * Hkv) * HD;
    const float scale = 1.0f / sqrtf((float)HD);
    const int d0 = DPL * lane, ci = d0 % HALF;
    const bool upper = d0 >= HALF;
    bf16_t *stash_k = reinterpret_cast<bf16_t *>(r.red) + (size_t)warp * (2 * MAXM * HD);   // [MAXM][HD] new K rows
    bf16_t *stash_v = stash_k + MAXM * HD;                                                  // [MAXM][HD] new V rows

    for (int t = warp * n_cta + cta; t < n_tasks; t += NCW * n_cta) {
        const int seg = t / H, h = t % H, kvh = h / G;
        const int p_begin = seg * SEGP, p_end = min(p_begin + SEGP, Ttot);
        const int m_first = max(0, p_begin - P0);
        const bool writer = (h % G) == 0;
        bf16_t *kbase = op.kc + (size_t)kvh * md.max_seq * HD;
        bf16_t *vbase = op.vc + (size_t)kvh * md.max_seq * HD;

        // new K/V rows that fall into this segment: rotate, round, stash (and store if this warp is the writer)
        __syncwarp();
        for (int mp = m_first; mp < M && P0 + mp < p_end; ++mp) {
            const float *kraw = md.qkv + (size_t)mp * qstride + (size_t)(H + kvh) * HD + d0;
            const float *vraw = md.qkv + (size_t)mp * qstride + (size_t)(H + Hkv + kvh) * HD + d0;
            float kf[DPL], vf[DPL];
#pragma unroll
            for (int e = 0; e < DPL; ++e) { kf[e] = __ldcg(kraw + e); vf[e] = __ldcg(vraw + e); }
#pragma unroll
            for (int e = 0; e < DPL; ++e) {
                const float partner = __shfl_xor_sync(0xffffffffu, kf[e], 16);
                const float2 cs = __ldcg(md.rope_cs + mp * HALF + ci + e);
                kf[e] = upper ? (kf[e] * cs.x + partner * cs.y) : (kf[e] * cs.x - partner * cs.y);
            }
            const VT kp = kv_pack<HD>(kf), vp = kv_pack<HD>(vf);
            *reinterpret_cast<VT *>(stash_k + mp * HD + d0) = kp;
            *reinterpret_cast<VT *>(stash_v + mp * HD + d0) = vp;
            if (writer) {
                *reinterpret_cast<VT *>(kbase + (size_t)(P0 + mp) * HD + d0) = kp;
                *reinterpret_cast<VT *>(vbase + (size_t)(P0 + mp) * HD + d0) = vp;
            }
        }
        __syncwarp();

        // rotated queries of the rows that see this segment
        float q[MR][DPL], o[MR][DPL], mx[MR], l[MR], sreg[MR];
#pragma unroll
        for (int m = 0; m < MR; ++m) {
            mx[m] = -INFINITY; l[m] = 0.f; sreg[m] = 0.f;
#pragma unroll
            for (int e = 0; e < DPL; ++e) { q[m][e] = 0.f; o[m][e] = 0.f; }
            if (m >= m_first && m < M) {
                const float *qraw = md.qkv + (size_t)m * qstride + (size_t)h * HD + d0;
#pragma unroll
                for (int e = 0; e < DPL; ++e) q[m][e] = __ldcg(qraw + e);
#pragma unroll
                for (int e = 0; e < DPL; ++e) {
                    const float partner = __shfl_xor_sync(0xffffffffu, q[m][e], 16);
                    const float2 cs = __ldcg(md.rope_cs + m * HALF + ci + e);
                    q[m][e] = upper ? (q[m][e] * cs.x + partner * cs.y) : (q[m][e] * cs.x - partner * cs.y);
                }
            }
        }

        // The segment as a flat list of register batches: per 32-position chunk, K rows 0-15, K rows 16-31, V rows
        // 0-15, V rows 16-31.  Batch it + 1 is loading while batch it is being used.
        auto load_batch = [&](int it, VT (&dst)[ATT_B]) {
            const int sub = it & 3, pb = p_begin + (it >> 2) * 32 + (sub & 1) * ATT_B;
            const bf16_t *cache = (sub >> 1) ? vbase : kbase;
            const bf16_t *stash = (sub >> 1) ? stash_v : stash_k;
#pragma unroll
            for (int j = 0; j < ATT_B; ++j) {
                const int p = pb + j;
                const bf16_t *src = p < P0 ? cache + (size_t)p * HD + d0 : stash + (p - P0) * HD + d0;
                dst[j] = p < p_end ? *reinterpret_cast<const VT *>(src) : kv_zero<HD>();
            }
        };
        const int n_it = 4 * ((p_end - p_begin + 31) >> 5);
        VT cur[ATT_B], nxt[ATT_B];
        load_batch(0, cur);
        for (int it = 0; it < n_it; ++it) {
            if (it + 1 < n_it) load_batch(it + 1, nxt);
            const int sub = it & 3, half = sub & 1, p0 = p_begin + (it >> 2) * 32;
            if (sub < 2) {
                // ---- scores of 16 positions: lane (half * 16 + i) keeps position i's score ----
#pragma unroll
                for (int m = 0; m < MR; ++m) {
                    if (m < m_first || m >= M || p0 > P0 + m) continue;      // row does not see this chunk
                    float part[ATT_B];
#pragma unroll
                    for (int j = 0; j < ATT_B; ++j) {
                        float kf[DPL];
                        kv_unpack<HD>(cur[j], kf);
                        float s = 0.f;
#pragma unroll
                        for (int e = 0; e < DPL; ++e) s = fmaf(q[m][e], kf[e], s);
                        part[j] = s;
                    }
                    const float tot = transposed_sum16(part, lane);
                    if ((lane >> 4) == half) sreg[m] = tot;
                }
                if (sub == 1) {
                    // ---- online softmax over the chunk's 32 positions (lane = position) ----
#pragma unroll
                    for (int m = 0; m < MR; ++m) {
                        if (m < m_first || m >= M || p0 > P0 + m) continue;
                        const bool valid = p0 + lane <= P0 + m;
                        const float s = valid ? sreg[m] * scale : -INFINITY;
                        const float mnew = fmaxf(mx[m], warp_max(s));
                        const float corr = expf(mx[m] - mnew);
                        const float pj = valid ? expf(s - mnew) : 0.f;
                        l[m] = fmaf(l[m], corr, warp_sum(pj));
#pragma unroll
                        for (int e = 0; e < DPL; ++e) o[m][e] *= corr;
                        mx[m] = mnew;
                        sreg[m] = pj;
                    }
                }
            } else {
                // ---- o += p V over 16 positions ----
#pragma unroll
                for (int j = 0; j < ATT_B; ++j) {
                    float vf[DPL];
                    kv_unpack<HD>(cur[j], vf);
#pragma unroll
                    for (int m = 0; m < MR; ++m) {
                        if (m < m_first || m >= M || p0 > P0 + m) continue;
                        const float pj = __shfl_sync(0xffffffffu, sreg[m], half * ATT_B + j);
#pragma unroll
                        for (int e = 0; e < DPL; ++e) o[m][e] = fmaf(pj, vf[e], o[m][e]);
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < ATT_B; ++j) cur[j] = nxt[j];
        }

        // ---- partials out; the last warp of a (row, head) merges ----
#pragma unroll
        for (int m = 0; m < MR; ++m) {
            if (m < m_first || m >= M) continue;
            const size_t pidx = ((size_t)m * H + h) * md.n_seg_max + seg;
            if (lane == 0) __stcg(md.part_ml + pidx, make_float2(mx[m], l[m]));
#pragma unroll
            for (int e = 0; e < DPL; ++e) __stcg(md.part_o + pidx * HD + d0 + e, o[m][e]);
        }
        __threadfence();
        __syncwarp();
        unsigned last_mask = 0;
        if (lane == 0) {
            for (int m = m_first; m < M; ++m) {
                const int n_seg_m = (P0 + m + SEGP) / SEGP;              // segments row m sees
                if (atomicAdd(md.attn_cnt + m * H + h, 1) == n_seg_m - 1) last_mask |= 1u << m;
            }
        }
        last_mask = __shfl_sync(0xffffffffu, last_mask, 0);
        if (last_mask) {
            __threadfence();
            for (int m = m_first; m < M; ++m) {
                if (!((last_mask >> m) & 1u)) continue;
                const int n_seg_m = (P0 + m + SEGP) / SEGP;
                const size_t base = ((size_t)m * H + h) * md.n_seg_max;
                float gm = -INFINITY;
                for (int s = 0; s < n_seg_m; ++s) gm = fmaxf(gm, __ldcg(md.part_ml + base + s).x);
                float L = 0.f, acc[DPL];
#pragma unroll
                for (int e = 0; e < DPL; ++e) acc[e] = 0.f;
                for (int s = 0; s < n_seg_m; ++s) {
                    const float2 ml = __ldcg(md.part_ml + base + s);
                    const float w = expf(ml.x - gm);
                    L = fmaf(ml.y, w, L);
#pragma unroll
                    for (int e = 0; e < DPL; ++e) acc[e] = fmaf(__ldcg(md.part_o + (base + s) * HD + d0 + e), w, acc[e]);
                }
#pragma unroll
                for (int e = 0; e < DPL; ++e) __stcg(md.attn + (size_t)m * H * HD + (size_t)h * HD + d0 + e, acc[e] / L);
                if (lane == 0) md.attn_cnt[m * H + h] = 0;
            }
        }
    }
}

// ---- the pass ---------------------------------------------------------------------------------------------------
template <int HD>
__global__ void __launch_bounds__(stream::NTHREADS, 1) pass_kernel(const Model md, const Params pr) {
    extern __shared__ __align__(128) unsigned char smem[];
    Ring r;
    stream::ring_setup(r, smem, md.err);
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cta = blockIdx.x, n_cta = gridDim.x;
    int w_use = 0;
    bool alive = true;
    if (warp >= NCW) {
        stream::regs_dec<stream::REGS_PRODUCER>();
        if (warp == NCW) {
            for (int i = 0; i < pr.n_ops && alive; ++i) {
                const Op &op = pr.ops[i];
                if (op.type != OP_LINEAR) continue;
                LinPhase lp = op.lin;
                lp.M = pr.M;
                if (op.is_head) { if (pr.head_row0 >= pr.M) continue; }
                stream::produce_linear(lp, r, cta, n_cta, lane, w_use, alive);
            }
            if (!alive) stream::producer_drain_after_abort();
        }
        return;
    }
    stream::regs_inc<stream::REGS_CONSUMER>();
    const int tid = threadIdx.x;
    unsigned long long n_bar = 0;
    for (int i = 0; i < pr.n_ops; ++i) {
        const Op &op = pr.ops[i];
        bool ran = true;
        if (op.type == OP_LINEAR) {
            LinPhase lp = op.lin;
            lp.M = pr.M;
            if (op.is_head) {
                if (pr.head_row0 >= pr.M) ran = false;
                lp.M = pr.M - pr.head_row0;
                lp.x += (size_t)pr.head_row0 * lp.K;
                lp.y += (size_t)pr.head_row0 * lp.units;
            }
            if (ran) stream::consume_linear(lp, r, cta, n_cta, warp, lane, w_use, alive);
        } else if (alive) {
            if (op.type == OP_EMBED) embed_phase(md, pr, cta, tid);
            else if (op.type == OP_ATTN) {
                if (pr.M == 1) attn_phase<HD, 1>(md, op, pr, r, cta, n_cta, warp, lane);
                else attn_phase<HD, MAXM>(md, op, pr, r, cta, n_cta, warp, lane);
            }
            else if (op.type == OP_HIDDEN) { if (pr.want_hidden) hidden_phase(md, pr, r, cta, tid); else ran = false; }
            else if (op.type == OP_ARGMAX) { if (pr.head_row0 < pr.M) argmax_phase(md, pr, r, cta, n_cta, tid); else ran = false; }
        }
        if (md.trace && cta == 0 && tid == 0) md.trace[2 * i] = globaltimer_ns();
        if (op.barrier_after && ran) {
            ++n_bar;
            alive = grid_barrier(md, r, pr.bar_base + n_bar * (unsigned long long)n_cta, tid, alive);
        }
        if (md.trace && cta == 0 && tid == 0) md.trace[2 * i + 1] = globaltimer_ns();
    }
}

}  // namespace pass
}  // namespace knnssd
