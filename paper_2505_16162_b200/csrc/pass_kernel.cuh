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
#include "linear_presplit.cuh"

namespace knnssd {
namespace pass {

using stream::LinPhase;
using stream::Ring;
using stream::NCW;

constexpr int MAXM = 16;           // rows per pass this kernel handles
constexpr int BLKM = 8;            // rows per tensor-core row block (linear maps take two blocks at once, attention one at a time)
constexpr int SEGP = 64;           // attention: positions per segment (fixed absolute boundaries)
constexpr unsigned BAR_SPIN_LIMIT = 4000000u;

enum { OP_EMBED = 0, OP_LINEAR = 1, OP_ATTN = 2, OP_HIDDEN = 3, OP_ARGMAX = 4, OP_ATTN_MERGE = 5, OP_KV_APPEND = 6 };
constexpr int MERGE_ROWS = 3;      // tasks with at least this many (row, head) pairs leave the merge to a separate operation

struct Op {
    int type;
    int barrier_after;   // 1: all CTAs meet before the next operation starts
    int is_head;         // OP_LINEAR: the LM head (runs on rows head_row0.. only)
    int layer;
    LinPhase lin;        // OP_LINEAR; OP_EMBED and OP_ATTN use its ys / next_gain / ss_out fields for their output
    bf16_t *kc, *vc;     // OP_ATTN: this layer's cache [n_kv_heads][max_seq][head_dim]
};

struct Model {           // what does not change from pass to pass
    const bf16_t *tok_embed;
    const float *final_norm;
    float rms_eps;
    int d_model, H, Hkv, hd, vocab, max_seq, n_seg_max;
    const double *inv_freq;    // [hd/2]
    float *x, *qkv, *attn, *logits, *hfinal;
    float2 *rope_cs;           // [grid][MAXM][hd/2]: one copy per CTA, written and read by that CTA only
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
    int out_row0;              // row of the logits / hidden-state buffers that this pass's row 0 goes to
    unsigned long long bar_base;   // value of *bar when this launch starts
    int merge_op;              // the attention partials are merged by the separate merge operation (merge_rows_separately)
    unsigned bar_spin_limit;   // polls a grid-barrier wait may take before the pass is aborted (0 = BAR_SPIN_LIMIT)
};

// Whether a pass of M rows merges its attention partials in the separate operation: when an attention task carries
// at least MERGE_ROWS (row, head) pairs - all G query heads of a K/V head for passes of up to BLKM rows.
__host__ __device__ inline bool merge_rows_separately(int M, int G);

__host__ __device__ inline bool merge_rows_separately(int M, int G) { return M > BLKM || M * G >= MERGE_ROWS; }

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
__device__ __forceinline__ bool grid_barrier(const Model &md, const Ring &r, unsigned long long target, int tid, bool alive,
                                             unsigned spin_limit) {
    asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
    if (tid == 0 && alive) {
        __threadfence();                       // cumulative: covers the writes of the CTA's other threads ordered by the bar.sync
        atomicAdd(md.bar, 1ULL);
        unsigned spins = 0;
        while (ld_acquire_u64(md.bar) < target) {
            if (*r.abort_flag || *reinterpret_cast<volatile int *>(md.gabort)) { *r.abort_flag = 1; break; }
            if (++spins > spin_limit) {
                *r.abort_flag = 1;
                atomicExch(md.gabort, 1);
                atomicExch(md.err, 7);
                break;
            }
            __nanosleep(32);
        }
    }
    asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
    return alive && !*r.abort_flag;
}

// ---- embedding gather + rotary table ----------------------------------------------------------------------
__device__ __forceinline__ void embed_phase(const Model &md, const Op &op, const Params &pr, const Ring &r, int cta, int n_cta,
                                            int tid) {
    const int d = md.d_model, half = md.hd >> 1;
    {   // every CTA fills its own copy of the (cos, sin) table of all rows: 148 readers of one copy would queue up at L2
        const int p0 = md.state->len + pr.pos_off;
        float2 *mine = md.rope_cs + (size_t)cta * MAXM * half;
        for (int idx = tid; idx < pr.M * half; idx += NCW * 32) {
            const int m = idx / half, i = idx % half;
            double s, c;
            sincos((double)(p0 + m) * md.inv_freq[i], &s, &c);
            mine[idx] = make_float2((float)c, (float)s);
        }
    }
    if (cta >= pr.M) return;                               // whole CTAs only: the named barrier below is CTA-local
    // row m = cta: residual stream in fp32, its pre-split form times the first RMSNorm's gain, its sum of squares
    const int m = cta, lane = tid & 31, warp = tid >> 5;
    int t = pr.tok[m];
    if (t < 0 || t >= md.vocab) {                          // never gather outside the table: report and read row 0 instead
        if (tid == 0) atomicExch(md.err, ERR_BAD_TOKEN);
        t = 0;
    }
    const bf16_t *row = md.tok_embed + (size_t)t * d;
    float ss = 0.f;
    for (int i = tid; i < d; i += NCW * 32) {
        const float v = bf16_bits_to_float(row[i]);
        __stcg(md.x + (size_t)m * d + i, v);
        stream::store_split(op.lin.ys, d >> 7, m, i, op.lin.next_gain ? v * __ldg(op.lin.next_gain + i) : v);
        ss = fmaf(v, v, ss);
    }
    ss = warp_sum(ss);
    if (lane == 0) r.red_ss[32 + warp] = ss;
    asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
    if (tid == 0) {
        float tot = 0.f;
        for (int w = 0; w < NCW; ++w) tot += r.red_ss[32 + w];
        __stcg(op.lin.ss_out + (size_t)m * n_cta, tot);
    }
    for (int c = 1 + tid; c < n_cta; c += NCW * 32) __stcg(op.lin.ss_out + (size_t)m * n_cta + c, 0.f);
    asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
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
    for (int i = tid; i < d; i += NCW * 32) __stcg(md.hfinal + (size_t)(pr.out_row0 + m) * d + i, __ldcg(xr + i) * rinv * md.final_norm[i]);
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
        const float *row = md.logits + (size_t)(pr.out_row0 + pr.head_row0 + m) * V;
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
                if (lane == 0) pr.argmax_out[m] = argmax_checked(bi, V, md.err);
            }
        }
        if (tid == 0) *md.amax_cnt = 0;
    }
    asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
}

// ---- attention over the KV cache ------------------------------------------------------------------------------
// Rows m = 0..M-1 sit at positions P0 + m; row m attends to positions [0, P0 + m].  The context is cut at fixed
// absolute boundaries into segments of SEGP positions; one warp handles one (query head, segment) for all rows: it
// reads each K and V row of the segment once, keeps the segment's scores in registers, takes a plain softmax over
// the segment and writes an un-normalised partial (max, sum, o).  The warp that completes the last segment of a
// (row, head) merges the partials in segment order and writes the result pre-split for the output projection.
// K/V of the M new positions come from the projection buffer (rotated, rounded to bf16 exactly as they are stored,
// staged in shared memory); the warp of the first query head of each KV group also writes them to the cache.
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

__device__ __forceinline__ void mma_tf32(float (&c)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
    // rows 8..15 of the 16-row operand are not used: their registers are zero
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_bf16_top(float (&c)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}

// The same with both halves of the 16-row operand: rows 0..7 from (a0, a2), rows 8..15 from (a1, a3).
__device__ __forceinline__ void mma_bf16_rows(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Merge the segment partials of one (row m, head h) in segment order and write the result pre-split (one warp).
template <int HD>
__device__ __forceinline__ void attn_merge_row(const Model &md, const Op &op, int P0, int m, int h, int lane) {
    constexpr int DPL = HD / 32;
    const int H = md.H, d0 = DPL * lane;
    const int n_seg_m = (P0 + m + SEGP) / SEGP;
    const size_t base = ((size_t)m * H + h) * md.n_seg_max;
    // segment statistics: lane s holds segments s and s + 32 (contexts up to 4096); fixed-order warp reductions
    const float2 ml0 = lane < n_seg_m ? __ldcg(md.part_ml + base + lane) : make_float2(-INFINITY, 0.f);
    const float2 ml1 = lane + 32 < n_seg_m ? __ldcg(md.part_ml + base + lane + 32) : make_float2(-INFINITY, 0.f);
    const float gm = warp_max(fmaxf(ml0.x, ml1.x));
    const float w0 = ml0.x == -INFINITY ? 0.f : expf(ml0.x - gm), w1 = ml1.x == -INFINITY ? 0.f : expf(ml1.x - gm);
    const float L = warp_sum(fmaf(ml1.y, w1, ml0.y * w0));
    // weighted sum of the partial outputs in segment order, sixteen segments in flight at a time
    float acc[DPL];
#pragma unroll
    for (int e = 0; e < DPL; ++e) acc[e] = 0.f;
    for (int s0 = 0; s0 < n_seg_m; s0 += 16) {
        float pv[16][DPL];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            // one vector load per segment (DPL = 4: 16 bytes, DPL = 2: 8 bytes)
            const float *src = md.part_o + (base + s0 + i) * HD + d0;
            if (DPL == 4) {
                const float4 v = s0 + i < n_seg_m ? __ldcg(reinterpret_cast<const float4 *>(src)) : make_float4(0.f, 0.f, 0.f, 0.f);
                pv[i][0] = v.x; pv[i][1] = v.y; pv[i][DPL - 2] = v.z; pv[i][DPL - 1] = v.w;
            } else {
                const float2 v = s0 + i < n_seg_m ? __ldcg(reinterpret_cast<const float2 *>(src)) : make_float2(0.f, 0.f);
                pv[i][0] = v.x; pv[i][DPL - 1] = v.y;
            }
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int sg = s0 + i;
            const float w = __shfl_sync(0xffffffffu, sg < 32 ? w0 : w1, sg & 31);
#pragma unroll
            for (int e = 0; e < DPL; ++e) acc[e] = fmaf(pv[i][e], w, acc[e]);
        }
    }
#pragma unroll
    for (int e = 0; e < DPL; ++e) stream::store_split(op.lin.ys, (H * HD) >> 7, m, h * HD + d0 + e, acc[e] / L);
}


// Tensor-core form.  Lane (g8, t4) = (lane / 4, lane % 4).  The pass's rows are the rows 0..7 of the 16-row MMA
// operand (row m = g8), so the cost does not depend on how many rows the pass carries.
//   scores  S = Q K^T   m16n8k16 bf16: the 8 columns of a tile are 8 consecutive positions (column n = g8 of the K
//           operand = position 8*nt + g8).  A dot product does not care in which order its terms are taken, so k-step
//           s pairs k-indices with the dimensions (DL*t4 + 4s .. + 3): every lane then reads one contiguous run of
//           DL = HD/4 dimensions of "its" K row (16-byte loads) and holds the same run of q, split into two bf16
//           terms (hi + lo, 16-17 bits); products are exact.
//   output  O += P V    m16n8k16 bf16 over pairs of tiles: k-indices 2t4, 2t4+1 stand for positions 2t4, 2t4+1 of the
//           first tile and 2t4+8, 2t4+9 for the same positions of the second - exactly the four scores the lane already
//           holds - and column n = g8 of V-tile j is dimension (HD/8)*g8 + j, so a lane reads HD/8 contiguous
//           dimensions of four V rows; an operand register (two positions of one dimension) is one byte-permute of two
//           loaded words.  p is split into two bf16 terms.
// A lane ends up with output dimensions [DL*t4, DL*t4 + DL) of row g8, the run it holds of q.
template <int HD, bool R16>
__device__ __forceinline__ void attn_phase(const Model &md, const Op &op, const Params &pr, const Ring &r, int cta, int n_cta,
                                           int warp, int lane, bool defer_merge, int row0, bool all_cached) {
    constexpr int DL = HD / 4;         // dimensions of q / o per lane
    constexpr int NW = HD / 8;         // 32-bit words of a K row per lane
    constexpr int VW = HD / 16;        // 32-bit words of a V row per lane
    constexpr int VJ = HD / 8;         // V tiles (8 dimensions each)
    constexpr int HALF = HD / 2;
    constexpr int NT = SEGP / 8;       // position tiles per segment
    constexpr int NR = R16 ? 2 : 1;    // pass rows per lane: row0 + g8 and, with R16, row0 + g8 + 8 (rows 8..15 of the MMA operand)
    const int g8 = lane >> 2, t4 = lane & 3;
    const int M = pr.M, H = md.H, Hkv = md.Hkv, G = H / Hkv;
    const int P0 = md.state->len + pr.pos_off, Ttot = P0 + M;
    const int Pc = all_cached ? Ttot : P0;                   // positions below Pc are read from the cache
    // A task = (segment, head group, block of 8 rows).  Passes of up to BLKM rows (all_cached false) take the G query
    // heads that share a K/V head together: the rows of a group are the (head-in-group, pass row) pairs rr = hg M + m,
    // eight per block, so that a K/V segment is read once per block instead of once per head and a GQA model has
    // G times fewer tasks.  With all_cached a task is one head and the block is given by row0.
    const int Gt = all_cached ? 1 : G;                       // query heads per group
    const int n_grp = H / Gt;
    const int R = all_cached ? M : M * Gt;                   // rows of a group
    const int nblk = all_cached ? 1 : (R + BLKM - 1) / BLKM;
    const int n_seg = (Ttot + SEGP - 1) / SEGP, n_tasks = n_grp * n_seg * nblk;
    const int qstride = (H + 2 * Hkv) * HD;
    const float scale = 1.0f / sqrtf((float)HD);
    const bool upper = t4 >= 2;                              // this lane's run lies in the second half of the head
    const int ci = DL * (t4 & 1);                            // its offset in the (cos, sin) table
    bf16_t *stash_k = reinterpret_cast<bf16_t *>(r.red) + (size_t)warp * (2 * BLKM * HD);   // [BLKM][HD] new K rows
    bf16_t *stash_v = stash_k + BLKM * HD;                                                  // [BLKM][HD] new V rows
    const float2 *my_cs = md.rope_cs + (size_t)cta * MAXM * HALF;                           // this CTA's copy

    for (int t = warp * n_cta + cta; t < n_tasks; t += NCW * n_cta) {
        const int blk = t % nblk, tt = t / nblk, seg = tt / n_grp, grp = tt % n_grp;
        const int kvh = all_cached ? grp / G : grp;
        const int rr = blk * BLKM + g8;                      // this lane's row of the group (grouped tasks)
        const int rm = all_cached ? row0 + g8 : rr % M;      // the pass row this lane's MMA row stands for
        const int h = all_cached ? grp : kvh * G + min(rr / M, G - 1);   // and its query head
        const bool row_in = all_cached ? rm < M : rr < R;
        const int rm2 = rm + BLKM;                           // R16: the lane's second row (MMA row g8 + 8), same head
        const int p_begin = seg * SEGP, p_end = min(p_begin + SEGP, Ttot);
        const int m_first = max(0, p_begin - P0);           // first row that sees this segment
        const bool writer = !all_cached && blk == 0;         // one task per (segment, K/V head) puts the new rows into the cache
        bf16_t *kbase = op.kc + (size_t)kvh * md.max_seq * HD;
        bf16_t *vbase = op.vc + (size_t)kvh * md.max_seq * HD;
        if (all_cached && row0 + NR * BLKM <= m_first) continue;  // none of this block's rows sees the segment
        // pass row g8's own position lies in this segment and is not in the cache yet: this lane rotates / rounds its K, V
        const bool row_new = !all_cached && g8 < M && P0 + g8 >= p_begin && P0 + g8 < p_end;
        const bool row_live = row_in && rm >= m_first;
        const bool row_live2 = R16 && rm2 < M && rm2 >= m_first;
        // ---- this lane's run of q (row g8), of the new K row and of the new V row: load, rotate, round / split ----
        float qf[DL], kf[DL];
        float qf2[R16 ? DL : 1];                             // R16: the second row's run of q, rotated like the first
        {
            const float *qraw = md.qkv + (size_t)min(rm, M - 1) * qstride + (size_t)h * HD + DL * t4;
            const float *kraw = md.qkv + (size_t)min(g8, M - 1) * qstride + (size_t)(H + kvh) * HD + DL * t4;
#pragma unroll
            for (int e = 0; e < DL; e += 4) {
                const float4 a = row_live ? __ldcg(reinterpret_cast<const float4 *>(qraw + e)) : make_float4(0.f, 0.f, 0.f, 0.f);
                const float4 b = row_new ? __ldcg(reinterpret_cast<const float4 *>(kraw + e)) : make_float4(0.f, 0.f, 0.f, 0.f);
                qf[e] = a.x; qf[e + 1] = a.y; qf[e + 2] = a.z; qf[e + 3] = a.w;
                kf[e] = b.x; kf[e + 1] = b.y; kf[e + 2] = b.z; kf[e + 3] = b.w;
            }
            if constexpr (R16) {
                const float *qraw2 = md.qkv + (size_t)min(rm2, M - 1) * qstride + (size_t)h * HD + DL * t4;
#pragma unroll
                for (int e = 0; e < DL; e += 4) {
                    const float4 a = row_live2 ? __ldcg(reinterpret_cast<const float4 *>(qraw2 + e)) : make_float4(0.f, 0.f, 0.f, 0.f);
                    qf2[e] = a.x; qf2[e + 1] = a.y; qf2[e + 2] = a.z; qf2[e + 3] = a.w;
                }
            }
#pragma unroll
            for (int e = 0; e < DL; ++e) {
                const float qp = __shfl_xor_sync(0xffffffffu, qf[e], 2), kp = __shfl_xor_sync(0xffffffffu, kf[e], 2);
                const float2 cq = row_live ? my_cs[rm * HALF + ci + e] : make_float2(1.f, 0.f);
                const float2 ck = row_new ? my_cs[g8 * HALF + ci + e] : make_float2(1.f, 0.f);
                qf[e] = upper ? (qf[e] * cq.x + qp * cq.y) : (qf[e] * cq.x - qp * cq.y);
                kf[e] = upper ? (kf[e] * ck.x + kp * ck.y) : (kf[e] * ck.x - kp * ck.y);
            }
            if constexpr (R16) {
#pragma unroll
                for (int e = 0; e < DL; ++e) {
                    const float qp = __shfl_xor_sync(0xffffffffu, qf2[e], 2);
                    const float2 cq = row_live2 ? my_cs[rm2 * HALF + ci + e] : make_float2(1.f, 0.f);
                    qf2[e] = upper ? (qf2[e] * cq.x + qp * cq.y) : (qf2[e] * cq.x - qp * cq.y);
                }
            }
        }
        __syncwarp();
        if (row_new) {
            const float *vraw = md.qkv + (size_t)g8 * qstride + (size_t)(H + Hkv + kvh) * HD + DL * t4;
#pragma unroll
            for (int e = 0; e < DL; e += 8) {
                const float4 a = __ldcg(reinterpret_cast<const float4 *>(vraw + e)), b = __ldcg(reinterpret_cast<const float4 *>(vraw + e + 4));
                uint4 kp, vp;
                kp.x = (uint32_t)float_to_bf16_rne(kf[e]) | ((uint32_t)float_to_bf16_rne(kf[e + 1]) << 16);
                kp.y = (uint32_t)float_to_bf16_rne(kf[e + 2]) | ((uint32_t)float_to_bf16_rne(kf[e + 3]) << 16);
                kp.z = (uint32_t)float_to_bf16_rne(kf[e + 4]) | ((uint32_t)float_to_bf16_rne(kf[e + 5]) << 16);
                kp.w = (uint32_t)float_to_bf16_rne(kf[e + 6]) | ((uint32_t)float_to_bf16_rne(kf[e + 7]) << 16);
                vp.x = (uint32_t)float_to_bf16_rne(a.x) | ((uint32_t)float_to_bf16_rne(a.y) << 16);
                vp.y = (uint32_t)float_to_bf16_rne(a.z) | ((uint32_t)float_to_bf16_rne(a.w) << 16);
                vp.z = (uint32_t)float_to_bf16_rne(b.x) | ((uint32_t)float_to_bf16_rne(b.y) << 16);
                vp.w = (uint32_t)float_to_bf16_rne(b.z) | ((uint32_t)float_to_bf16_rne(b.w) << 16);
                *reinterpret_cast<uint4 *>(stash_k + g8 * HD + DL * t4 + e) = kp;
                *reinterpret_cast<uint4 *>(stash_v + g8 * HD + DL * t4 + e) = vp;
                if (writer) {
                    *reinterpret_cast<uint4 *>(kbase + (size_t)(P0 + g8) * HD + DL * t4 + e) = kp;
                    *reinterpret_cast<uint4 *>(vbase + (size_t)(P0 + g8) * HD + DL * t4 + e) = vp;
                }
            }
        }
        __syncwarp();
        uint32_t qh[NW], ql[NW];                             // word w = dimensions (2w, 2w + 1) of the run; q = hi + lo
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            const uint32_t h0 = float_to_bf16_rne(qf[2 * w]), h1 = float_to_bf16_rne(qf[2 * w + 1]);
            const uint32_t l0 = float_to_bf16_rne(qf[2 * w] - __uint_as_float(h0 << 16));
            const uint32_t l1 = float_to_bf16_rne(qf[2 * w + 1] - __uint_as_float(h1 << 16));
            qh[w] = h0 | (h1 << 16); ql[w] = l0 | (l1 << 16);
        }
        uint32_t qh2[R16 ? NW : 1], ql2[R16 ? NW : 1];       // R16: the second row's words
        if constexpr (R16) {
#pragma unroll
            for (int w = 0; w < NW; ++w) {
                const uint32_t h0 = float_to_bf16_rne(qf2[2 * w]), h1 = float_to_bf16_rne(qf2[2 * w + 1]);
                const uint32_t l0 = float_to_bf16_rne(qf2[2 * w] - __uint_as_float(h0 << 16));
                const uint32_t l1 = float_to_bf16_rne(qf2[2 * w + 1] - __uint_as_float(h1 << 16));
                qh2[w] = h0 | (h1 << 16); ql2[w] = l0 | (l1 << 16);
            }
        }
        // ---- scores: one tile = 8 positions; K rows are fetched two tiles ahead ----
        auto load_k = [&](int nt, uint4 (&dst)[NW / 4]) {
            const int p = p_begin + 8 * nt + g8;
            const bf16_t *src = p < Pc ? kbase + (size_t)p * HD + DL * t4 : stash_k + (p - P0) * HD + DL * t4;
#pragma unroll
            for (int q = 0; q < NW / 4; ++q)
                dst[q] = p < p_end ? (p < Pc ? __ldcs(reinterpret_cast<const uint4 *>(src + 8 * q)) : *reinterpret_cast<const uint4 *>(src + 8 * q)) : make_uint4(0u, 0u, 0u, 0u);
        };
        float sc[NT][2 * NR];                                // scores of (row g8, positions 8*nt + 2*t4 + {0, 1}); R16: [2], [3] = row g8 + 8
        {
            constexpr int KR = NT < 4 ? NT : 4;              // tiles in flight
            uint4 kb[KR][NW / 4];
#pragma unroll
            for (int i = 0; i < KR; ++i) load_k(i, kb[i]);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                uint4(&kq)[NW / 4] = kb[nt % KR];
                float ch[4] = {}, cl[4] = {};
#pragma unroll
                for (int q = 0; q < NW / 4; ++q) {
                    // words 4q .. 4q+3 of the run: k-steps 2q (x, y) and 2q + 1 (z, w)
                    if constexpr (R16) {
                        mma_bf16_rows(cl, ql[4 * q], ql2[4 * q], ql[4 * q + 1], ql2[4 * q + 1], kq[q].x, kq[q].y);
                        mma_bf16_rows(ch, qh[4 * q], qh2[4 * q], qh[4 * q + 1], qh2[4 * q + 1], kq[q].x, kq[q].y);
                        mma_bf16_rows(cl, ql[4 * q + 2], ql2[4 * q + 2], ql[4 * q + 3], ql2[4 * q + 3], kq[q].z, kq[q].w);
                        mma_bf16_rows(ch, qh[4 * q + 2], qh2[4 * q + 2], qh[4 * q + 3], qh2[4 * q + 3], kq[q].z, kq[q].w);
                    } else {
                        mma_bf16_top(cl, ql[4 * q], ql[4 * q + 1], kq[q].x, kq[q].y);
                        mma_bf16_top(ch, qh[4 * q], qh[4 * q + 1], kq[q].x, kq[q].y);
                        mma_bf16_top(cl, ql[4 * q + 2], ql[4 * q + 3], kq[q].z, kq[q].w);
                        mma_bf16_top(ch, qh[4 * q + 2], qh[4 * q + 3], kq[q].z, kq[q].w);
                    }
                }
                sc[nt][0] = cl[0] + ch[0];
                sc[nt][1] = cl[1] + ch[1];
                if constexpr (R16) { sc[nt][2] = cl[2] + ch[2]; sc[nt][3] = cl[3] + ch[3]; }
                if (nt + KR < NT) load_k(nt + KR, kq);
            }
        }
        // ---- V rows of the first tiles start moving while the softmax runs ----
        auto load_v = [&](int nt, uint4 (&dst)[2][(VW + 3) / 4]) {
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) {
                const int p = p_begin + 8 * nt + 2 * t4 + rr;
                const bf16_t *src = p < Pc ? vbase + (size_t)p * HD + 2 * VW * g8 : stash_v + (p - P0) * HD + 2 * VW * g8;
                if (VW >= 4) {
#pragma unroll
                    for (int q = 0; q < VW / 4; ++q)
                        dst[rr][q] = p < p_end ? (p < Pc ? __ldcs(reinterpret_cast<const uint4 *>(src + 8 * q)) : *reinterpret_cast<const uint4 *>(src + 8 * q)) : make_uint4(0u, 0u, 0u, 0u);
                } else {
                    const uint2 v = p < p_end ? *reinterpret_cast<const uint2 *>(src) : make_uint2(0u, 0u);
                    dst[rr][0] = make_uint4(v.x, v.y, 0u, 0u);
                }
            }
        };
        constexpr int VR = NT < 4 ? NT : 4;                  // tiles in flight
        uint4 vb[VR][2][(VW + 3) / 4];
#pragma unroll
        for (int i = 0; i < VR; ++i) load_v(i, vb[i]);
        // ---- softmax over the segment for row g8 (the four lanes of a row share it); R16: and for row g8 + 8 ----
        float mx_r[NR], lsum_r[NR];
#pragma unroll
        for (int r = 0; r < NR; ++r) {
            const bool live_r = r == 0 ? row_live : row_live2;
            const int rm_r = r == 0 ? rm : rm2;
            float mx = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int p = p_begin + 8 * nt + 2 * t4 + e;
                    const bool valid = live_r && p <= P0 + rm_r;             // causal; also excludes p >= p_end
                    sc[nt][2 * r + e] = valid ? sc[nt][2 * r + e] * scale : -INFINITY;
                    mx = fmaxf(mx, sc[nt][2 * r + e]);
                }
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            float lsum = 0.f;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const float pj = sc[nt][2 * r + e] == -INFINITY ? 0.f : expf(sc[nt][2 * r + e] - mx);
                    sc[nt][2 * r + e] = pj;
                    lsum += pj;
                }
            lsum += __shfl_xor_sync(0xffffffffu, lsum, 1);
            lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
            mx_r[r] = mx; lsum_r[r] = lsum;
        }
        const float mx = mx_r[0], lsum = lsum_r[0];
        // ---- o += p V ----
        float o[VJ][4];
#pragma unroll
        for (int j = 0; j < VJ; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
#pragma unroll
        for (int np = 0; np < NT; np += 2) {
            // k-indices 2t4, 2t4+1 stand for this lane's two positions of tile np, 2t4+8, 2t4+9 for those of tile np + 1
            uint32_t ah[2], al[2];
            uint32_t ah2[2] = {0u, 0u}, al2[2] = {0u, 0u};  // R16: the same for row g8 + 8
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const uint32_t h0 = float_to_bf16_rne(sc[np + i][0]), h1 = float_to_bf16_rne(sc[np + i][1]);
                const uint32_t l0 = float_to_bf16_rne(sc[np + i][0] - __uint_as_float(h0 << 16));
                const uint32_t l1 = float_to_bf16_rne(sc[np + i][1] - __uint_as_float(h1 << 16));
                ah[i] = h0 | (h1 << 16); al[i] = l0 | (l1 << 16);
                if constexpr (R16) {
                    const uint32_t g0 = float_to_bf16_rne(sc[np + i][2]), g1 = float_to_bf16_rne(sc[np + i][3]);
                    const uint32_t m0 = float_to_bf16_rne(sc[np + i][2] - __uint_as_float(g0 << 16));
                    const uint32_t m1 = float_to_bf16_rne(sc[np + i][3] - __uint_as_float(g1 << 16));
                    ah2[i] = g0 | (g1 << 16); al2[i] = m0 | (m1 << 16);
                }
            }
#pragma unroll
            for (int j = 0; j < VJ; ++j) {
                const int wi = (j >> 1) & 3;
                uint32_t b[2];
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const uint4 &wa = vb[(np + i) % VR][0][j / 8], &wb = vb[(np + i) % VR][1][j / 8];
                    const uint32_t xa = wi == 0 ? wa.x : wi == 1 ? wa.y : wi == 2 ? wa.z : wa.w;
                    const uint32_t xb = wi == 0 ? wb.x : wi == 1 ? wb.y : wi == 2 ? wb.z : wb.w;
                    b[i] = __byte_perm(xa, xb, (j & 1) ? 0x7632 : 0x5410);     // dimension j of the two positions' rows
                }
                if constexpr (R16) {
                    mma_bf16_rows(o[j], al[0], al2[0], al[1], al2[1], b[0], b[1]);
                    mma_bf16_rows(o[j], ah[0], ah2[0], ah[1], ah2[1], b[0], b[1]);
                } else {
                    mma_bf16_top(o[j], al[0], al[1], b[0], b[1]);
                    mma_bf16_top(o[j], ah[0], ah[1], b[0], b[1]);
                }
            }
            if (np + VR < NT) load_v(np + VR, vb[np % VR]);
            if (np + 1 + VR < NT) load_v(np + 1 + VR, vb[(np + 1) % VR]);
        }
        // ---- partials out (row g8: dimensions DL*t4 + j and DL*t4 + VJ + j); the last warp of a (row, head) merges ----
        if (row_live) {
            const size_t pidx = ((size_t)rm * H + h) * md.n_seg_max + seg;
            if (t4 == 0) __stcg(md.part_ml + pidx, make_float2(mx, lsum));
            float *po = md.part_o + pidx * HD + DL * t4;
#pragma unroll
            for (int j = 0; j < VJ; j += 4) {
                __stcg(reinterpret_cast<float4 *>(po + j), make_float4(o[j][0], o[j + 1][0], o[j + 2][0], o[j + 3][0]));
                __stcg(reinterpret_cast<float4 *>(po + VJ + j), make_float4(o[j][1], o[j + 1][1], o[j + 2][1], o[j + 3][1]));
            }
        }
        if constexpr (R16) {
            if (row_live2) {                                  // row g8 + 8: accumulator registers 2, 3
                const size_t pidx = ((size_t)rm2 * H + h) * md.n_seg_max + seg;
                if (t4 == 0) __stcg(md.part_ml + pidx, make_float2(mx_r[NR - 1], lsum_r[NR - 1]));
                float *po = md.part_o + pidx * HD + DL * t4;
#pragma unroll
                for (int j = 0; j < VJ; j += 4) {
                    __stcg(reinterpret_cast<float4 *>(po + j), make_float4(o[j][2], o[j + 1][2], o[j + 2][2], o[j + 3][2]));
                    __stcg(reinterpret_cast<float4 *>(po + VJ + j), make_float4(o[j][3], o[j + 1][3], o[j + 2][3], o[j + 3][3]));
                }
            }
        }
        if (defer_merge) continue;                            // a separate merge operation follows a grid barrier
        __threadfence();
        __syncwarp();
        bool last = false;
        if (row_live && t4 == 0) {
            const int n_seg_m = (P0 + rm + SEGP) / SEGP;                  // segments row rm sees
            last = atomicAdd(md.attn_cnt + rm * H + h, 1) == n_seg_m - 1;
        }
        const unsigned last_mask = __ballot_sync(0xffffffffu, last);     // bit 4*g set: this warp finishes the (row, head) of lane row g
        if (last_mask) {
            __threadfence();
            for (int g = 0; g < BLKM; ++g) {
                if (!((last_mask >> (4 * g)) & 1u)) continue;
                const int rg = blk * BLKM + g;
                const int mg = all_cached ? row0 + g : rg % M, hg = all_cached ? grp : kvh * G + rg / M;
                attn_merge_row<HD>(md, op, P0, mg, hg, lane);
                if (lane == 0) md.attn_cnt[mg * H + hg] = 0;
            }
        }
    }
}

// Passes of more than BLKM rows first put the K/V rows of all their new positions into the cache (rotated, rounded),
// one (row, KV head) per warp, so that the attention operation - which then takes the rows one block at a time - reads
// every position from the cache.  Lane l holds dimensions [DPL*l, DPL*l + DPL); its rotation partner is lane l ^ 16.
template <int HD>
__device__ __forceinline__ void kv_append_phase(const Model &md, const Op &op, const Params &pr, int cta, int n_cta, int warp,
                                                int lane) {
    constexpr int DPL = HD / 32, HALF = HD / 2;
    typedef typename KVVec<HD>::T VT;
    const int H = md.H, Hkv = md.Hkv, P0 = md.state->len + pr.pos_off, jobs = pr.M * Hkv;
    const int qstride = (H + 2 * Hkv) * HD, d0 = DPL * lane, ci = d0 % HALF;
    const bool upper = d0 >= HALF;
    const float2 *my_cs = md.rope_cs + (size_t)cta * MAXM * HALF;
    for (int j = warp * n_cta + cta; j < jobs; j += NCW * n_cta) {
        const int m = j / Hkv, kvh = j % Hkv;
        const float *kraw = md.qkv + (size_t)m * qstride + (size_t)(H + kvh) * HD + d0;
        const float *vraw = md.qkv + (size_t)m * qstride + (size_t)(H + Hkv + kvh) * HD + d0;
        float kf[DPL], vf[DPL];
#pragma unroll
        for (int e = 0; e < DPL; ++e) { kf[e] = __ldcg(kraw + e); vf[e] = __ldcg(vraw + e); }
#pragma unroll
        for (int e = 0; e < DPL; ++e) {
            const float partner = __shfl_xor_sync(0xffffffffu, kf[e], 16);
            const float2 cs = my_cs[m * HALF + ci + e];
            kf[e] = upper ? (kf[e] * cs.x + partner * cs.y) : (kf[e] * cs.x - partner * cs.y);
        }
        *reinterpret_cast<VT *>(op.kc + ((size_t)kvh * md.max_seq + P0 + m) * HD + d0) = kv_pack<HD>(kf);
        *reinterpret_cast<VT *>(op.vc + ((size_t)kvh * md.max_seq + P0 + m) * HD + d0) = kv_pack<HD>(vf);
    }
}

// With several rows the warp that finishes a head last would merge all its rows one after the other; the merges
// then run as an operation of their own instead, one (row, head) per warp across the whole grid.
template <int HD>
__device__ __forceinline__ void attn_merge_phase(const Model &md, const Op &op, const Params &pr, int cta, int n_cta, int warp,
                                                 int lane) {
    const int P0 = md.state->len + pr.pos_off, jobs = pr.M * md.H;
    for (int j = warp * n_cta + cta; j < jobs; j += NCW * n_cta) attn_merge_row<HD>(md, op, P0, j / md.H, j % md.H, lane);
}

// ---- the pass ---------------------------------------------------------------------------------------------------
// NB = 1: passes of up to BLKM rows; NB = 2: 9..16 rows (a kernel of its own, so that the common one stays small).
// NP > 0: the linear maps take the rows four at a time with both terms in one operand (NP = 1: passes of up to 4 rows -
// every draft step; NP = 3 with NB = 2: passes of 9..12 rows); NP = 0: eight at a time, one operand per term.
template <int HD, int NB, int NP>
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
                lp.gb = stream::groups_per_batch<NB, NP>();
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
            lp.gb = stream::groups_per_batch<NB, NP>();
            if (op.is_head) {
                if (pr.head_row0 >= pr.M) ran = false;
                lp.M = pr.M - pr.head_row0;
                lp.xs += (size_t)pr.head_row0 * (lp.K >> 7) * stream::SLOT_WORDS;
                lp.ss_in += (size_t)pr.head_row0 * n_cta;
                lp.y += (size_t)(pr.out_row0 + pr.head_row0) * lp.units;
            }
            if (ran) stream::consume_linear_pre<NB, NP>(lp, r, cta, n_cta, warp, lane, w_use, alive);
        } else if (alive) {
            if (op.type == OP_EMBED) embed_phase(md, op, pr, r, cta, n_cta, tid);
            else if (op.type == OP_KV_APPEND) { if (NB > 1) kv_append_phase<HD>(md, op, pr, cta, n_cta, warp, lane); else ran = false; }
            else if (op.type == OP_ATTN) {
                if (NB == 1) {
                    attn_phase<HD, false>(md, op, pr, r, cta, n_cta, warp, lane, pr.merge_op != 0, 0, false);
                } else {
                    attn_phase<HD, true>(md, op, pr, r, cta, n_cta, warp, lane, true, 0, true);
                }
            }
            else if (op.type == OP_ATTN_MERGE) { if (pr.merge_op) attn_merge_phase<HD>(md, op, pr, cta, n_cta, warp, lane); else ran = false; }
            else if (op.type == OP_HIDDEN) { if (pr.want_hidden) hidden_phase(md, pr, r, cta, tid); else ran = false; }
            else if (op.type == OP_ARGMAX) { if (pr.head_row0 < pr.M) argmax_phase(md, pr, r, cta, n_cta, tid); else ran = false; }
        }
        if (md.trace && cta == 0 && tid == 0) md.trace[2 * i] = globaltimer_ns();
        if (op.barrier_after && ran) {
            ++n_bar;
            alive = grid_barrier(md, r, pr.bar_base + n_bar * (unsigned long long)n_cta, tid, alive,
                                 pr.bar_spin_limit ? pr.bar_spin_limit : BAR_SPIN_LIMIT);
        }
        if (md.trace && cta == 0 && tid == 0) md.trace[2 * i + 1] = globaltimer_ns();
    }
}

}  // namespace pass
}  // namespace knnssd
