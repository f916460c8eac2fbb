// Weight-streaming linear engine for bf16 weights and up to 8 activation rows (sm_100a).
//
// One persistent CTA per SM: a producer warp and eight consumer warps around a shared-memory ring.
//
// The producer streams the CTA's share of a weight matrix through the ring with bulk asynchronous copies
// (cp.async.bulk + mbarrier transaction counts), one 2 KB row segment per copy, sixteen per stage.  It needs
// nothing but free ring stages, so it runs ahead of the consumers - across the end of one linear map and
// into the next when several are chained in one kernel.
//
// The consumers turn each 16-row x 1024-column stage into tensor-core work: ldmatrix for the weight
// fragments, mma.sync m16n8k16 with the weights as the 16-row operand and the (at most 8) activation rows as
// the 8-column operand.  Activations are fp32 and are read straight from global memory (L2) by the warp that
// needs them; each value is split into three bf16 terms (hi + mid + lo, 24 mantissa bits together) that are
// multiplied separately into separate accumulators, so products are exact, the chains are independent and the
// result has fp32-accumulate accuracy.  The contraction is HBM-bound: the tensor pipe is used because it makes
// the per-byte instruction cost independent of the number of rows, not for FLOPs.
//
// Work split: the CTA owns a contiguous range of output units (balanced to +-1 across CTAs), cut into groups
// of at most 16 rows (8 gate + 8 up rows for the SwiGLU pair), processed in batches of up to 8 groups.  Inside
// a batch the loop runs over column tiles (outer) and groups (inner), so an activation slice is fetched and
// split once per column tile.  The 8 consumer warps each own a 128-column slot of every tile; their partial
// sums meet in shared memory in warp order at the end of a batch.  The sum order of an output therefore
// depends only on K, never on the row count M or on the grid.
//
// Every wait on an mbarrier is bounded: after SPIN_LIMIT polls the thread raises a CTA-wide abort flag,
// records a code in *err, and all threads fall through to the end of the kernel without further waits.
#pragma once
#include "kernels.cuh"

namespace knnssd {
namespace stream {

constexpr int SEG = 1024;                    // bf16 columns per tile
constexpr int WROWS = 16;                    // rows per weight tile (one mma M)
constexpr int WPITCH = SEG * 2 + 16;         // bytes; (pitch / 16) odd -> ldmatrix rows hit distinct banks
constexpr int WSTAGE = WROWS * WPITCH;
constexpr int NCW = 8;                       // consumer warps
constexpr int SLOT = SEG / NCW;              // columns per consumer warp per tile (128 = 8 k16 steps)
constexpr int KSTEPS = SLOT / 16;
constexpr int GB = 4;                        // groups per batch
constexpr int NTHREADS = (NCW + 4) * 32;      // two consumer warpgroups + the producer's warpgroup (one warp of it works)
constexpr int REGS_PRODUCER = 40, REGS_CONSUMER = 232;
constexpr int RED_BYTES = NCW * 8 * 32 * 4 * 4;  // reduction buffer (sized for 8 groups; attention keeps its K/V stash here)
constexpr int SS_BYTES = NCW * 8 * 4;
constexpr int BAR_BYTES = 1024;
constexpr int MAX_SMEM = 232448;             // 227 KB
constexpr int WS = (MAX_SMEM - RED_BYTES - SS_BYTES - BAR_BYTES) / WSTAGE;   // ring stages
constexpr int SMEM_BYTES = WS * WSTAGE + RED_BYTES + SS_BYTES + BAR_BYTES;
constexpr unsigned SPIN_LIMIT = 20000000u;
constexpr int NTERM = 2;                     // bf16 terms a pre-split activation is carried in (2: hi + lo, 16-17 significant bits)
constexpr int SLOT_WORDS = NTERM * 64;       // 32-bit words of one row's 128-column slot in a pre-split buffer
static_assert(WS >= 4 && 2 * WS * 8 + 16 <= BAR_BYTES, "ring layout");

// One linear map  y[m][u] = epilogue( sum_i W[u][i] * gain[i] * x[m][i] ).
struct LinPhase {
    const bf16_t *W[3];
    int rows[3];
    int units;          // outputs (SWIGLU: d_ff, each unit = one gate row + one up row)
    int K;              // n_in, multiple of 128
    const float *x;     // [M][K]
    const float *gain;  // [K] or nullptr
    float eps;
    float *y;           // [M][units]
    int epi;
    int M;              // 1..8 (stand-alone kernel), 1..16 (pass kernel)
    int gb;             // groups per batch, 1..GB (0 = GB); producer and consumers must use the same value
    // Pre-split form (persistent pass kernel): the producer of an activation writes it already split into the three
    // bf16 terms, in the order the tensor-core operand wants, so the consuming map only loads fragments.
    const uint32_t *xs;      // input  [M][K/128][NTERM terms][4][16] words (see split_index); nullptr = read x / gain
    const float *ss_in;      // [M][n_cta] partial sums of squares of the input rows (maps behind an RMSNorm); or nullptr
    uint32_t *ys;            // output in the same form for the next map (EPI_ADD: y * next_gain, SWIGLU: y); or nullptr
    const float *next_gain;  // [units] RMSNorm gain of the next map that reads y (EPI_ADD); nullptr = none
    float *ss_out;           // [M][n_cta] this CTA's partial sum of squares of each y row (EPI_ADD); or nullptr
};

// Word index of term 0 of column `col` of row m in a pre-split buffer with nslots = K / 128 column slots; the terms
// of one value sit 64 words apart (NTERM terms per value).  A lane (group t4) needs 16 words per term and slot: word
// 2j + h packs columns (16j + 8h + 2t4, 16j + 8h + 2t4 + 1) of the slot - the pair an m16n8k16 "col" operand register
// holds for k-step j.  They are stored as four 16-byte pieces q = 0..3, and piece q of the four lane groups is
// contiguous (64 bytes), so one warp-wide 16-byte load touches whole 32-byte sectors only.
__host__ __device__ __forceinline__ size_t split_index(int nslots, int m, int col) {
    const int s = col >> 7, within = col & 127, j = within >> 4, r = within & 15, h = r >> 3, t4 = (r & 7) >> 1;
    const int wr = 2 * j + h;                 // word of the lane's 16-word run: q = wr / 4 is the 16-byte piece it lies in
    return (((size_t)m * nslots + s) * NTERM) * 64 + (wr >> 2) * 16 + t4 * 4 + (wr & 3);
}

// Shared-memory ring and its barriers, carved out of the CTA's dynamic shared memory.
struct Ring {
    unsigned char *wring;
    float *red, *red_ss;
    uint64_t *full_w, *empty_w;
    volatile int *abort_flag;
    int *err;           // device int: set non-zero if a bounded wait gave up
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t *b, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *b, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *b) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *b, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false (and raises the abort flag) if the barrier never flipped.
__device__ __forceinline__ bool mbar_wait(uint64_t *b, uint32_t parity, volatile int *abort_flag, int *err, int code) {
    if (mbar_try_wait(b, parity)) return true;
    unsigned spins = 0;
    while (!mbar_try_wait(b, parity)) {
        if (*abort_flag) return false;
        if (++spins > SPIN_LIMIT) {
            *abort_flag = 1;
            atomicExch(err, code);
            return false;
        }
    }
    return true;
}
// Weight rows are read once per pass: they go through L2 marked evict-first, so that the 26 GB stream does not push
// out what every CTA reads again and again from there (activation fragments, partial sums, the projection buffer).
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, uint64_t *b) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(b)), "l"(l2_evict_first_policy())
                 : "memory");
}
// Register hand-over between warpgroups: the producer's warpgroup gives most of its registers back and the two
// consumer warpgroups take them (every warp of a warpgroup must execute the instruction).
template <int N> __device__ __forceinline__ void regs_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void regs_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &a0, uint32_t &a1, uint32_t &a2, uint32_t &a3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// Activations may have been written by other CTAs earlier in the same kernel: read them at L2, never from L1.
__device__ __forceinline__ float2 ld_act2(const float *p) { return __ldcg(reinterpret_cast<const float2 *>(p)); }

// v = hi + mid + lo with each term a bf16 (round to nearest even); residuals are exact in fp32.
__device__ __forceinline__ void split3(float v, uint32_t &hi, uint32_t &mid, uint32_t &lo) {
    hi = float_to_bf16_rne(v);
    const float r1 = v - __uint_as_float(hi << 16);
    mid = float_to_bf16_rne(r1);
    const float r2 = r1 - __uint_as_float(mid << 16);
    lo = float_to_bf16_rne(r2);
}

// Write one activation value in pre-split form: hi = bf16(v), then the bf16 roundings of the successive residuals
// (each residual is exact in fp32).
__device__ __forceinline__ void store_split(uint32_t *buf, int nslots, int m, int col, float v) {
    bf16_t *b = reinterpret_cast<bf16_t *>(buf) + 2 * split_index(nslots, m, col) + (col & 1);
#pragma unroll
    for (int t = 0; t < NTERM; ++t) {
        const uint32_t h = float_to_bf16_rne(v);
        __stcg(b + 128 * t, (bf16_t)h);
        v -= __uint_as_float(h << 16);
    }
}

// The CTA's share of a linear map: units [u_lo, u_lo + n_units) in n_groups groups whose sizes differ by at
// most one (the first g_rem groups hold g_base + 1 units).
struct Share {
    int u_lo, n_units, n_groups, g_base, g_rem, n_batches, n_kt, gsz, gb;
    bool swiglu;
    __device__ __forceinline__ int group_lo(int g) const { return g * g_base + min(g, g_rem); }
    __device__ __forceinline__ int group_size(int g) const { return g_base + (g < g_rem ? 1 : 0); }
};

__device__ __forceinline__ Share make_share(const LinPhase &p, int cta, int n_cta) {
    Share s;
    s.swiglu = p.epi == EPI_SWIGLU;
    s.gsz = s.swiglu ? 8 : 16;
    s.u_lo = (int)(((long long)p.units * cta) / n_cta);
    const int u_hi = (int)(((long long)p.units * (cta + 1)) / n_cta);
    s.n_units = u_hi - s.u_lo;
    s.n_groups = (s.n_units + s.gsz - 1) / s.gsz;
    s.g_base = s.n_groups ? s.n_units / s.n_groups : 0;
    s.g_rem = s.n_groups ? s.n_units % s.n_groups : 0;
    s.gb = p.gb > 0 && p.gb < GB ? p.gb : GB;
    s.n_batches = (s.n_groups + s.gb - 1) / s.gb;
    s.n_kt = (p.K + SEG - 1) / SEG;
    return s;
}

__device__ __forceinline__ void ring_setup(Ring &r, unsigned char *smem, int *err) {
    r.wring = smem;
    r.red = reinterpret_cast<float *>(smem + WS * WSTAGE);
    r.red_ss = r.red + RED_BYTES / 4;
    uint64_t *bars = reinterpret_cast<uint64_t *>(reinterpret_cast<unsigned char *>(r.red_ss) + SS_BYTES);
    r.full_w = bars;
    r.empty_w = bars + WS;
    r.abort_flag = reinterpret_cast<volatile int *>(bars + 2 * WS);
    r.err = err;
    if (threadIdx.x == 0) {
        for (int s = 0; s < WS; ++s) { mbar_init(&r.full_w[s], 1); mbar_init(&r.empty_w[s], NCW); }
        *r.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
}

// ------------------------------------------------------------------------------------------------------------
// Producer warp: streams this CTA's share of the weights of one linear map into the ring.  w_use counts the
// stages this CTA has filled since the kernel began (the consumers keep the same count).
// ------------------------------------------------------------------------------------------------------------
__device__ __forceinline__ void produce_linear(const LinPhase &p, const Ring &r, int cta, int n_cta, int lane, int &w_use,
                                               bool &alive) {
    const Share s = make_share(p, cta, n_cta);
    int ws = w_use % WS, it = w_use / WS;
    for (int b = 0; b < s.n_batches && alive; ++b) {
        const int g0 = b * s.gb, ng = min(s.n_groups - g0, s.gb);
        // source row of this lane in each group of the batch, and the row count of each group
        const bf16_t *src[GB];
        int nrows[GB];
#pragma unroll
        for (int gi = 0; gi < GB; ++gi) {
            src[gi] = nullptr;
            nrows[gi] = 0;
            if (gi < ng) {
                const int lo = s.group_lo(g0 + gi), nu = s.group_size(g0 + gi);
                nrows[gi] = s.swiglu ? 2 * nu : nu;
                const int rr = s.swiglu ? (lane & 7) : lane;
                if (lane < WROWS && rr < nu) {
                    int u = s.u_lo + lo + rr;
                    if (s.swiglu) {
                        src[gi] = p.W[lane >> 3] + (size_t)u * p.K;
                    } else {
                        int which = 0;
                        if (u >= p.rows[0]) { u -= p.rows[0]; which = 1; }
                        if (which == 1 && u >= p.rows[1]) { u -= p.rows[1]; which = 2; }
                        src[gi] = p.W[which] + (size_t)u * p.K;
                    }
                }
            }
        }
        for (int kt = 0; kt < s.n_kt && alive; ++kt) {
            const int c0 = kt * SEG, segc = min(SEG, p.K - c0);
#pragma unroll
            for (int gi = 0; gi < GB; ++gi) {
                if (gi >= ng || !alive) break;
                if (it > 0) alive = mbar_wait(&r.empty_w[ws], (it - 1) & 1, r.abort_flag, r.err, 3);
                if (!alive) break;
                if (lane == 0) mbar_expect_tx(&r.full_w[ws], (uint32_t)nrows[gi] * segc * 2);
                __syncwarp();
                if (src[gi]) bulk_g2s(r.wring + ws * WSTAGE + lane * WPITCH, src[gi] + c0, segc * 2, &r.full_w[ws]);
                ++w_use;
                if (++ws == WS) { ws = 0; ++it; }
            }
        }
    }
}

// After an abort: give copies already in flight time to land before the CTA's shared memory goes away.
__device__ __forceinline__ void producer_drain_after_abort() {
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
}

// ------------------------------------------------------------------------------------------------------------
// Consumer warps (warp 0..NCW-1, 256 threads, named barrier 1): the matching half.
// ------------------------------------------------------------------------------------------------------------
__device__ __forceinline__ void consume_linear(const LinPhase &p, const Ring &r, int cta, int n_cta, int warp, int lane,
                                               int &w_use, bool &alive) {
    const Share s = make_share(p, cta, n_cta);
    const int tid = warp * 32 + lane;
    const int g8 = lane >> 2, t4 = lane & 3;
    const int lm_row = (lane & 7) + ((lane >> 3) & 1) * 8, lm_col = (lane >> 4) * 8;   // ldmatrix source of this lane
    const bool normed = p.gain != nullptr;
    const bool row_live = g8 < p.M;
    const float *xrow = p.x + (size_t)min(g8, p.M - 1) * p.K + warp * SLOT + 2 * t4;
    const float *grow = normed ? p.gain + warp * SLOT + 2 * t4 : nullptr;
    int ws = w_use % WS, it = w_use / WS;
    float *red = r.red, *red_ss = r.red_ss;
    for (int b = 0; b < s.n_batches; ++b) {
        const int g0 = b * s.gb, ng = min(s.n_groups - g0, s.gb);
        float acc[GB][4];
#pragma unroll
        for (int i = 0; i < GB; ++i) { acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f; }
        float ss = 0.f;
        // raw activations (and gains) of the next column tile: fetched one tile ahead so that the L2 latency
        // hides behind the tensor-core work of the current tile
        float2 xv[KSTEPS][2], gv[KSTEPS][2];
        auto fetch = [&](int kt) {
            const int c0 = kt * SEG, segc = min(SEG, p.K - c0);
            const bool ld = alive && row_live && warp * SLOT < segc;
#pragma unroll
            for (int j = 0; j < KSTEPS; ++j) {
                xv[j][0] = xv[j][1] = make_float2(0.f, 0.f);
                gv[j][0] = gv[j][1] = make_float2(1.f, 1.f);
                if (ld) {
                    xv[j][0] = ld_act2(xrow + c0 + j * 16);
                    xv[j][1] = ld_act2(xrow + c0 + j * 16 + 8);
                    if (normed) {
                        gv[j][0] = __ldg(reinterpret_cast<const float2 *>(grow + c0 + j * 16));
                        gv[j][1] = __ldg(reinterpret_cast<const float2 *>(grow + c0 + j * 16 + 8));
                    }
                }
            }
        };
        fetch(0);
        for (int kt = 0; kt < s.n_kt; ++kt) {
            const int c0 = kt * SEG, segc = min(SEG, p.K - c0);
            const bool slot_valid = warp * SLOT < segc;
            uint32_t bh[KSTEPS][2], bm[KSTEPS][2], bl[KSTEPS][2];
#pragma unroll
            for (int j = 0; j < KSTEPS; ++j) {
                float v[4] = {xv[j][0].x, xv[j][0].y, xv[j][1].x, xv[j][1].y};
                if (normed) {
                    ss = fmaf(v[0], v[0], ss); ss = fmaf(v[1], v[1], ss);
                    ss = fmaf(v[2], v[2], ss); ss = fmaf(v[3], v[3], ss);
                    v[0] *= gv[j][0].x; v[1] *= gv[j][0].y; v[2] *= gv[j][1].x; v[3] *= gv[j][1].y;
                }
                uint32_t h[4], m[4], l[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) split3(v[e], h[e], m[e], l[e]);
                bh[j][0] = h[0] | (h[1] << 16); bh[j][1] = h[2] | (h[3] << 16);
                bm[j][0] = m[0] | (m[1] << 16); bm[j][1] = m[2] | (m[3] << 16);
                bl[j][0] = l[0] | (l[1] << 16); bl[j][1] = l[2] | (l[3] << 16);
            }
            if (kt + 1 < s.n_kt) fetch(kt + 1);
#pragma unroll
            for (int gi = 0; gi < GB; ++gi) {
                if (gi >= ng) break;
                if (alive) alive = mbar_wait(&r.full_w[ws], it & 1, r.abort_flag, r.err, 5);
                if (alive && slot_valid) {
                    const uint32_t base = smem_u32(r.wring + ws * WSTAGE) + lm_row * WPITCH + (warp * SLOT + lm_col) * 2;
                    float tl[4] = {0.f, 0.f, 0.f, 0.f}, tm[4] = {0.f, 0.f, 0.f, 0.f}, th[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int j = 0; j < KSTEPS; ++j) {
                        uint32_t a0, a1, a2, a3;
                        ldmatrix_x4(base + j * 32, a0, a1, a2, a3);
                        mma_bf16(tl, a0, a1, a2, a3, bl[j][0], bl[j][1]);
                        mma_bf16(tm, a0, a1, a2, a3, bm[j][0], bm[j][1]);
                        mma_bf16(th, a0, a1, a2, a3, bh[j][0], bh[j][1]);
                    }
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[gi][e] += (tl[e] + tm[e]) + th[e];
                }
                __syncwarp();
                if (alive && lane == 0) mbar_arrive(&r.empty_w[ws]);
                ++w_use;
                if (++ws == WS) { ws = 0; ++it; }
            }
        }
        // ---- batch end: partial sums of the 8 column slots meet in shared memory, in warp order ----
#pragma unroll
        for (int gi = 0; gi < GB; ++gi)
            *reinterpret_cast<float4 *>(red + ((warp * GB + gi) * 32 + lane) * 4) =
                make_float4(acc[gi][0], acc[gi][1], acc[gi][2], acc[gi][3]);
        if (normed) {
            ss += __shfl_xor_sync(0xffffffffu, ss, 1);
            ss += __shfl_xor_sync(0xffffffffu, ss, 2);
            if (t4 == 0) red_ss[warp * 8 + g8] = ss;
        }
        asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
        if (alive) {
            const int per_group = s.gsz * 8;                        // (unit, token) pairs per group
            for (int idx = tid; idx < ng * per_group; idx += NCW * 32) {
                const int gi = idx / per_group, rem = idx % per_group;
                const int rr = rem >> 3, n = rem & 7;             // unit within group, token
                if (rr >= s.group_size(g0 + gi) || n >= p.M) continue;
                // rows 0..7 of the tile: regs 0,1; rows 8..15: regs 2,3
                const int src_lane = (rr & 7) * 4 + (n >> 1), reg = n & 1;
                float s0 = 0.f, s1 = 0.f;
#pragma unroll
                for (int w = 0; w < NCW; ++w) {
                    const float *q = red + ((w * GB + gi) * 32 + src_lane) * 4;
                    if (s.swiglu) { s0 += q[reg]; s1 += q[2 + reg]; }
                    else s0 += q[(rr >> 3) * 2 + reg];
                }
                float ri = 1.0f;
                if (normed) {
                    float tot = 0.f;
#pragma unroll
                    for (int w = 0; w < NCW; ++w) tot += red_ss[w * 8 + n];
                    ri = 1.0f / sqrtf(tot / (float)p.K + p.eps);
                }
                float *yp = p.y + (size_t)n * p.units + (s.u_lo + s.group_lo(g0 + gi) + rr);
                if (s.swiglu) {
                    const float gt = s0 * ri, up = s1 * ri;
                    __stcg(yp, gt / (1.0f + expf(-gt)) * up);
                } else if (p.epi == EPI_ADD) {
                    __stcg(yp, __ldcg(yp) + s0 * ri);
                } else {
                    __stcg(yp, s0 * ri);
                }
            }
        }
        asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
    }
}

// Stand-alone launch of one linear map: grid = one CTA per SM.
__global__ void __launch_bounds__(NTHREADS, 1) linear_stream_kernel(const LinPhase p, int *err) {
    extern __shared__ __align__(128) unsigned char smem[];
    Ring r;
    ring_setup(r, smem, err);
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int w_use = 0;
    bool alive = true;
    if (warp >= NCW) {
        regs_dec<REGS_PRODUCER>();
        if (warp == NCW) {
            produce_linear(p, r, blockIdx.x, gridDim.x, lane, w_use, alive);
            if (!alive) producer_drain_after_abort();
        }
    } else {
        regs_inc<REGS_CONSUMER>();
        consume_linear(p, r, blockIdx.x, gridDim.x, warp, lane, w_use, alive);
    }
}

}  // namespace stream
}  // namespace knnssd
