// Host side of libknnssd.so: the C ABI declared in include/knnssd.h, the session state and the
// sequencing of one decoder pass (which sublayers run, on how many rows, at which positions).
// Every step of the path runs in the kernels of kernels.cuh; the host only enqueues them.
#include "../../include/knnssd.h"
#include "kernels.cuh"
#include "linear_stream.cuh"
#include "pass_kernel.cuh"
#include "prefill_host.cuh"
#include "anchors.cuh"
#include "linear_tc.cuh"
#include "sampling.cuh"

#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

using namespace knnssd;

namespace {

constexpr int kMaxRows = 16;       // most rows one pass carries (prefill chunk; verify uses k+1 <= 16)
constexpr int kArgmaxBlocks = 64;  // slices per row in the arg-max

struct Layer {
    const float *attn_norm, *mlp_norm;
    const void *wq, *wk, *wv, *wo, *w_gate, *w_up, *w_down;
};

}  // namespace

struct knnssd_ctx {
    knnssd_config cfg{};
    std::vector<Layer> layers;
    const void *tok_embed = nullptr, *lm_head = nullptr;
    const float *final_norm = nullptr;
    const float *anchors = nullptr;
    std::vector<unsigned char> domain_masks;  // [n_domains][2L]
    std::vector<unsigned char> active_mask;   // [2L]
    bool has_mask = false, prefilled = false;
    cudaStream_t stream = nullptr;
    int device = 0, n_sms = 148;
    size_t wbytes = 2;

    // device buffers (owned)
    void *kcache = nullptr, *vcache = nullptr;
    float *x = nullptr, *qkv = nullptr, *attn = nullptr, *act = nullptr, *logits = nullptr, *hfinal = nullptr;
    float *part_o = nullptr, *pooled = nullptr, *anchor_inv_norm = nullptr, *cosines = nullptr, *amax_v = nullptr;
    float2 *part_ml = nullptr, *rope_cs = nullptr;
    double *pool_sum = nullptr, *inv_freq = nullptr;
    int *chain = nullptr, *target = nullptr, *prompt = nullptr, *out_tokens = nullptr, *accept_log = nullptr;
    int *amax_i = nullptr, *flag = nullptr, *knn_out = nullptr;
    DeviceState *state = nullptr;
    float *samp_p = nullptr, *samp_q = nullptr;   // sampled decoding: filtered distributions [kMaxRows][vocab], made on first use
    int *samp_res = nullptr;                      // [2] result of a keep-or-resample round
    int *err_word = nullptr;   // this device's error word (bounded waits that gave up, bad token ids, non-finite logits)
    bool enqueue_failed = false;   // a pass could not be enqueued (its operation list did not reach the device)
    unsigned bar_spin_limit = 0;   // grid-barrier poll limit handed to the pass kernel (0 = its default)
    int *pinned = nullptr;  // host, pinned: small read-backs
    int n_splits = 1;

    // host mirror of the session
    int len = 0, pending = -1;
    knnssd_stats stats{};
    cudaEvent_t ev0 = nullptr, ev1 = nullptr, ev2 = nullptr;
    std::string err;

    // persistent pass kernel (bf16 models whose widths are multiples of 128)
    bool mega_ok = false;
    pass::Model model{};
    pass::Op *ops_full = nullptr, *ops_draft = nullptr;     // device op lists
    int n_ops_full = 0, n_ops_draft = 0, bar_full = 0, bar_draft = 0;   // ops and barriers (without head / hidden parts)
    int attn_full = 0, attn_draft = 0;                                  // attention sublayers in each list
    std::vector<unsigned char> ops_draft_mask;              // the mask ops_draft was built for
    unsigned long long *bar = nullptr, bar_total = 0;
    int *gabort = nullptr, *attn_cnt = nullptr, *amax_cnt = nullptr;
    float *mpart_o = nullptr, *mamax_v = nullptr;
    float2 *mpart_ml = nullptr;
    int *mamax_i = nullptr;
    unsigned long long *trace = nullptr;
    uint32_t *xs_x = nullptr, *xs_attn = nullptr, *xs_act = nullptr;   // pre-split activations (see LinPhase::xs)
    float *ssp = nullptr;                                              // [MAXM][n_sms] partial sums of squares of x rows

    // tensor-core prompt pass (same eligibility as the pass kernel): activations of up to pf_cap rows
    bool pf_ok = false;
    int pf_cap = 0;                                          // rows per chunk, a multiple of 128
    float *pf_x = nullptr, *pf_qkv = nullptr;                // residual stream [cap][d]; q, k, v [cap][nq + 2 nkv]
    float2 *pf_cs = nullptr;                                 // rotary (cos, sin) of the chunk's rows [cap][hd / 2]
    float *pf_rinv = nullptr;                                // RMSNorm scale of the chunk's rows [cap]
    bf16_t *pf_ad = nullptr, *pf_aq = nullptr, *pf_af = nullptr;   // hi / lo planes [2][cap][d], [2][cap][nq], [2][cap][d_ff]
    CUtensorMap pf_map_d{}, pf_map_q{}, pf_map_f{};

    // instrumentation
    long long launches = 0;
    bool time_linear = false;
    std::vector<cudaEvent_t> lin_events;
    size_t lin_used = 0;
};

namespace {

knnssd_status fail(knnssd_ctx *c, knnssd_status s, const std::string &msg) {
    if (c) c->err = msg;
    return s;
}

#define CUDA_TRY(ctx, expr)                                                                          \
    do {                                                                                             \
        cudaError_t e_ = (expr);                                                                     \
        if (e_ != cudaSuccess)                                                                       \
            return fail(ctx, KNNSSD_ERR_CUDA, std::string(#expr) + ": " + cudaGetErrorString(e_));   \
    } while (0)

template <typename T> cudaError_t dev_alloc(T **p, size_t count) {
    return cudaMalloc(reinterpret_cast<void **>(p), count * sizeof(T));
}

int pick_mt(int M) {
    static const int opts[] = {1, 2, 3, 4, 5, 6, 7, 8, 9, 16};
    for (int o : opts)
        if (M <= o) return o;
    return -1;
}

template <typename WT> void launch_linear_t(const LinearArgs &a, int grid, cudaStream_t s) {
    switch (pick_mt(a.M)) {
        case 1: linear_kernel<WT, 1><<<grid, 256, 0, s>>>(a); break;
        case 2: linear_kernel<WT, 2><<<grid, 256, 0, s>>>(a); break;
        case 3: linear_kernel<WT, 3><<<grid, 256, 0, s>>>(a); break;
        case 4: linear_kernel<WT, 4><<<grid, 256, 0, s>>>(a); break;
        case 5: linear_kernel<WT, 5><<<grid, 256, 0, s>>>(a); break;
        case 6: linear_kernel<WT, 6><<<grid, 256, 0, s>>>(a); break;
        case 7: linear_kernel<WT, 7><<<grid, 256, 0, s>>>(a); break;
        case 8: linear_kernel<WT, 8><<<grid, 256, 0, s>>>(a); break;
        case 9: linear_kernel<WT, 9><<<grid, 256, 0, s>>>(a); break;
        default: linear_kernel<WT, 16><<<grid, 256, 0, s>>>(a); break;
    }
}

// Set by the streaming kernel if one of its bounded waits ever gives up (never in normal operation).
__device__ int g_stream_err;

constexpr int kMaxDevices = 64;

// Index of the current device in the per-device tables below (0 if it cannot be read or is out of range).
int current_device_slot() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) dev = 0;
    return dev;
}

// Address of the error word on the CURRENT device (every device that loads the library has its own copy).
int *stream_err_ptr() {
    static int *addr[kMaxDevices] = {};
    static std::mutex mu;
    const int dev = current_device_slot();
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) cudaGetSymbolAddress(reinterpret_cast<void **>(&addr[dev]), g_stream_err);
    return addr[dev];
}

bool stream_eligible(int dtype, const LinearArgs &a) {
    return dtype == 1 && a.M <= 8 && a.n_in % 128 == 0 && a.n_in >= 256;
}

stream::LinPhase to_phase(const LinearArgs &a) {
    stream::LinPhase p{};
    for (int i = 0; i < 3; ++i) { p.W[i] = reinterpret_cast<const bf16_t *>(a.W[i]); p.rows[i] = a.rows[i]; }
    p.units = a.units; p.K = a.n_in; p.x = a.x; p.gain = a.gain; p.eps = a.eps; p.y = a.y; p.epi = a.epi; p.M = a.M;
    return p;
}

void launch_stream(const LinearArgs &a, int n_sms, cudaStream_t s) {
    static bool configured[kMaxDevices] = {};          // function attributes are per device
    const int dev = current_device_slot();
    if (!configured[dev]) {
        cudaFuncSetAttribute(stream::linear_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, stream::SMEM_BYTES);
        configured[dev] = true;
    }
    stream::linear_stream_kernel<<<n_sms, stream::NTHREADS, stream::SMEM_BYTES, s>>>(to_phase(a), stream_err_ptr());
}

void launch_linear(int dtype, const LinearArgs &a, int n_sms, cudaStream_t s) {
    if (stream_eligible(dtype, a)) { launch_stream(a, n_sms, s); return; }
    // generic kernel: enough warps that every SM holds 8 blocks of 8 warps, but never more warps than units
    long long blocks = (long long)n_sms * 8;
    const long long max_blocks = (a.units + 7) / 8;
    if (blocks > max_blocks) blocks = max_blocks;
    if (blocks < 1) blocks = 1;
    if (dtype) launch_linear_t<bf16_t>(a, (int)blocks, s); else launch_linear_t<float>(a, (int)blocks, s);
}

void ctx_linear(knnssd_ctx *c, const LinearArgs &a) {
    if (c->time_linear) {
        if (c->lin_used + 2 > c->lin_events.size()) {
            for (int i = 0; i < 2; ++i) {
                cudaEvent_t e;
                cudaEventCreate(&e);
                c->lin_events.push_back(e);
            }
        }
        cudaEventRecord(c->lin_events[c->lin_used], c->stream);
    }
    launch_linear(c->cfg.dtype, a, c->n_sms, c->stream);
    if (c->time_linear) {
        cudaEventRecord(c->lin_events[c->lin_used + 1], c->stream);
        c->lin_used += 2;
    }
    c->launches++;
}

LinearArgs make_args(const void *W0, int rows0, int n_in, const float *x, const float *gain, float eps, float *y,
                     int epi, int M) {
    LinearArgs a{};
    a.W[0] = W0; a.rows[0] = rows0; a.units = rows0; a.n_in = n_in; a.x = x; a.gain = gain; a.eps = eps; a.y = y;
    a.epi = epi; a.M = M;
    return a;
}

// ---- persistent pass kernel: op lists and launch ----------------------------------------------------------------
// The list of one pass under a skip mask (nullptr = full model).  n_bar receives the number of grid barriers of the
// body; the head part (when rows get logits) adds one more.
std::vector<pass::Op> build_ops(const knnssd_ctx *c, const unsigned char *mask, int *n_bar, int *n_attn) {
    const knnssd_config &g = c->cfg;
    const int d = g.d_model, hd = g.head_dim, nq = g.n_heads * hd, nkv = g.n_kv_heads * hd, F = g.d_ff, V = g.vocab;
    std::vector<pass::Op> ops;
    int bars = 0, attn = 0;
    auto lin = [&](const void *W0, int rows0, int K, const float *x, const float *gain, float *y, int epi) {
        pass::Op o{};
        o.type = pass::OP_LINEAR; o.barrier_after = 1;
        o.lin.W[0] = reinterpret_cast<const bf16_t *>(W0); o.lin.rows[0] = rows0; o.lin.units = rows0; o.lin.K = K;
        o.lin.x = x; o.lin.gain = gain; o.lin.eps = g.rms_eps; o.lin.y = y; o.lin.epi = epi; o.lin.M = 1;
        return o;
    };
    pass::Op e{};
    e.type = pass::OP_EMBED; e.barrier_after = 1;
    e.lin.K = d; e.lin.ys = c->xs_x; e.lin.ss_out = c->ssp;
    ops.push_back(e); ++bars;
    const size_t layer_stride = (size_t)g.n_kv_heads * g.max_seq * hd;
    for (int l = 0; l < g.n_layers; ++l) {
        const Layer &ly = c->layers[l];
        if (!mask || !mask[2 * l]) {
            pass::Op q = lin(ly.wq, nq, d, c->x, ly.attn_norm, c->qkv, EPI_STORE);
            q.lin.W[1] = reinterpret_cast<const bf16_t *>(ly.wk); q.lin.rows[1] = nkv;
            q.lin.W[2] = reinterpret_cast<const bf16_t *>(ly.wv); q.lin.rows[2] = nkv;
            q.lin.units = nq + 2 * nkv; q.layer = l;
            q.lin.xs = c->xs_x; q.lin.ss_in = c->ssp;
            ops.push_back(q);
            pass::Op ap{};                               // runs (and its barrier counts) only in passes of > BLKM rows
            ap.type = pass::OP_KV_APPEND; ap.barrier_after = 1; ap.layer = l;
            ap.kc = reinterpret_cast<bf16_t *>(c->kcache) + (size_t)l * layer_stride;
            ap.vc = reinterpret_cast<bf16_t *>(c->vcache) + (size_t)l * layer_stride;
            ops.push_back(ap);
            pass::Op a{};
            a.type = pass::OP_ATTN; a.barrier_after = 1; a.layer = l;
            a.kc = reinterpret_cast<bf16_t *>(c->kcache) + (size_t)l * layer_stride;
            a.vc = reinterpret_cast<bf16_t *>(c->vcache) + (size_t)l * layer_stride;
            a.lin.ys = c->xs_attn;
            ops.push_back(a);
            pass::Op mg{};                               // runs (and its barrier counts) only in passes of >= MERGE_ROWS rows
            mg.type = pass::OP_ATTN_MERGE; mg.barrier_after = 1; mg.layer = l; mg.lin.ys = c->xs_attn;
            ops.push_back(mg);
            ++attn;
            pass::Op o = lin(ly.wo, d, nq, c->attn, nullptr, c->x, EPI_ADD);
            o.layer = l;
            o.lin.xs = c->xs_attn; o.lin.ys = c->xs_x; o.lin.ss_out = c->ssp;
            ops.push_back(o);
            bars += 3;
        }
        if (!mask || !mask[2 * l + 1]) {
            pass::Op gu = lin(ly.w_gate, F, d, c->x, ly.mlp_norm, c->act, EPI_SWIGLU);
            gu.lin.W[1] = reinterpret_cast<const bf16_t *>(ly.w_up); gu.lin.rows[1] = F; gu.layer = l;
            gu.lin.xs = c->xs_x; gu.lin.ss_in = c->ssp; gu.lin.ys = c->xs_act;
            ops.push_back(gu);
            pass::Op dn = lin(ly.w_down, d, F, c->act, nullptr, c->x, EPI_ADD);
            dn.layer = l;
            dn.lin.xs = c->xs_act; dn.lin.ys = c->xs_x; dn.lin.ss_out = c->ssp;
            ops.push_back(dn);
            bars += 2;
        }
    }
    pass::Op hdn{};
    hdn.type = pass::OP_HIDDEN;                      // runs only when the pass wants hidden states; no barrier: reads x only
    ops.push_back(hdn);
    pass::Op head = lin(c->lm_head, V, d, c->x, c->final_norm, c->logits, EPI_STORE);
    head.is_head = 1;                                // runs only when rows get logits; its barrier counts only then
    head.lin.xs = c->xs_x; head.lin.ss_in = c->ssp;
    ops.push_back(head);
    pass::Op am{};
    am.type = pass::OP_ARGMAX;
    ops.push_back(am);
    // whoever writes the residual stream also writes it pre-split, times the gain of the RMSNorm that reads it next
    const float *next_gain = nullptr;
    for (int i = (int)ops.size() - 1; i >= 0; --i) {
        pass::Op &o = ops[i];
        if (o.type == pass::OP_EMBED || (o.type == pass::OP_LINEAR && o.lin.epi == EPI_ADD)) o.lin.next_gain = next_gain;
        if (o.type == pass::OP_LINEAR && o.lin.gain) next_gain = o.lin.gain;
    }
    *n_bar = bars;
    *n_attn = attn;
    return ops;
}

knnssd_status upload_ops(knnssd_ctx *c, const std::vector<pass::Op> &ops, pass::Op *dst) {
    CUDA_TRY(c, cudaMemcpyAsync(dst, ops.data(), ops.size() * sizeof(pass::Op), cudaMemcpyHostToDevice, c->stream));
    // the host vector goes away after this call: wait for the copy (mask changes are rare)
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    return KNNSSD_OK;
}

template <int HD, int NB, int NP> cudaError_t launch_pass_t(knnssd_ctx *c, const pass::Params &pr) {
    static bool configured[kMaxDevices] = {};          // function attributes are per device
    const int dev = current_device_slot();
    if (!configured[dev]) {
        cudaFuncSetAttribute(pass::pass_kernel<HD, NB, NP>, cudaFuncAttributeMaxDynamicSharedMemorySize, stream::SMEM_BYTES);
        configured[dev] = true;
    }
    void *args[] = {const_cast<pass::Model *>(&c->model), const_cast<pass::Params *>(&pr)};
    return cudaLaunchCooperativeKernel(reinterpret_cast<void *>(pass::pass_kernel<HD, NB, NP>), dim3(c->n_sms),
                                       dim3(stream::NTHREADS), args, stream::SMEM_BYTES, c->stream);
}

// One pass through the persistent kernel.  Errors surface at the caller's next synchronisation.
void run_pass_mega(knnssd_ctx *c, int M, const int *tok_dev, int pos_off, const unsigned char *mask, int head_row0,
                   int *argmax_out, bool want_hidden, int out_row0 = 0) {
    pass::Params pr{};
    int bars, n_attn;
    if (!mask) {
        pr.ops = c->ops_full; pr.n_ops = c->n_ops_full; bars = c->bar_full; n_attn = c->attn_full;
    } else {
        const size_t n = 2 * (size_t)c->cfg.n_layers;
        if (c->ops_draft_mask.size() != n || std::memcmp(c->ops_draft_mask.data(), mask, n) != 0) {
            const std::vector<pass::Op> ops = build_ops(c, mask, &c->bar_draft, &c->attn_draft);
            c->n_ops_draft = (int)ops.size();
            if (upload_ops(c, ops, c->ops_draft) != KNNSSD_OK) { c->enqueue_failed = true; return; }
            c->ops_draft_mask.assign(mask, mask + n);
        }
        pr.ops = c->ops_draft; pr.n_ops = c->n_ops_draft; bars = c->bar_draft; n_attn = c->attn_draft;
    }
    pr.M = M; pr.tok = tok_dev; pr.pos_off = pos_off; pr.head_row0 = head_row0; pr.argmax_out = argmax_out;
    pr.want_hidden = want_hidden ? 1 : 0;
    pr.out_row0 = out_row0;
    pr.bar_spin_limit = c->bar_spin_limit;
    pr.bar_base = c->bar_total;
    if (head_row0 < M) bars += 1;
    pr.merge_op = pass::merge_rows_separately(M, c->cfg.n_heads / c->cfg.n_kv_heads) ? 1 : 0;
    if (pr.merge_op) bars += n_attn;
    if (M > pass::BLKM) bars += n_attn;
    cudaError_t e;
    if (M > 12) e = c->cfg.head_dim == 128 ? launch_pass_t<128, 2, 0>(c, pr) : launch_pass_t<64, 2, 0>(c, pr);
    else if (M > pass::BLKM) e = c->cfg.head_dim == 128 ? launch_pass_t<128, 2, 3>(c, pr) : launch_pass_t<64, 2, 3>(c, pr);
    else if (M > pass::BLKM / 2) e = c->cfg.head_dim == 128 ? launch_pass_t<128, 1, 0>(c, pr) : launch_pass_t<64, 1, 0>(c, pr);
    else e = c->cfg.head_dim == 128 ? launch_pass_t<128, 1, 1>(c, pr) : launch_pass_t<64, 1, 1>(c, pr);
    if (e == cudaSuccess) c->bar_total += (unsigned long long)bars * (unsigned long long)c->n_sms;
    c->launches++;
}

// After a pass kernel gave up: bring the barrier counter and the work counters back to their idle state.
void reset_mega_state(knnssd_ctx *c) {
    if (!c->mega_ok) return;
    cudaMemset(c->bar, 0, sizeof(unsigned long long));
    cudaMemset(c->gabort, 0, sizeof(int));
    cudaMemset(c->attn_cnt, 0, sizeof(int) * pass::MAXM * c->cfg.n_heads);
    cudaMemset(c->amax_cnt, 0, sizeof(int));
    c->bar_total = 0;
}

// One decoder pass over M rows whose token ids are tok_dev[0..M) at positions state.len + pos_off + m.
//   mask       nullptr = full model, else [2L] with 1 = skipped
//   head_row0  first row that gets logits and an arg-max (M = no head at all)
//   argmax_out device ints, entry (m - head_row0) receives row m's greedy token
//   want_hidden  also write RMSNorm_final(x) of all rows to c->hfinal
template <typename WT>
void run_pass_t(knnssd_ctx *c, int M, const int *tok_dev, int pos_off, const unsigned char *mask, int head_row0,
                int *argmax_out, bool want_hidden) {
    const knnssd_config &g = c->cfg;
    const int d = g.d_model, H = g.n_heads, Hkv = g.n_kv_heads, hd = g.head_dim, F = g.d_ff, V = g.vocab;
    const int nq = H * hd, nkv = Hkv * hd;
    cudaStream_t s = c->stream;
    embed_rope_kernel<WT><<<M, 256, 0, s>>>(reinterpret_cast<const WT *>(c->tok_embed), tok_dev, d, c->x, c->state, pos_off,
                                            c->inv_freq, hd / 2, c->rope_cs, g.vocab, c->err_word);
    c->launches++;
    const size_t layer_stride = (size_t)Hkv * g.max_seq * hd;
    for (int l = 0; l < g.n_layers; ++l) {
        const Layer &ly = c->layers[l];
        if (!mask || !mask[2 * l]) {
            LinearArgs a = make_args(ly.wq, nq, d, c->x, ly.attn_norm, g.rms_eps, c->qkv, EPI_STORE, M);
            a.W[1] = ly.wk; a.rows[1] = nkv; a.W[2] = ly.wv; a.rows[2] = nkv; a.units = nq + 2 * nkv;
            ctx_linear(c, a);
            WT *kc = reinterpret_cast<WT *>(c->kcache) + (size_t)l * layer_stride;
            WT *vc = reinterpret_cast<WT *>(c->vcache) + (size_t)l * layer_stride;
            rope_kv_kernel<WT><<<dim3(H + 2 * Hkv, M), hd / 2, 0, s>>>(c->qkv, H, Hkv, hd, c->rope_cs, kc, vc, g.max_seq,
                                                                      c->state, pos_off);
            const dim3 ag(H, M, c->n_splits);
            if (hd == 128) {
                attn_partial_kernel<WT, 128><<<ag, 128, 0, s>>>(c->qkv, H, Hkv, kc, vc, g.max_seq, c->state, pos_off,
                                                                 c->part_o, c->part_ml, c->n_splits);
                attn_merge_kernel<128><<<dim3(H, M), 128, 0, s>>>(c->part_o, c->part_ml, H, c->state, pos_off, c->n_splits,
                                                                   c->attn);
            } else {
                attn_partial_kernel<WT, 64><<<ag, 128, 0, s>>>(c->qkv, H, Hkv, kc, vc, g.max_seq, c->state, pos_off,
                                                                c->part_o, c->part_ml, c->n_splits);
                attn_merge_kernel<64><<<dim3(H, M), 64, 0, s>>>(c->part_o, c->part_ml, H, c->state, pos_off, c->n_splits,
                                                                 c->attn);
            }
            c->launches += 3;
            ctx_linear(c, make_args(ly.wo, d, nq, c->attn, nullptr, 0.f, c->x, EPI_ADD, M));
        }
        if (!mask || !mask[2 * l + 1]) {
            LinearArgs a = make_args(ly.w_gate, F, d, c->x, ly.mlp_norm, g.rms_eps, c->act, EPI_SWIGLU, M);
            a.W[1] = ly.w_up; a.rows[1] = F; a.units = F;
            ctx_linear(c, a);
            ctx_linear(c, make_args(ly.w_down, d, F, c->act, nullptr, 0.f, c->x, EPI_ADD, M));
        }
    }
    if (want_hidden) {
        rmsnorm_rows_kernel<<<M, 256, 0, s>>>(c->x, c->final_norm, d, g.rms_eps, c->hfinal);
        c->launches++;
    }
    if (head_row0 < M) {
        const int hm = M - head_row0;
        ctx_linear(c, make_args(c->lm_head, V, d, c->x + (size_t)head_row0 * d, c->final_norm, g.rms_eps,
                                c->logits + (size_t)head_row0 * V, EPI_STORE, hm));
        argmax_partial_kernel<<<dim3(kArgmaxBlocks, hm), 256, 0, s>>>(c->logits + (size_t)head_row0 * V, V, kArgmaxBlocks,
                                                                      c->amax_v, c->amax_i);
        argmax_final_kernel<<<hm, 32, 0, s>>>(c->amax_v, c->amax_i, kArgmaxBlocks, argmax_out, V, c->err_word);
        c->launches += 2;
    }
}

void run_pass(knnssd_ctx *c, int M, const int *tok_dev, int pos_off, const unsigned char *mask, int head_row0,
              int *argmax_out, bool want_hidden) {
    if (c->mega_ok && M <= pass::MAXM) { run_pass_mega(c, M, tok_dev, pos_off, mask, head_row0, argmax_out, want_hidden); return; }
    if (c->cfg.dtype) run_pass_t<bf16_t>(c, M, tok_dev, pos_off, mask, head_row0, argmax_out, want_hidden);
    else run_pass_t<float>(c, M, tok_dev, pos_off, mask, head_row0, argmax_out, want_hidden);
}

knnssd_status sync_check(knnssd_ctx *c, const char *what) {
    cudaError_t e = cudaStreamSynchronize(c->stream);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return fail(c, KNNSSD_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
    if (c->enqueue_failed) {
        c->enqueue_failed = false;
        c->prefilled = false;
        return fail(c, KNNSSD_ERR_CUDA, std::string(what) + ": a pass could not be enqueued (prefill again): " + c->err);
    }
    return KNNSSD_OK;
}

// What a non-zero device error word means.  Whatever it was, the pass that raised it did not finish: the session's
// cache and pending token are no longer trustworthy, so the caller has to prefill again.
knnssd_status fail_device_code(knnssd_ctx *c, const char *what, int code) {
    cudaMemset(c->err_word, 0, sizeof(int));
    reset_mega_state(c);
    c->prefilled = false;
    if (code == ERR_BAD_LOGITS)
        return fail(c, KNNSSD_ERR_DEGENERATE, std::string(what) + ": a row of logits holds no finite value (prefill again)");
    if (code == ERR_BAD_TOKEN)
        return fail(c, KNNSSD_ERR_INVALID_ARG, std::string(what) + ": a token id on the device was out of range (prefill again)");
    return fail(c, KNNSSD_ERR_TIMEOUT, std::string(what) + ": a device-side wait gave up (code " + std::to_string(code) +
                                       "); prefill again");
}

// Read the device error word (synchronises); reports it once and clears it.
knnssd_status check_stream_err(knnssd_ctx *c, const char *what) {
    int code = 0;
    if (cudaMemcpy(&code, c->err_word, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
        return fail(c, KNNSSD_ERR_CUDA, std::string(what) + ": cannot read the device error word");
    if (code) return fail_device_code(c, what, code);
    return KNNSSD_OK;
}

void free_all(knnssd_ctx *c) {
    void *ptrs[] = {c->kcache, c->vcache, c->x, c->qkv, c->attn, c->act, c->logits, c->hfinal, c->part_o, c->pooled,
                    c->anchor_inv_norm, c->cosines, c->amax_v, c->part_ml, c->rope_cs, c->pool_sum, c->inv_freq, c->chain,
                    c->target, c->prompt, c->out_tokens, c->accept_log, c->amax_i, c->flag, c->knn_out, c->state,
                    c->ops_full, c->ops_draft, c->bar, c->gabort, c->attn_cnt, c->amax_cnt, c->mpart_o, c->mamax_v, c->mpart_ml,
                    c->mamax_i, c->trace, c->xs_x, c->xs_attn, c->xs_act, c->ssp, c->pf_x, c->pf_qkv, c->pf_ad, c->pf_aq, c->pf_af, c->pf_cs, c->pf_rinv,
                    c->samp_p, c->samp_q, c->samp_res};
    for (void *p : ptrs)
        if (p) cudaFree(p);
    if (c->pinned) cudaFreeHost(c->pinned);
    if (c->ev0) cudaEventDestroy(c->ev0);
    if (c->ev1) cudaEventDestroy(c->ev1);
    if (c->ev2) cudaEventDestroy(c->ev2);
    for (cudaEvent_t e : c->lin_events) cudaEventDestroy(e);
}

struct DeviceGuard {
    int prev = 0;
    explicit DeviceGuard(int dev) { cudaGetDevice(&prev); if (prev != dev) cudaSetDevice(dev); else prev = -1; }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

float elapsed_ms(knnssd_ctx *c) {
    float ms = 0.f;
    cudaEventElapsedTime(&ms, c->ev0, c->ev1);
    return ms;
}

// The prompt pass on the tensor cores: rows [t0, t0 + T) of the prompt at a time, every linear map one contraction
// over all T rows.  Leaves K/V of all layers in the cache, the pooled numerator in pool_sum and the last row's greedy
// token in chain[0].  Returns false if a tensor map could not be made.
template <int HD>
bool prefill_tensor(knnssd_ctx *c, int n) {
    const knnssd_config &g = c->cfg;
    const int d = g.d_model, H = g.n_heads, Hkv = g.n_kv_heads, F = g.d_ff, V = g.vocab;
    const int nq = H * HD, nkv = Hkv * HD, ldq = nq + 2 * nkv, cap = c->pf_cap;
    cudaStream_t s = c->stream;
    int *err = c->err_word;
    const size_t layer_stride = (size_t)Hkv * g.max_seq * HD;
    bool ok = true;
    for (int t0 = 0; t0 < n && ok; t0 += cap) {
        const int T = n - t0 < cap ? n - t0 : cap;
        const bool last = t0 + T == n;
        prefill::embed_rows_kernel<<<T, 256, 0, s>>>(reinterpret_cast<const bf16_t *>(c->tok_embed), c->prompt + t0, d, c->pf_x);
        prefill::rope_table_kernel<<<T, HD / 2, 0, s>>>(c->inv_freq, t0, c->pf_cs);
        c->launches += 2;
        for (int l = 0; l < g.n_layers && ok; ++l) {
            const Layer &ly = c->layers[l];
            bf16_t *kc = reinterpret_cast<bf16_t *>(c->kcache) + (size_t)l * layer_stride;
            bf16_t *vc = reinterpret_cast<bf16_t *>(c->vcache) + (size_t)l * layer_stride;
            prefill::norm_split_kernel<<<T, 256, 0, s>>>(c->pf_x, d, ly.attn_norm, g.rms_eps, c->pf_ad, c->pf_ad + (size_t)cap * d, c->pf_rinv);
            bool heads_done = false;     // rotary embedding and K / V rows done by the q / k / v launch's epilogue
            if (nq % prefill::BOX_N == 0 && nkv % prefill::BOX_N == 0) {
                // q, k and v in one launch over the stacked units (their columns of the projection buffer are adjacent)
                const prefill::QkvFuse fuse{c->pf_cs, kc, vc, g.max_seq, t0, HD};
                ok = ok && prefill::launch_gemm(c->pf_map_d, cap, ly.wq, ly.wk, ldq, d, T, prefill::PF_STORE, c->pf_qkv, ldq, 0, nullptr,
                                                nullptr, 0, err, c->n_sms, s, ly.wv, nq, nkv, &fuse, &heads_done, c->pf_rinv);
            } else {
                ok = ok && prefill::launch_gemm(c->pf_map_d, cap, ly.wq, nullptr, nq, d, T, prefill::PF_STORE, c->pf_qkv, ldq, 0, nullptr,
                                                nullptr, 0, err, c->n_sms, s, nullptr, 0, 0, nullptr, nullptr, c->pf_rinv);
                ok = ok && prefill::launch_gemm(c->pf_map_d, cap, ly.wk, nullptr, nkv, d, T, prefill::PF_STORE, c->pf_qkv, ldq, nq, nullptr,
                                                nullptr, 0, err, c->n_sms, s, nullptr, 0, 0, nullptr, nullptr, c->pf_rinv);
                ok = ok && prefill::launch_gemm(c->pf_map_d, cap, ly.wv, nullptr, nkv, d, T, prefill::PF_STORE, c->pf_qkv, ldq, nq + nkv,
                                                nullptr, nullptr, 0, err, c->n_sms, s, nullptr, 0, 0, nullptr, nullptr, c->pf_rinv);
            }
            if (!heads_done) prefill::rope_kv_rows_kernel<<<T, 256, 0, s>>>(c->pf_qkv, H, Hkv, HD, c->pf_cs, kc, vc, g.max_seq, t0);
            prefill::attn_prompt_kernel<HD><<<dim3(H, (T + 63) / 64), 128, prefill::attn_smem_bytes<HD>(), s>>>(
                c->pf_qkv, H, Hkv, kc, vc, g.max_seq, t0, T, c->pf_aq, c->pf_aq + (size_t)cap * nq);
            ok = ok && prefill::launch_gemm(c->pf_map_q, cap, ly.wo, nullptr, d, nq, T, prefill::PF_ADD, c->pf_x, d, 0, nullptr, nullptr, 0,
                                            err, c->n_sms, s);
            prefill::norm_split_kernel<<<T, 256, 0, s>>>(c->pf_x, d, ly.mlp_norm, g.rms_eps, c->pf_ad, c->pf_ad + (size_t)cap * d, c->pf_rinv);
            ok = ok && prefill::launch_gemm(c->pf_map_d, cap, ly.w_gate, ly.w_up, F, d, T, prefill::PF_SWIGLU, nullptr, 0, 0, c->pf_af,
                                            c->pf_af + (size_t)cap * F, F, err, c->n_sms, s, nullptr, 0, 0, nullptr, nullptr, c->pf_rinv);
            ok = ok && prefill::launch_gemm(c->pf_map_f, cap, ly.w_down, nullptr, d, F, T, prefill::PF_ADD, c->pf_x, d, 0, nullptr, nullptr,
                                            0, err, c->n_sms, s);
            c->launches += ((nq % prefill::BOX_N == 0 && nkv % prefill::BOX_N == 0) ? 9 : 11) - (heads_done ? 1 : 0);
        }
        // pooled numerator: every row's final hidden state (mean pooling) or the last row's
        if (g.pool_mode == 0) {
            rmsnorm_rows_kernel<<<T, 256, 0, s>>>(c->pf_x, c->final_norm, d, g.rms_eps, c->pf_qkv);     // [T][d] scratch
            pool_accumulate_kernel<<<(d + 255) / 256, 256, 0, s>>>(c->pf_qkv, T, d, c->pool_sum, t0 == 0);
            c->launches += 2;
        } else if (last) {
            rmsnorm_rows_kernel<<<1, 256, 0, s>>>(c->pf_x + (size_t)(T - 1) * d, c->final_norm, d, g.rms_eps, c->hfinal);
            pool_accumulate_kernel<<<(d + 255) / 256, 256, 0, s>>>(c->hfinal, 1, d, c->pool_sum, 1);
            c->launches += 2;
        }
        if (last) {
            ctx_linear(c, make_args(c->lm_head, V, d, c->pf_x + (size_t)(T - 1) * d, c->final_norm, g.rms_eps, c->logits, EPI_STORE, 1));
            argmax_partial_kernel<<<dim3(kArgmaxBlocks, 1), 256, 0, s>>>(c->logits, V, kArgmaxBlocks, c->amax_v, c->amax_i);
            argmax_final_kernel<<<1, 32, 0, s>>>(c->amax_v, c->amax_i, kArgmaxBlocks, c->chain, V, c->err_word);
            c->launches += 2;
        }
    }
    return ok;
}

knnssd_status do_prefill(knnssd_ctx *c, const int *tokens_host, int n, float *pooled_dev, int *first_token) {
    const knnssd_config &g = c->cfg;
    if (!tokens_host || n < 1) return fail(c, KNNSSD_ERR_INVALID_ARG, "prefill: need at least one prompt token");
    if (n > g.max_seq - 1) return fail(c, KNNSSD_ERR_CAPACITY, "prefill: prompt does not fit in max_seq - 1");
    for (int i = 0; i < n; ++i)
        if (tokens_host[i] < 0 || tokens_host[i] >= g.vocab)
            return fail(c, KNNSSD_ERR_INVALID_ARG, "prefill: token id out of range");
    cudaStream_t s = c->stream;
    c->prefilled = false;
    CUDA_TRY(c, cudaMemcpyAsync(c->prompt, tokens_host, sizeof(int) * n, cudaMemcpyHostToDevice, s));
    set_state_kernel<<<1, 1, 0, s>>>(c->state, 0, 0);
    cudaEventRecord(c->ev0, s);
    const int d = g.d_model;
    const int chunk = c->mega_ok ? pass::MAXM : kMaxRows;   // rows per pass: what the faster path takes
    // prompts longer than one pass's rows go through the tensor-core prompt pass where the model is eligible for it
    const bool tensor_path = c->pf_ok && n > pass::MAXM;
    if (tensor_path) {
        const bool made = g.head_dim == 128 ? prefill_tensor<128>(c, n) : prefill_tensor<64>(c, n);
        if (!made) { cudaStreamSynchronize(s); return fail(c, KNNSSD_ERR_CUDA, "prefill: cannot encode a tensor map"); }
    }
    for (int t0 = 0; t0 < n && !tensor_path; t0 += chunk) {
        const int M = (n - t0 < chunk) ? n - t0 : chunk;
        const bool last = t0 + M == n;
        // mean pooling needs every row's final hidden state; last-token pooling only the last row's
        const bool hidden = g.pool_mode == 0 || last;
        run_pass(c, M, c->prompt + t0, t0, nullptr, last ? M - 1 : M, c->chain, hidden);
        if (g.pool_mode == 0) {
            pool_accumulate_kernel<<<(d + 255) / 256, 256, 0, s>>>(c->hfinal, M, d, c->pool_sum, t0 == 0);
        } else if (last) {
            pool_accumulate_kernel<<<(d + 255) / 256, 256, 0, s>>>(c->hfinal + (size_t)(M - 1) * d, 1, d, c->pool_sum, 1);
        }
    }
    pool_finish_kernel<<<(d + 255) / 256, 256, 0, s>>>(c->pool_sum, d, g.pool_mode == 0 ? 1.0 / (double)n : 1.0, c->pooled);
    emit_first_token_kernel<<<1, 1, 0, s>>>(c->chain, c->state, c->out_tokens, n);
    cudaEventRecord(c->ev1, s);
    if (pooled_dev) CUDA_TRY(c, cudaMemcpyAsync(pooled_dev, c->pooled, sizeof(float) * d, cudaMemcpyDeviceToDevice, s));
    CUDA_TRY(c, cudaMemcpyAsync(c->pinned, c->chain, sizeof(int), cudaMemcpyDeviceToHost, s));
    knnssd_status st = sync_check(c, "prefill");
    if (st == KNNSSD_OK) st = check_stream_err(c, "prefill");
    if (st != KNNSSD_OK) return st;
    c->len = n;
    c->pending = c->pinned[0];
    c->prefilled = true;
    c->stats = knnssd_stats{};
    c->stats.tokens = 1;
    c->stats.ms_prefill = elapsed_ms(c);
    if (first_token) *first_token = c->pending;
    return KNNSSD_OK;
}

knnssd_status do_select(knnssd_ctx *c, const float *query_dev, int *domain, int *anchor, float *cosine) {
    const knnssd_config &g = c->cfg;
    if (g.n_domains <= 0) return fail(c, KNNSSD_ERR_STATE, "select_skipset: the context has no anchors");
    if (!query_dev && !c->prefilled) return fail(c, KNNSSD_ERR_STATE, "select_skipset: no pooled vector (prefill first)");
    const int n = g.n_domains * g.anchors_per_domain;
    cudaStream_t s = c->stream;
    CUDA_TRY(c, cudaMemsetAsync(c->flag, 0, sizeof(int), s));
    cudaEventRecord(c->ev0, s);
    cosine_scores_kernel<<<(n + 7) / 8, 256, 0, s>>>(query_dev ? query_dev : c->pooled, c->anchors, c->anchor_inv_norm, n,
                                                     g.d_model, c->cosines, c->flag);
    cosine_argmax_kernel<<<1, 256, 0, s>>>(c->cosines, n, c->knn_out);
    cudaEventRecord(c->ev1, s);
    CUDA_TRY(c, cudaMemcpyAsync(c->pinned, c->knn_out, 2 * sizeof(int), cudaMemcpyDeviceToHost, s));
    CUDA_TRY(c, cudaMemcpyAsync(c->pinned + 2, c->flag, sizeof(int), cudaMemcpyDeviceToHost, s));
    knnssd_status st = sync_check(c, "select_skipset");
    if (st != KNNSSD_OK) return st;
    if (c->pinned[2]) return fail(c, KNNSSD_ERR_DEGENERATE, "select_skipset: query has zero or non-finite norm");
    const int best = c->pinned[0];
    float cs;
    std::memcpy(&cs, &c->pinned[1], sizeof(float));
    const int dom = best / g.anchors_per_domain;
    c->active_mask.assign(c->domain_masks.begin() + (size_t)dom * 2 * g.n_layers,
                          c->domain_masks.begin() + (size_t)(dom + 1) * 2 * g.n_layers);
    c->has_mask = true;
    c->stats.ms_select = elapsed_ms(c);
    if (domain) *domain = dom;
    if (anchor) *anchor = best % g.anchors_per_domain;
    if (cosine) *cosine = cs;
    return KNNSSD_OK;
}

// Enqueue k draft steps: step j reads chain[j] at position len + j and writes chain[j + 1].
void enqueue_draft(knnssd_ctx *c, int k) {
    for (int j = 0; j < k; ++j) run_pass(c, 1, c->chain + j, j, c->active_mask.data(), 0, c->chain + j + 1, false);
}

// Enqueue the verification pass over chain[0..k] and the accept/rollback step.
void enqueue_verify(knnssd_ctx *c, int k, bool want_hidden, int round_idx) {
    run_pass(c, k + 1, c->chain, 0, nullptr, 0, c->target, want_hidden);
    accept_kernel<<<1, 32, 0, c->stream>>>(c->chain, c->target, k, c->state, c->out_tokens, c->cfg.max_seq, c->accept_log,
                                           round_idx);
    c->launches++;
}

}  // namespace

extern "C" {

knnssd_status knnssd_init(const knnssd_config *cfg, const knnssd_weights *w, const float *anchors_dev,
                          const unsigned char *skip_masks_host, void *cuda_stream, knnssd_ctx **out) {
    if (!cfg || !w || !out) return KNNSSD_ERR_INVALID_ARG;
    *out = nullptr;
    const knnssd_config &g = *cfg;
    if (g.n_layers < 1 || g.d_model < 8 || g.n_heads < 1 || g.n_kv_heads < 1 || g.d_ff < 8 || g.vocab < 2 ||
        g.max_seq < 2 || g.max_draft < 1 || g.n_domains < 0 || (g.n_domains > 0 && g.anchors_per_domain < 1) ||
        (g.dtype != 0 && g.dtype != 1) || (g.pool_mode != 0 && g.pool_mode != 1) || !(g.rms_eps > 0.f) ||
        !(g.rope_theta > 0.f))
        return KNNSSD_ERR_INVALID_ARG;
    if ((g.head_dim != 64 && g.head_dim != 128) || g.n_heads % g.n_kv_heads != 0 || g.d_model % 8 != 0 ||
        g.d_ff % 8 != 0 || g.max_draft > kMaxRows - 1)
        return KNNSSD_ERR_SHAPE;
    if ((g.n_domains > 0) != (anchors_dev != nullptr) || (g.n_domains > 0) != (skip_masks_host != nullptr))
        return KNNSSD_ERR_INVALID_ARG;
    if (!w->tok_embed || !w->final_norm || !w->lm_head || !w->attn_norm || !w->wq || !w->wk || !w->wv || !w->wo ||
        !w->mlp_norm || !w->w_gate || !w->w_up || !w->w_down)
        return KNNSSD_ERR_INVALID_ARG;
    knnssd_ctx *c = new (std::nothrow) knnssd_ctx();
    if (!c) return KNNSSD_ERR_CUDA;
    c->cfg = g;
    c->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    c->wbytes = g.dtype ? 2 : 4;
    c->tok_embed = w->tok_embed; c->final_norm = w->final_norm; c->lm_head = w->lm_head;
    for (int l = 0; l < g.n_layers; ++l) {
        Layer ly{w->attn_norm[l], w->mlp_norm[l], w->wq[l], w->wk[l], w->wv[l], w->wo[l], w->w_gate[l], w->w_up[l],
                 w->w_down[l]};
        const void *all[] = {ly.attn_norm, ly.mlp_norm, ly.wq, ly.wk, ly.wv, ly.wo, ly.w_gate, ly.w_up, ly.w_down};
        for (const void *p : all)
            if (!p || (reinterpret_cast<uintptr_t>(p) & 15u)) { delete c; return KNNSSD_ERR_INVALID_ARG; }
        c->layers.push_back(ly);
    }
    if ((reinterpret_cast<uintptr_t>(w->tok_embed) & 15u) || (reinterpret_cast<uintptr_t>(w->lm_head) & 15u) ||
        (reinterpret_cast<uintptr_t>(w->final_norm) & 15u)) { delete c; return KNNSSD_ERR_INVALID_ARG; }
    c->anchors = anchors_dev;
    const int L2 = 2 * g.n_layers;
    if (g.n_domains > 0) {
        c->domain_masks.assign(skip_masks_host, skip_masks_host + (size_t)g.n_domains * L2);
        for (unsigned char b : c->domain_masks)
            if (b > 1) { delete c; return KNNSSD_ERR_INVALID_ARG; }
    }
    auto bail = [&](knnssd_status s) { free_all(c); delete c; return s; };
    if (cudaGetDevice(&c->device) != cudaSuccess) return bail(KNNSSD_ERR_CUDA);
    cudaDeviceGetAttribute(&c->n_sms, cudaDevAttrMultiProcessorCount, c->device);
    c->err_word = stream_err_ptr();
    if (!c->err_word) return bail(KNNSSD_ERR_CUDA);
    const int d = g.d_model, hd = g.head_dim, nq = g.n_heads * hd, nkv = g.n_kv_heads * hd;
    const size_t cache_elems = (size_t)g.n_layers * g.n_kv_heads * g.max_seq * hd;
    c->n_splits = (g.max_seq + ATT_CHUNK - 1) / ATT_CHUNK;
    const int na = g.n_domains * g.anchors_per_domain;
    bool ok = true;
    ok &= cudaMalloc(&c->kcache, cache_elems * c->wbytes) == cudaSuccess;
    ok &= cudaMalloc(&c->vcache, cache_elems * c->wbytes) == cudaSuccess;
    ok &= dev_alloc(&c->x, (size_t)kMaxRows * d) == cudaSuccess;
    ok &= dev_alloc(&c->qkv, (size_t)kMaxRows * (nq + 2 * nkv)) == cudaSuccess;
    ok &= dev_alloc(&c->attn, (size_t)kMaxRows * nq) == cudaSuccess;
    ok &= dev_alloc(&c->act, (size_t)kMaxRows * g.d_ff) == cudaSuccess;
    ok &= dev_alloc(&c->logits, (size_t)kMaxRows * g.vocab) == cudaSuccess;
    ok &= dev_alloc(&c->hfinal, (size_t)kMaxRows * d) == cudaSuccess;
    ok &= dev_alloc(&c->part_o, (size_t)kMaxRows * g.n_heads * c->n_splits * hd) == cudaSuccess;
    ok &= dev_alloc(&c->part_ml, (size_t)kMaxRows * g.n_heads * c->n_splits) == cudaSuccess;
    ok &= dev_alloc(&c->rope_cs, (size_t)(c->n_sms > 1 ? c->n_sms : 1) * kMaxRows * (hd / 2)) == cudaSuccess;   // one copy per CTA of the pass kernel
    ok &= dev_alloc(&c->pooled, (size_t)d) == cudaSuccess;
    ok &= dev_alloc(&c->pool_sum, (size_t)d) == cudaSuccess;
    ok &= dev_alloc(&c->inv_freq, (size_t)hd / 2) == cudaSuccess;
    ok &= dev_alloc(&c->amax_v, (size_t)kMaxRows * kArgmaxBlocks) == cudaSuccess;
    ok &= dev_alloc(&c->amax_i, (size_t)kMaxRows * kArgmaxBlocks) == cudaSuccess;
    ok &= dev_alloc(&c->chain, (size_t)kMaxRows + 1) == cudaSuccess;
    ok &= dev_alloc(&c->target, (size_t)kMaxRows) == cudaSuccess;
    ok &= dev_alloc(&c->prompt, (size_t)g.max_seq) == cudaSuccess;
    ok &= dev_alloc(&c->out_tokens, (size_t)g.max_seq) == cudaSuccess;
    ok &= dev_alloc(&c->accept_log, (size_t)g.max_seq) == cudaSuccess;
    ok &= dev_alloc(&c->flag, 1) == cudaSuccess;
    ok &= dev_alloc(&c->knn_out, 2) == cudaSuccess;
    ok &= dev_alloc(&c->state, 1) == cudaSuccess;
    ok &= dev_alloc(&c->cosines, (size_t)(na > 0 ? na : 1)) == cudaSuccess;
    ok &= dev_alloc(&c->anchor_inv_norm, (size_t)(na > 0 ? na : 1)) == cudaSuccess;
    ok &= cudaMallocHost(reinterpret_cast<void **>(&c->pinned), 64 * sizeof(int)) == cudaSuccess;
    ok &= cudaEventCreate(&c->ev0) == cudaSuccess && cudaEventCreate(&c->ev1) == cudaSuccess &&
          cudaEventCreate(&c->ev2) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return bail(KNNSSD_ERR_CUDA); }
    // K/V start at zero so that no kernel ever reads uninitialised memory
    cudaMemsetAsync(c->kcache, 0, cache_elems * c->wbytes, c->stream);
    cudaMemsetAsync(c->vcache, 0, cache_elems * c->wbytes, c->stream);
    std::vector<double> inv_freq(hd / 2);
    for (int i = 0; i < hd / 2; ++i) inv_freq[i] = std::pow((double)g.rope_theta, -2.0 * (double)i / (double)hd);
    cudaMemcpyAsync(c->inv_freq, inv_freq.data(), sizeof(double) * inv_freq.size(), cudaMemcpyHostToDevice, c->stream);
    set_state_kernel<<<1, 1, 0, c->stream>>>(c->state, 0, 0);
    cudaMemsetAsync(c->flag, 0, sizeof(int), c->stream);
    // token buffers start at a valid id, so that a pass that ends early never leaves garbage ids behind
    cudaMemsetAsync(c->chain, 0, sizeof(int) * (kMaxRows + 1), c->stream);
    cudaMemsetAsync(c->target, 0, sizeof(int) * kMaxRows, c->stream);
    if (na > 0) anchor_inv_norm_kernel<<<(na + 7) / 8, 256, 0, c->stream>>>(c->anchors, na, d, c->anchor_inv_norm, c->flag);
    cudaMemcpyAsync(c->pinned, c->flag, sizeof(int), cudaMemcpyDeviceToHost, c->stream);
    if (sync_check(c, "init") != KNNSSD_OK) return bail(KNNSSD_ERR_CUDA);
    if (c->pinned[0]) return bail(KNNSSD_ERR_DEGENERATE);
    // the persistent pass kernel serves bf16 models whose linear maps all have inputs that are multiples of 128
    int coop = 0;
    cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device);
    if (g.dtype == 1 && coop && d % 128 == 0 && nq % 128 == 0 && g.d_ff % 128 == 0 && d >= 256 && nq >= 256 && g.d_ff >= 256 &&
        g.max_seq <= 64 * pass::SEGP) {            // the attention merge keeps at most 64 segment statistics per warp
        const int n_seg_max = (g.max_seq + pass::SEGP - 1) / pass::SEGP;
        const int n_ops_cap = 7 * g.n_layers + 8;
        bool ok2 = true;
        ok2 &= dev_alloc(&c->ops_full, (size_t)n_ops_cap) == cudaSuccess;
        ok2 &= dev_alloc(&c->ops_draft, (size_t)n_ops_cap) == cudaSuccess;
        ok2 &= dev_alloc(&c->bar, 1) == cudaSuccess;
        ok2 &= dev_alloc(&c->gabort, 1) == cudaSuccess;
        ok2 &= dev_alloc(&c->attn_cnt, (size_t)pass::MAXM * g.n_heads) == cudaSuccess;
        ok2 &= dev_alloc(&c->amax_cnt, 1) == cudaSuccess;
        ok2 &= dev_alloc(&c->mpart_o, (size_t)pass::MAXM * g.n_heads * n_seg_max * hd) == cudaSuccess;
        ok2 &= dev_alloc(&c->mpart_ml, (size_t)pass::MAXM * g.n_heads * n_seg_max) == cudaSuccess;
        ok2 &= dev_alloc(&c->mamax_v, (size_t)pass::MAXM * c->n_sms) == cudaSuccess;
        ok2 &= dev_alloc(&c->mamax_i, (size_t)pass::MAXM * c->n_sms) == cudaSuccess;
        ok2 &= dev_alloc(&c->trace, (size_t)2 * n_ops_cap) == cudaSuccess;
        ok2 &= dev_alloc(&c->xs_x, (size_t)pass::MAXM * (d / 128) * stream::SLOT_WORDS) == cudaSuccess;
        ok2 &= dev_alloc(&c->xs_attn, (size_t)pass::MAXM * (nq / 128) * stream::SLOT_WORDS) == cudaSuccess;
        ok2 &= dev_alloc(&c->xs_act, (size_t)pass::MAXM * (g.d_ff / 128) * stream::SLOT_WORDS) == cudaSuccess;
        ok2 &= dev_alloc(&c->ssp, (size_t)pass::MAXM * c->n_sms) == cudaSuccess;
        if (!ok2) { cudaGetLastError(); return bail(KNNSSD_ERR_CUDA); }
        // tensor-core prompt pass: needs the driver's tensor-map encoder; without it prompts go through the pass kernel
        if (prefill::encode_tiled_fn() && prefill::gemm_attrs_once()) {
            const int cap_seq = (g.max_seq + prefill::BM - 1) / prefill::BM * prefill::BM;
            c->pf_cap = cap_seq < 1024 ? cap_seq : 1024;
            const size_t cap = (size_t)c->pf_cap;
            bool ok3 = true;
            ok3 &= dev_alloc(&c->pf_x, cap * d) == cudaSuccess;
            ok3 &= dev_alloc(&c->pf_qkv, cap * (nq + 2 * nkv)) == cudaSuccess;
            ok3 &= dev_alloc(&c->pf_cs, cap * (hd / 2)) == cudaSuccess;
            ok3 &= dev_alloc(&c->pf_rinv, cap) == cudaSuccess;
            ok3 &= dev_alloc(&c->pf_ad, 2 * cap * d) == cudaSuccess;
            ok3 &= dev_alloc(&c->pf_aq, 2 * cap * nq) == cudaSuccess;
            ok3 &= dev_alloc(&c->pf_af, 2 * cap * g.d_ff) == cudaSuccess;
            if (!ok3) { cudaGetLastError(); return bail(KNNSSD_ERR_CUDA); }
            cudaMemsetAsync(c->pf_ad, 0, 2 * cap * d * sizeof(bf16_t), c->stream);
            cudaMemsetAsync(c->pf_aq, 0, 2 * cap * nq * sizeof(bf16_t), c->stream);
            cudaMemsetAsync(c->pf_af, 0, 2 * cap * g.d_ff * sizeof(bf16_t), c->stream);
            c->pf_ok = prefill::make_map(&c->pf_map_d, c->pf_ad, 2 * cap, (size_t)d, prefill::BM) &&
                       prefill::make_map(&c->pf_map_q, c->pf_aq, 2 * cap, (size_t)nq, prefill::BM) &&
                       prefill::make_map(&c->pf_map_f, c->pf_af, 2 * cap, (size_t)g.d_ff, prefill::BM);
        }
        pass::Model &md = c->model;
        md.tok_embed = reinterpret_cast<const bf16_t *>(c->tok_embed); md.final_norm = c->final_norm; md.rms_eps = g.rms_eps;
        md.d_model = d; md.H = g.n_heads; md.Hkv = g.n_kv_heads; md.hd = hd; md.vocab = g.vocab; md.max_seq = g.max_seq;
        md.n_seg_max = n_seg_max; md.inv_freq = c->inv_freq;
        md.x = c->x; md.qkv = c->qkv; md.attn = c->attn; md.logits = c->logits; md.hfinal = c->hfinal; md.rope_cs = c->rope_cs;
        md.part_o = c->mpart_o; md.part_ml = c->mpart_ml; md.attn_cnt = c->attn_cnt; md.amax_v = c->mamax_v; md.amax_i = c->mamax_i;
        md.amax_cnt = c->amax_cnt; md.state = c->state; md.bar = c->bar; md.gabort = c->gabort; md.err = c->err_word;
        c->mega_ok = true;
        reset_mega_state(c);
        const std::vector<pass::Op> ops = build_ops(c, nullptr, &c->bar_full, &c->attn_full);
        c->n_ops_full = (int)ops.size();
        if (upload_ops(c, ops, c->ops_full) != KNNSSD_OK) return bail(KNNSSD_ERR_CUDA);
    }
    *out = c;
    return KNNSSD_OK;
}

void knnssd_destroy(knnssd_ctx *c) {
    if (!c) return;
    DeviceGuard dg(c->device);
    cudaStreamSynchronize(c->stream);
    free_all(c);
    delete c;
}

knnssd_status knnssd_prefill(knnssd_ctx *c, const int *tokens_host, int n_tokens, float *pooled_dev_or_null,
                             int *first_token_or_null) {
    if (!c) return KNNSSD_ERR_INVALID_ARG;
    DeviceGuard dg(c->device);
    return do_prefill(c, tokens_host, n_tokens, pooled_dev_or_null, first_token_or_null);
}

knnssd_status knnssd_select_skipset(knnssd_ctx *c, const float *query_dev_or_null, int *domain, int *anchor,
                                    float *cosine) {
    if (!c) return KNNSSD_ERR_INVALID_ARG;
    DeviceGuard dg(c->device);
    return do_select(c, query_dev_or_null, domain, anchor, cosine);
}

knnssd_status knnssd_set_skipmask(knnssd_ctx *c, const unsigned char *mask_host) {
    if (!c) return KNNSSD_ERR_INVALID_ARG;
    if (!mask_host) return fail(c, KNNSSD_ERR_INVALID_ARG, "set_skipmask: NULL mask");
    const int n = 2 * c->cfg.n_layers;
    for (int j = 0; j < n; ++j)
        if (mask_host[j] > 1) return fail(c, KNNSSD_ERR_INVALID_ARG, "set_skipmask: entries must be 0 or 1");
    c->active_mask.assign(mask_host, mask_host + n);
    c->has_mask = true;
    return KNNSSD_OK;
}

knnssd_status knnssd_draft(knnssd_ctx *c, int k, int *draft_tokens_host, float *logits_dev_or_null) {
    if (!c) return KNNSSD_ERR_INVALID_ARG;
    DeviceGuard dg(c->device);
    if (!draft_tokens_host || k < 1 || k > c->cfg.max_draft) return fail(c, KNNSSD_ERR_INVALID_ARG, "draft: bad k or NULL output");
    if (!c->prefilled) return fail(c, KNNSSD_ERR_STATE, "draft: prefill first");
    if (!c->has_mask) return fail(c, KNNSSD_ERR_STATE, "draft: no active skip mask (select_skipset or set_skipmask first)");
    if (c->len + k + 1 > c->cfg.max_seq) return fail(c, KNNSSD_ERR_CAPACITY, "draft: len + k + 1 exceeds max_seq");
    cudaStream_t s = c->stream;
    cudaEventRecord(c->ev0, s);
    for (int j = 0; j < k; ++j) {
        run_pass(c, 1, c->chain + j, j, c->active_mask.data(), 0, c->chain + j + 1, false);
        if (logits_dev_or_null)
            CUDA_TRY(c, cudaMemcpyAsync(logits_dev_or_null + (size_t)j * c->cfg.vocab, c->logits, sizeof(float) * c->cfg.vocab,
                                        cudaMemcpyDeviceToDevice, s));
    }
    cudaEventRecord(c->ev1, s);
    CUDA_TRY(c, cudaMemcpyAsync(c->pinned, c->chain + 1, sizeof(int) * k, cudaMemcpyDeviceToHost, s));
    knnssd_status st = sync_check(c, "draft");
    if (st == KNNSSD_OK) st = check_stream_err(c, "draft");
    if (st != KNNSSD_OK) return st;
    for (int j = 0; j < k; ++j) draft_tokens_host[j] = c->pinned[j];
    c->stats.ms_draft += elapsed_ms(c);
    return KNNSSD_OK;
}

knnssd_status knnssd_verify(knnssd_ctx *c, const int *draft_tokens_host, int k, int *n_accepted, int *next_token,
                            float *logits_dev_or_null, float *hidden_dev_or_null) {
    if (!c) return KNNSSD_ERR_INVALID_ARG;
    DeviceGuard dg(c->device);
    const knnssd_config &g = c->cfg;
    if (k < 0 || k > g.max_draft || (k > 0 && !draft_tokens_host)) return fail(c, KNNSSD_ERR_INVALID_ARG, "verify: bad k or NULL drafts");
    if (!c->prefilled) return fail(c, KNNSSD_ERR_STATE, "verify: prefill first");
    if (c->len + k + 1 > g.max_seq) return fail(c, KNNSSD_ERR_CAPACITY, "verify: len + k + 1 exceeds max_seq");
    for (int j = 0; j < k; ++j)
        if (draft_tokens_host[j] < 0 || draft_tokens_host[j] >= g.vocab)
            return fail(c, KNNSSD_ERR_INVALID_ARG, "verify: draft token id out of range");
    cudaStream_t s = c->stream;
    if (k > 0) CUDA_TRY(c, cudaMemcpyAsync(c->chain + 1, draft_tokens_host, sizeof(int) * k, cudaMemcpyHostToDevice, s));
    cudaEventRecord(c->ev0, s);
    enqueue_verify(c, k, hidden_dev_or_null != nullptr, c->stats.rounds % g.max_seq);
    cudaEventRecord(c->ev1, s);
    if (logits_dev_or_null)
        CUDA_TRY(c, cudaMemcpyAsync(logits_dev_or_null, c->logits, sizeof(float) * (size_t)(k + 1) * g.vocab,
                                    cudaMemcpyDeviceToDevice, s));
    if (hidden_dev_or_null)
        CUDA_TRY(c, cudaMemcpyAsync(hidden_dev_or_null, c->hfinal, sizeof(float) * (size_t)(k + 1) * g.d_model,
                                    cudaMemcpyDeviceToDevice, s));
    CUDA_TRY(c, cudaMemcpyAsync(c->pinned, c->state, sizeof(DeviceState), cudaMemcpyDeviceToHost, s));
    knnssd_status st = sync_check(c, "verify");
    if (st == KNNSSD_OK) st = check_stream_err(c, "verify");
    if (st != KNNSSD_OK) return st;
    const DeviceState *hs = reinterpret_cast<const DeviceState *>(c->pinned);
    c->len = hs->len;
    c->pending = hs->last_next;
    c->stats.rounds += 1;
    c->stats.drafted += k;
    c->stats.accepted += hs->last_accept;
    c->stats.tokens += hs->last_accept + 1;
    c->stats.ms_verify += elapsed_ms(c);
    if (n_accepted) *n_accepted = hs->last_accept;
    if (next_token) *next_token = hs->last_next;
    return KNNSSD_OK;
}

static knnssd_status do_decode(knnssd_ctx *c, int max_new, int k, int use_selection, int *out_tokens_host, int *n_out,
                               int *accepts_host_or_null, int *domain_or_null, knnssd_stats *stats_or_null) {
    const knnssd_config &g = c->cfg;
    if (!out_tokens_host || !n_out || max_new < 1 || k < 0 || k > g.max_draft)
        return fail(c, KNNSSD_ERR_INVALID_ARG, "decode: bad arguments");
    if (!c->prefilled) return fail(c, KNNSSD_ERR_STATE, "decode: prefill first");
    if (c->len + max_new + 1 > g.max_seq) return fail(c, KNNSSD_ERR_CAPACITY, "decode: length + max_new + 1 exceeds max_seq");
    const bool select = use_selection && g.n_domains > 0;
    if (!select && !c->has_mask) return fail(c, KNNSSD_ERR_STATE, "decode: no active skip mask and no selection");
    knnssd_status st;
    int domain = -1;
    if (select) {
        st = do_select(c, nullptr, &domain, nullptr, nullptr);
        if (st != KNNSSD_OK) return st;
    }
    cudaStream_t s = c->stream;
    // the pending token is the first token of this call's output
    emit_first_token_kernel<<<1, 1, 0, s>>>(c->chain, c->state, c->out_tokens, c->len);
    c->launches++;
    int produced = 1, round = 0;
    c->stats.rounds = c->stats.drafted = c->stats.accepted = 0;
    c->stats.ms_draft = c->stats.ms_verify = 0.f;
    while (produced < max_new) {
        const int remaining = max_new - produced;
        const int keff = k < remaining - 1 ? k : remaining - 1;
        cudaEventRecord(c->ev0, s);
        enqueue_draft(c, keff);
        cudaEventRecord(c->ev1, s);
        enqueue_verify(c, keff, false, round);
        cudaEventRecord(c->ev2, s);
        CUDA_TRY(c, cudaMemcpyAsync(c->pinned, c->state, sizeof(DeviceState), cudaMemcpyDeviceToHost, s));
        CUDA_TRY(c, cudaMemcpyAsync(c->pinned + 8, c->err_word, sizeof(int), cudaMemcpyDeviceToHost, s));
        st = sync_check(c, "decode");
        if (st != KNNSSD_OK) return st;
        // a pass that gave up (or met a bad id / non-finite logits) must not be committed to the session
        if (c->pinned[8]) return fail_device_code(c, "decode", c->pinned[8]);
        const DeviceState *hs = reinterpret_cast<const DeviceState *>(c->pinned);
        float ms = 0.f;
        cudaEventElapsedTime(&ms, c->ev0, c->ev1);
        c->stats.ms_draft += ms;
        cudaEventElapsedTime(&ms, c->ev1, c->ev2);
        c->stats.ms_verify += ms;
        produced = hs->produced;
        c->len = hs->len;
        c->pending = hs->last_next;
        c->stats.rounds += 1;
        c->stats.drafted += keff;
        c->stats.accepted += hs->last_accept;
        ++round;
    }
    c->stats.tokens = produced;
    CUDA_TRY(c, cudaMemcpyAsync(out_tokens_host, c->out_tokens, sizeof(int) * max_new, cudaMemcpyDeviceToHost, s));
    if (accepts_host_or_null && round > 0)
        CUDA_TRY(c, cudaMemcpyAsync(accepts_host_or_null, c->accept_log, sizeof(int) * round, cudaMemcpyDeviceToHost, s));
    st = sync_check(c, "decode");
    if (st == KNNSSD_OK) st = check_stream_err(c, "decode");
    if (st != KNNSSD_OK) return st;
    *n_out = max_new;
    if (domain_or_null) *domain_or_null = domain;
    if (stats_or_null) *stats_or_null = c->stats;
    return KNNSSD_OK;
}

knnssd_status knnssd_decode(knnssd_ctx *c, int max_new, int k, int use_selection, int *out_tokens_host, int *n_out,
                            int *accepts_host_or_null, int *domain_or_null, knnssd_stats *stats_or_null) {
    if (!c) return KNNSSD_ERR_INVALID_ARG;
    DeviceGuard dg(c->device);
    return do_decode(c, max_new, k, use_selection, out_tokens_host, n_out, accepts_host_or_null, domain_or_null,
                     stats_or_null);
}

knnssd_status knnssd_decode_sampled(knnssd_ctx *c, int max_new, int k, float temperature, float top_p, const float *uniforms_host,
                                    int n_uniforms, int *out_tokens_host, int *n_out, int *accepts_host_or_null,
                                    knnssd_stats *stats_or_null) {
    if (!c) return KNNSSD_ERR_INVALID_ARG;
    DeviceGuard dg(c->device);
    const knnssd_config &g = c->cfg;
    const int stride = 2 * k + 1;
    if (!out_tokens_host || !n_out || !uniforms_host || max_new < 1 || k < 0 || k > g.max_draft || !(temperature > 0.f) ||
        !(top_p > 0.f) || !std::isfinite(temperature) || !std::isfinite(top_p) || (long long)n_uniforms < (long long)(max_new - 1) * stride)
        return fail(c, KNNSSD_ERR_INVALID_ARG, "decode_sampled: bad arguments (need (max_new - 1) * (2k + 1) uniforms)");
    for (int i = 0; i < (max_new - 1) * stride; ++i)
        if (!(uniforms_host[i] >= 0.f) || !(uniforms_host[i] < 1.f))
            return fail(c, KNNSSD_ERR_INVALID_ARG, "decode_sampled: uniforms must lie in [0, 1)");
    if (!c->prefilled) return fail(c, KNNSSD_ERR_STATE, "decode_sampled: prefill first");
    if (!c->has_mask) return fail(c, KNNSSD_ERR_STATE, "decode_sampled: no active skip mask");
    if (c->len + max_new + 1 > g.max_seq) return fail(c, KNNSSD_ERR_CAPACITY, "decode_sampled: length + max_new + 1 exceeds max_seq");
    const size_t V = (size_t)g.vocab;
    if (!c->samp_p) {
        if (dev_alloc(&c->samp_p, (size_t)kMaxRows * V) != cudaSuccess || dev_alloc(&c->samp_q, (size_t)kMaxRows * V) != cudaSuccess ||
            dev_alloc(&c->samp_res, 2) != cudaSuccess) {
            cudaGetLastError();
            return fail(c, KNNSSD_ERR_CUDA, "decode_sampled: cannot allocate the distribution buffers");
        }
    }
    cudaStream_t s = c->stream;
    float *u_dev = nullptr;
    const size_t n_u = (size_t)(max_new > 1 ? (max_new - 1) * stride : 1);
    if (dev_alloc(&u_dev, n_u) != cudaSuccess) { cudaGetLastError(); return fail(c, KNNSSD_ERR_CUDA, "decode_sampled: cannot allocate the uniforms"); }
    knnssd_status st = KNNSSD_OK;
    auto finish = [&](knnssd_status r) { cudaStreamSynchronize(s); cudaFree(u_dev); return r; };
    if (max_new > 1 && cudaMemcpyAsync(u_dev, uniforms_host, sizeof(float) * n_u, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return finish(fail(c, KNNSSD_ERR_CUDA, "decode_sampled: cannot copy the uniforms"));
    emit_first_token_kernel<<<1, 1, 0, s>>>(c->chain, c->state, c->out_tokens, c->len);
    c->launches++;
    int produced = 1, round = 0;
    c->stats.rounds = c->stats.drafted = c->stats.accepted = 0;
    c->stats.ms_draft = c->stats.ms_verify = 0.f;
    const float inv_t = 1.0f / temperature;
    while (produced < max_new) {
        const int remaining = max_new - produced;
        const int keff = k < remaining - 1 ? k : remaining - 1;
        const float *u = u_dev + (size_t)round * stride;
        cudaEventRecord(c->ev0, s);
        for (int j = 0; j < keff; ++j) {
            // draft step j: the draft model's logits of the row, filtered into q_j, the draft drawn from it
            run_pass(c, 1, c->chain + j, j, c->active_mask.data(), 0, c->target, false);
            sampling::filtered_probs_kernel<<<1, sampling::NT, 0, s>>>(c->logits, g.vocab, inv_t, top_p, c->samp_q + (size_t)j * V);
            sampling::sample_kernel<<<1, sampling::NT, 0, s>>>(c->samp_q + (size_t)j * V, g.vocab, u + j, 0.f, c->chain + j + 1);
            c->launches += 2;
        }
        cudaEventRecord(c->ev1, s);
        run_pass(c, keff + 1, c->chain, 0, nullptr, 0, c->target, false);
        sampling::filtered_probs_kernel<<<keff + 1, sampling::NT, 0, s>>>(c->logits, g.vocab, inv_t, top_p, c->samp_p);
        sampling::spec_accept_kernel<<<1, sampling::NT, 0, s>>>(c->samp_p, c->samp_q, c->chain + 1, keff, g.vocab, u + k, u + 2 * k, 0.f,
                                                                c->samp_res);
        sampling::commit_sampled_kernel<<<1, 32, 0, s>>>(c->chain, c->samp_res, c->state, c->out_tokens, g.max_seq, c->accept_log, round);
        c->launches += 3;
        cudaEventRecord(c->ev2, s);
        if (cudaMemcpyAsync(c->pinned, c->state, sizeof(DeviceState), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
            cudaMemcpyAsync(c->pinned + 8, c->err_word, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess)
            return finish(fail(c, KNNSSD_ERR_CUDA, "decode_sampled: read-back failed"));
        st = sync_check(c, "decode_sampled");
        if (st != KNNSSD_OK) return finish(st);
        if (c->pinned[8]) return finish(fail_device_code(c, "decode_sampled", c->pinned[8]));
        const DeviceState *hs = reinterpret_cast<const DeviceState *>(c->pinned);
        float ms = 0.f;
        cudaEventElapsedTime(&ms, c->ev0, c->ev1);
        c->stats.ms_draft += ms;
        cudaEventElapsedTime(&ms, c->ev1, c->ev2);
        c->stats.ms_verify += ms;
        produced = hs->produced;
        c->len = hs->len;
        c->pending = hs->last_next;
        c->stats.rounds += 1;
        c->stats.drafted += keff;
        c->stats.accepted += hs->last_accept;
        ++round;
    }
    c->stats.tokens = produced;
    if (cudaMemcpyAsync(out_tokens_host, c->out_tokens, sizeof(int) * max_new, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return finish(fail(c, KNNSSD_ERR_CUDA, "decode_sampled: read-back failed"));
    if (accepts_host_or_null && round > 0 &&
        cudaMemcpyAsync(accepts_host_or_null, c->accept_log, sizeof(int) * round, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return finish(fail(c, KNNSSD_ERR_CUDA, "decode_sampled: read-back failed"));
    st = sync_check(c, "decode_sampled");
    if (st == KNNSSD_OK) st = check_stream_err(c, "decode_sampled");
    if (st != KNNSSD_OK) return finish(st);
    *n_out = max_new;
    if (stats_or_null) *stats_or_null = c->stats;
    return finish(KNNSSD_OK);
}

knnssd_status knnssd_generate(knnssd_ctx *c, const int *prompt_host, int n_prompt, int max_new, int k, int use_selection,
                              int *out_tokens_host, int *n_out, int *accepts_host_or_null, int *domain_or_null,
                              knnssd_stats *stats_or_null) {
    if (!c) return KNNSSD_ERR_INVALID_ARG;
    DeviceGuard dg(c->device);
    const knnssd_config &g = c->cfg;
    if (!out_tokens_host || !n_out || max_new < 1 || k < 0 || k > g.max_draft)
        return fail(c, KNNSSD_ERR_INVALID_ARG, "generate: bad arguments");
    if (n_prompt + max_new + 1 > g.max_seq) return fail(c, KNNSSD_ERR_CAPACITY, "generate: prompt + max_new + 1 exceeds max_seq");
    if (!(use_selection && g.n_domains > 0) && !c->has_mask)
        return fail(c, KNNSSD_ERR_STATE, "generate: no active skip mask and no selection");
    knnssd_status st = do_prefill(c, prompt_host, n_prompt, nullptr, nullptr);
    if (st != KNNSSD_OK) return st;
    return do_decode(c, max_new, k, use_selection, out_tokens_host, n_out, accepts_host_or_null, domain_or_null,
                     stats_or_null);
}

long long knnssd_get_launch_count(const knnssd_ctx *c) { return c ? c->launches : -1; }

int knnssd_get_length(const knnssd_ctx *c) { return c ? c->len : -1; }

knnssd_status knnssd_set_length(knnssd_ctx *c, int new_len) {
    if (!c) return KNNSSD_ERR_INVALID_ARG;
    DeviceGuard dg(c->device);
    if (!c->prefilled) return fail(c, KNNSSD_ERR_STATE, "set_length: prefill first");
    if (new_len < 1 || new_len > c->len) return fail(c, KNNSSD_ERR_INVALID_ARG, "set_length: can only roll back (1 <= new_len <= length)");
    CUDA_TRY(c, cudaMemcpyAsync(&c->state->len, &new_len, sizeof(int), cudaMemcpyHostToDevice, c->stream));
    knnssd_status st = sync_check(c, "set_length");
    if (st != KNNSSD_OK) return st;
    c->len = new_len;
    return KNNSSD_OK;
}

knnssd_status knnssd_set_pending(knnssd_ctx *c, int token) {
    if (!c) return KNNSSD_ERR_INVALID_ARG;
    DeviceGuard dg(c->device);
    if (!c->prefilled) return fail(c, KNNSSD_ERR_STATE, "set_pending: prefill first");
    if (token < 0 || token >= c->cfg.vocab) return fail(c, KNNSSD_ERR_INVALID_ARG, "set_pending: token id out of range");
    CUDA_TRY(c, cudaMemcpyAsync(c->chain, &token, sizeof(int), cudaMemcpyHostToDevice, c->stream));
    knnssd_status st = sync_check(c, "set_pending");
    if (st != KNNSSD_OK) return st;
    c->pending = token;
    return KNNSSD_OK;
}

knnssd_status knnssd_mask_objective(knnssd_ctx *c, const unsigned char *masks_host, int n_masks, const int *tokens_host,
                                    const int *lens_host, int n_samples, int max_new, int k, float *ms_per_token_host,
                                    int *accepted_host, int *drafted_host) {
    if (!c) return KNNSSD_ERR_INVALID_ARG;
    DeviceGuard dg(c->device);
    if (!masks_host || !tokens_host || !lens_host || !ms_per_token_host || n_masks < 1 || n_samples < 1 || max_new < 1)
        return fail(c, KNNSSD_ERR_INVALID_ARG, "mask_objective: bad arguments");
    const int L2 = 2 * c->cfg.n_layers;
    for (size_t j = 0; j < (size_t)n_masks * L2; ++j)
        if (masks_host[j] > 1) return fail(c, KNNSSD_ERR_INVALID_ARG, "mask_objective: mask entries must be 0 or 1");
    std::vector<double> ms(n_masks, 0.0);
    std::vector<long long> tok(n_masks, 0), acc(n_masks, 0), drf(n_masks, 0);
    std::vector<int> out(max_new);
    size_t off = 0;
    for (int sidx = 0; sidx < n_samples; ++sidx) {
        const int P = lens_host[sidx];
        int first = 0;
        // the prompt pass does not depend on the mask: once per sample, then every mask decodes from the state it left
        knnssd_status st = do_prefill(c, tokens_host + off, P, nullptr, &first);
        if (st != KNNSSD_OK) return st;
        off += (size_t)P;
        for (int m = 0; m < n_masks; ++m) {
            if (m > 0) {
                st = knnssd_set_length(c, P);
                if (st == KNNSSD_OK) st = knnssd_set_pending(c, first);
                if (st != KNNSSD_OK) return st;
            }
            c->active_mask.assign(masks_host + (size_t)m * L2, masks_host + (size_t)(m + 1) * L2);
            c->has_mask = true;
            int n_out = 0;
            knnssd_stats stt{};
            st = do_decode(c, max_new, k, 0, out.data(), &n_out, nullptr, nullptr, &stt);
            if (st != KNNSSD_OK) return st;
            ms[m] += (double)stt.ms_draft + (double)stt.ms_verify;
            tok[m] += n_out - 1;                              // the first token of the output came from the prompt pass
            acc[m] += stt.accepted;
            drf[m] += stt.drafted;
        }
    }
    for (int m = 0; m < n_masks; ++m) {
        ms_per_token_host[m] = tok[m] > 0 ? (float)(ms[m] / (double)tok[m]) : 0.f;
        if (accepted_host) accepted_host[m] = (int)acc[m];
        if (drafted_host) drafted_host[m] = (int)drf[m];
    }
    return KNNSSD_OK;
}

knnssd_status knnssd_get_stats(const knnssd_ctx *c, knnssd_stats *out) {
    if (!c || !out) return KNNSSD_ERR_INVALID_ARG;
    *out = c->stats;
    return KNNSSD_OK;
}

const char *knnssd_last_error(const knnssd_ctx *c) { return c ? c->err.c_str() : "NULL context"; }

knnssd_status knnssd_time_pass(knnssd_ctx *c, int which, int k, int iters, float *ms_per_pass, int *launches_per_pass,
                               float *ms_linear_per_pass, int *linear_launches_per_pass) {
    if (!c) return KNNSSD_ERR_INVALID_ARG;
    DeviceGuard dg(c->device);
    const knnssd_config &g = c->cfg;
    if ((which != 0 && which != 1) || iters < 1 || k < 0 || k > g.max_draft) return fail(c, KNNSSD_ERR_INVALID_ARG, "time_pass: bad arguments");
    if (!c->prefilled) return fail(c, KNNSSD_ERR_STATE, "time_pass: prefill first");
    if (which == 0 && !c->has_mask) return fail(c, KNNSSD_ERR_STATE, "time_pass: no active skip mask");
    if (c->len + k + 1 > g.max_seq) return fail(c, KNNSSD_ERR_CAPACITY, "time_pass: len + k + 1 exceeds max_seq");
    cudaStream_t s = c->stream;
    // the chain must hold valid token ids for the rows a verify pass reads
    std::vector<int> fill(k + 1, c->pending);
    CUDA_TRY(c, cudaMemcpyAsync(c->chain, fill.data(), sizeof(int) * (k + 1), cudaMemcpyHostToDevice, s));
    auto one = [&]() {
        if (which == 0) run_pass(c, 1, c->chain, 0, c->active_mask.data(), 0, c->target, false);
        else run_pass(c, k + 1, c->chain, 0, nullptr, 0, c->target, false);
    };
    const long long l0 = c->launches;
    one();
    const int launches = (int)(c->launches - l0);
    knnssd_status st = sync_check(c, "time_pass warm-up");
    if (st != KNNSSD_OK) return st;
    cudaEventRecord(c->ev0, s);
    for (int i = 0; i < iters; ++i) one();
    cudaEventRecord(c->ev1, s);
    st = sync_check(c, "time_pass");
    if (st != KNNSSD_OK) return st;
    if (ms_per_pass) *ms_per_pass = elapsed_ms(c) / (float)iters;
    if (launches_per_pass) *launches_per_pass = launches;
    // separate replay with events around every linear kernel
    c->time_linear = true;
    c->lin_used = 0;
    one();
    c->time_linear = false;
    st = sync_check(c, "time_pass linear replay");
    if (st != KNNSSD_OK) return st;
    float tot = 0.f;
    for (size_t i = 0; i + 1 < c->lin_used; i += 2) {
        float ms = 0.f;
        cudaEventElapsedTime(&ms, c->lin_events[i], c->lin_events[i + 1]);
        tot += ms;
    }
    if (ms_linear_per_pass) *ms_linear_per_pass = tot;
    if (linear_launches_per_pass) *linear_launches_per_pass = (int)(c->lin_used / 2);
    // restore the pending token the chain held
    CUDA_TRY(c, cudaMemcpyAsync(c->chain, &c->pending, sizeof(int), cudaMemcpyHostToDevice, s));
    st = sync_check(c, "time_pass restore");
    if (st == KNNSSD_OK) st = check_stream_err(c, "time_pass");
    return st;
}

knnssd_status knnssd_trace_pass(knnssd_ctx *c, int which, int k, int cap, int *op_types, int *op_layers, float *us_work,
                                float *us_barrier, int *n_ops) {
    if (!c || !op_types || !op_layers || !us_work || !us_barrier || !n_ops) return KNNSSD_ERR_INVALID_ARG;
    DeviceGuard dg(c->device);
    const knnssd_config &g = c->cfg;
    if ((which != 0 && which != 1) || k < 0 || k > g.max_draft || cap < 1) return fail(c, KNNSSD_ERR_INVALID_ARG, "trace_pass: bad arguments");
    if (!c->mega_ok || (which == 1 && k + 1 > pass::MAXM)) return fail(c, KNNSSD_ERR_SHAPE, "trace_pass: this pass does not run in the persistent kernel");
    if (!c->prefilled) return fail(c, KNNSSD_ERR_STATE, "trace_pass: prefill first");
    if (which == 0 && !c->has_mask) return fail(c, KNNSSD_ERR_STATE, "trace_pass: no active skip mask");
    if (c->len + k + 1 > g.max_seq) return fail(c, KNNSSD_ERR_CAPACITY, "trace_pass: len + k + 1 exceeds max_seq");
    cudaStream_t s = c->stream;
    std::vector<int> fill(k + 1, c->pending);
    CUDA_TRY(c, cudaMemcpyAsync(c->chain, fill.data(), sizeof(int) * (k + 1), cudaMemcpyHostToDevice, s));
    auto one = [&]() {
        if (which == 0) run_pass(c, 1, c->chain, 0, c->active_mask.data(), 0, c->target, false);
        else run_pass(c, k + 1, c->chain, 0, nullptr, 0, c->target, false);
    };
    one();                                       // warm-up (also builds the draft list for the active mask)
    knnssd_status st = sync_check(c, "trace_pass warm-up");
    if (st != KNNSSD_OK) return st;
    std::vector<pass::Op> ops;
    int bars = 0;
    int n_attn_unused = 0;
    ops = build_ops(c, which == 0 ? c->active_mask.data() : nullptr, &bars, &n_attn_unused);
    const int n = (int)ops.size();
    CUDA_TRY(c, cudaMemsetAsync(c->trace, 0, sizeof(unsigned long long) * 2 * n, s));
    c->model.trace = c->trace;
    one();
    c->model.trace = nullptr;
    std::vector<unsigned long long> t(2 * (size_t)n);
    CUDA_TRY(c, cudaMemcpyAsync(t.data(), c->trace, sizeof(unsigned long long) * 2 * n, cudaMemcpyDeviceToHost, s));
    st = sync_check(c, "trace_pass");
    if (st != KNNSSD_OK) return st;
    unsigned long long prev = 0;
    int out = 0;
    for (int i = 0; i < n && out < cap; ++i) {
        if (t[2 * i] == 0) continue;
        if (prev == 0) prev = t[2 * i];          // the first operation's start is not stamped: its work reads as 0
        op_types[out] = ops[i].type == pass::OP_LINEAR ? (ops[i].is_head ? 14 : 10 + ops[i].lin.epi) : ops[i].type;
        op_layers[out] = ops[i].layer;
        us_work[out] = (float)((double)(t[2 * i] - prev) * 1e-3);
        us_barrier[out] = (float)((double)(t[2 * i + 1] - t[2 * i]) * 1e-3);
        prev = t[2 * i + 1];
        ++out;
    }
    *n_ops = out;
    CUDA_TRY(c, cudaMemcpyAsync(c->chain, &c->pending, sizeof(int), cudaMemcpyHostToDevice, s));
    st = sync_check(c, "trace_pass restore");
    if (st == KNNSSD_OK) st = check_stream_err(c, "trace_pass");
    return st;
}

knnssd_status knnssd_debug_barrier_timeout(knnssd_ctx *c, unsigned spin_limit) {
    if (!c) return KNNSSD_ERR_INVALID_ARG;
    DeviceGuard dg(c->device);
    if (spin_limit < 1 || spin_limit > 1000000u) return fail(c, KNNSSD_ERR_INVALID_ARG, "debug_barrier_timeout: spin_limit must be 1..1000000");
    if (!c->mega_ok) return fail(c, KNNSSD_ERR_SHAPE, "debug_barrier_timeout: this model does not run in the persistent kernel");
    // an operation list holding just the embedding (no linear map: the producer warp issues no copy) whose barrier
    // waits for one more round of arrivals than there are CTAs; every CTA runs out of polls, raises the abort word and
    // falls through to the end of the kernel
    pass::Op e{};
    e.type = pass::OP_EMBED; e.barrier_after = 1;
    e.lin.K = c->cfg.d_model; e.lin.ys = c->xs_x; e.lin.ss_out = c->ssp;
    std::vector<pass::Op> ops(1, e);
    c->ops_draft_mask.clear();                       // the draft list's slot is reused: it is rebuilt on the next draft
    knnssd_status st = upload_ops(c, ops, c->ops_draft);
    if (st != KNNSSD_OK) return st;
    pass::Params pr{};
    pr.ops = c->ops_draft; pr.n_ops = 1; pr.M = 1; pr.tok = c->chain; pr.pos_off = 0; pr.head_row0 = 1;
    pr.argmax_out = c->target; pr.bar_spin_limit = spin_limit;
    pr.bar_base = c->bar_total + (unsigned long long)c->n_sms;   // one CTA-count beyond what this launch can reach
    const cudaError_t le = c->cfg.head_dim == 128 ? launch_pass_t<128, 1, 0>(c, pr) : launch_pass_t<64, 1, 0>(c, pr);
    c->launches++;
    if (le != cudaSuccess) return fail(c, KNNSSD_ERR_CUDA, std::string("debug_barrier_timeout: ") + cudaGetErrorString(le));
    st = sync_check(c, "debug_barrier_timeout");
    if (st != KNNSSD_OK) return st;
    // the launch left n_sms arrivals on the counter: without an error the next pass would be off by them
    st = check_stream_err(c, "debug_barrier_timeout");
    if (st == KNNSSD_OK) { reset_mega_state(c); c->prefilled = false; }
    return st;
}

knnssd_status knnssd_linear(const void *W_dev, int dtype, int n_out, int n_in, const float *x_dev, int M, float *y_dev,
                            void *cuda_stream) {
    if (!W_dev || !x_dev || !y_dev || n_out < 1 || n_in < 8 || M < 1 || M > kMaxRows || (dtype != 0 && dtype != 1))
        return KNNSSD_ERR_INVALID_ARG;
    if (n_in % 8 != 0 || (reinterpret_cast<uintptr_t>(W_dev) & 15u) || (reinterpret_cast<uintptr_t>(x_dev) & 15u))
        return KNNSSD_ERR_SHAPE;
    int dev = 0, n_sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess) return KNNSSD_ERR_CUDA;
    cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev);
    LinearArgs a = make_args(W_dev, n_out, n_in, x_dev, nullptr, 0.f, y_dev, EPI_STORE, M);
    launch_linear(dtype, a, n_sms, reinterpret_cast<cudaStream_t>(cuda_stream));
    return cudaGetLastError() == cudaSuccess ? KNNSSD_OK : KNNSSD_ERR_CUDA;
}

knnssd_status knnssd_gemm_split(const void *W0_dev, const void *W1_dev, int n_out, int n_in, const float *x_dev, int T,
                                int mode, float *y_dev, void *cuda_stream) {
    if (!W0_dev || !x_dev || !y_dev || T < 1 || n_out < 1 || n_in < 1 || mode < 0 || mode > 2 || (mode == 2 && !W1_dev))
        return KNNSSD_ERR_INVALID_ARG;
    if (n_in % prefill::BK != 0 || n_out % 8 != 0 || (reinterpret_cast<uintptr_t>(W0_dev) & 15u) ||
        (reinterpret_cast<uintptr_t>(W1_dev) & 15u) || (reinterpret_cast<uintptr_t>(x_dev) & 15u) ||
        (reinterpret_cast<uintptr_t>(y_dev) & 15u))
        return KNNSSD_ERR_SHAPE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    int dev = 0, n_sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess) return KNNSSD_ERR_CUDA;
    cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev);
    const int cap = (T + prefill::BM - 1) / prefill::BM * prefill::BM;
    bf16_t *planes = nullptr, *outp = nullptr;
    const size_t plane = (size_t)cap * n_in, oplane = (size_t)T * n_out;
    if (dev_alloc(&planes, 2 * plane) != cudaSuccess) { cudaGetLastError(); return KNNSSD_ERR_CUDA; }
    if (mode == 2 && dev_alloc(&outp, 2 * oplane) != cudaSuccess) { cudaGetLastError(); cudaFree(planes); return KNNSSD_ERR_CUDA; }
    knnssd_status st = KNNSSD_OK;
    cudaMemsetAsync(planes, 0, 2 * plane * sizeof(bf16_t), s);
    prefill::split_rows_kernel<<<T, 256, 0, s>>>(x_dev, n_in, planes, planes + plane);
    CUtensorMap ta;
    if (!prefill::make_map(&ta, planes, (size_t)2 * cap, (size_t)n_in, prefill::BM) ||
        !prefill::launch_gemm(ta, cap, W0_dev, W1_dev, n_out, n_in, T, mode, y_dev, n_out, 0, outp, outp ? outp + oplane : nullptr,
                              n_out, stream_err_ptr(), n_sms, s))
        st = KNNSSD_ERR_CUDA;
    if (st == KNNSSD_OK && mode == 2) prefill::join_planes_kernel<<<T, 256, 0, s>>>(outp, outp + oplane, n_out, y_dev);
    cudaError_t e = cudaStreamSynchronize(s);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) st = KNNSSD_ERR_CUDA;
    if (st == KNNSSD_OK) {
        int code = 0;
        if (cudaMemcpy(&code, stream_err_ptr(), sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) st = KNNSSD_ERR_CUDA;
        else if (code) { cudaMemset(stream_err_ptr(), 0, sizeof(int)); st = KNNSSD_ERR_TIMEOUT; }
    }
    cudaFree(planes);
    if (outp) cudaFree(outp);
    return st;
}

knnssd_status knnssd_linear_tc(const void *W_dev, int n_out, int n_in, const float *x_dev, int M, float *y_dev,
                               float *ms_kernels_host, void *cuda_stream) {
    if (!W_dev || !x_dev || !y_dev || n_out < 1 || n_in < 1 || M < 1) return KNNSSD_ERR_INVALID_ARG;
    if (M > lintc::TN) return KNNSSD_ERR_CAPACITY;
    if (n_in % lintc::BK != 0 || (reinterpret_cast<uintptr_t>(W_dev) & 15u)) return KNNSSD_ERR_SHAPE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    int dev = 0, n_sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess) return KNNSSD_ERR_CUDA;
    cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev);
    const int tiles = (n_out + lintc::TM - 1) / lintc::TM, nkb = n_in / lintc::BK;
    // chunks of the input columns: enough work items for every SM when the matrix has few 128-unit tiles, at least
    // 8 k-blocks per item
    int kc = tiles >= n_sms ? 1 : (n_sms + tiles - 1) / tiles;
    if (kc > nkb / 8) kc = nkb / 8 > 0 ? nkb / 8 : 1;
    const int kb_per = (nkb + kc - 1) / kc;
    kc = (nkb + kb_per - 1) / kb_per;
    bf16_t *planes = nullptr;
    float *part = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    const size_t plane_elems = (size_t)2 * lintc::TN * n_in, part_elems = (size_t)kc * M * n_out;
    bool ok = dev_alloc(&planes, plane_elems) == cudaSuccess && dev_alloc(&part, part_elems) == cudaSuccess &&
              cudaEventCreate(&e0) == cudaSuccess && cudaEventCreate(&e1) == cudaSuccess;
    auto cleanup = [&]() {
        if (planes) cudaFree(planes);
        if (part) cudaFree(part);
        if (e0) cudaEventDestroy(e0);
        if (e1) cudaEventDestroy(e1);
    };
    if (!ok) { cudaGetLastError(); cleanup(); return KNNSSD_ERR_CUDA; }
    knnssd_status st = KNNSSD_OK;
    CUtensorMap tw, tx;
    if (cudaFuncSetAttribute(lintc::linear_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, lintc::SMEM) != cudaSuccess ||
        !prefill::make_map(&tw, W_dev, (size_t)n_out, (size_t)n_in, lintc::TM) ||
        !prefill::make_map(&tx, planes, (size_t)2 * lintc::TN, (size_t)n_in, lintc::TN)) {
        cudaGetLastError();
        cleanup();
        return KNNSSD_ERR_CUDA;
    }
    cudaMemsetAsync(planes, 0, plane_elems * sizeof(bf16_t), s);
    lintc::split_x_kernel<<<M, 256, 0, s>>>(x_dev, n_in, planes);
    lintc::Args a{M, n_in, n_out, kc, kb_per, part, stream_err_ptr()};
    cudaEventRecord(e0, s);
    lintc::linear_tc_kernel<<<dim3(tiles, kc), lintc::THREADS, lintc::SMEM, s>>>(tw, tx, a);
    const size_t n = (size_t)M * n_out;
    lintc::reduce_chunks_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(part, kc, n, y_dev);
    cudaEventRecord(e1, s);
    cudaError_t e = cudaStreamSynchronize(s);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) st = KNNSSD_ERR_CUDA;
    if (st == KNNSSD_OK) {
        int code = 0;
        if (cudaMemcpy(&code, stream_err_ptr(), sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) st = KNNSSD_ERR_CUDA;
        else if (code) { cudaMemset(stream_err_ptr(), 0, sizeof(int)); st = KNNSSD_ERR_TIMEOUT; }
    }
    if (st == KNNSSD_OK && ms_kernels_host) cudaEventElapsedTime(ms_kernels_host, e0, e1);
    cleanup();
    return st;
}

namespace {
__global__ void widen_kernel(const float *__restrict__ a, size_t n, double *__restrict__ b) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) b[i] = (double)a[i];
}
}  // namespace

knnssd_status knnssd_build_anchors(const float *x_dev, int n_points, int d, int n_clusters,
                                   const float *init_centroids_dev, int max_rounds, int k, int *labels_host,
                                   double *centroids_out_dev, int *anchors_host, int *rounds_host, float *ms_rounds_host,
                                   void *cuda_stream) {
    if (!x_dev || !init_centroids_dev || !anchors_host || n_points < 1 || d < 1 || n_clusters < 1 || max_rounds < 1 || k < 1 ||
        n_points < n_clusters)
        return KNNSSD_ERR_INVALID_ARG;
    if (n_clusters > anchors::MAXC) return KNNSSD_ERR_CAPACITY;
    if (reinterpret_cast<uintptr_t>(x_dev) & 15u) return KNNSSD_ERR_SHAPE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    const int N = n_points, n = n_clusters;
    int S = (N + 63) / 64;                        // slices of the centroid sums: at least 64 points each, at most 64 slices
    if (S > 64) S = 64;
    const int per = (N + S - 1) / S;
    double *mu = nullptr, *dist = nullptr, *part = nullptr;
    int *labels = nullptr, *small = nullptr, *out = nullptr;     // small: [0] changed, [1 .. n] counts
    unsigned char *taken = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    bool ok = dev_alloc(&mu, (size_t)n * d) == cudaSuccess && dev_alloc(&dist, (size_t)N) == cudaSuccess &&
              dev_alloc(&part, (size_t)S * n * d) == cudaSuccess && dev_alloc(&labels, (size_t)N) == cudaSuccess &&
              dev_alloc(&small, (size_t)n + 1) == cudaSuccess && dev_alloc(&out, (size_t)n * k) == cudaSuccess &&
              dev_alloc(&taken, (size_t)N) == cudaSuccess && cudaEventCreate(&e0) == cudaSuccess &&
              cudaEventCreate(&e1) == cudaSuccess;
    auto cleanup = [&]() {
        void *ptrs[] = {mu, dist, part, labels, small, out, taken};
        for (void *p : ptrs)
            if (p) cudaFree(p);
        if (e0) cudaEventDestroy(e0);
        if (e1) cudaEventDestroy(e1);
    };
    if (!ok) { cudaGetLastError(); cleanup(); return KNNSSD_ERR_CUDA; }
    widen_kernel<<<(unsigned)(((size_t)n * d + 255) / 256), 256, 0, s>>>(init_centroids_dev, (size_t)n * d, mu);
    cudaMemsetAsync(labels, 0xFF, sizeof(int) * N, s);           // -1: the first round changes every assignment
    const dim3 cols((d + 255) / 256);
    const int agrid = (N + anchors::PTS - 1) / anchors::PTS;
    const bool vec = d % 4 == 0;                                 // rows stay 16-byte aligned
    auto launch_assign = [&](int relabel) {
#define KNNSSD_ASSIGN(V, NC) anchors::assign_kernel<V, NC><<<agrid, 256, 0, s>>>(x_dev, N, d, mu, n, relabel, labels, dist, small + 1, small)
        if (vec) { if (n <= 4) KNNSSD_ASSIGN(true, 4); else if (n <= 8) KNNSSD_ASSIGN(true, 8); else KNNSSD_ASSIGN(true, 16); }
        else { if (n <= 4) KNNSSD_ASSIGN(false, 4); else if (n <= 8) KNNSSD_ASSIGN(false, 8); else KNNSSD_ASSIGN(false, 16); }
#undef KNNSSD_ASSIGN
    };
    int rounds = 0, changed = 1;
    float ms_total = 0.f;
    cudaError_t e = cudaSuccess;
    while (rounds < max_rounds && e == cudaSuccess) {
        cudaMemsetAsync(small, 0, sizeof(int) * (n + 1), s);
        cudaEventRecord(e0, s);
        launch_assign(1);
        cudaEventRecord(e1, s);
        e = cudaMemcpyAsync(&changed, small, sizeof(int), cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) break;
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        ms_total += ms;
        ++rounds;
        if (!changed) break;
        cudaEventRecord(e0, s);
        anchors::partial_sums_kernel<<<dim3(cols.x, S), 256, 0, s>>>(x_dev, N, d, labels, n, per, part);
        anchors::fold_centroids_kernel<<<dim3(cols.x, n), 256, 0, s>>>(part, small + 1, n, d, S, mu);
        cudaEventRecord(e1, s);
        e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) break;
        cudaEventElapsedTime(&ms, e0, e1);
        ms_total += ms;
    }
    if (e == cudaSuccess) {
        // the anchors are ranked by fp64 distances to the final fp64 centroids (which moved after the last assignment
        // if the round limit ended the iteration)
        anchors::member_dist_kernel<<<(N + 7) / 8, 256, 0, s>>>(x_dev, N, d, mu, labels, dist);
        cudaMemsetAsync(taken, 0, (size_t)N, s);
        anchors::select_anchors_kernel<<<n, 256, 0, s>>>(dist, labels, N, k, taken, out);
        e = cudaMemcpyAsync(anchors_host, out, sizeof(int) * n * k, cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess && labels_host) e = cudaMemcpyAsync(labels_host, labels, sizeof(int) * N, cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess && centroids_out_dev)
            e = cudaMemcpyAsync(centroids_out_dev, mu, sizeof(double) * n * d, cudaMemcpyDeviceToDevice, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        if (e == cudaSuccess) e = cudaGetLastError();
    }
    cleanup();
    if (e != cudaSuccess) { cudaGetLastError(); return KNNSSD_ERR_CUDA; }
    if (rounds_host) *rounds_host = rounds;
    if (ms_rounds_host) *ms_rounds_host = ms_total;
    return KNNSSD_OK;
}

knnssd_status knnssd_filtered_probs(const float *logits_dev, int rows, int vocab, float temperature, float top_p,
                                    float *probs_dev, void *cuda_stream) {
    if (!logits_dev || !probs_dev || rows < 1 || vocab < 1 || !(temperature > 0.f) || !(top_p > 0.f) || !std::isfinite(temperature) ||
        !std::isfinite(top_p))
        return KNNSSD_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    sampling::filtered_probs_kernel<<<rows, sampling::NT, 0, s>>>(logits_dev, vocab, 1.0f / temperature, top_p, probs_dev);
    return cudaGetLastError() == cudaSuccess ? KNNSSD_OK : KNNSSD_ERR_CUDA;
}

knnssd_status knnssd_sample_token(const float *weights_dev, int vocab, float u, int *token_host, void *cuda_stream) {
    if (!weights_dev || !token_host || vocab < 1 || !(u >= 0.f) || !(u < 1.f)) return KNNSSD_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    int *tok = nullptr;
    if (cudaMalloc(reinterpret_cast<void **>(&tok), sizeof(int)) != cudaSuccess) { cudaGetLastError(); return KNNSSD_ERR_CUDA; }
    sampling::sample_kernel<<<1, sampling::NT, 0, s>>>(weights_dev, vocab, nullptr, u, tok);
    cudaError_t e = cudaMemcpyAsync(token_host, tok, sizeof(int), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e == cudaSuccess) e = cudaGetLastError();
    cudaFree(tok);
    return e == cudaSuccess ? KNNSSD_OK : KNNSSD_ERR_CUDA;
}

knnssd_status knnssd_spec_accept(const float *p_dev, const float *q_dev, const int *drafts_host, int k, int vocab,
                                 const float *u_accept_host, float u_final, int *n_accepted, int *next_token, void *cuda_stream) {
    if (!p_dev || !n_accepted || !next_token || k < 0 || k > kMaxRows - 1 || vocab < 1 || !(u_final >= 0.f) || !(u_final < 1.f) ||
        (k > 0 && (!q_dev || !drafts_host || !u_accept_host)))
        return KNNSSD_ERR_INVALID_ARG;
    for (int j = 0; j < k; ++j)
        if (drafts_host[j] < 0 || drafts_host[j] >= vocab || !(u_accept_host[j] >= 0.f) || !(u_accept_host[j] < 1.f))
            return KNNSSD_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    int *buf = nullptr;                       // [0..1] result, [2 .. 2 + k) drafts, then k floats of uniforms
    if (cudaMalloc(reinterpret_cast<void **>(&buf), sizeof(int) * (2 + 2 * (size_t)kMaxRows)) != cudaSuccess) {
        cudaGetLastError();
        return KNNSSD_ERR_CUDA;
    }
    int *d_dev = buf + 2;
    float *u_dev = reinterpret_cast<float *>(buf + 2 + kMaxRows);
    cudaError_t e = cudaSuccess;
    if (k > 0) {
        e = cudaMemcpyAsync(d_dev, drafts_host, sizeof(int) * k, cudaMemcpyHostToDevice, s);
        if (e == cudaSuccess) e = cudaMemcpyAsync(u_dev, u_accept_host, sizeof(float) * k, cudaMemcpyHostToDevice, s);
    }
    int host[2] = {0, 0};
    if (e == cudaSuccess) {
        sampling::spec_accept_kernel<<<1, sampling::NT, 0, s>>>(p_dev, q_dev, d_dev, k, vocab, u_dev, nullptr, u_final, buf);
        e = cudaMemcpyAsync(host, buf, sizeof(int) * 2, cudaMemcpyDeviceToHost, s);
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e == cudaSuccess) e = cudaGetLastError();
    cudaFree(buf);
    if (e != cudaSuccess) return KNNSSD_ERR_CUDA;
    *n_accepted = host[0];
    *next_token = host[1];
    return KNNSSD_OK;
}

knnssd_status knnssd_cosine_top1(const float *query_dev, const float *anchors_dev, int n, int d, int *best, float *cosine,
                                 void *cuda_stream) {
    if (!query_dev || !anchors_dev || n < 1 || d < 1) return KNNSSD_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    float *cos_dev = nullptr;
    int *small = nullptr;  // [0..1] result, [2] flag
    if (cudaMalloc(reinterpret_cast<void **>(&cos_dev), sizeof(float) * n) != cudaSuccess) return KNNSSD_ERR_CUDA;
    if (cudaMalloc(reinterpret_cast<void **>(&small), sizeof(int) * 4) != cudaSuccess) { cudaFree(cos_dev); return KNNSSD_ERR_CUDA; }
    cudaMemsetAsync(small, 0, sizeof(int) * 4, s);
    cosine_scores_kernel<<<(n + 7) / 8, 256, 0, s>>>(query_dev, anchors_dev, nullptr, n, d, cos_dev, small + 2);
    cosine_argmax_kernel<<<1, 256, 0, s>>>(cos_dev, n, small);
    int host[4] = {0, 0, 0, 0};
    cudaError_t e = cudaMemcpyAsync(host, small, sizeof(int) * 4, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    cudaFree(cos_dev);
    cudaFree(small);
    if (e != cudaSuccess) return KNNSSD_ERR_CUDA;
    if (host[2]) return KNNSSD_ERR_DEGENERATE;
    if (best) *best = host[0];
    if (cosine) std::memcpy(cosine, &host[1], sizeof(float));
    return KNNSSD_OK;
}

}  // extern "C"

// ---- cosine top-1 without any allocation ------------------------------------------------------------------------
// Scratch of knnssd_cosine_top1_static: the per-anchor cosines, then four result words (best index, cosine bits,
// degenerate-input flag, spare).  It lives in the library's device image, one copy per GPU that loads the library.
// In host code the name below is only a handle for cudaGetSymbolAddress; kernels get the address that call returns.
namespace {
constexpr int kStaticWords = KNNSSD_STATIC_MAX_ANCHORS + 4;
}  // namespace
static __device__ __align__(256) float g_top1_static_scratch[kStaticWords];

namespace {
// Device address of the array on the current device, looked up once per device.
cudaError_t static_scratch_address(int dev, float **out) {
    static float *addr[kMaxDevices] = {};
    static std::mutex mu;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        float *p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void **>(&p), g_top1_static_scratch);
        if (e != cudaSuccess) return e;
        addr[dev] = p;
    }
    *out = addr[dev];
    return cudaSuccess;
}
}  // namespace

extern "C" knnssd_status knnssd_cosine_top1_static(const float *query_dev, const float *anchors_dev, int n, int d,
                                                   int *best, float *cosine, void *cuda_stream) {
    if (!query_dev || !anchors_dev || n < 1 || d < 1) return KNNSSD_ERR_INVALID_ARG;
    if (n > KNNSSD_STATIC_MAX_ANCHORS) return KNNSSD_ERR_CAPACITY;   // beyond the fixed scratch: refuse, touch nothing
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return KNNSSD_ERR_CUDA;
    float *scratch = nullptr;
    if (static_scratch_address(dev, &scratch) != cudaSuccess) { cudaGetLastError(); return KNNSSD_ERR_CUDA; }
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    float *cos_dev = scratch;
    int *small = reinterpret_cast<int *>(scratch + KNNSSD_STATIC_MAX_ANCHORS);   // [0..1] result, [2] flag
    // the array still holds the previous call's result and flag: the words that must start at zero are cleared here
    if (cudaMemsetAsync(small, 0, sizeof(int) * 4, s) != cudaSuccess) return KNNSSD_ERR_CUDA;
    cosine_scores_kernel<<<(n + 7) / 8, 256, 0, s>>>(query_dev, anchors_dev, nullptr, n, d, cos_dev, small + 2);
    cosine_argmax_kernel<<<1, 256, 0, s>>>(cos_dev, n, small);
    int host[4] = {0, 0, 0, 0};
    cudaError_t e = cudaMemcpyAsync(host, small, sizeof(int) * 4, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return KNNSSD_ERR_CUDA;
    if (host[2]) return KNNSSD_ERR_DEGENERATE;
    if (best) *best = host[0];
    if (cosine) std::memcpy(cosine, &host[1], sizeof(float));
    return KNNSSD_OK;
}
