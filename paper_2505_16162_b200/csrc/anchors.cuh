// Anchor construction of the pre-inference stage (Sec. 4.1): the sampled last hidden vectors of all domains are
// clustered with K-means (Lloyd's iteration, as many clusters as domains), and each cluster's k members nearest to
// its centroid become its anchors (Eq. (2): the k smallest distances minimise the sum over size-k subsets).
//
// The points are fp32 [N][d] (d = the model width, N = domains x samples per domain: 5 x 1000 in the paper's
// set-up, 100 MB at d = 5120).  Centroids and their sums are fp64.  A squared distance is formed from fp32
// differences to the fp32-rounded centroid, squared and added eight at a time in fp32, and those short sums are
// accumulated without loss in pairs of floats (fp64 only for the final reductions): the fp64 pipe of this GPU issues
// a few lanes per clock per SM, so per-element fp64 arithmetic made the assignment 15x slower than its memory
// traffic, while this form keeps ~1e-8 relative accuracy (error of a
// distance^2 of ~1e3: ~1e-5, four orders below the gaps that decide nearest centroids and nearest members).  A round
// reads the points twice (assignment, centroid sums).  Every reduction has a fixed order: results do not depend on
// timing.
#pragma once

#include "kernels.cuh"

namespace knnssd {
namespace anchors {

constexpr int MAXC = 16;       // most clusters (domains)
constexpr int CHUNK = 256;     // columns of the centroids staged in shared memory per step
constexpr int PTS = 16;        // points per block of assign_kernel: two per warp

// For each point: the squared distances to all n centroids; relabel != 0: labels[p] <- the nearest centroid (lowest
// index among equal distances), *changed set if that differs from the old label, counts[c] incremented; in both modes
// dist[p] <- the distance to the centroid of labels[p].  grid = ceil(N / PTS), 256 threads: a warp owns two points, the
// block shares the staged columns of the centroids.  Per step of 256 columns a lane holds 8 columns of each of its
// points (VEC: two 16-byte loads per point, d % 4 == 0), fetched one step ahead; the centroids' next columns are
// fetched into registers under the arithmetic as well.  In shared memory the centroid values are ordered
// [cluster][i][lane] (i = which of the lane's 8 columns), so that a warp reads consecutive words.
// NC = the cluster count rounded up to 4, 8 or 16: the per-cluster registers (and with them the CTAs per SM) follow it.
template <bool VEC, int NC>
__global__ void __launch_bounds__(256, NC <= 8 ? 3 : 2) assign_kernel(const float *__restrict__ x, int N, int d, const double *__restrict__ mu, int n,
                                                     int relabel, int *__restrict__ labels, double *__restrict__ dist,
                                                     int *__restrict__ counts, int *__restrict__ changed) {
    __shared__ float smu[NC][8][32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int pa = blockIdx.x * PTS + 2 * warp, pb = pa + 1;
    const bool la = pa < N, lb = pb < N;
    // running sums as unevaluated pairs of floats (hi + lo, hi the rounded sum, lo the rounding errors collected by
    // the error-free two-sum): ~48 bits without touching the fp64 pipe in the loop
    float hi[2][NC], lo[2][NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) hi[0][c] = hi[1][c] = lo[0][c] = lo[1][c] = 0.f;
    auto add_pair = [](float &h, float &l, float v) {
        const float s = __fadd_rn(h, v);
        const float bb = __fsub_rn(s, h);
        l = __fadd_rn(l, __fadd_rn(__fsub_rn(h, __fsub_rn(s, bb)), __fsub_rn(v, bb)));
        h = s;
    };
    const float *xa = x + (size_t)(la ? pa : 0) * d, *xb = x + (size_t)(lb ? pb : 0) * d;
    // the lane's i-th column within a step: VEC: (i / 4) 128 + 4 lane + i % 4; else lane + 32 i
    auto col_of = [&](int i, int ln) { return VEC ? (i >> 2) * 128 + 4 * ln + (i & 3) : ln + 32 * i; };
    auto fetch = [&](const float *xr, bool live, int col0, float (&v)[8]) {
        if (VEC) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int c0 = col0 + h * 128 + 4 * lane;
                const float4 t = (live && c0 < d) ? __ldg(reinterpret_cast<const float4 *>(xr + c0)) : make_float4(0.f, 0.f, 0.f, 0.f);
                v[4 * h] = t.x; v[4 * h + 1] = t.y; v[4 * h + 2] = t.z; v[4 * h + 3] = t.w;
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = (live && col0 + lane + 32 * i < d) ? __ldg(xr + col0 + lane + 32 * i) : 0.f;
        }
    };
    // this thread stages slot (i, ln) = (threadIdx.x / 32, threadIdx.x % 32) of every cluster
    const int my_col = col_of(warp, lane);
    auto fetch_mu = [&](int col0, float (&m)[NC]) {
#pragma unroll
        for (int c = 0; c < NC; ++c) m[c] = (c < n && col0 + my_col < d) ? (float)mu[(size_t)c * d + col0 + my_col] : 0.f;
    };
    float ca[8], cb[8], na[8], nb[8];
    float mreg[NC];
    fetch(xa, la, 0, ca);
    fetch(xb, lb, 0, cb);
    fetch_mu(0, mreg);
    for (int col0 = 0; col0 < d; col0 += CHUNK) {
#pragma unroll
        for (int c = 0; c < NC; ++c)
            if (c < n) smu[c][warp][lane] = mreg[c];
        __syncthreads();
        if (col0 + CHUNK < d) {
            fetch(xa, la, col0 + CHUNK, na);
            fetch(xb, lb, col0 + CHUNK, nb);
            fetch_mu(col0 + CHUNK, mreg);
        }
#pragma unroll
        for (int c = 0; c < NC; ++c)
            if (c < n) {
                // columns past the end hold zeros on both sides: they add nothing
                float sa = 0.f, sb = 0.f;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float m = smu[c][i][lane];
                    const float da = ca[i] - m, db = cb[i] - m;
                    sa = fmaf(da, da, sa);
                    sb = fmaf(db, db, sb);
                }
                add_pair(hi[0][c], lo[0][c], sa);
                add_pair(hi[1][c], lo[1][c], sb);
            }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < 8; ++i) { ca[i] = na[i]; cb[i] = nb[i]; }
    }
    double acc[2][NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) { acc[0][c] = (double)hi[0][c] + (double)lo[0][c]; acc[1][c] = (double)hi[1][c] + (double)lo[1][c]; }
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        const int p = q ? pb : pa;
        if (p >= N) continue;                                  // warp-uniform
#pragma unroll
        for (int c = 0; c < NC; ++c)
            if (c < n) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) acc[q][c] += __shfl_xor_sync(0xffffffffu, acc[q][c], o);
            }
        if (lane == 0) {
            int best = labels[p];
            if (relabel) {
                best = 0;
                double bv = acc[q][0];
#pragma unroll
                for (int c = 1; c < NC; ++c)
                    if (c < n && acc[q][c] < bv) { bv = acc[q][c]; best = c; }
                if (best != labels[p]) { labels[p] = best; atomicOr(changed, 1); }
                atomicAdd(counts + best, 1);
            }
            double own = acc[q][0];
#pragma unroll
            for (int c = 1; c < NC; ++c)
                if (c == best) own = acc[q][c];
            dist[p] = sqrt(own);
        }
    }
}

// part[s][c][j] = sum of x[p][j] over the points p of slice s (S slices of `per` consecutive points) labelled c, added
// in index order.  grid = (ceil(d / 256), S), 256 threads: a thread owns one column.
__global__ void __launch_bounds__(256) partial_sums_kernel(const float *__restrict__ x, int N, int d, const int *__restrict__ labels,
                                                           int n, int per, double *__restrict__ part) {
    __shared__ double acc[MAXC][256];
    const int j = blockIdx.x * 256 + threadIdx.x, s = blockIdx.y;
    for (int c = 0; c < n; ++c) acc[c][threadIdx.x] = 0.0;
    const int p0 = s * per, p1 = min(N, p0 + per);
    if (j < d) {
        int p = p0;
        for (; p + 8 <= p1; p += 8) {                          // eight loads in flight, added in index order
            float v[8];
            int l[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) { v[i] = __ldg(x + (size_t)(p + i) * d + j); l[i] = labels[p + i]; }
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[l[i]][threadIdx.x] += (double)v[i];
        }
        for (; p < p1; ++p) acc[labels[p]][threadIdx.x] += (double)__ldg(x + (size_t)p * d + j);
    }
    if (j < d)
        for (int c = 0; c < n; ++c) part[((size_t)s * n + c) * d + j] = acc[c][threadIdx.x];
}

// mu[c][j] = (sum over slices, in slice order, of part[s][c][j]) / counts[c]; a cluster without members keeps its
// centroid.  grid = (ceil(d / 256), n), 256 threads.
__global__ void fold_centroids_kernel(const double *__restrict__ part, const int *__restrict__ counts, int n, int d, int S,
                                      double *__restrict__ mu) {
    const int j = blockIdx.x * 256 + threadIdx.x, c = blockIdx.y;
    if (j >= d || counts[c] == 0) return;
    double s = 0.0;
    int i = 0;
    for (; i + 8 <= S; i += 8) {                              // eight loads in flight, added in slice order
        double v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = part[((size_t)(i + e) * n + c) * d + j];
#pragma unroll
        for (int e = 0; e < 8; ++e) s += v[e];
    }
    for (; i < S; ++i) s += part[((size_t)i * n + c) * d + j];
    mu[(size_t)c * d + j] = s / (double)counts[c];
}

// dist[p] = ||x_p - mu_{labels[p]}|| with every difference, square and sum in fp64 against the fp64 centroid: the
// distances Eq. (2) ranks the members by.  Points at equal distance in exact arithmetic (duplicates, or points mirrored
// about their centroid) then get equal values, so the lowest index decides among them.  One warp per point, lanes
// stride over the columns, fixed-order reduction.  Runs once per call.  grid = ceil(N / 8), 256 threads.
__global__ void __launch_bounds__(256) member_dist_kernel(const float *__restrict__ x, int N, int d, const double *__restrict__ mu,
                                                          const int *__restrict__ labels, double *__restrict__ dist) {
    const int lane = threadIdx.x & 31, p = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (p >= N) return;
    const float *xr = x + (size_t)p * d;
    const double *m = mu + (size_t)labels[p] * d;
    double s = 0.0;
    for (int j = lane; j < d; j += 32) {
        const double df = (double)__ldg(xr + j) - m[j];
        s = fma(df, df, s);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) dist[p] = sqrt(s);
}

// Eq. (2) for cluster c = blockIdx.x: k times, the not yet taken member with the smallest (distance, index);
// out[c][r] = its index, -1 once the cluster has run out of members.  taken[N] starts at zero.  256 threads.
__global__ void __launch_bounds__(256) select_anchors_kernel(const double *__restrict__ dist, const int *__restrict__ labels, int N, int k,
                                                             unsigned char *__restrict__ taken, int *__restrict__ out) {
    __shared__ double sv[256];
    __shared__ int si[256];
    const int c = blockIdx.x, tid = threadIdx.x;
    for (int r = 0; r < k; ++r) {
        double bv = INFINITY;
        int bi = -1;
        for (int p = tid; p < N; p += 256)
            if (labels[p] == c && !taken[p] && (bi < 0 || dist[p] < bv)) { bv = dist[p]; bi = p; }   // ascending p: first of equals wins
        sv[tid] = bv;
        si[tid] = bi;
        __syncthreads();
        for (int o = 128; o > 0; o >>= 1) {
            if (tid < o) {
                const double ov = sv[tid + o];
                const int oi = si[tid + o];
                if (oi >= 0 && (si[tid] < 0 || ov < sv[tid] || (ov == sv[tid] && oi < si[tid]))) { sv[tid] = ov; si[tid] = oi; }
            }
            __syncthreads();
        }
        if (tid == 0) {
            out[c * k + r] = si[0];
            if (si[0] >= 0) taken[si[0]] = 1;
        }
        __syncthreads();
    }
}

}  // namespace anchors
}  // namespace knnssd
