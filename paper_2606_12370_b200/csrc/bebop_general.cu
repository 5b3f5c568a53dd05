// General path of the verify step: works for any V, dtype and row stride the
// C ABI admits.  Split-row fp32 sweeps (stats, then TV with the normalisers
// known), a warp-per-sequence accept scan, and an fp64 inverse-CDF draw at the
// stop row.  The pipelined kernel (bebop_pipe.cu) covers the common shapes faster; this
// path serves the remaining shapes, bebop_tv and the greedy mode.
#include "bebop_kernels.h"

namespace bebop {

namespace {

constexpr int kThreads = 256;
constexpr float kNegInf = -INFINITY;

__device__ __forceinline__ float tau_of(const RowArgs& a, int b) {
    return a.temperature ? a.temperature[b] : a.temperature_all;
}
__device__ __forceinline__ bool tau_ok(float t) { return t > 0.f && t < INFINITY; }
__device__ __forceinline__ int len_of(const RowArgs& a, int b) {
    int L = a.draft_len ? a.draft_len[b] : a.K;
    return max(0, min(L, a.K));
}
__device__ __forceinline__ const char* target_row(const RowArgs& a, int b, int k) {
    return a.target + ((int64_t)b * a.t_seq_rows + k) * a.t_row_bytes;
}
__device__ __forceinline__ const char* draft_row(const RowArgs& a, int b, int k) {
    return a.draft + ((int64_t)b * a.d_seq_rows + k) * a.d_row_bytes;
}
__device__ __forceinline__ int ms_status(MS v) {
    if (v.m != v.m || v.m == INFINITY || v.s != v.s) return ST_NONFINITE;
    if (v.m == kNegInf) return ST_EMPTY;
    return 0;
}

__device__ __forceinline__ MS ms_block(MS v, float c, MS* sh) {
    v = ms_warp(v, c);
    int w = threadIdx.x >> 5, l = threadIdx.x & 31;
    if (l == 0) sh[w] = v;
    __syncthreads();
    if (w == 0) {
        MS t = (l < (int)(blockDim.x >> 5)) ? sh[l] : MS{kNegInf, 0.f};
        t = ms_warp(t, c);
        if (l == 0) sh[0] = t;
    }
    __syncthreads();
    MS r = sh[0];
    __syncthreads();
    return r;
}

template <typename T> __device__ __forceinline__ T sum_block(T v, T* sh) {
    v = warp_sum(v);
    int w = threadIdx.x >> 5, l = threadIdx.x & 31;
    if (l == 0) sh[w] = v;
    __syncthreads();
    if (w == 0) {
        T t = (l < (int)(blockDim.x >> 5)) ? sh[l] : T(0);
        t = warp_sum(t);
        if (l == 0) sh[0] = t;
    }
    __syncthreads();
    T r = sh[0];
    __syncthreads();
    return r;
}

// ---------------------------------------------------------------- fp32 sweep 1
// (m, S) of one slice of one logit row: S = sum exp2((z - m) * log2e / tau).
template <int DT>
__global__ void __launch_bounds__(kThreads) k_row_stats(RowArgs a, float2* __restrict__ stats) {
    constexpr int VEC = Elem<DT>::VEC, U = 4;
    __shared__ MS sh[kThreads / 32];
    int x = blockIdx.x;
    int split = x % a.nsplit; x /= a.nsplit;
    int r = x % (2 * a.K);
    int b = x / (2 * a.K);
    int k = r >> 1, which = r & 1;
    if (k >= len_of(a, b)) return;
    float tau = tau_of(a, b);
    if (!tau_ok(tau)) return;
    const float c = kLog2e / tau;
    const char* row = which ? draft_row(a, b, k) : target_row(a, b, k);
    int begin, end;
    slice_range(a.nvec, a.nsplit, split, begin, end);

    MS acc{kNegInf, 0.f};
    for (int i0 = begin + (int)threadIdx.x; i0 < end; i0 += kThreads * U) {
        float f[U][VEC];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            int iv = i0 + u * kThreads;
            if (iv < end) load_vec<DT>(row, iv, a.V, f[u]);
            else {
#pragma unroll
                for (int j = 0; j < VEC; ++j) f[u][j] = kNegInf;
            }
        }
        float bm = f[0][0];
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
            for (int j = 0; j < VEC; ++j) bm = max_nan(bm, f[u][j]);
        float mn = max_nan(acc.m, bm);
        if (mn == kNegInf) continue;
        float s = 0.f;
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
            for (int j = 0; j < VEC; ++j) s += ex2f((f[u][j] - mn) * c);
        acc.s = acc.s * ex2f((acc.m - mn) * c) + s;
        acc.m = mn;
    }
    MS tot = ms_block(acc, c, sh);
    if (threadIdx.x == 0)
        stats[(((int64_t)b * a.K + k) * 2 + which) * a.nsplit + split] = make_float2(tot.m, tot.s);
}

// Merge the nsplit partials of one row (warp 0 of the block), broadcast via smem.
__device__ __forceinline__ void merged_stats(const RowArgs& a, const float2* stats, int b, int k,
                                             float c, MS* out_p, MS* out_q, MS* sh2) {
    if (threadIdx.x < 32) {
        const float2* sp = stats + (((int64_t)b * a.K + k) * 2) * a.nsplit;
        MS p{kNegInf, 0.f}, q{kNegInf, 0.f};
        if ((int)threadIdx.x < a.nsplit) {
            float2 v = sp[threadIdx.x], w = sp[a.nsplit + threadIdx.x];
            p = MS{v.x, v.y}; q = MS{w.x, w.y};
        }
        p = ms_warp(p, c); q = ms_warp(q, c);
        if (threadIdx.x == 0) { sh2[0] = p; sh2[1] = q; }
    }
    __syncthreads();
    *out_p = sh2[0]; *out_q = sh2[1];
}

// ---------------------------------------------------------------- fp32 sweep 2
// Slice partial of Z = sum max(0, p - q) and of S_aux = sum q 1[q <= p].
template <int DT>
__global__ void __launch_bounds__(kThreads) k_row_tv(RowArgs a, const float2* __restrict__ stats,
                                                     float2* __restrict__ zpart) {
    constexpr int VEC = Elem<DT>::VEC, U = 2;
    __shared__ MS sh2[2];
    __shared__ float shf[kThreads / 32];
    int x = blockIdx.x;
    int split = x % a.nsplit; x /= a.nsplit;
    int k = x % a.K;
    int b = x / a.K;
    if (k >= len_of(a, b)) return;
    float tau = tau_of(a, b);
    if (!tau_ok(tau)) return;
    const float c = kLog2e / tau;
    MS P, Q;
    merged_stats(a, stats, b, k, c, &P, &Q, sh2);
    float2* out = zpart + ((int64_t)b * a.K + k) * a.nsplit + split;
    if (ms_status(P) | ms_status(Q)) { if (threadIdx.x == 0) *out = make_float2(0.f, 0.f); return; }
    const float ip = 1.f / P.s, iq = 1.f / Q.s;
    const char* prow = target_row(a, b, k);
    const char* qrow = draft_row(a, b, k);
    int begin, end;
    slice_range(a.nvec, a.nsplit, split, begin, end);
    float z0 = 0.f, z1 = 0.f, s0 = 0.f, s1 = 0.f;
    for (int i0 = begin + (int)threadIdx.x; i0 < end; i0 += kThreads * U) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            int iv = i0 + u * kThreads;
            if (iv < end) {
                float fp[VEC], fq[VEC];
                load_vec<DT>(prow, iv, a.V, fp);
                load_vec<DT>(qrow, iv, a.V, fq);
#pragma unroll
                for (int j = 0; j < VEC; ++j) {
                    float p = __fmul_rn(ex2f((fp[j] - P.m) * c), ip);
                    float q = __fmul_rn(ex2f((fq[j] - Q.m) * c), iq);
                    float d = fmaxf(p - q, 0.f);
                    float sq = (q <= p) ? q : 0.f;
                    if (j & 1) { z1 += d; s1 += sq; } else { z0 += d; s0 += sq; }
                }
            }
        }
    }
    float z = sum_block(z0 + z1, shf);
    float s = sum_block(s0 + s1, shf);
    if (threadIdx.x == 0) *out = make_float2(z, s);
}

// ------------------------------------------------------------------ accept scan
// One warp per sequence, lane k owns draft position k: gathers p(x_k), q(x_k),
// tests u*q < p in double, finds the first reject with a ballot, writes TV.
__global__ void __launch_bounds__(128) k_accept(RowArgs a, const float2* __restrict__ stats,
                                                const float2* __restrict__ zpart, VerifyOut o,
                                                const int32_t* __restrict__ draft_tokens,
                                                const float* __restrict__ u_accept,
                                                int* __restrict__ stop, int dt) {
    int b = (int)((blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5);
    int lane = threadIdx.x & 31;
    if (b >= a.B) return;
    const int K = a.K, L = len_of(a, b);
    float tau = tau_of(a, b);
    const bool active = lane < L;
    int tok = active ? draft_tokens[(int64_t)b * K + lane] : 0;
    // precedence of the fatal conditions: bad temperature, then bad token id, then the
    // first position whose rows are non-finite or empty
    int st = 0;
    if (!tau_ok(tau)) st = ST_BAD_TEMP;
    else if (__ballot_sync(0xffffffffu, active && (tok < 0 || tok >= a.V))) st = ST_BAD_TOKEN;
    MS P{0.f, 1.f}, Q{0.f, 1.f};
    float z = 0.f;
    int row_st = 0;
    if (active && st == 0) {
        const float c = kLog2e / tau;
        const float2* sp = stats + (((int64_t)b * K + lane) * 2) * a.nsplit;
        const float2* zp = zpart + ((int64_t)b * K + lane) * a.nsplit;
        P = MS{kNegInf, 0.f}; Q = MS{kNegInf, 0.f};
        for (int s = 0; s < a.nsplit; ++s) {
            float2 v = sp[s], w = sp[a.nsplit + s];
            P = ms_merge(P, MS{v.x, v.y}, c);
            Q = ms_merge(Q, MS{w.x, w.y}, c);
            z += zp[s].x;
        }
        row_st = ms_status(P) | ms_status(Q);
    }
    {
        unsigned badrows = __ballot_sync(0xffffffffu, row_st != 0);
        if (badrows) st |= __shfl_sync(0xffffffffu, row_st, __ffs(badrows) - 1);
    }
    if (st & ST_FATAL) {
        if (lane < K) {
            if (o.tv) o.tv[(int64_t)b * K + lane] = 0.f;
            if (o.p_draft) o.p_draft[(int64_t)b * K + lane] = 0.f;
            if (o.q_draft) o.q_draft[(int64_t)b * K + lane] = 0.f;
        }
        for (int j = lane; j <= K; j += 32) o.out_tokens[(int64_t)b * (K + 1) + j] = -1;
        if (lane == 0) { o.accept_len[b] = 0; stop[b] = -1; if (o.row_status) o.row_status[b] = st; }
        return;
    }
    double px = 0.0, qx = 0.0;
    bool acc = false;
    if (active) {
        const double td = (double)tau;
        float zpx = dt == 0 ? load_one<0>(target_row(a, b, lane), tok) : load_one<1>(target_row(a, b, lane), tok);
        float zqx = dt == 0 ? load_one<0>(draft_row(a, b, lane), tok) : load_one<1>(draft_row(a, b, lane), tok);
        px = exp(((double)zpx - (double)P.m) / td) / (double)P.s;
        qx = exp(((double)zqx - (double)Q.m) / td) / (double)Q.s;
        acc = (double)u_accept[(int64_t)b * K + lane] * qx < px;
    }
    unsigned rej = __ballot_sync(0xffffffffu, active && !acc);
    int n = rej ? (__ffs(rej) - 1) : L;
    if (lane < K) {
        if (o.tv) o.tv[(int64_t)b * K + lane] = active ? fminf(fmaxf(z, 0.f), 1.f) : 0.f;
        if (o.p_draft) o.p_draft[(int64_t)b * K + lane] = (float)px;
        if (o.q_draft) o.q_draft[(int64_t)b * K + lane] = (float)qx;
    }
    for (int j = lane; j <= K; j += 32) o.out_tokens[(int64_t)b * (K + 1) + j] = j < n ? tok : -1;
    if (lane == 0) { o.accept_len[b] = n; stop[b] = n; if (o.row_status) o.row_status[b] = st; }
}

// ------------------------------------------------------------------ fp64 draw
struct DrawRow {
    const char* prow; const char* qrow;
    double inv_tau, mp, ip, mq, iq;
    bool resid;
};

// residual (or bonus) mass of the VEC elements of vector iv, in double
template <int DT>
__device__ __forceinline__ void draw_vec(const DrawRow& d, int iv, int V, double* r) {
    constexpr int VEC = Elem<DT>::VEC;
    float fp[VEC], fq[VEC];
    load_vec<DT>(d.prow, iv, V, fp);
    if (d.resid) load_vec<DT>(d.qrow, iv, V, fq);
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
        // explicit roundings: a contracted p*ip - q would leave rounding dust when p == q
        double p = __dmul_rn(exp((double)fp[j] * d.inv_tau - d.mp), d.ip);
        if (d.resid) {
            double q = __dmul_rn(exp((double)fq[j] * d.inv_tau - d.mq), d.iq);
            double df = p - q;
            r[j] = df > 0.0 ? df : 0.0;
        } else {
            r[j] = p;
        }
    }
}

__device__ __forceinline__ bool draw_setup(const RowArgs& a, const int* stop, int b, int* n_out,
                                           bool* resid, const char** prow, const char** qrow) {
    int n = stop[b];
    if (n < 0) return false;
    int L = len_of(a, b);
    *n_out = n;
    *resid = n < L;
    *prow = target_row(a, b, n);
    *qrow = *resid ? draft_row(a, b, n) : nullptr;
    return true;
}

// (m, S) in double of one slice of the stop row(s): S = sum exp(z/tau - m).
template <int DT>
__device__ __forceinline__ void draw_stats_body(const RowArgs& a, const int* __restrict__ stop, int b,
                                                int split, int nsplit_d, double2* __restrict__ dstats,
                                                double* shm, double* shs) {
    constexpr int VEC = Elem<DT>::VEC;
    int n; bool resid; const char *prow, *qrow;
    if (!draw_setup(a, stop, b, &n, &resid, &prow, &qrow)) return;
    const double inv_tau = 1.0 / (double)tau_of(a, b);
    int begin, end;
    slice_range(a.nvec, nsplit_d, split, begin, end);
    for (int which = 0; which < (resid ? 2 : 1); ++which) {
        const char* row = which ? qrow : prow;
        MSd acc{-INFINITY, 0.0};
        for (int iv = begin + (int)threadIdx.x; iv < end; iv += kThreads) {
            float f[VEC];
            load_vec<DT>(row, iv, a.V, f);
            float bmf = f[0];
#pragma unroll
            for (int j = 1; j < VEC; ++j) bmf = max_nan(bmf, f[j]);
            double bm = (double)bmf * inv_tau;
            double mn = (bm != bm || acc.m != acc.m) ? (bm + acc.m) : fmax(acc.m, bm);
            if (mn == -INFINITY) continue;
            double s = 0.0;
#pragma unroll
            for (int j = 0; j < VEC; ++j) s += exp((double)f[j] * inv_tau - mn);
            acc.s = acc.s * exp(acc.m - mn) + s;
            acc.m = mn;
        }
        // block merge
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            MSd w;
            w.m = __shfl_xor_sync(0xffffffffu, acc.m, off);
            w.s = __shfl_xor_sync(0xffffffffu, acc.s, off);
            acc = msd_merge(acc, w);
        }
        int wid = threadIdx.x >> 5, l = threadIdx.x & 31;
        if (l == 0) { shm[wid] = acc.m; shs[wid] = acc.s; }
        __syncthreads();
        if (threadIdx.x == 0) {
            MSd t{shm[0], shs[0]};
            for (int i = 1; i < kThreads / 32; ++i) t = msd_merge(t, MSd{shm[i], shs[i]});
            // store the partial against an integer power of two, sum = s2 * 2^e, so that the merge of
            // the slices is an exact rescaling (no exponentials)
            double e = t.m, s2 = t.s;
            if (t.m == t.m && t.m != INFINITY && t.m != -INFINITY) {
                e = ceil(t.m * 1.4426950408889634);
                s2 = t.s * exp(t.m - e * 0.6931471805599453);
            }
            dstats[((int64_t)b * 2 + which) * nsplit_d + split] = make_double2(e, s2);
        }
        __syncthreads();
    }
}

// Sequences to draw for: all B, or the entries of a device-side list.
struct DrawList {
    const int* list;    // nullptr: every sequence 0..B-1
    const int* count;   // number of list entries (device memory)
};
__device__ __forceinline__ int draw_items(const DrawList& dl, int B) { return dl.list ? min(*dl.count, B) : B; }
__device__ __forceinline__ int draw_seq(const DrawList& dl, int i) { return dl.list ? dl.list[i] : i; }

template <int DT>
__global__ void __launch_bounds__(kThreads) k_draw_stats(RowArgs a, const int* __restrict__ stop,
                                                         int nsplit_d, double2* __restrict__ dstats,
                                                         DrawList dl) {
    __shared__ double shm[kThreads / 32], shs[kThreads / 32];
    const int split = blockIdx.x % nsplit_d, items = draw_items(dl, a.B);
    for (int i = blockIdx.x / nsplit_d; i < items; i += gridDim.x / nsplit_d)
        draw_stats_body<DT>(a, stop, draw_seq(dl, i), split, nsplit_d, dstats, shm, shs);
}

// Merge the fp64 partials of the stop row(s); returns status bits.
__device__ __forceinline__ int draw_merge(const double2* dstats, int b, int nsplit_d, bool resid,
                                          DrawRow* d) {
    // partials are (e, s2) with sum = s2 * 2^e, e an integer (or NaN / +-inf for a bad or empty slice)
    MSd P{-INFINITY, 0.0}, Q{-INFINITY, 0.0};
    const double2* sp = dstats + (int64_t)b * 2 * nsplit_d;
    for (int w = 0; w < (resid ? 2 : 1); ++w) {
        double em = -INFINITY;
        bool nan = false;
        for (int s = 0; s < nsplit_d; ++s) { const double e = sp[w * nsplit_d + s].x; if (e != e) nan = true; else em = fmax(em, e); }
        double sum = 0.0;
        if (!nan && em != INFINITY && em != -INFINITY)
            for (int s = 0; s < nsplit_d; ++s) {
                const double2 v = sp[w * nsplit_d + s];
                if (v.x != -INFINITY) sum += scalbn(v.y, (int)fmax(v.x - em, -2000.0));
            }
        MSd& R_ = w ? Q : P;
        R_.m = nan ? NAN : (em == INFINITY || em == -INFINITY ? em : em * 0.6931471805599453);
        R_.s = (nan || em == INFINITY) ? NAN : sum;
    }
    int st = 0;
    if (P.m != P.m || P.m == INFINITY || P.s != P.s) st |= ST_NONFINITE;
    else if (P.m == -INFINITY) st |= ST_EMPTY;
    if (resid) {
        if (Q.m != Q.m || Q.m == INFINITY || Q.s != Q.s) st |= ST_NONFINITE;
        else if (Q.m == -INFINITY) st |= ST_EMPTY;
    }
    d->mp = P.m; d->ip = 1.0 / P.s; d->mq = Q.m; d->iq = resid ? 1.0 / Q.s : 0.0;
    return st;
}

template <int DT>
__device__ __forceinline__ double slice_mass(const DrawRow& d, int V, int begin, int end, double* sh) {
    constexpr int VEC = Elem<DT>::VEC;
    double acc = 0.0;
    for (int iv = begin + (int)threadIdx.x; iv < end; iv += kThreads) {
        double r[VEC];
        draw_vec<DT>(d, iv, V, r);
#pragma unroll
        for (int j = 0; j < VEC; ++j) acc += r[j];
    }
    return sum_block(acc, sh);
}

template <int DT>
__device__ __forceinline__ void draw_mass_body(const RowArgs& a, const int* __restrict__ stop, int b,
                                               int split, int nsplit_d, const double2* __restrict__ dstats,
                                               double* __restrict__ dmass, double* sh) {
    int n; DrawRow d;
    if (!draw_setup(a, stop, b, &n, &d.resid, &d.prow, &d.qrow)) return;
    d.inv_tau = 1.0 / (double)tau_of(a, b);
    int st = draw_merge(dstats, b, nsplit_d, d.resid, &d);
    double* out = dmass + (int64_t)b * nsplit_d + split;
    if (st) { if (threadIdx.x == 0) *out = 0.0; return; }
    int begin, end;
    slice_range(a.nvec, nsplit_d, split, begin, end);
    double m = slice_mass<DT>(d, a.V, begin, end, sh);
    if (threadIdx.x == 0) *out = m;
}

template <int DT>
__global__ void __launch_bounds__(kThreads) k_draw_mass(RowArgs a, const int* __restrict__ stop,
                                                        int nsplit_d, const double2* __restrict__ dstats,
                                                        double* __restrict__ dmass, DrawList dl) {
    __shared__ double sh[kThreads / 32];
    const int split = blockIdx.x % nsplit_d, items = draw_items(dl, a.B);
    for (int i = blockIdx.x / nsplit_d; i < items; i += gridDim.x / nsplit_d)
        draw_mass_body<DT>(a, stop, draw_seq(dl, i), split, nsplit_d, dstats, dmass, sh);
}

// Locate y = min{v : C(v) >= u * Z}: slice from the partials, thread chunk by a
// scan of chunk sums, element by a sequential walk.  One block per sequence.
struct PickShared {
    double sh[kThreads / 32];
    double part[32];
    double cs[kThreads];
    double t, c0;
    int split, thread;
};

template <int DT>
__device__ __forceinline__ void draw_pick_body(const RowArgs& a, const int* __restrict__ stop, int b,
                                               int nsplit_d, const double2* __restrict__ dstats,
                                               const double* __restrict__ dmass,
                                               const float* __restrict__ u_final, const VerifyOut& o,
                                               PickShared& S) {
    constexpr int VEC = Elem<DT>::VEC;
    double* sh = S.sh; double* part = S.part; double* cs = S.cs;
    double& sh_t = S.t; double& sh_c0 = S.c0; int& sh_split = S.split; int& sh_thread = S.thread;
    const int K = a.K;
    int n; DrawRow d;
    if (!draw_setup(a, stop, b, &n, &d.resid, &d.prow, &d.qrow)) return;
    d.inv_tau = 1.0 / (double)tau_of(a, b);
    int st = draw_merge(dstats, b, nsplit_d, d.resid, &d);
    if (st & ST_FATAL) {   // only the bonus row can still turn out bad here
        if ((int)threadIdx.x < K) {
            if (o.tv) o.tv[(int64_t)b * K + threadIdx.x] = 0.f;
            if (o.p_draft) o.p_draft[(int64_t)b * K + threadIdx.x] = 0.f;
            if (o.q_draft) o.q_draft[(int64_t)b * K + threadIdx.x] = 0.f;
        }
        if ((int)threadIdx.x <= K) o.out_tokens[(int64_t)b * (K + 1) + threadIdx.x] = -1;
        if (threadIdx.x == 0) { o.accept_len[b] = 0; if (o.row_status) o.row_status[b] |= st; }
        return;
    }
    if ((int)threadIdx.x < nsplit_d) part[threadIdx.x] = dmass[(int64_t)b * nsplit_d + threadIdx.x];
    __syncthreads();
    double Z = 0.0;
    for (int s = 0; s < nsplit_d; ++s) Z += part[s];
    if (!(Z > 0.0) && d.resid) {
        // residual mass vanished at a rejected position: draw from p of that position
        d.resid = false;
        __syncthreads();
        for (int s = 0; s < nsplit_d; ++s) {
            int sb, se;
            slice_range(a.nvec, nsplit_d, s, sb, se);
            double m = slice_mass<DT>(d, a.V, sb, se, sh);
            if (threadIdx.x == 0) part[s] = m;
        }
        __syncthreads();
        Z = 0.0;
        for (int s = 0; s < nsplit_d; ++s) Z += part[s];
        if (threadIdx.x == 0 && o.row_status) o.row_status[b] |= ST_ZERO_RESID;
    }
    if (threadIdx.x == 0) {
        double t = (double)u_final[b] * Z, C = 0.0;
        int sel = -1;
        for (int s = 0; s < nsplit_d; ++s) {
            if (C + part[s] >= t) { sel = s; break; }
            C += part[s];
        }
        if (sel < 0) {   // rounding only: take the last slice that holds mass
            C = 0.0;
            int last = 0;
            for (int s = 0; s < nsplit_d; ++s) if (part[s] > 0.0) last = s;
            for (int s = 0; s < last; ++s) C += part[s];
            sel = last;
        }
        sh_t = t; sh_c0 = C; sh_split = sel;
    }
    __syncthreads();
    int begin, end;
    slice_range(a.nvec, nsplit_d, sh_split, begin, end);
    const int per = (end - begin + kThreads - 1) / kThreads;
    const int cb = min(begin + (int)threadIdx.x * per, end), ce = min(cb + per, end);
    double mine = 0.0;
    for (int iv = cb; iv < ce; ++iv) {
        double r[VEC];
        draw_vec<DT>(d, iv, a.V, r);
#pragma unroll
        for (int j = 0; j < VEC; ++j) mine += r[j];
    }
    cs[threadIdx.x] = mine;
    __syncthreads();
    if (threadIdx.x == 0) {
        double C = sh_c0;
        int sel = -1;
        for (int j = 0; j < kThreads; ++j) {
            if (cs[j] > 0.0 && C + cs[j] >= sh_t) { sel = j; break; }
            C += cs[j];
        }
        if (sel < 0) {
            C = sh_c0;
            int last = 0;
            for (int j = 0; j < kThreads; ++j) if (cs[j] > 0.0) last = j;
            for (int j = 0; j < last; ++j) C += cs[j];
            sel = last;
        }
        sh_c0 = C; sh_thread = sel;
    }
    __syncthreads();
    if ((int)threadIdx.x == sh_thread) {
        double C = sh_c0;
        const double t = sh_t;
        int y = -1, lastpos = -1;
        for (int iv = cb; iv < ce && y < 0; ++iv) {
            double r[VEC];
            draw_vec<DT>(d, iv, a.V, r);
#pragma unroll
            for (int j = 0; j < VEC; ++j) {
                if (y < 0) {
                    C += r[j];
                    if (r[j] > 0.0) lastpos = iv * VEC + j;
                    if (C >= t && r[j] > 0.0) y = iv * VEC + j;
                }
            }
        }
        if (y < 0) y = lastpos;
        o.out_tokens[(int64_t)b * (K + 1) + n] = y;
    }
}

template <int DT>
__global__ void __launch_bounds__(kThreads) k_draw_pick(RowArgs a, const int* __restrict__ stop,
                                                        int nsplit_d, const double2* __restrict__ dstats,
                                                        const double* __restrict__ dmass,
                                                        const float* __restrict__ u_final, VerifyOut o,
                                                        DrawList dl) {
    __shared__ PickShared S;
    const int items = draw_items(dl, a.B);
    for (int i = blockIdx.x; i < items; i += gridDim.x) {
        draw_pick_body<DT>(a, stop, draw_seq(dl, i), nsplit_d, dstats, dmass, u_final, o, S);
        __syncthreads();
    }
}

// ---------------------------------------------------------------------- TV only
__global__ void k_tv_finalize(RowArgs a, const float2* __restrict__ stats,
                              const float2* __restrict__ zpart, float* __restrict__ tv,
                              float* __restrict__ s_aux, int32_t* __restrict__ row_status) {
    int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= a.B) return;
    float tau = tau_of(a, n);
    int st = tau_ok(tau) ? 0 : ST_BAD_TEMP;
    float z = 0.f, s = 0.f;
    if (!st) {
        const float c = kLog2e / tau;
        MS P{kNegInf, 0.f}, Q{kNegInf, 0.f};
        const float2* sp = stats + (int64_t)n * 2 * a.nsplit;
        const float2* zp = zpart + (int64_t)n * a.nsplit;
        for (int i = 0; i < a.nsplit; ++i) {
            P = ms_merge(P, MS{sp[i].x, sp[i].y}, c);
            Q = ms_merge(Q, MS{sp[a.nsplit + i].x, sp[a.nsplit + i].y}, c);
            z += zp[i].x; s += zp[i].y;
        }
        st = ms_status(P) | ms_status(Q);
    }
    if (st) { z = 0.f; s = 0.f; }
    tv[n] = fminf(fmaxf(z, 0.f), 1.f);
    if (s_aux) s_aux[n] = s;
    if (row_status) row_status[n] = st;
}

// ----------------------------------------------------------------------- greedy
// Slice argmax (value, lowest index) of one target row; NaN / +inf poison it.
template <int DT>
__global__ void __launch_bounds__(kThreads) k_argmax(RowArgs a, float2* __restrict__ amax) {
    constexpr int VEC = Elem<DT>::VEC;
    __shared__ float shv[kThreads / 32];
    __shared__ int shi[kThreads / 32];
    int x = blockIdx.x;
    int split = x % a.nsplit; x /= a.nsplit;
    int k = x % (a.K + 1);
    int b = x / (a.K + 1);
    if (k > len_of(a, b)) return;
    const char* row = target_row(a, b, k);
    int begin, end;
    slice_range(a.nvec, a.nsplit, split, begin, end);
    float best = kNegInf;
    int bidx = INT_MAX;
    bool bad = false;
    // branch-free over the vectors (so that several loads are on their way per thread): the best vector first,
    // the index inside it from one more look at that vector
    int bvec = -1;
#pragma unroll 4
    for (int iv = begin + (int)threadIdx.x; iv < end; iv += kThreads) {
        float f[VEC];
        load_vec<DT>(row, iv, a.V, f);
        float vm = f[0];
#pragma unroll
        for (int j = 1; j < VEC; ++j) vm = max_nan(vm, f[j]);
        bad = bad || !(vm < INFINITY);                 // NaN or +inf
        const bool better = vm > best;                 // strictly: the lowest vector wins a tie
        best = better ? vm : best;
        bvec = better ? iv : bvec;
    }
    if (bvec >= 0) {
        float f[VEC];
        load_vec<DT>(row, bvec, a.V, f);
        int jj = 0;
#pragma unroll
        for (int j = VEC - 1; j >= 0; --j) if (f[j] == best) jj = j;
        bidx = bvec * VEC + jj;
    }
    if (bad) { best = __int_as_float(0x7fc00000); bidx = INT_MAX; }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        float ov = __shfl_xor_sync(0xffffffffu, best, off);
        int oi = __shfl_xor_sync(0xffffffffu, bidx, off);
        bool take = (ov != ov) || (!(best != best) && (ov > best || (ov == best && oi < bidx)));
        if (take) { best = ov; bidx = oi; }
    }
    int w = threadIdx.x >> 5, l = threadIdx.x & 31;
    if (l == 0) { shv[w] = best; shi[w] = bidx; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < kThreads / 32; ++i) {
            float ov = shv[i]; int oi = shi[i];
            bool take = (ov != ov) || (!(best != best) && (ov > best || (ov == best && oi < bidx)));
            if (take) { best = ov; bidx = oi; }
        }
        amax[((int64_t)b * (a.K + 1) + k) * a.nsplit + split] = make_float2(best, __int_as_float(bidx));
    }
}

__global__ void __launch_bounds__(128) k_greedy_finalize(RowArgs a, const float2* __restrict__ amax,
                                                         const int32_t* __restrict__ draft_tokens,
                                                         int32_t* __restrict__ accept_len,
                                                         int32_t* __restrict__ out_tokens,
                                                         int32_t* __restrict__ row_status) {
    int b = (int)((blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5);
    int lane = threadIdx.x & 31;
    if (b >= a.B) return;
    const int K = a.K, L = len_of(a, b);
    int st = 0;
    int tok = lane < L ? draft_tokens[(int64_t)b * K + lane] : -1;
    if (lane < L && (tok < 0 || tok >= a.V)) st |= ST_BAD_TOKEN;
    // lanes 0..L merge the target rows 0..L (two rounds when L + 1 > 32)
    int g = -1, g_bonus = -1;
    for (int round = 0; round < 2; ++round) {
        int k = round == 0 ? lane : 32 + lane;
        if (k <= L && k <= K) {
            const float2* ap = amax + ((int64_t)b * (K + 1) + k) * a.nsplit;
            float best = kNegInf; int bidx = INT_MAX;
            for (int s = 0; s < a.nsplit; ++s) {
                float ov = ap[s].x; int oi = __float_as_int(ap[s].y);
                if (ov != ov) { best = ov; break; }
                if (ov > best) { best = ov; bidx = oi; }
            }
            if (best != best) st |= ST_NONFINITE;
            else if (best == kNegInf) st |= ST_EMPTY;
            if (round == 0) g = bidx; else g_bonus = bidx;
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) st |= __shfl_xor_sync(0xffffffffu, st, off);
    if (st & ST_FATAL) {
        if (lane <= K) out_tokens[(int64_t)b * (K + 1) + lane] = -1;
        if (K == 32 && lane == 0) out_tokens[(int64_t)b * (K + 1) + 32] = -1;
        if (lane == 0) { accept_len[b] = 0; if (row_status) row_status[b] = st; }
        return;
    }
    unsigned mis = __ballot_sync(0xffffffffu, lane < L && tok != g);
    int n = mis ? (__ffs(mis) - 1) : L;
    int y = n < 32 ? __shfl_sync(0xffffffffu, g, n & 31) : __shfl_sync(0xffffffffu, g_bonus, 0);
    if (lane <= K && lane < 32) out_tokens[(int64_t)b * (K + 1) + lane] = lane < n ? tok : (lane == n ? y : -1);
    if (K == 32 && lane == 0) out_tokens[(int64_t)b * (K + 1) + 32] = (n == 32) ? y : -1;
    if (lane == 0) { accept_len[b] = n; if (row_status) row_status[b] = st; }
}

}  // namespace

// ---------------------------------------------------------------------- launchers
#define LAUNCH_DT(dt, kern, grid, block, stream, ...)                                   \
    do {                                                                                \
        if ((dt) == 0) kern<0><<<(grid), (block), 0, (stream)>>>(__VA_ARGS__);          \
        else kern<1><<<(grid), (block), 0, (stream)>>>(__VA_ARGS__);                    \
    } while (0)

cudaError_t general_verify(const RowArgs& a, const Plan& p, const int32_t* draft_tokens,
                           const float* u_accept, const float* u_final, VerifyOut o, char* ws,
                           cudaStream_t stream) {
    float2* stats = reinterpret_cast<float2*>(ws + p.off_stats);
    float2* zpart = reinterpret_cast<float2*>(ws + p.off_zpart);
    int* stop = reinterpret_cast<int*>(ws + p.off_stop);
    double2* dstats = reinterpret_cast<double2*>(ws + p.off_dstats);
    double* dmass = reinterpret_cast<double*>(ws + p.off_dmass);
    if (a.K > 0) {
        LAUNCH_DT(a.dt, k_row_stats, (unsigned)((int64_t)a.B * 2 * a.K * a.nsplit), kThreads, stream, a, stats);
        LAUNCH_DT(a.dt, k_row_tv, (unsigned)((int64_t)a.B * a.K * a.nsplit), kThreads, stream, a, stats, zpart);
    }
    k_accept<<<(a.B + 3) / 4, 128, 0, stream>>>(a, stats, zpart, o, draft_tokens, u_accept, stop, a.dt);
    DrawList all{nullptr, nullptr};
    LAUNCH_DT(a.dt, k_draw_stats, (unsigned)((int64_t)a.B * p.nsplit_d), kThreads, stream, a, stop, p.nsplit_d, dstats, all);
    LAUNCH_DT(a.dt, k_draw_mass, (unsigned)((int64_t)a.B * p.nsplit_d), kThreads, stream, a, stop, p.nsplit_d, dstats, dmass, all);
    LAUNCH_DT(a.dt, k_draw_pick, (unsigned)a.B, kThreads, stream, a, stop, p.nsplit_d, dstats, dmass, u_final, o, all);
    return cudaGetLastError();
}

cudaError_t general_tv(const RowArgs& a, const Plan& p, float* tv, float* s_aux, int32_t* row_status,
                       char* ws, cudaStream_t stream) {
    float2* stats = reinterpret_cast<float2*>(ws + p.off_stats);
    float2* zpart = reinterpret_cast<float2*>(ws + p.off_zpart);
    LAUNCH_DT(a.dt, k_row_stats, (unsigned)((int64_t)a.B * 2 * a.nsplit), kThreads, stream, a, stats);
    LAUNCH_DT(a.dt, k_row_tv, (unsigned)((int64_t)a.B * a.nsplit), kThreads, stream, a, stats, zpart);
    k_tv_finalize<<<(a.B + 127) / 128, 128, 0, stream>>>(a, stats, zpart, tv, s_aux, row_status);
    return cudaGetLastError();
}

cudaError_t general_greedy(const RowArgs& a, const Plan& p, const int32_t* draft_tokens,
                           int32_t* accept_len, int32_t* out_tokens, int32_t* row_status, char* ws,
                           cudaStream_t stream) {
    float2* amax = reinterpret_cast<float2*>(ws + p.off_amax);
    LAUNCH_DT(a.dt, k_argmax, (unsigned)((int64_t)a.B * (a.K + 1) * a.nsplit), kThreads, stream, a, amax);
    k_greedy_finalize<<<(a.B + 3) / 4, 128, 0, stream>>>(a, amax, draft_tokens, accept_len, out_tokens, row_status);
    return cudaGetLastError();
}

}  // namespace bebop
