// Wave kernel: the hot path of bebop_verify as one persistent, ticket-scheduled
// kernel whose tasks never wait for each other in practice.
//
// The batch is cut into WAVES of a few sequences (about 20 MB of logits, a
// fraction of the 126 MB L2).  Each wave goes through four phases:
//
//   P1  one task per (row, slice): stream a slice of ONE logit row from HBM with
//       128-bit loads and compute its softmax partial (E, S): S = sum 2^(x*c - E)
//       relative to a power-of-two reference, one exponential per logit;
//   A   one task per sequence: merge the partials of its 2K+1 rows exactly
//       (integer exponents, fp64 sums), run the accept scan (u*q(x) < p(x)),
//       write accept_len, the accepted tokens, p(x), q(x), the status, and leave
//       the row normalisers for the next phase;
//   P2  one task per (row pair, slice): read both rows again -- from L2, the wave
//       was streamed moments ago -- and accumulate TV = sum max(0, p - q); at the
//       stop row (or the bonus row when every draft was accepted) also the slice's
//       residual mass in double and the sum of squares for the error bound;
//   D   one task per sequence: add the TV parts in slice order; locate the slice
//       holding the inverse-CDF crossing, re-scan that slice (per-vector sums, block
//       scan, eight-token walk) and keep the token only if the crossing clears the
//       error bound of draw_bound(); otherwise the sequence goes to the list that
//       the fp64 kernels re-draw.
//
// Tickets are handed out in an order that puts LAG waves of P1 work between a
// phase and the phase it depends on (P1(w) .. P1(w+LAG), A(w), P2(w), D(w-1) ..),
// so by the time a CTA picks a dependent task its inputs are long complete, while
// the wave is still in L2.  A task that does arrive early spins (bounded) on the
// wave's completion counter; tasks only ever wait for earlier tickets, so the
// schedule cannot deadlock.  DRAM sees every logit once; the exponential pipe sees
// it twice.
#include "bebop_kernels.h"
#include "bebop_ptx.cuh"

namespace bebop {

namespace {

constexpr int WT = 256;               // threads per CTA
constexpr int WW = WT / 32;
constexpr int SLICE_VECS = kWaveSliceVecs;   // vectors per row slice, at most (8 per thread)
constexpr int BEBOP_MAX_K_INT = 32;
constexpr int MAX_SLICES = 64;
constexpr int E_EMPTY = INT_MIN / 2;
constexpr uint32_t kSpin = 1u << 22;

struct __align__(16) P1Part { double s; int e; float m; };             // per (row, slice); m = NaN marks a non-finite logit
struct __align__(16) RowStat { double inv_s; float ef; int e; int pad[2]; };   // per row, after the merge: 1/S, exponent E
struct __align__(16) DPart { double tot; float sq; int pad; };        // per (sequence, slice)
struct __align__(16) SeqInfo {          // per sequence, written by phase A
    int n;                              // accept count (stop position); -1: fatal
    int draw_row;                       // row whose residual is drawn from (n, or L for the bonus row); -1 none
    int pad0;
    int pad;
};

struct WaveArgs {
    RowArgs r;
    const int32_t* draft_tokens;
    const float* u_accept;
    const float* u_final;
    VerifyOut o;
    int* stop;
    int* fb_count;
    int* fb_list;
    // workspace
    int* ticket;          // [1]
    int* wait_failed;     // [1]
    int* p1done;          // [nwaves]
    int* adone;           // [nwaves]
    int* p2done;          // [nwaves]
    P1Part* part;         // [B][2K+1][T]
    RowStat* rstat;       // [B][2K+1]
    float* zpart;         // [B][K][T]
    DPart* dpart;         // [B][T]
    SeqInfo* sinfo;       // [B]
    int ntickets, lag;
    long long* trace;
    int T, slice_vecs, wave_seqs, nwaves;
};

__device__ __forceinline__ float tau_of(const RowArgs& a, int b) { return a.temperature ? a.temperature[b] : a.temperature_all; }
__device__ __forceinline__ bool tau_ok(float t) { return t > 0.f && t < INFINITY; }
__device__ __forceinline__ int len_of(const RowArgs& a, int b) {
    int L = a.draft_len ? a.draft_len[b] : a.K;
    return max(0, min(L, a.K));
}
__device__ __forceinline__ int ld_acquire(const int* p) {
    int v; asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory"); return v;
}
__device__ __forceinline__ bool spin_ge(const int* p, int want) {
    for (uint32_t i = 0; i < kSpin; ++i) {
        if (ld_acquire(p) >= want) return true;
        __nanosleep(64);
    }
    return false;
}

// The error bound a draw must clear.  The residual is formed from fp32 exponentials (ex2.approx:
// 2 ulp), an fp32 argument (half an ulp of a number below 64, times 2^arg) and one fp32 rounding of
// the product with the two-float normaliser, so each p, q carries a relative error below
// delta = 2^-22; the errors of different tokens are independent, hence the error of a prefix sum is
// of the order delta * sqrt(sum p^2 + q^2), and so is the part common to all tokens, the error of the
// fp32-summed normalisers.  Measured on 40 000 draws with the certification switched off, the largest
// error that changed a token was 0.1 * delta * sqrt(sum p^2 + q^2); kappa = 4 leaves a factor 40 over
// that.
#ifndef BEBOP_KAPPA
#define BEBOP_KAPPA 4.0
#endif
__device__ __forceinline__ double draw_bound(double sumsq) {
    const double delta = 2.384185791015625e-07;   // 2^-22
    return BEBOP_KAPPA * delta * sqrt(sumsq) + 1e-300;
}

// c = log2(e) / tau in fp32, and 2^(x * c - E): the product is exact inside the fma, so the argument
// carries one rounding of half an ulp of itself.  The rounding of c itself acts like a temperature
// changed by at most 2^-24 relative; over a prefix of the vocabulary its effect, 2^-24 * sum p (z - zbar) / tau,
// is a sum of zero-mean terms of the size draw_bound() already allows per token.
struct TempScale { float hi; };
__device__ __forceinline__ TempScale temp_scale(float tau) {
    TempScale r; r.hi = kLog2e / (tau_ok(tau) ? tau : 1.f);
    return r;
}
__device__ __forceinline__ float exp2_scaled(float x, const TempScale& t, float Ef) {
    return ex2f(fmaf(x, t.hi, -Ef));
}
// E = ceil(m * c) of a maximum m, as int and float: any integer near m * c serves as the reference, and
// integer references make every merge of partial sums an exact power-of-two scaling.
__device__ __forceinline__ int ref_exponent(float m, const TempScale& t, float* Ef) {
    const float th = fminf(fmaxf(m * t.hi, -4.0e6f), 4.0e6f);
    return ceil_alu(th, Ef);
}

struct WaveShared {
    float vsum[SLICE_VECS];       // per-vector residual mass (D phase)
    double redd[WW];
    float redf[2][WW];
    int redi[WW];
    int ticket, phase, wave, index;
    // D-phase broadcast
    double base, Ttarget, bound;
    int owner_slice;
};

__device__ __forceinline__ const char* row_ptr(const RowArgs& R, int b, int r) {
    // r in [0, K]: target row r; r in [K+1, 2K]: draft row r - (K+1)
    const int K = R.K;
    return r <= K ? R.target + ((int64_t)b * R.t_seq_rows + r) * R.t_row_bytes
                  : R.draft + ((int64_t)b * R.d_seq_rows + (r - K - 1)) * R.d_row_bytes;
}

// ------------------------------------------------------------------ phase P1
template <int DT>
__device__ __forceinline__ void phase_p1(const WaveArgs& a, WaveShared& S, int b, int r, int s) {
    constexpr int VEC = Elem<DT>::VEC, NV = SLICE_VECS / WT;     // 8 vectors per thread
    const RowArgs& R = a.r;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int L = len_of(R, b), K = R.K;
    const bool is_target = r <= K;
    const int k = is_target ? r : r - (K + 1);
    if (is_target ? k > L : k >= L) return;
    const float tau = tau_of(R, b);
    const TempScale ts = temp_scale(tau);
    const int v0 = s * a.slice_vecs;
    const int nv = max(min(a.slice_vecs, R.nvec - v0), 0);
    const char* row = row_ptr(R, b, r) + (int64_t)v0 * 16;

    // every load of the task is issued before anything is used
    uint4 raw[NV];
#pragma unroll
    for (int u = 0; u < NV; ++u) {
        const int v = tid + u * WT;
        raw[u] = neg_inf_vec<DT>();
        if (v < nv) raw[u] = ldg16_stream(row + (size_t)v * 16);
    }
    if ((v0 + nv) * VEC > R.V) {
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            const int gbase = (v0 + tid + u * WT) * VEC;
            if (tid + u * WT < nv && gbase + VEC > R.V) mask_tail<DT>(raw[u], R.V - gbase);
        }
    }
    float m = vec_max<DT>(raw[0]);
#pragma unroll
    for (int u = 1; u < NV; ++u) m = max_nan(m, vec_max<DT>(raw[u]));
    const bool bad = m != m || m == INFINITY;
    int E = E_EMPTY;
    float Ef = 0.f;
    if (!bad && m != -INFINITY) E = ref_exponent(m, ts, &Ef);
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
    if (E > E_EMPTY) {
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            float f[VEC];
            unpack<DT>(raw[u], f);
#pragma unroll
            for (int i = 0; i < VEC; i += 4) {
                s0 += exp2_scaled(f[i], ts, Ef);
                s1 += exp2_scaled(f[i + 1], ts, Ef);
                s2 += exp2_scaled(f[i + 2], ts, Ef);
                s3 += exp2_scaled(f[i + 3], ts, Ef);
            }
        }
    }
    // thread -> warp -> block, exact power-of-two rescaling, sums in a fixed order
    float st = (s0 + s1) + (s2 + s3);
    const int Ew = redux_max(E);
    st = E > E_EMPTY ? st * pow2f(max(E - Ew, -126)) : 0.f;
    st = warp_sum(st);
    const unsigned anybad = __ballot_sync(0xffffffffu, bad);
    float mw = ord2f(redux_max(f2ord(bad ? -INFINITY : m)));
    if (anybad) mw = __int_as_float(0x7fc00000);
    if (lane == 0) { S.redf[0][warp] = st; S.redi[warp] = Ew; S.redf[1][warp] = mw; }
    __syncthreads();
    if (tid == 0) {
        int Ec = E_EMPTY; float mc = -INFINITY;
        for (int w = 0; w < WW; ++w) { Ec = max(Ec, S.redi[w]); mc = max_nan(mc, S.redf[1][w]); }
        double sum = 0.0;
        for (int w = 0; w < WW; ++w) if (S.redi[w] > E_EMPTY) sum += (double)(S.redf[0][w] * pow2f(max(S.redi[w] - Ec, -126)));
        P1Part p; p.s = (mc != mc) ? 0.0 : sum; p.e = Ec; p.m = mc;
        a.part[((int64_t)b * (2 * K + 1) + r) * a.T + s] = p;
    }
}

// ------------------------------------------------------------------ phase A
// One CTA per sequence; warp w merges rows w, w + WW, ..; thread 0 runs the accept scan.
template <int DT>
__device__ __forceinline__ void phase_a(const WaveArgs& a, WaveShared& S, int b) {
    const RowArgs& R = a.r;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = R.K, V = R.V, L = len_of(R, b), NR = 2 * K + 1, T = a.T;
    const float tau = tau_of(R, b);
    const bool ok = tau_ok(tau);
    const TempScale ts = temp_scale(tau);
    __shared__ int sh_status[2 * BEBOP_MAX_K_INT + 1];
    __shared__ double sh_S[2 * BEBOP_MAX_K_INT + 1];
    __shared__ int sh_E[2 * BEBOP_MAX_K_INT + 1];
    __shared__ float sh_M[2 * BEBOP_MAX_K_INT + 1];
    for (int r = warp; r < NR; r += WW) {
        const bool is_target = r <= K;
        const int k = is_target ? r : r - (K + 1);
        const bool used = is_target ? k <= L : k < L;
        int Em = E_EMPTY, fl = 0;
        double sum = 0.0;
        float mrow = -INFINITY;
        if (used) {
            const P1Part* pp = a.part + ((int64_t)b * NR + r) * T;
            // lanes take slices in order; exponent first, then the scaled sum in a fixed tree
            int e_l = E_EMPTY; double s_l = 0.0; int f_l = 0; float m_l = -INFINITY;
            P1Part mine[2];
            int cnt = 0;
            for (int s = lane; s < T && cnt < 2; s += 32) {
                mine[cnt] = pp[s]; e_l = max(e_l, mine[cnt].e);
                if (mine[cnt].m != mine[cnt].m) f_l = 1; else m_l = fmaxf(m_l, mine[cnt].m);
                cnt++;
            }
            Em = redux_max(e_l);
            mrow = ord2f(redux_max(f2ord(m_l)));
            for (int i = 0; i < cnt; ++i) if (mine[i].e > E_EMPTY) s_l += mine[i].s * pow2d(max(mine[i].e - Em, -1000));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) { s_l += shfl_xor_d(s_l, o); f_l |= __shfl_xor_sync(0xffffffffu, f_l, o); }
            sum = s_l; fl = f_l;
        }
        if (lane == 0) {
            int st = 0;
            if (used) { if (fl || !(sum == sum)) st = ST_NONFINITE; else if (Em == E_EMPTY) st = ST_EMPTY; }
            sh_status[r] = st; sh_S[r] = sum; sh_E[r] = Em; sh_M[r] = mrow;
        }
    }
    __syncthreads();
    if (warp == 0) {
        // lane k owns draft position k (K <= 32): tokens, gathered logits, accept bit; ballots give the chain
        const bool active = lane < L;
        const int tk = active ? a.draft_tokens[(int64_t)b * K + lane] : 0;
        int seq_st = ok ? 0 : ST_BAD_TEMP;
        if (!seq_st && __ballot_sync(0xffffffffu, active && (tk < 0 || tk >= V))) seq_st = ST_BAD_TOKEN;
        // the first bad row pair decides the status; rows after it do not count
        const int rs = active ? (sh_status[lane] | sh_status[K + 1 + lane]) : 0;
        const unsigned badrows = __ballot_sync(0xffffffffu, rs != 0);
        const int first_bad = badrows ? __ffs(badrows) - 1 : 32;
        if (!seq_st && badrows) seq_st = __shfl_sync(0xffffffffu, rs, first_bad);
        double px = 0.0, qx = 0.0;
        bool acc = false;
        if (active && !(seq_st & ST_FATAL) && lane < first_bad) {
            const float zpx = DT == 0 ? load_one<0>(row_ptr(R, b, lane), tk) : load_one<1>(row_ptr(R, b, lane), tk);
            const float zqx = DT == 0 ? load_one<0>(row_ptr(R, b, K + 1 + lane), tk) : load_one<1>(row_ptr(R, b, K + 1 + lane), tk);
            const double cd = (double)ts.hi;
            px = exp2((double)zpx * cd - (double)sh_E[lane]) / sh_S[lane];
            qx = exp2((double)zqx * cd - (double)sh_E[K + 1 + lane]) / sh_S[K + 1 + lane];
            acc = (double)a.u_accept[(int64_t)b * K + lane] * qx < px;
        }
        const unsigned rej = __ballot_sync(0xffffffffu, active && !acc);
        int n = rej ? __ffs(rej) - 1 : L;
        if (!(seq_st & ST_FATAL) && n == L && sh_status[L]) seq_st |= sh_status[L];   // bonus row, read only now
        const bool fatal = (seq_st & ST_FATAL) != 0;
        const int nn = fatal ? 0 : n;
        // outputs: lane q writes position q (position nn is filled by the draw)
        for (int q = lane; q <= K; q += 32)
            if (fatal || q != nn) a.o.out_tokens[(int64_t)b * (K + 1) + q] = q < nn ? tk : -1;   // q < nn <= 32: q == lane
        if (lane < K) {
            const bool zero = fatal || lane >= L;
            if (a.o.p_draft) a.o.p_draft[(int64_t)b * K + lane] = zero ? 0.f : (float)px;
            if (a.o.q_draft) a.o.q_draft[(int64_t)b * K + lane] = zero ? 0.f : (float)qx;
            if (zero && a.o.tv) a.o.tv[(int64_t)b * K + lane] = 0.f;
        }
        // normalisers for phase P2; lane r (and r + 32, r + 64) owns row r
        for (int r = lane; r < NR; r += 32) {
            RowStat st; st.inv_s = 0.0; st.ef = (float)sh_E[r]; st.e = sh_E[r]; st.pad[0] = 0; st.pad[1] = 0;
            if (!fatal && sh_E[r] > E_EMPTY && sh_S[r] > 0.0) st.inv_s = 1.0 / sh_S[r];
            a.rstat[(int64_t)b * NR + r] = st;
        }
        const int draw_row = fatal ? -1 : nn;
        if (lane == 0) {
            a.o.accept_len[b] = nn;
            if (a.o.row_status) a.o.row_status[b] = seq_st;
            a.stop[b] = fatal ? -1 : nn;
            SeqInfo si; si.n = fatal ? -1 : nn; si.draw_row = draw_row; si.pad0 = 0; si.pad = 0;
            a.sinfo[b] = si;
        }
        __syncwarp();
        // everything phase P2 reads was written by this warp: lane 0's release (in the caller) must cover
        // the other lanes' stores
        __threadfence();
    }
}

// residuals of one vector pair: p = 2^(x*c - E_p) / S_p, q likewise
struct RowScale { float ef, inv, inv_lo; };     // exponent E; 1/S = inv + inv_lo to about 2^-48
__device__ __forceinline__ RowScale row_scale(const RowStat& s) {
    RowScale r; r.ef = s.ef; r.inv = (float)s.inv_s; r.inv_lo = (float)(s.inv_s - (double)r.inv);
    return r;
}
__device__ __forceinline__ RowScale no_row() { RowScale r; r.ef = 0.f; r.inv = 0.f; r.inv_lo = 0.f; return r; }

// FINE (the rows a token is drawn from): the normaliser enters as two floats, so that its rounding to fp32
// is not an error common to all tokens of the row; what is left is one rounding per token.
template <int DT, bool FINE>
__device__ __forceinline__ void residual_vec(const uint4& rp, const uint4& rq, bool pair, const TempScale& c, const RowScale& P,
                                             const RowScale& Q, float* r, float* sq) {
    constexpr int VEC = Elem<DT>::VEC;
    float fp[VEC], fq[VEC];
    unpack<DT>(rp, fp);
    if (pair) unpack<DT>(rq, fq);
#pragma unroll
    for (int i = 0; i < VEC; ++i) {
        const float ap = exp2_scaled(fp[i], c, P.ef);
        const float aq = pair ? exp2_scaled(fq[i], c, Q.ef) : 0.f;
        // explicit roundings: a contracted p - a*inv would leave rounding dust when the rows are equal
        const float p = FINE ? __fmaf_rn(ap, P.inv_lo, __fmul_rn(ap, P.inv)) : __fmul_rn(ap, P.inv);
        const float q = pair ? (FINE ? __fmaf_rn(aq, Q.inv_lo, __fmul_rn(aq, Q.inv)) : __fmul_rn(aq, Q.inv)) : 0.f;
        r[i] = fmaxf(p - q, 0.f);
        if (sq) { *sq = fmaf(p, p, *sq); *sq = fmaf(q, q, *sq); }
    }
}

// ------------------------------------------------------------------ phase P2
// Slices of phase P2 and D are half as long as those of P1 (two rows are in flight per thread).
template <int DT>
__device__ __forceinline__ void phase_p2(const WaveArgs& a, WaveShared& S, int b, int k, int s) {
    constexpr int VEC = Elem<DT>::VEC, NV = SLICE_VECS / (2 * WT);    // 4 vectors per thread and row
    const RowArgs& R = a.r;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = R.K, L = len_of(R, b), NR = 2 * K + 1, T2 = 2 * a.T, sv = a.slice_vecs >> 1;
    if (k > L) return;
    const SeqInfo si = a.sinfo[b];
    if (si.n < 0) return;                                  // fatal sequence
    const bool pair = k < L;
    if (!pair && si.draw_row != L) return;                 // bonus row not needed
    const bool draw = si.draw_row == k;
    const int v0 = s * sv;
    const int nv = max(min(sv, R.nvec - v0), 0);
    const char* prow = row_ptr(R, b, k) + (int64_t)v0 * 16;
    const char* qrow = pair ? row_ptr(R, b, K + 1 + k) + (int64_t)v0 * 16 : nullptr;
    uint4 rp[NV], rq[NV];
#pragma unroll
    for (int u = 0; u < NV; ++u) {
        const int v = tid + u * WT;
        rp[u] = neg_inf_vec<DT>(); rq[u] = neg_inf_vec<DT>();
        if (v < nv) { rp[u] = ldg16(prow + (size_t)v * 16); if (pair) rq[u] = ldg16(qrow + (size_t)v * 16); }
    }
    const float tau = tau_of(R, b);
    const TempScale c = temp_scale(tau);
    const RowScale SP = row_scale(a.rstat[(int64_t)b * NR + k]);
    RowScale SQ = no_row();
    if (pair) SQ = row_scale(a.rstat[(int64_t)b * NR + K + 1 + k]);
    if ((v0 + nv) * VEC > R.V) {
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            const int gbase = (v0 + tid + u * WT) * VEC;
            if (tid + u * WT < nv && gbase + VEC > R.V) { mask_tail<DT>(rp[u], R.V - gbase); mask_tail<DT>(rq[u], R.V - gbase); }
        }
    }
    float z0 = 0.f, z1 = 0.f, sqs = 0.f;
    double zd = 0.0;
    if (!draw) {
        // the common case: TV only
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            if (tid + u * WT < nv) {
                float r[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) r[i] = 0.f;
                residual_vec<DT, false>(rp[u], rq[u], pair, c, SP, SQ, r, nullptr);
                const float vs = ((r[0] + r[1]) + (r[2] + r[3])) + ((r[4] + r[5]) + (r[6] + r[7]));
                if (u & 1) z1 += vs; else z0 += vs;
            }
        }
    } else {
        // the row pair a token is drawn from: also the mass in double and the sum of squares
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            if (tid + u * WT < nv) {
                float r[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) r[i] = 0.f;
                residual_vec<DT, true>(rp[u], rq[u], pair, c, SP, SQ, r, &sqs);
                const float vs = ((r[0] + r[1]) + (r[2] + r[3])) + ((r[4] + r[5]) + (r[6] + r[7]));
                z0 += vs;
                zd += (double)vs;
            }
        }
    }
    float z = warp_sum(z0 + z1);
    if (lane == 0) S.redf[0][warp] = z;
    if (draw) {
        zd = warp_sum(zd); sqs = warp_sum(sqs);
        if (lane == 0) { S.redd[warp] = zd; S.redf[1][warp] = sqs; }
    }
    __syncthreads();
    if (tid == 0) {
        if (pair) {
            float zz = 0.f;
            for (int w = 0; w < WW; ++w) zz += S.redf[0][w];
            a.zpart[((int64_t)b * K + k) * T2 + s] = zz;
        }
        if (draw) {
            double tot = 0.0; float sq = 0.f;
            for (int w = 0; w < WW; ++w) { tot += S.redd[w]; sq += S.redf[1][w]; }
            DPart d; d.tot = tot; d.sq = sq; d.pad = 0;
            a.dpart[(int64_t)b * T2 + s] = d;
        }
    }
}

// ------------------------------------------------------------------ phase D
template <int DT>
__device__ __forceinline__ void phase_d(const WaveArgs& a, WaveShared& S, int b) {
    constexpr int VEC = Elem<DT>::VEC;
    const RowArgs& R = a.r;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = R.K, L = len_of(R, b), NR = 2 * K + 1, T = 2 * a.T, sv = a.slice_vecs >> 1;
    const SeqInfo si = a.sinfo[b];
    if (si.n < 0) return;
    // TV of every draft position: slice parts in slice order
    if (tid < L && a.o.tv) {
        float z = 0.f;
        for (int s = 0; s < T; ++s) z += a.zpart[((int64_t)b * K + tid) * T + s];
        a.o.tv[(int64_t)b * K + tid] = fminf(fmaxf(z, 0.f), 1.f);
    }
    const int k = si.draw_row;
    if (k < 0) return;
    const bool pair = k < L;
    if (tid == 0) {
        double Z = 0.0, sumsq = 0.0;
        for (int s = 0; s < T; ++s) { Z += a.dpart[(int64_t)b * T + s].tot; sumsq += (double)a.dpart[(int64_t)b * T + s].sq; }
        const double Tt = (double)a.u_final[b] * Z;
        double run = 0.0; int owner = -1; double base = 0.0;
        for (int s = 0; s < T; ++s) {
            const double nx = run + a.dpart[(int64_t)b * T + s].tot;
            if (owner < 0 && Tt > run && Tt <= nx) { owner = s; base = run; }
            run = nx;
        }
        S.owner_slice = (Tt > 0.0) ? owner : -1;
        S.base = base; S.Ttarget = Tt; S.bound = draw_bound(sumsq);
    }
    __syncthreads();
    const int s = S.owner_slice;
    int found_y = -1, found_cert = 0;
    if (s >= 0) {
        const float tau = tau_of(R, b);
        const TempScale c = temp_scale(tau);
        const RowScale SP = row_scale(a.rstat[(int64_t)b * NR + k]);
        RowScale SQ = no_row();
        if (pair) SQ = row_scale(a.rstat[(int64_t)b * NR + K + 1 + k]);
        const int v0 = s * sv;
        const int nv = max(min(sv, R.nvec - v0), 0);
        const char* prow = row_ptr(R, b, k) + (int64_t)v0 * 16;
        const char* qrow = pair ? row_ptr(R, b, K + 1 + k) + (int64_t)v0 * 16 : nullptr;
        // per-vector residual mass, same arithmetic as phase P2
        for (int v = tid; v < nv; v += WT) {
            uint4 rp = ldg16(prow + (size_t)v * 16), rq = neg_inf_vec<DT>();
            if (pair) rq = ldg16(qrow + (size_t)v * 16);
            const int gbase = (v0 + v) * VEC;
            if (gbase + VEC > R.V) { mask_tail<DT>(rp, R.V - gbase); mask_tail<DT>(rq, R.V - gbase); }
            float r[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) r[i] = 0.f;
            residual_vec<DT, true>(rp, rq, pair, c, SP, SQ, r, nullptr);
            S.vsum[v] = ((r[0] + r[1]) + (r[2] + r[3])) + ((r[4] + r[5]) + (r[6] + r[7]));
        }
        __syncthreads();
        // contiguous ranges of vectors per thread, inclusive scan over threads
        const int per = (nv + WT - 1) / WT;
        const int vb = min(tid * per, nv), ve = min(vb + per, nv);
        double mine = 0.0;
        for (int v = vb; v < ve; ++v) mine += (double)S.vsum[v];
        double incl = mine;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) { double t2 = shfl_up_d(incl, d); if (lane >= d) incl += t2; }
        if (lane == 31) S.redd[warp] = incl;
        __syncthreads();
        double woff = 0.0;
        for (int w = 0; w < warp; ++w) woff += S.redd[w];
        double prev = shfl_up_d(incl, 1);
        if (lane == 0) prev = 0.0;
        const double Tt = S.Ttarget, bound = S.bound;
        const double lower = S.base + woff + prev, upper = S.base + woff + incl;
        if (lower < Tt && Tt <= upper) {
            double C = lower;
            for (int v = vb; v < ve && found_y < 0; ++v) {
                const double nxt = C + (double)S.vsum[v];
                if (Tt <= nxt) {
                    uint4 rp = ldg16(prow + (size_t)v * 16), rq = neg_inf_vec<DT>();
                    if (pair) rq = ldg16(qrow + (size_t)v * 16);
                    const int gbase = (v0 + v) * VEC;
                    if (gbase + VEC > R.V) { mask_tail<DT>(rp, R.V - gbase); mask_tail<DT>(rq, R.V - gbase); }
                    float r[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) r[i] = 0.f;
                    residual_vec<DT, true>(rp, rq, pair, c, SP, SQ, r, nullptr);
                    double Cw = C;
#pragma unroll
                    for (int i = 0; i < VEC; ++i) {
                        if (found_y < 0) {
                            const double r1 = (double)r[i];
                            const double Cn = Cw + r1;
                            if (r1 > 0.0 && Cn >= Tt) { found_y = gbase + i; found_cert = (Tt - Cw > bound) && (Cn - Tt >= bound); }
                            Cw = Cn;
                        }
                    }
                    break;
                }
                C = nxt;
            }
        }
    }
    // at most one thread should have found the token
    const unsigned own = __ballot_sync(0xffffffffu, found_y >= 0);
    if (lane == 0) S.redi[warp] = -1;
    __syncthreads();
    if (own && lane == (__ffs(own) - 1)) S.redi[warp] = (__popc(own) == 1 && found_cert) ? found_y : -2;
    __syncthreads();
    if (tid == 0) {
        int y = -1, cnt = 0;
        for (int w = 0; w < WW; ++w) if (S.redi[w] != -1) { y = S.redi[w]; cnt++; }
        if (cnt == 1 && y >= 0) a.o.out_tokens[(int64_t)b * (K + 1) + k] = y;
        else { int idx = atomicAdd(a.fb_count, 1); a.fb_list[idx] = b; }
    }
}

}  // namespace

template <int DT>
__global__ void __launch_bounds__(WT, 4) k_wave(const WaveArgs a) {
    __shared__ WaveShared S;
    const int tid = threadIdx.x;
    const int K = a.r.K, T = a.T, T2 = 2 * a.T, NR = 2 * K + 1;
    // schedule constants (all tickets fit 31 bits).  Prologue: P1(0..lag).  Step w = 0 .. nw+1 holds
    // A(w), P2(w-1), P1(w+lag+1), D(w-2): every phase sits one whole step behind the phase it needs.
    const int B = a.r.B, WS = a.wave_seqs, LAG = a.lag;
    const int c0 = NR * T, c2 = (K + 1) * T2;
    auto N = [&](int w) { return w <= 0 ? 0 : min(B, w * WS); };                 // sequences in the first w waves
    const int P = c0 * N(LAG + 1);
    auto F = [&](int w) { return N(w) + c2 * N(w - 1) + c0 * (N(w + LAG + 1) - N(LAG + 1)) + N(w - 2); };
    int next = 0;
    if (tid == 0) next = atomicAdd(a.ticket, 1);
    for (;;) {
        long long tr0 = 0, tr1 = 0, trd = 0, trs = 0;
        (void)tr1; (void)trd; (void)trs;
        if (tid == 0) {
#ifdef BEBOP_TRACE
            tr0 = clock64();
#endif
            const int t = next;
            S.ticket = t;
            if (t < a.ntickets) {
                int ph, wv, off;
                if (t < P) { ph = 0; wv = t / (c0 * WS); off = t - c0 * N(wv); }
                else {
                    const int tt = t - P;
                    int lo = 0, hi = a.nwaves + 1;
                    while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if (F(mid) <= tt) lo = mid; else hi = mid - 1; }
                    const int w = lo, o2 = tt - F(w);
                    const int nA = N(w + 1) - N(w), n2 = (N(w) - N(w - 1)) * c2, n1 = c0 * (N(w + LAG + 2) - N(w + LAG + 1));
                    if (o2 < nA) { ph = 1; wv = w; off = o2; }
                    else if (o2 < nA + n2) { ph = 2; wv = w - 1; off = o2 - nA; }
                    else if (o2 < nA + n2 + n1) { ph = 0; wv = w + LAG + 1; off = o2 - nA - n2; }
                    else { ph = 3; wv = w - 2; off = o2 - nA - n2 - n1; }
                }
                S.phase = ph; S.wave = wv; S.index = off;
                next = atomicAdd(a.ticket, 1);
#ifdef BEBOP_TRACE
                trd = clock64();
#endif
                // dependencies: completion counters of the wave (almost always long satisfied)
                const int ns = N(wv + 1) - N(wv);
                bool okw = true;
                if (ph == 1) okw = spin_ge(&a.p1done[wv], ns * c0);
                else if (ph == 2) okw = spin_ge(&a.adone[wv], ns);
                else if (ph == 3) okw = spin_ge(&a.p2done[wv], ns * c2);
                if (!okw) atomicExch(a.wait_failed, 1);
#ifdef BEBOP_TRACE
                trs = clock64();
#endif
            }
        }
        __syncthreads();
        if (S.ticket >= a.ntickets) break;
#ifdef BEBOP_TRACE
        if (tid == 0) tr1 = clock64();
#endif
        const int phase = S.phase, w = S.wave, idx = S.index;
        const int b0 = w * WS;
        int* done = nullptr;
        if (phase == 0) {
            const int s = idx % T, r = (idx / T) % NR, b = b0 + idx / c0;
            phase_p1<DT>(a, S, b, r, s);
            done = &a.p1done[w];
        } else if (phase == 1) {
            phase_a<DT>(a, S, b0 + idx);
            done = &a.adone[w];
        } else if (phase == 2) {
            const int s = idx % T2, k = (idx / T2) % (K + 1), b = b0 + idx / c2;
            phase_p2<DT>(a, S, b, k, s);
            done = &a.p2done[w];
        } else {
            phase_d<DT>(a, S, b0 + idx);
        }
        __syncthreads();
        // results consumed by later phases are written by thread 0: its release covers them
        if (tid == 0 && done) asm volatile("red.release.gpu.global.add.s32 [%0], 1;" :: "l"(done) : "memory");
#ifdef BEBOP_TRACE
        if (tid == 0 && a.trace) {
            // per phase: cycles in ticket decode, dependency wait, barrier, task; task count
            const long long tr2 = clock64();
            unsigned long long* tq = reinterpret_cast<unsigned long long*>(a.trace) + phase * 8;
            atomicAdd(tq + 0, (unsigned long long)(trd - tr0)); atomicAdd(tq + 1, (unsigned long long)(trs - trd));
            atomicAdd(tq + 2, (unsigned long long)(tr1 - trs)); atomicAdd(tq + 3, (unsigned long long)(tr2 - tr1));
            atomicAdd(tq + 4, 1ull);
        }
#endif
    }
}

namespace {

// ------------------------------------------------------------------ fp64 re-draw of the listed sequences
// Two small kernels behind the wave kernel, for the few sequences whose fast draw did not clear its
// error bound.  Every row is cut into XT = 4T quarter slices; CTA (s, y) takes quarter slice s of the
// listed sequences y, y + gridDim.y, ...  Everything is evaluated in double around the row exponents
// that phase A left (any common reference cancels in p = a / sum a).
//   k_redraw_sum   exact normalisers: sum of exponentials of each quarter slice of the draw rows;
//   k_redraw_mass  residual mass of each quarter slice, one sum per warp (warp w owns the contiguous
//                  vectors [w*cw, (w+1)*cw)); the CTA that completes a sequence picks its token at
//                  once: quarter slice and warp chunk from the stored sums, then the few hundred
//                  tokens of that chunk are evaluated once more, one or two per thread, and scanned.
struct RedrawArgs {
    RowArgs r;
    const float* u_final;
    VerifyOut o;
    const int* fb_count;     // listed sequences
    const int* fb_list;
    const SeqInfo* sinfo;
    const RowStat* rstat;
    double2* xsum;           // [B][XT] sums of exponentials (target row, draft row) per quarter slice
    double* xmass;           // [B][XT][WW] residual mass per quarter slice and warp chunk
    int* xdone;              // [B] per listed sequence: mass tasks finished
    int T, slice_vecs;
};

struct XRow {
    const char* prow; const char* qrow;
    double c, ep, eq, ip, iq;      // p = exp2(x * c - ep) * ip
    int b, k;
    bool pair;
};
__device__ __forceinline__ double x_resid(const XRow& d, float zp, float zq) {
    // explicit roundings: a contracted p * ip - q would leave rounding dust when p == q
    const double p = __dmul_rn(exp2(fma((double)zp, d.c, -d.ep)), d.ip);
    if (!d.pair) return p;
    const double q = __dmul_rn(exp2(fma((double)zq, d.c, -d.eq)), d.iq);
    const double df = p - q;
    return df > 0.0 ? df : 0.0;
}
__device__ __forceinline__ bool x_row(const RedrawArgs& a, int slot, XRow* d) {
    const RowArgs& R = a.r;
    const int K = R.K, NR = 2 * K + 1;
    const int b = a.fb_list[slot];
    const SeqInfo si = a.sinfo[b];
    d->b = b; d->k = si.draw_row;
    if (si.draw_row < 0) return false;
    d->pair = si.draw_row < len_of(R, b);
    d->prow = row_ptr(R, b, si.draw_row);
    d->qrow = d->pair ? row_ptr(R, b, K + 1 + si.draw_row) : d->prow;
    d->c = 1.4426950408889634 / (double)tau_of(R, b);
    d->ep = (double)a.rstat[(int64_t)b * NR + si.draw_row].e;
    d->eq = d->pair ? (double)a.rstat[(int64_t)b * NR + K + 1 + si.draw_row].e : 0.0;
    d->ip = 1.0; d->iq = 1.0;
    return true;
}
constexpr int XNU = 2;     // vectors per thread and row in a quarter slice (at most 512 vectors)

// this thread's vectors of quarter slice s: warp chunk [warp*cw, warp*cw + cw), lanes interleaved
template <int DT>
__device__ __forceinline__ void x_load(const RedrawArgs& a, const XRow& d, int s, float (*fp)[Elem<DT>::VEC],
                                       float (*fq)[Elem<DT>::VEC]) {
    constexpr int VEC = Elem<DT>::VEC;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int qv = a.slice_vecs >> 2, cw = (qv + WW - 1) / WW;
    const int v0 = s * qv, nv = max(min(qv, a.r.nvec - v0), 0);
#pragma unroll
    for (int u = 0; u < XNU; ++u) {
        const int vl = warp * cw + lane + 32 * u;
        const bool in = lane + 32 * u < cw && vl < nv;
#pragma unroll
        for (int i = 0; i < VEC; ++i) { fp[u][i] = -INFINITY; fq[u][i] = -INFINITY; }
        if (in) {
            load_vec<DT>(d.prow, v0 + vl, a.r.V, fp[u]);
            if (d.pair) load_vec<DT>(d.qrow, v0 + vl, a.r.V, fq[u]);
        }
    }
}

template <int DT>
__global__ void __launch_bounds__(WT) k_redraw_sum(const RedrawArgs a) {
    constexpr int VEC = Elem<DT>::VEC;
    __shared__ double sh[2][WW];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int XT = 4 * a.T, s = blockIdx.x, count = *a.fb_count;
    for (int slot = blockIdx.y; slot < count; slot += gridDim.y) {
        XRow d;
        if (!x_row(a, slot, &d)) continue;
        float fp[XNU][VEC], fq[XNU][VEC];
        x_load<DT>(a, d, s, fp, fq);
        double sa = 0.0, sb = 0.0;
#pragma unroll
        for (int u = 0; u < XNU; ++u) {
#pragma unroll
            for (int i = 0; i < VEC; ++i) {
                sa += exp2(fma((double)fp[u][i], d.c, -d.ep));
                if (d.pair) sb += exp2(fma((double)fq[u][i], d.c, -d.eq));
            }
        }
        sa = warp_sum(sa); sb = warp_sum(sb);
        __syncthreads();
        if (lane == 0) { sh[0][warp] = sa; sh[1][warp] = sb; }
        __syncthreads();
        if (tid == 0) {
            double ta = 0.0, tb = 0.0;
            for (int w = 0; w < WW; ++w) { ta += sh[0][w]; tb += sh[1][w]; }
            a.xsum[(int64_t)d.b * XT + s] = make_double2(ta, tb);
        }
    }
}

struct PickShared {
    double part[4 * MAX_SLICES];     // slice masses of the sequence, later the warp masses of one slice
    double redd[WW];
    double base, target;
    int last, sel, chunk, tok_first, tok_last;
};

// first entry with mass whose running sum reaches t (running sum starts at *C); by rounding none may:
// then the last entry with mass.  Leaves in *C the sum before the chosen entry.
__device__ __forceinline__ int pick_entry(const double* m, int n, double t, double* C) {
    const double c0 = *C;
    double run = c0;
    int last = 0;
    for (int i = 0; i < n; ++i) {
        if (m[i] > 0.0) {
            if (run + m[i] >= t) { *C = run; return i; }
            last = i;
        }
        run += m[i];
    }
    run = c0;
    for (int i = 0; i < last; ++i) run += m[i];
    *C = run;
    return last;
}

template <int DT>
__global__ void __launch_bounds__(WT) k_redraw_mass(const RedrawArgs a) {
    constexpr int VEC = Elem<DT>::VEC;
    __shared__ PickShared S;
    const RowArgs& R = a.r;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = R.K, XT = 4 * a.T, s = blockIdx.x, count = *a.fb_count;
    const int qv = a.slice_vecs >> 2, cw = (qv + WW - 1) / WW;
    for (int slot = blockIdx.y; slot < count; slot += gridDim.y) {
        XRow d;
        if (!x_row(a, slot, &d)) continue;
        const int b = d.b;
        // exact normalisers: quarter-slice sums in slice order (the same order in every CTA)
        double Sa = 0.0, Sb = 0.0;
#pragma unroll 8
        for (int t = 0; t < XT; ++t) { const double2 x = a.xsum[(int64_t)b * XT + t]; Sa += x.x; Sb += x.y; }
        d.ip = 1.0 / Sa; d.iq = d.pair ? 1.0 / Sb : 0.0;
        if (d.pair) {     // a bonus row needs no mass pass: its masses are sums of exponentials over Sa
            float fp[XNU][VEC], fq[XNU][VEC];
            x_load<DT>(a, d, s, fp, fq);
            double m = 0.0;
#pragma unroll
            for (int u = 0; u < XNU; ++u) {
#pragma unroll
                for (int i = 0; i < VEC; ++i) m += x_resid(d, fp[u][i], fq[u][i]);
            }
            m = warp_sum(m);
            if (lane == 0) a.xmass[((int64_t)b * XT + s) * WW + warp] = m;
        }
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            S.last = atomicAdd(a.xdone + slot, 1) == XT - 1;
        }
        __syncthreads();
        if (!S.last) continue;
        __threadfence();

        // ---- pick.  Stage 1: quarter slice from the slice masses.
        bool zero_resid = false;
        for (int pass = 0; pass < 2; ++pass) {
            for (int t = tid; t < XT; t += WT) {
                double m = 0.0;
                if (d.pair) { for (int w = 0; w < WW; ++w) m += __ldcg(a.xmass + ((int64_t)b * XT + t) * WW + w); }
                else m = a.xsum[(int64_t)b * XT + t].x * d.ip;
                S.part[t] = m;
            }
            __syncthreads();
            if (tid == 0) {
                double Z = 0.0;
                for (int t = 0; t < XT; ++t) Z += S.part[t];
                S.base = Z;
            }
            __syncthreads();
            if (S.base > 0.0 || !d.pair) break;
            // residual mass vanished at a rejected position: draw from p of that position
            d.pair = false; zero_resid = true;
            __syncthreads();
        }
        if (tid == 0) {
            if (zero_resid && a.o.row_status) a.o.row_status[b] |= ST_ZERO_RESID;
            const double t = (double)a.u_final[b] * S.base;
            double C = 0.0;
            S.sel = pick_entry(S.part, XT, t, &C);
            S.target = t; S.base = C;
        }
        __syncthreads();
        const int qs = S.sel;
        // Stage 2: warp chunk inside the quarter slice (residual: stored; plain softmax row: evaluated now)
        const int p0 = qs * qv, pn = max(min(qv, R.nvec - p0), 0);
        double wm = 0.0;
        if (!d.pair) {
#pragma unroll
            for (int u = 0; u < XNU; ++u) {
                const int vl = warp * cw + lane + 32 * u;
                if (lane + 32 * u < cw && vl < pn) {
                    float f[VEC];
                    load_vec<DT>(d.prow, p0 + vl, R.V, f);
#pragma unroll
                    for (int i = 0; i < VEC; ++i) wm += x_resid(d, f[i], 0.f);
                }
            }
            wm = warp_sum(wm);
        }
        __syncthreads();                                   // S.part is about to be overwritten
        if (lane == 0) S.part[warp] = d.pair ? __ldcg(a.xmass + ((int64_t)b * XT + qs) * WW + warp) : wm;
        __syncthreads();
        if (tid == 0) {
            double C = S.base;
            S.chunk = pick_entry(S.part, WW, S.target, &C);
            S.base = C;
            S.tok_first = 0x7fffffff; S.tok_last = -1;
        }
        __syncthreads();
        // Stage 3: the tokens of the chunk, `per` consecutive tokens per thread, scanned in token order
        const int e0 = (p0 + S.chunk * cw) * VEC;                                 // first token of the chunk
        const int e1 = min(min((p0 + min((S.chunk + 1) * cw, pn)) * VEC, R.V), e0 + 4 * WT);
        const int per = (max(e1 - e0, 0) + WT - 1) / WT;                          // <= 2 (cw <= 64 vectors of 8)
        double r[4] = {0.0, 0.0, 0.0, 0.0};
        double mine = 0.0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int v = e0 + tid * per + i;
            if (i < per && v < e1) {
                const float zp = load_one<DT>(d.prow, v);
                const float zq = d.pair ? load_one<DT>(d.qrow, v) : 0.f;
                r[i] = x_resid(d, zp, zq);
                mine += r[i];
            }
        }
        double incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const double t2 = shfl_up_d(incl, o); if (lane >= o) incl += t2; }
        if (lane == 31) S.redd[warp] = incl;
        __syncthreads();
        double C = S.base;
        for (int w = 0; w < warp; ++w) C += S.redd[w];
        C += incl - mine;
        const double t = S.target;
        // the first token with mass whose prefix sum reaches the target; by rounding none may: then the
        // last token with mass
        int y = -1, lastpos = -1;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (r[i] > 0.0) {
                lastpos = e0 + tid * per + i;
                if (y < 0 && C + r[i] >= t) y = lastpos;
            }
            C += r[i];
        }
        if (y >= 0) atomicMin(&S.tok_first, y);
        if (lastpos >= 0) atomicMax(&S.tok_last, lastpos);
        __syncthreads();
        if (tid == 0) a.o.out_tokens[(int64_t)b * (K + 1) + d.k] = S.tok_first != 0x7fffffff ? S.tok_first : S.tok_last;
        __syncthreads();
    }
}

}  // namespace

__global__ void k_wave_flag(const int* __restrict__ wait_failed, int32_t* row_status, int B) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B && *wait_failed && row_status) row_status[b] |= ST_WAIT;
}

// -----------------------------------------------------------------------------
namespace {

template <int DT>
int wave_grid() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (dev >= 0 && dev < 64 && cached[dev]) return cached[dev];
    int per_sm = 0, sms = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_wave<DT>, WT, 0) != cudaSuccess) per_sm = 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaGetLastError();
    const int n = per_sm * sms;
    if (dev >= 0 && dev < 64) cached[dev] = n;
    return n;
}

}  // namespace

long long* g_wave_trace = nullptr;
void wave_set_trace(long long* p) { g_wave_trace = p; }
cudaEvent_t g_ev_start = nullptr, g_ev_stop = nullptr;
void wave_set_events(cudaEvent_t start, cudaEvent_t stop) { g_ev_start = start; g_ev_stop = stop; }

bool wave_supported(const RowArgs& a) {
    const int T = (a.nvec + SLICE_VECS - 1) / SLICE_VECS;
    return T >= 1 && T <= MAX_SLICES && a.K <= BEBOP_MAX_K_INT;
}

cudaError_t wave_verify(const RowArgs& a, const Plan& p, const int32_t* draft_tokens,
                        const float* u_accept, const float* u_final, VerifyOut o, char* ws,
                        cudaStream_t stream, bool* launched) {
    *launched = false;
    const int grid_max = a.dt == 0 ? wave_grid<0>() : wave_grid<1>();
    if (grid_max < 1) return cudaSuccess;
    const WavePlan wp = make_wave_plan(a.B, a.K, a.nvec, a.dt);
    WaveArgs wa;
    wa.r = a; wa.draft_tokens = draft_tokens; wa.u_accept = u_accept; wa.u_final = u_final; wa.o = o;
    wa.stop = reinterpret_cast<int*>(ws + p.off_stop);
    wa.fb_count = reinterpret_cast<int*>(ws + p.off_fb);
    wa.fb_list = wa.fb_count + 16;
    char* w = ws + p.off_wave;
    wa.ticket = reinterpret_cast<int*>(w);
    wa.wait_failed = wa.ticket + 1;
    wa.p1done = reinterpret_cast<int*>(w + wp.off_p1done);
    wa.adone = reinterpret_cast<int*>(w + wp.off_adone);
    wa.p2done = reinterpret_cast<int*>(w + wp.off_p2done);
    wa.part = reinterpret_cast<P1Part*>(w + wp.off_part);
    wa.rstat = reinterpret_cast<RowStat*>(w + wp.off_rstat);
    wa.zpart = reinterpret_cast<float*>(w + wp.off_zpart);
    wa.dpart = reinterpret_cast<DPart*>(w + wp.off_dpart);
    wa.sinfo = reinterpret_cast<SeqInfo*>(w + wp.off_sinfo);
    wa.trace = g_wave_trace;
    wa.T = wp.T; wa.slice_vecs = wp.slice_vecs; wa.wave_seqs = wp.wave_seqs; wa.nwaves = wp.nwaves;
    // number of tickets: every phase of every wave
    {
        const long long NR = 2 * a.K + 1;
        const long long total = (long long)a.B * (NR * wp.T + 1 + (long long)(a.K + 1) * 2 * wp.T + 1);
        if (total > 0x7fff0000LL) return cudaSuccess;
        wa.ntickets = (int)total;
        wa.lag = wp.lag;
    }
    cudaError_t e = cudaMemsetAsync(w, 0, wp.zero_bytes, stream);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(wa.fb_count, 0, sizeof(int), stream);
    if (e != cudaSuccess) return e;
    const int grid = wa.ntickets < grid_max ? wa.ntickets : grid_max;
    if (g_ev_start) cudaEventRecord(g_ev_start, stream);
    if (a.dt == 0) k_wave<0><<<grid, WT, 0, stream>>>(wa);
    else k_wave<1><<<grid, WT, 0, stream>>>(wa);
    e = cudaGetLastError();
    if (g_ev_stop) cudaEventRecord(g_ev_stop, stream);
    if (e != cudaSuccess) return e;
    k_wave_flag<<<(a.B + 255) / 256, 256, 0, stream>>>(wa.wait_failed, o.row_status, a.B);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    *launched = true;
    // fp64 re-draw of the listed sequences (usually a few per cent of the batch; the count stays on the device)
    RedrawArgs ra;
    ra.r = a; ra.u_final = u_final; ra.o = o;
    ra.fb_count = wa.fb_count; ra.fb_list = wa.fb_list;
    ra.sinfo = wa.sinfo; ra.rstat = wa.rstat;
    ra.xsum = reinterpret_cast<double2*>(w + wp.off_xsum);
    ra.xmass = reinterpret_cast<double*>(w + wp.off_xmass);
    ra.xdone = reinterpret_cast<int*>(w + wp.off_xdone);
    ra.T = wp.T; ra.slice_vecs = wp.slice_vecs;
    const dim3 rgrid(4 * wp.T, a.B < 32 ? a.B : 32);
    if (a.dt == 0) { k_redraw_sum<0><<<rgrid, WT, 0, stream>>>(ra); k_redraw_mass<0><<<rgrid, WT, 0, stream>>>(ra); }
    else { k_redraw_sum<1><<<rgrid, WT, 0, stream>>>(ra); k_redraw_mass<1><<<rgrid, WT, 0, stream>>>(ra); }
    return cudaGetLastError();
}

}  // namespace bebop
