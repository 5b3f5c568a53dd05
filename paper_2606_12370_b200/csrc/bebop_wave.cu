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
struct __align__(16) RowStat { double inv_s; float m_ref, frac; int e; int pad; };   // per row, after the merge
struct __align__(16) DPart { double tot; float sq; int pad; };        // per (sequence, slice)
struct __align__(16) SeqInfo {          // per sequence, written by phase A
    int n;                              // accept count (stop position); -1: fatal
    int draw_row;                       // row whose residual is drawn from (n, or L for the bonus row); -1 none
    float sys;                          // systematic part of the error bound (rounding of the normalisers)
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

// The error bound a draw must clear.  The residual is formed from fp32
// exponentials (ex2.approx: 2 ulp) and fp32 products, so each p, q carries a
// relative error of a few 2^-24; the errors of different tokens are independent,
// hence the error of a prefix sum is of the order delta * sqrt(sum p^2 + q^2).
// kappa leaves a wide safety factor over that root-sum-square.  `sys` adds the
// part that is common to all tokens: the rounding of 1/S_p and 1/S_q to fp32.
__device__ __forceinline__ double draw_bound(double sumsq, double sys) {
    const double delta = 2.384185791015625e-07;   // 2^-22
    const double kappa = 16.0;
    return kappa * delta * sqrt(sumsq) + sys + 1e-300;
}

// E = ceil(m * c), frac = E - m * c in [0, 1] without rounding loss, so that
// 2^((x - m) * c - frac) equals 2^(x * c - E) whatever reference point m is used.
__device__ __forceinline__ void reference(float m, float c, int* E, float* frac) {
    float th = fminf(fmaxf(m * c, -4.0e6f), 4.0e6f);
    float te = fmaf(m, c, -th);
    if (th != m * c) te = 0.f;
    float Ef;
    int Ei = ceil_alu(th, &Ef);
    float f = (Ef - th) - te;
    if (f < 0.f) { f += 1.f; Ei += 1; }
    *E = Ei; *frac = f;
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
    constexpr int VEC = Elem<DT>::VEC, U = 4;
    const RowArgs& R = a.r;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int L = len_of(R, b), K = R.K;
    const bool is_target = r <= K;
    const int k = is_target ? r : r - (K + 1);
    if (is_target ? k > L : k >= L) return;
    const float tau = tau_of(R, b);
    const float c = kLog2e / (tau_ok(tau) ? tau : 1.f);
    const int v0 = s * a.slice_vecs;
    const int nv = max(min(a.slice_vecs, R.nvec - v0), 0);
    const char* row = row_ptr(R, b, r) + (int64_t)v0 * 16;

    float m_ref = -INFINITY, frac = 0.f;
    int E = E_EMPTY;
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
    bool bad = false;
    for (int i0 = tid; i0 < nv; i0 += WT * U) {
        uint4 raw[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int v = i0 + u * WT;
            raw[u] = neg_inf_vec<DT>();
            if (v < nv) {
                raw[u] = ldg16_stream(row + (size_t)v * 16);
                const int gbase = (v0 + v) * VEC;
                if (gbase + VEC > R.V) mask_tail<DT>(raw[u], R.V - gbase);
            }
        }
        float bm = max_nan(max_nan(vec_max<DT>(raw[0]), vec_max<DT>(raw[1])), max_nan(vec_max<DT>(raw[2]), vec_max<DT>(raw[3])));
        if (bm != bm || bm == INFINITY) bad = true;
        else if (bm > m_ref) {
            // new reference point: rescale the running sums by an exact power of two
            int En; float fn;
            reference(bm, c, &En, &fn);
            const float sc = E > E_EMPTY ? pow2f(max(E - En, -126)) : 0.f;
            s0 *= sc; s1 *= sc; s2 *= sc; s3 *= sc;
            E = En; frac = fn; m_ref = bm;
        }
        if (E > E_EMPTY) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float f[VEC];
                unpack<DT>(raw[u], f);
#pragma unroll
                for (int i = 0; i < VEC; i += 4) {
                    s0 += ex2f(fmaf(f[i] - m_ref, c, -frac));
                    s1 += ex2f(fmaf(f[i + 1] - m_ref, c, -frac));
                    s2 += ex2f(fmaf(f[i + 2] - m_ref, c, -frac));
                    s3 += ex2f(fmaf(f[i + 3] - m_ref, c, -frac));
                }
            }
        }
    }
    // thread -> warp -> block, exact power-of-two rescaling, sums in a fixed order
    float st = (s0 + s1) + (s2 + s3);
    const int Ew = redux_max(E);
    st = E > E_EMPTY ? st * pow2f(max(E - Ew, -126)) : 0.f;
    st = warp_sum(st);
    const unsigned anybad = __ballot_sync(0xffffffffu, bad);
    float mw = ord2f(redux_max(f2ord(m_ref)));
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
    const float c = kLog2e / (ok ? tau : 1.f);
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
    if (tid == 0) {
        int seq_st = ok ? 0 : ST_BAD_TEMP;
        if (!seq_st)
            for (int j = 0; j < L; ++j) { int tk = a.draft_tokens[(int64_t)b * K + j]; if (tk < 0 || tk >= V) seq_st = ST_BAD_TOKEN; }
        int n = L, alive = 1;
        for (int k = 0; k < L && !(seq_st & ST_FATAL); ++k) {
            const int rs = sh_status[k] | sh_status[K + 1 + k];
            if (rs) { seq_st |= rs; break; }              // the first bad row pair decides
            const int tk = a.draft_tokens[(int64_t)b * K + k];
            const float zpx = DT == 0 ? load_one<0>(row_ptr(R, b, k), tk) : load_one<1>(row_ptr(R, b, k), tk);
            const float zqx = DT == 0 ? load_one<0>(row_ptr(R, b, K + 1 + k), tk) : load_one<1>(row_ptr(R, b, K + 1 + k), tk);
            const double cd = (double)c;
            const double px = exp2((double)zpx * cd - (double)sh_E[k]) / sh_S[k];
            const double qx = exp2((double)zqx * cd - (double)sh_E[K + 1 + k]) / sh_S[K + 1 + k];
            if (a.o.p_draft) a.o.p_draft[(int64_t)b * K + k] = (float)px;
            if (a.o.q_draft) a.o.q_draft[(int64_t)b * K + k] = (float)qx;
            if (alive && !((double)a.u_accept[(int64_t)b * K + k] * qx < px)) { alive = 0; n = k; }
        }
        if (!(seq_st & ST_FATAL) && alive && sh_status[L]) seq_st |= sh_status[L];   // bonus row, read only now
        const bool fatal = (seq_st & ST_FATAL) != 0;
        // integer outputs (position n is filled by the draw)
        const int nn = fatal ? 0 : n;
        a.o.accept_len[b] = nn;
        for (int q = 0; q <= K; ++q)
            if (fatal || q != nn) a.o.out_tokens[(int64_t)b * (K + 1) + q] = q < nn ? a.draft_tokens[(int64_t)b * K + q] : -1;
        if (a.o.row_status) a.o.row_status[b] = seq_st;
        a.stop[b] = fatal ? -1 : nn;
        for (int q = 0; q < K; ++q) {
            if (fatal || q >= L) {
                if (a.o.tv) a.o.tv[(int64_t)b * K + q] = 0.f;
                if (a.o.p_draft) a.o.p_draft[(int64_t)b * K + q] = 0.f;
                if (a.o.q_draft) a.o.q_draft[(int64_t)b * K + q] = 0.f;
            }
        }
        // normalisers for phase P2: 2^(x*c - E) is evaluated as 2^((x - m_ref)*c - frac) around the row maximum
        float sys = 0.f;
        for (int r = 0; r < NR; ++r) {
            RowStat rs; rs.inv_s = 0.0; rs.m_ref = 0.f; rs.frac = 0.f; rs.e = sh_E[r]; rs.pad = 0;
            if (!fatal && sh_E[r] > E_EMPTY && sh_S[r] > 0.0) {
                rs.inv_s = 1.0 / sh_S[r];
                int Er; float fr;
                reference(sh_M[r], c, &Er, &fr);           // Er == sh_E[r]: the row maximum fixes the exponent
                rs.m_ref = sh_M[r]; rs.frac = fr + (float)(sh_E[r] - Er);
            }
            a.rstat[(int64_t)b * NR + r] = rs;
        }
        const int draw_row = fatal ? -1 : nn;
        if (draw_row >= 0) {
            // |fl(1/S) - 1/S| / (1/S), an upper bound of what the fp32 scale factors add to a prefix sum
            const double ip = a.rstat[(int64_t)b * NR + draw_row].inv_s;
            sys += (float)(fabs((double)(float)ip - ip) / ip);
            if (draw_row < L) { const double iq = a.rstat[(int64_t)b * NR + K + 1 + draw_row].inv_s; sys += (float)(fabs((double)(float)iq - iq) / iq); }
        }
        SeqInfo si; si.n = fatal ? -1 : nn; si.draw_row = draw_row; si.sys = sys; si.pad = 0;
        a.sinfo[b] = si;
    }
}

// residuals of one vector pair: p = 2^(x*c - E_p) / S_p, q likewise
struct RowScale { float m, frac, inv; };
__device__ __forceinline__ RowScale row_scale(const RowStat& s) { RowScale r; r.m = s.m_ref; r.frac = s.frac; r.inv = (float)s.inv_s; return r; }

template <int DT>
__device__ __forceinline__ void residual_vec(const uint4& rp, const uint4& rq, bool pair, float c, const RowScale& P,
                                             const RowScale& Q, float* r, float* sq) {
    constexpr int VEC = Elem<DT>::VEC;
    float fp[VEC], fq[VEC];
    unpack<DT>(rp, fp);
    if (pair) unpack<DT>(rq, fq);
#pragma unroll
    for (int i = 0; i < VEC; ++i) {
        const float p = __fmul_rn(ex2f(fmaf(fp[i] - P.m, c, -P.frac)), P.inv);
        const float q = pair ? __fmul_rn(ex2f(fmaf(fq[i] - Q.m, c, -Q.frac)), Q.inv) : 0.f;
        r[i] = fmaxf(p - q, 0.f);
        if (sq) { *sq = fmaf(p, p, *sq); *sq = fmaf(q, q, *sq); }
    }
}

// ------------------------------------------------------------------ phase P2
template <int DT>
__device__ __forceinline__ void phase_p2(const WaveArgs& a, WaveShared& S, int b, int k, int s) {
    constexpr int VEC = Elem<DT>::VEC;
    const RowArgs& R = a.r;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = R.K, L = len_of(R, b), NR = 2 * K + 1;
    if (k > L) return;
    const SeqInfo si = a.sinfo[b];
    if (si.n < 0) return;                                  // fatal sequence
    const bool pair = k < L;
    if (!pair && si.draw_row != L) return;                 // bonus row not needed
    const bool draw = si.draw_row == k;
    const float tau = tau_of(R, b);
    const float c = kLog2e / tau;
    const RowScale SP = row_scale(a.rstat[(int64_t)b * NR + k]);
    RowScale SQ; SQ.m = 0.f; SQ.frac = 0.f; SQ.inv = 0.f;
    if (pair) SQ = row_scale(a.rstat[(int64_t)b * NR + K + 1 + k]);
    const int v0 = s * a.slice_vecs;
    const int nv = max(min(a.slice_vecs, R.nvec - v0), 0);
    const char* prow = row_ptr(R, b, k) + (int64_t)v0 * 16;
    const char* qrow = pair ? row_ptr(R, b, K + 1 + k) + (int64_t)v0 * 16 : nullptr;
    float z0 = 0.f, z1 = 0.f, sqs = 0.f;
    double zd = 0.0;
    for (int i0 = tid; i0 < nv; i0 += WT * 2) {
        uint4 rp[2], rq[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int v = i0 + u * WT;
            rp[u] = neg_inf_vec<DT>(); rq[u] = neg_inf_vec<DT>();
            if (v < nv) {
                rp[u] = ldg16(prow + (size_t)v * 16);
                if (pair) rq[u] = ldg16(qrow + (size_t)v * 16);
                const int gbase = (v0 + v) * VEC;
                if (gbase + VEC > R.V) { mask_tail<DT>(rp[u], R.V - gbase); mask_tail<DT>(rq[u], R.V - gbase); }
            }
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            if (i0 + u * WT < nv) {
                float r[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) r[i] = 0.f;
                residual_vec<DT>(rp[u], rq[u], pair, c, SP, SQ, r, draw ? &sqs : nullptr);
                const float vs = ((r[0] + r[1]) + (r[2] + r[3])) + ((r[4] + r[5]) + (r[6] + r[7]));
                if (u) z1 += vs; else z0 += vs;
                if (draw) zd += (double)vs;
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
            a.zpart[((int64_t)b * K + k) * a.T + s] = zz;
        }
        if (draw) {
            double tot = 0.0; float sq = 0.f;
            for (int w = 0; w < WW; ++w) { tot += S.redd[w]; sq += S.redf[1][w]; }
            DPart d; d.tot = tot; d.sq = sq; d.pad = 0;
            a.dpart[(int64_t)b * a.T + s] = d;
        }
    }
}

// ------------------------------------------------------------------ phase D
template <int DT>
__device__ __forceinline__ void phase_d(const WaveArgs& a, WaveShared& S, int b) {
    constexpr int VEC = Elem<DT>::VEC;
    const RowArgs& R = a.r;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = R.K, L = len_of(R, b), NR = 2 * K + 1, T = a.T;
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
        S.base = base; S.Ttarget = Tt; S.bound = draw_bound(sumsq, (double)si.sys);
    }
    __syncthreads();
    const int s = S.owner_slice;
    int found_y = -1, found_cert = 0;
    if (s >= 0) {
        const float tau = tau_of(R, b);
        const float c = kLog2e / tau;
        const RowScale SP = row_scale(a.rstat[(int64_t)b * NR + k]);
        RowScale SQ; SQ.m = 0.f; SQ.frac = 0.f; SQ.inv = 0.f;
        if (pair) SQ = row_scale(a.rstat[(int64_t)b * NR + K + 1 + k]);
        const int v0 = s * a.slice_vecs;
        const int nv = max(min(a.slice_vecs, R.nvec - v0), 0);
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
            residual_vec<DT>(rp, rq, pair, c, SP, SQ, r, nullptr);
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
                    residual_vec<DT>(rp, rq, pair, c, SP, SQ, r, nullptr);
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
    const int K = a.r.K, T = a.T, NR = 2 * K + 1;
    int next = 0;
    if (tid == 0) next = atomicAdd(a.ticket, 1);
    for (;;) {
        if (tid == 0) {
            const int t = next;
            S.ticket = t;
            if (t < a.ntickets) {
                // closed-form schedule: P1(0..lag), then per wave w: A(w), P2(w), P1(w+lag+1), D(w-1); last D(nw-1)
                const int B = a.r.B, WS = a.wave_seqs, LAG = a.lag;
                auto N = [&](int w) { return w <= 0 ? 0 : min(B, w * WS); };           // sequences in the first w waves
                const long long c0 = (long long)NR * T, c2 = (long long)(K + 1) * T;
                const long long P = c0 * N(LAG + 1);
                int ph, wv; long long off;
                if (t < P) { ph = 0; wv = (int)(t / (c0 * WS)); off = t - c0 * N(wv); }
                else {
                    auto F = [&](int w) { return (long long)N(w) * (1 + c2) + c0 * (N(w + LAG + 1) - N(LAG + 1)) + N(w - 1); };
                    const long long tt = t - P;
                    int lo = 0, hi = a.nwaves;
                    while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if (F(mid) <= tt) lo = mid; else hi = mid - 1; }
                    const int w = lo;
                    long long o2 = tt - F(w);
                    const long long nA = N(w + 1) - N(w), n2 = nA * c2, n1 = c0 * (N(w + LAG + 2) - N(w + LAG + 1));
                    if (o2 < nA) { ph = 1; wv = w; off = o2; }
                    else if (o2 < nA + n2) { ph = 2; wv = w; off = o2 - nA; }
                    else if (o2 < nA + n2 + n1) { ph = 0; wv = w + LAG + 1; off = o2 - nA - n2; }
                    else { ph = 3; wv = w - 1; off = o2 - nA - n2 - n1; }
                }
                struct { int phase, wave; } sg = {ph, wv};
                S.phase = ph; S.wave = wv; S.index = (int)off;
                next = atomicAdd(a.ticket, 1);
                // dependencies: counters of the wave (almost always long satisfied)
                const int w = sg.wave;
                const int b0 = w * a.wave_seqs, ns = min(a.wave_seqs, a.r.B - b0);
                bool okw = true;
                if (sg.phase == 1) okw = spin_ge(&a.p1done[w], ns * NR * T);
                else if (sg.phase == 2) okw = spin_ge(&a.adone[w], ns);
                else if (sg.phase == 3) okw = spin_ge(&a.p2done[w], ns * (K + 1) * T);
                if (!okw) atomicExch(a.wait_failed, 1);
            }
        }
        __syncthreads();
        if (S.ticket >= a.ntickets) break;
        const int phase = S.phase, w = S.wave, idx = S.index;
        const int b0 = w * a.wave_seqs;
        if (phase == 0) {
            const int s = idx % T, r = (idx / T) % NR, b = b0 + idx / (T * NR);
            phase_p1<DT>(a, S, b, r, s);
            __syncthreads();
            if (tid == 0) { __threadfence(); atomicAdd(&a.p1done[w], 1); }
        } else if (phase == 1) {
            phase_a<DT>(a, S, b0 + idx);
            __syncthreads();
            if (tid == 0) { __threadfence(); atomicAdd(&a.adone[w], 1); }
        } else if (phase == 2) {
            const int s = idx % T, k = (idx / T) % (K + 1), b = b0 + idx / (T * (K + 1));
            phase_p2<DT>(a, S, b, k, s);
            __syncthreads();
            if (tid == 0) { __threadfence(); atomicAdd(&a.p2done[w], 1); }
        } else {
            phase_d<DT>(a, S, b0 + idx);
        }
        __syncthreads();
    }
}

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
    wa.T = wp.T; wa.slice_vecs = wp.slice_vecs; wa.wave_seqs = wp.wave_seqs; wa.nwaves = wp.nwaves;
    // number of tickets: every phase of every wave
    {
        const long long NR = 2 * a.K + 1;
        const long long total = (long long)a.B * (NR * wp.T + 1 + (long long)(a.K + 1) * wp.T + 1);
        if (total > 0x7fff0000LL) return cudaSuccess;
        wa.ntickets = (int)total;
        wa.lag = wp.lag;
    }
    cudaError_t e = cudaMemsetAsync(w, 0, wp.zero_bytes, stream);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(wa.fb_count, 0, sizeof(int), stream);
    if (e != cudaSuccess) return e;
    const int grid = wa.ntickets < grid_max ? wa.ntickets : grid_max;
    if (a.dt == 0) k_wave<0><<<grid, WT, 0, stream>>>(wa);
    else k_wave<1><<<grid, WT, 0, stream>>>(wa);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    k_wave_flag<<<(a.B + 255) / 256, 256, 0, stream>>>(wa.wait_failed, o.row_status, a.B);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    *launched = true;
    return general_draw_list(a, p, u_final, o, ws, wa.fb_list, wa.fb_count, stream);
}

}  // namespace bebop
