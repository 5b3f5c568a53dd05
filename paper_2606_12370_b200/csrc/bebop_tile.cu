// Tile kernel: the single-read, one-exponential-per-logit hot path of bebop_verify.
//
// A logit row is cut into T tiles of at most TILE_VECS 16-byte vectors, each a
// multiple of 128 bytes.  One task = one tile of one row pair (target row k and
// draft row k of sequence b) or of one bonus row.  A persistent grid of 256-thread
// CTAs, several per SM, takes tasks in order from a ticket counter:
//
//   1. coalesced 128-bit loads of the tile (both rows) into registers;
//   2. block maximum -> power-of-two reference 2^E of the tile; one exponential
//      per logit, relative to 2^E, written to shared memory; block sum;
//   3. the tile's partial (E, S) goes to a workspace in global memory and a
//      per-row counter is bumped; the CTA waits (bounded) until the T partials
//      of its row are in.  Tiles of one row hold consecutive tickets, so they run
//      at the same time on different SMs; the other CTAs of the SM hide the wait;
//   4. every tile merges the T partials exactly (integer exponents, fp64 sums) and
//      evaluates the accept test of its row; the accept chain of the sequence is
//      read from flags the earlier rows left behind;
//   5. TV = sum max(0, p - q) from the exponentials in shared memory; the last
//      tile to finish adds the T parts in tile order;
//   6. at the stop row (or the bonus row) the tiles exchange their residual mass,
//      the tile holding the inverse-CDF crossing scans its per-vector sums and the
//      owning thread walks its eight tokens.  The draw is kept only if it clears
//      the error bound of draw_bound(); otherwise the sequence goes to the list
//      the fp64 kernels re-draw.
//
// Progress: tickets are handed out in order and a task only ever waits for tasks
// with smaller or equal row index, all of which hold tickets already; so the
// lowest unfinished row always runs to completion.  Every wait is bounded; an
// expired wait raises BEBOP_ROW_WAIT_EXPIRED and the CTA carries on.
#include "bebop_kernels.h"
#include "bebop_ptx.cuh"

namespace bebop {

namespace {

constexpr int TT = 256;              // threads per CTA
constexpr int TW = TT / 32;
constexpr int TILE_VECS = kTileVecs;  // vectors per row and tile, at most
constexpr int VPT = (TILE_VECS + TT - 1) / TT;   // vectors per thread and row (3)
constexpr int E_EMPTY = INT_MIN / 2;
constexpr uint32_t kSpin = 1u << 22; // bound of every spin on a global flag

struct __align__(16) TPart { double sp, sq; int ep, eq, flags, pad; };   // per-tile softmax partial
struct __align__(16) TDraw { double tot; float sq; int pad; };           // per-tile residual mass

// workspace of the tile kernel (all counters and flags are zeroed before the launch)
struct TileWs {
    int* ticket;          // [1]
    int* rowcnt;          // [B*(K+1)]  tiles whose partial is in
    int* zcnt;            // [B*(K+1)]  tiles whose Z part is in
    int* dcnt;            // [B]        tiles whose residual mass is in
    int* rcnt;            // [B]        tiles that reported the result of the walk
    int* rowres;          // [B*(K+1)]  1 accepted, 2 rejected, 3 first fatal row (0: not known yet)
    int* seqn;            // [B]        n + 1 once the accept scan of the sequence is over, -1 fatal
    int* dres;            // [B]        token found by the owner of the crossing (-1 none), certified flag in bit 30
    TPart* part;          // [B*(K+1)][T]
    float* zpart;         // [B*(K+1)][T]
    TDraw* dpart;         // [B][T]
};

struct TileArgs {
    RowArgs r;
    const int32_t* draft_tokens;
    const float* u_accept;
    const float* u_final;
    VerifyOut o;
    int* stop;
    int* fb_count;
    int* fb_list;
    int* wait_failed;
    TileWs w;
    int T, tile_vecs;
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
// spin until *p >= want (bounded); returns false if it gave up
__device__ __forceinline__ bool spin_ge(const int* p, int want) {
    for (uint32_t i = 0; i < kSpin; ++i) {
        if (ld_acquire(p) >= want) return true;
        __nanosleep(40);
    }
    return false;
}
__device__ __forceinline__ bool spin_nz(const int* p, int* out) {
    for (uint32_t i = 0; i < kSpin; ++i) {
        int v = ld_acquire(p);
        if (v != 0) { *out = v; return true; }
        __nanosleep(40);
    }
    *out = 0;
    return false;
}

// The error bound a draw must clear.  The residual is formed from fp32
// exponentials (ex2.approx: 2 ulp) and fp32 products, so each p, q carries a
// relative error of a few 2^-24; the errors of different tokens are independent,
// hence the error of a prefix sum is of the order delta * sqrt(sum p^2 + q^2).
// kappa leaves a wide safety factor over that root-sum-square.
__device__ __forceinline__ double draw_bound(double sumsq) {
    const double delta = 2.384185791015625e-07;   // 2^-22
    const double kappa = 16.0;
    return kappa * delta * sqrt(sumsq) + 1e-300;
}

__device__ __forceinline__ int row_status(int flagbit, int E, double S) {
    if (flagbit || !(S == S)) return ST_NONFINITE;
    return E == E_EMPTY ? ST_EMPTY : 0;
}

// E = ceil(m * c), frac = E - m * c in [0, 1] without rounding loss (see bebop_ring.cu)
__device__ __forceinline__ void tile_reference(float m, float c, int* E, float* frac) {
    float th = fminf(fmaxf(m * c, -4.0e6f), 4.0e6f);
    float te = fmaf(m, c, -th);
    if (th != m * c) te = 0.f;
    float Ef;
    int Ei = ceil_alu(th, &Ef);
    float f = (Ef - th) - te;
    if (f < 0.f) { f += 1.f; Ei += 1; }
    *E = Ei; *frac = f;
}

struct TileShared {
    float4 e[2][2][TILE_VECS];    // [row][half][vector]: exponentials (half 0: elements 0-3, half 1: 4-7)
    float vsum[TILE_VECS];        // per-vector residual mass (draw)
    float redf[2][TW];
    double redd[TW];
    int redi[2][TW];
    // broadcast block of the control thread
    int task;
    int Ep, Eq, bad, stop_here, do_draw, skip, alive;
    float a_hi, a_lo, b_hi, b_lo;
    double base, Ttarget, bound;
    int owner;
};

}  // namespace

template <int DT>
__global__ void __launch_bounds__(TT, 4) k_tile(const TileArgs a, int ntasks) {
    constexpr int VEC = Elem<DT>::VEC;
    __shared__ TileShared S;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const RowArgs& R = a.r;
    const int K = R.K, V = R.V, T = a.T;

    for (;;) {
        if (tid == 0) S.task = atomicAdd(a.w.ticket, 1);
        __syncthreads();
        const int task = S.task;
        if (task >= ntasks) break;
        const int tile = task % T, row = task / T;
        const int b = row / (K + 1), k = row % (K + 1);
        const int L = len_of(R, b);
        if (k > L) { __syncthreads(); continue; }
        const bool pair = k < L;
        const float tau = tau_of(R, b);
        const bool tok_ok = tau_ok(tau);
        const float c = kLog2e / (tok_ok ? tau : 1.f);

        // ---- bonus row: only when every draft of the sequence was accepted
        if (!pair) {
            if (tid == 0) {
                int n1 = 0, skip = 0;
                if (L > 0) { if (!spin_nz(&a.w.seqn[b], &n1)) { atomicExch(a.wait_failed, 1); skip = 1; } if (n1 != L + 1) skip = 1; }
                S.skip = skip;
            }
            __syncthreads();
            if (S.skip) { __syncthreads(); continue; }
        }

        // ---- 1. load the tile
        const int v0 = tile * a.tile_vecs;
        const int nv = max(min(a.tile_vecs, R.nvec - v0), 0);
        const char* prow = R.target + ((int64_t)b * R.t_seq_rows + k) * R.t_row_bytes + (int64_t)v0 * 16;
        const char* qrow = pair ? R.draft + ((int64_t)b * R.d_seq_rows + k) * R.d_row_bytes + (int64_t)v0 * 16 : nullptr;
        uint4 rp[VPT], rq[VPT];
#pragma unroll
        for (int j = 0; j < VPT; ++j) {
            const int v = j * TT + tid;
            rp[j] = neg_inf_vec<DT>(); rq[j] = neg_inf_vec<DT>();
            if (v < nv) {
                rp[j] = ldg16_stream(prow + (size_t)v * 16);
                if (pair) rq[j] = ldg16_stream(qrow + (size_t)v * 16);
            }
        }
        // gathered logits of the drafted token (thread 0, needed after the merge)
        float zpx = 0.f, zqx = 0.f, u_acc = 0.5f;
        int st0 = tok_ok ? 0 : ST_BAD_TEMP;
        if (tid == 0 && pair) {
            if (!st0)
                for (int j = 0; j < L; ++j) { int tk = a.draft_tokens[(int64_t)b * K + j]; if (tk < 0 || tk >= V) st0 = ST_BAD_TOKEN; }
            int tk = min(max(a.draft_tokens[(int64_t)b * K + k], 0), V - 1);
            const char* pr = R.target + ((int64_t)b * R.t_seq_rows + k) * R.t_row_bytes;
            const char* qr = R.draft + ((int64_t)b * R.d_seq_rows + k) * R.d_row_bytes;
            zpx = DT == 0 ? load_one<0>(pr, tk) : load_one<1>(pr, tk);
            zqx = DT == 0 ? load_one<0>(qr, tk) : load_one<1>(qr, tk);
            u_acc = a.u_accept[(int64_t)b * K + k];
        }
#pragma unroll
        for (int j = 0; j < VPT; ++j) {
            const int gbase = (v0 + j * TT + tid) * VEC;
            if (j * TT + tid < nv && gbase + VEC > V) { mask_tail<DT>(rp[j], V - gbase); mask_tail<DT>(rq[j], V - gbase); }
        }

        // ---- 2. block maximum, reference, exponentials, block sum
        float mp = vec_max<DT>(rp[0]), mq = vec_max<DT>(rq[0]);
#pragma unroll
        for (int j = 1; j < VPT; ++j) { mp = max_nan(mp, vec_max<DT>(rp[j])); mq = max_nan(mq, vec_max<DT>(rq[j])); }
        {
            int op = redux_max(f2ord(mp)), oq = redux_max(f2ord(mq));
            if (lane == 0) { S.redi[0][warp] = op; S.redi[1][warp] = oq; }
        }
        __syncthreads();
        {
            int op = S.redi[0][0], oq = S.redi[1][0];
#pragma unroll
            for (int w = 1; w < TW; ++w) { op = max(op, S.redi[0][w]); oq = max(oq, S.redi[1][w]); }
            mp = ord2f(op); mq = ord2f(oq);
        }
        int Ep = E_EMPTY, Eq = E_EMPTY, flags = 0;
        float fp_ = 0.f, fq_ = 0.f, mpu = 0.f, mqu = 0.f;
        if (mp != mp || mp == INFINITY) flags |= 1;
        else if (mp != -INFINITY) { tile_reference(mp, c, &Ep, &fp_); mpu = mp; }
        if (pair) {
            if (mq != mq || mq == INFINITY) flags |= 2;
            else if (mq != -INFINITY) { tile_reference(mq, c, &Eq, &fq_); mqu = mq; }
        }
        float s_p = 0.f, s_q = 0.f;
#pragma unroll
        for (int j = 0; j < VPT; ++j) {
            const int v = j * TT + tid;
            if (v < nv) {
                float f[VEC], e[8];
                unpack<DT>(rp[j], f);
#pragma unroll
                for (int i = 0; i < VEC; ++i) { e[i] = ex2f(fmaf(f[i] - mpu, c, -fp_)); s_p += e[i]; }
#pragma unroll
                for (int i = VEC; i < 8; ++i) e[i] = 0.f;
                S.e[0][0][v] = make_float4(e[0], e[1], e[2], e[3]);
                if (VEC == 8) S.e[0][1][v] = make_float4(e[4], e[5], e[6], e[7]);
                if (pair) {
                    unpack<DT>(rq[j], f);
#pragma unroll
                    for (int i = 0; i < VEC; ++i) { e[i] = ex2f(fmaf(f[i] - mqu, c, -fq_)); s_q += e[i]; }
                    S.e[1][0][v] = make_float4(e[0], e[1], e[2], e[3]);
                    if (VEC == 8) S.e[1][1][v] = make_float4(e[4], e[5], e[6], e[7]);
                }
            }
        }
        s_p = warp_sum(s_p); s_q = warp_sum(s_q);
        if (lane == 0) { S.redf[0][warp] = s_p; S.redf[1][warp] = s_q; }
        __syncthreads();

        // ---- 3. publish the partial, wait for the row, 4. merge, accept
        if (tid == 0) {
            double sp = 0.0, sq = 0.0;
            for (int w = 0; w < TW; ++w) { sp += (double)S.redf[0][w]; sq += (double)S.redf[1][w]; }
            TPart p; p.sp = (flags & 1) ? 0.0 : sp; p.sq = (flags & 2) ? 0.0 : sq; p.ep = Ep; p.eq = Eq; p.flags = flags; p.pad = 0;
            a.w.part[(int64_t)row * T + tile] = p;
            __threadfence();
            atomicAdd(&a.w.rowcnt[row], 1);
            if (!spin_ge(&a.w.rowcnt[row], T)) atomicExch(a.wait_failed, 1);
            // merge (in tile order)
            int Em_p = E_EMPTY, Em_q = E_EMPTY, fl = 0;
            const TPart* pp = a.w.part + (int64_t)row * T;
            for (int i = 0; i < T; ++i) { Em_p = max(Em_p, pp[i].ep); Em_q = max(Em_q, pp[i].eq); fl |= pp[i].flags; }
            double Sp = 0.0, Sq = 0.0;
            for (int i = 0; i < T; ++i) {
                if (pp[i].ep > E_EMPTY) Sp += pp[i].sp * pow2d(max(pp[i].ep - Em_p, -1000));
                if (pp[i].eq > E_EMPTY) Sq += pp[i].sq * pow2d(max(pp[i].eq - Em_q, -1000));
            }
            int bad = row_status(fl & 1, Em_p, Sp);
            if (pair) bad |= row_status(fl & 2, Em_q, Sq);
            double iSp = 0.0, iSq = 0.0;
            if (!bad) { iSp = 1.0 / Sp; if (pair) iSq = 1.0 / Sq; }
            // accept chain: rows before this one
            int alive = 1, seq_fatal = st0;
            if (pair) {
                for (int kk = 0; kk < k && alive && !seq_fatal; ++kk) {
                    int rr;
                    if (!spin_nz(&a.w.rowres[(int64_t)b * (K + 1) + kk], &rr)) { atomicExch(a.wait_failed, 1); rr = 2; }
                    if (rr == 2) alive = 0;
                    if (rr == 3) seq_fatal = 1;
                }
            }
            int stop_here = 0, acc = 0;
            double pxd = 0.0, qxd = 0.0;
            if (pair && !bad && !seq_fatal) {
                float pxf = ex2f(fmaf(zpx, c, -(float)Em_p)) * (float)iSp;
                float qxf = ex2f(fmaf(zqx, c, -(float)Em_q)) * (float)iSq;
                float lhs = u_acc * qxf;
                acc = lhs < pxf;
                pxd = pxf; qxd = qxf;
                if (fabsf(lhs - pxf) <= 1e-3f * fmaxf(lhs, pxf)) {
                    const double cd = (double)c;
                    pxd = exp2((double)zpx * cd - (double)Em_p) * iSp;
                    qxd = exp2((double)zqx * cd - (double)Em_q) * iSq;
                    acc = (double)u_acc * qxd < pxd;
                }
                if (alive && !acc) stop_here = 1;
            }
            const int fatal_here = (!seq_fatal && bad) ? 1 : 0;     // first fatal row of the sequence
            if (tile == 0) {
                // outputs and flags of this row (one writer per row)
                if (pair && !bad && !seq_fatal) {
                    if (a.o.p_draft) a.o.p_draft[(int64_t)b * K + k] = (float)pxd;
                    if (a.o.q_draft) a.o.q_draft[(int64_t)b * K + k] = (float)qxd;
                }
                const int status_now = seq_fatal ? st0 : bad;
                if (pair) {
                    if ((st0 && k == 0) || fatal_here) {
                        if (a.o.row_status) a.o.row_status[b] = status_now;
                        a.stop[b] = -1;
                        __threadfence();
                        atomicExch(&a.w.seqn[b], -1);
                    } else if (!seq_fatal && alive && (stop_here || k == L - 1)) {
                        const int n = stop_here ? k : L;
                        a.o.accept_len[b] = n;
                        a.stop[b] = n;
                        if (a.o.row_status) a.o.row_status[b] = 0;
                        for (int q = 0; q <= K; ++q)
                            if (q != n) a.o.out_tokens[(int64_t)b * (K + 1) + q] = q < n ? a.draft_tokens[(int64_t)b * K + q] : -1;
                        __threadfence();
                        atomicExch(&a.w.seqn[b], n + 1);
                    }
                    __threadfence();
                    atomicExch(&a.w.rowres[(int64_t)b * (K + 1) + k], (seq_fatal || bad) ? 3 : (acc ? 1 : 2));
                } else {
                    // bonus row: L == 0 sequences get their integer outputs here
                    if (L == 0) {
                        const int st = st0 | bad;
                        a.o.accept_len[b] = 0;
                        a.stop[b] = (st & ST_FATAL) ? -1 : 0;
                        if (a.o.row_status) a.o.row_status[b] = st;
                        for (int q = 1; q <= K; ++q) a.o.out_tokens[(int64_t)b * (K + 1) + q] = -1;
                        if (st & ST_FATAL) a.o.out_tokens[(int64_t)b * (K + 1)] = -1;
                    } else if (bad) {
                        // other tiles of this row may still be reading seqn: only stop[] marks the fatal state
                        if (a.o.row_status) a.o.row_status[b] |= bad;
                        a.stop[b] = -1;
                    }
                }
            }
            const bool fatal = seq_fatal || bad;
            S.bad = fatal ? 1 : 0;
            S.Ep = Em_p; S.Eq = Em_q;
            S.stop_here = stop_here;
            S.do_draw = (!fatal && (pair ? stop_here : 1)) ? 1 : 0;
            const double sa = Ep > E_EMPTY ? pow2d(max(Ep - Em_p, -1000)) * iSp : 0.0;
            const double sb = Eq > E_EMPTY ? pow2d(max(Eq - Em_q, -1000)) * iSq : 0.0;
            S.a_hi = (float)sa; S.a_lo = (float)(sa - (double)S.a_hi);
            S.b_hi = (float)sb; S.b_lo = (float)(sb - (double)S.b_hi);
        }
        __syncthreads();
        const int bad = S.bad, do_draw = S.do_draw;
        const float a_hi = S.a_hi, a_lo = S.a_lo, b_hi = S.b_hi, b_lo = S.b_lo;

        // ---- 5. TV part of this tile (and the per-vector sums of a draw)
        float z_t = 0.f, sq_t = 0.f;
        double zd_t = 0.0;
        if (!bad) {
#pragma unroll
            for (int j = 0; j < VPT; ++j) {
                const int v = j * TT + tid;
                if (v < nv) {
                    float ep[8], eq[8];
                    { float4 x = S.e[0][0][v]; ep[0] = x.x; ep[1] = x.y; ep[2] = x.z; ep[3] = x.w; }
                    if (VEC == 8) { float4 x = S.e[0][1][v]; ep[4] = x.x; ep[5] = x.y; ep[6] = x.z; ep[7] = x.w; }
                    if (pair) {
                        { float4 x = S.e[1][0][v]; eq[0] = x.x; eq[1] = x.y; eq[2] = x.z; eq[3] = x.w; }
                        if (VEC == 8) { float4 x = S.e[1][1][v]; eq[4] = x.x; eq[5] = x.y; eq[6] = x.z; eq[7] = x.w; }
                    } else {
#pragma unroll
                        for (int i = 0; i < 8; ++i) eq[i] = 0.f;
                    }
                    if (!do_draw) {
#pragma unroll
                        for (int i = 0; i < VEC; ++i) z_t += fmaxf(fmaf(ep[i], a_hi, -__fmul_rn(eq[i], b_hi)), 0.f);
                    } else {
                        float r[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) r[i] = 0.f;
#pragma unroll
                        for (int i = 0; i < VEC; ++i) {
                            const float p = fmaf(ep[i], a_lo, __fmul_rn(ep[i], a_hi));
                            const float q = fmaf(eq[i], b_lo, __fmul_rn(eq[i], b_hi));
                            r[i] = fmaxf(p - q, 0.f);
                            sq_t = fmaf(p, p, sq_t); sq_t = fmaf(q, q, sq_t);
                        }
                        const float vs = ((r[0] + r[1]) + (r[2] + r[3])) + ((r[4] + r[5]) + (r[6] + r[7]));
                        S.vsum[v] = vs;
                        z_t += vs;
                        zd_t += (double)vs;
                    }
                }
            }
        }
        z_t = warp_sum(z_t);
        if (lane == 0) S.redf[0][warp] = z_t;
        if (do_draw) {
            sq_t = warp_sum(sq_t);
            zd_t = warp_sum(zd_t);
            if (lane == 0) { S.redf[1][warp] = sq_t; S.redd[warp] = zd_t; }
        }
        __syncthreads();
        if (tid == 0) {
            if (pair) {
                float z = 0.f;
                for (int w = 0; w < TW; ++w) z += S.redf[0][w];
                a.w.zpart[(int64_t)row * T + tile] = z;
                __threadfence();
                if (atomicAdd(&a.w.zcnt[row], 1) == T - 1) {
                    __threadfence();
                    float zz = 0.f;
                    for (int i = 0; i < T; ++i) zz += a.w.zpart[(int64_t)row * T + i];
                    if (a.o.tv) a.o.tv[(int64_t)b * K + k] = bad ? 0.f : fminf(fmaxf(zz, 0.f), 1.f);
                }
            }
            // ---- 6. the draw: exchange the residual masses of the tiles
            int owner = 0;
            if (do_draw) {
                double tot = 0.0; float sq = 0.f;
                for (int w = 0; w < TW; ++w) { tot += S.redd[w]; sq += S.redf[1][w]; }
                TDraw d; d.tot = tot; d.sq = sq; d.pad = 0;
                a.w.dpart[(int64_t)b * T + tile] = d;
                __threadfence();
                atomicAdd(&a.w.dcnt[b], 1);
                if (!spin_ge(&a.w.dcnt[b], T)) atomicExch(a.wait_failed, 1);
                double base = 0.0, Z = 0.0, sumsq = 0.0, mytot = 0.0;
                for (int i = 0; i < T; ++i) {
                    const TDraw di = a.w.dpart[(int64_t)b * T + i];
                    if (i == tile) { base = Z; mytot = di.tot; }
                    Z += di.tot; sumsq += (double)di.sq;
                }
                const double Tt = (double)a.u_final[b] * Z;
                S.base = base; S.Ttarget = Tt; S.bound = draw_bound(sumsq);
                owner = (Tt > base && Tt <= base + mytot) ? 1 : 0;
            }
            S.owner = owner;
        }
        __syncthreads();
        if (do_draw) {
            int found_y = -1, found_cert = 0;
            if (S.owner) {
                // prefix over the per-vector sums in vector order: thread t scans vectors [t*VPT', ...)
                // Simple and exact in order: every warp takes a contiguous range of vectors.
                const int per = (nv + TT - 1) / TT;             // vectors per thread, contiguous ranges
                const int vb = min(tid * per, nv), ve = min(vb + per, nv);
                double mine = 0.0;
                for (int v = vb; v < ve; ++v) mine += (double)S.vsum[v];
                // inclusive scan over threads (warp scan + warp totals)
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
                            // walk the eight tokens of this vector
                            float ep[8], eq[8];
                            { float4 x = S.e[0][0][v]; ep[0] = x.x; ep[1] = x.y; ep[2] = x.z; ep[3] = x.w; }
                            { float4 x = S.e[0][1][v]; ep[4] = x.x; ep[5] = x.y; ep[6] = x.z; ep[7] = x.w; }
                            { float4 x = S.e[1][0][v]; eq[0] = x.x; eq[1] = x.y; eq[2] = x.z; eq[3] = x.w; }
                            { float4 x = S.e[1][1][v]; eq[4] = x.x; eq[5] = x.y; eq[6] = x.z; eq[7] = x.w; }
                            double Cw = C;
                            for (int i = 0; i < VEC && found_y < 0; ++i) {
                                const float p = fmaf(ep[i], a_lo, __fmul_rn(ep[i], a_hi));
                                const float q = pair ? fmaf(eq[i], b_lo, __fmul_rn(eq[i], b_hi)) : 0.f;
                                const double r1 = (double)fmaxf(p - q, 0.f);
                                const double Cn = Cw + r1;
                                if (r1 > 0.0 && Cn >= Tt) { found_y = (v0 + v) * VEC + i; found_cert = (Tt - Cw > bound) && (Cn - Tt >= bound); }
                                Cw = Cn;
                            }
                            break;
                        }
                        C = nxt;
                    }
                }
            }
            // block-level result -> global; the last tile to report settles the sequence
            unsigned ownmask = __ballot_sync(0xffffffffu, found_y >= 0);
            if (ownmask && lane == (__ffs(ownmask) - 1)) {
                const int cert = (__popc(ownmask) == 1) ? found_cert : 0;
                atomicMax(&a.w.dres[b], (found_y + 1) | (cert ? (1 << 30) : 0));
            }
            __syncthreads();
            if (tid == 0) {
                __threadfence();
                if (atomicAdd(&a.w.rcnt[b], 1) == T - 1) {
                    __threadfence();
                    const int res = ld_acquire(&a.w.dres[b]);
                    const int n = pair ? k : L;
                    const int y1 = res & ~(1 << 30);
                    if ((res & (1 << 30)) && y1 >= 1 && y1 <= V) a.o.out_tokens[(int64_t)b * (K + 1) + n] = y1 - 1;
                    else { int idx = atomicAdd(a.fb_count, 1); a.fb_list[idx] = b; }
                }
            }
        }
        __syncthreads();
    }
}

// Outputs that depend on the final state of a sequence: fatal rows and ragged padding.
__global__ void k_tile_fixup(RowArgs R, VerifyOut o, const int* __restrict__ stop, const int* __restrict__ wait_failed) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= R.B) return;
    const int K = R.K;
    const int L = max(0, min(R.draft_len ? R.draft_len[b] : K, K));
    const bool fatal = stop[b] < 0;
    if (fatal) {
        o.accept_len[b] = 0;
        for (int q = 0; q <= K; ++q) o.out_tokens[(int64_t)b * (K + 1) + q] = -1;
    }
    for (int q = 0; q < K; ++q) {
        if (fatal || q >= L) {
            if (o.tv) o.tv[(int64_t)b * K + q] = 0.f;
            if (o.p_draft) o.p_draft[(int64_t)b * K + q] = 0.f;
            if (o.q_draft) o.q_draft[(int64_t)b * K + q] = 0.f;
        }
    }
    if (*wait_failed && o.row_status) o.row_status[b] |= ST_WAIT;
}

// -----------------------------------------------------------------------------
namespace {

template <int DT>
int tile_grid() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (dev >= 0 && dev < 64 && cached[dev]) return cached[dev];
    int per_sm = 0, sms = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_tile<DT>, TT, 0) != cudaSuccess) per_sm = 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaGetLastError();
    const int n = per_sm * sms;
    if (dev >= 0 && dev < 64) cached[dev] = n;
    return n;
}

}  // namespace

bool tile_supported(const RowArgs& a) { return a.nvec >= 1; }

cudaError_t tile_verify(const RowArgs& a, const Plan& p, const int32_t* draft_tokens,
                        const float* u_accept, const float* u_final, VerifyOut o, char* ws,
                        cudaStream_t stream, bool* launched) {
    *launched = false;
    const int grid_max = a.dt == 0 ? tile_grid<0>() : tile_grid<1>();
    if (grid_max < 1) return cudaSuccess;
    TileArgs ta;
    ta.r = a; ta.draft_tokens = draft_tokens; ta.u_accept = u_accept; ta.u_final = u_final; ta.o = o;
    ta.stop = reinterpret_cast<int*>(ws + p.off_stop);
    ta.fb_count = reinterpret_cast<int*>(ws + p.off_fb);
    ta.fb_list = ta.fb_count + 16;
    ta.T = (a.nvec + TILE_VECS - 1) / TILE_VECS;
    ta.tile_vecs = (((a.nvec + ta.T - 1) / ta.T) + 7) & ~7;
    const size_t rows = (size_t)a.B * (a.K + 1);
    char* w = ws + p.off_tile;
    ta.w.ticket = reinterpret_cast<int*>(w);
    ta.wait_failed = ta.w.ticket + 1;
    size_t off = 256;
    ta.w.rowcnt = reinterpret_cast<int*>(w + off); off += align256(sizeof(int) * rows);
    ta.w.zcnt = reinterpret_cast<int*>(w + off); off += align256(sizeof(int) * rows);
    ta.w.rowres = reinterpret_cast<int*>(w + off); off += align256(sizeof(int) * rows);
    ta.w.dcnt = reinterpret_cast<int*>(w + off); off += align256(sizeof(int) * (size_t)a.B);
    ta.w.rcnt = reinterpret_cast<int*>(w + off); off += align256(sizeof(int) * (size_t)a.B);
    ta.w.seqn = reinterpret_cast<int*>(w + off); off += align256(sizeof(int) * (size_t)a.B);
    ta.w.dres = reinterpret_cast<int*>(w + off); off += align256(sizeof(int) * (size_t)a.B);
    const size_t zero_bytes = tile_ws_zero_bytes(a.B, a.K);
    ta.w.part = reinterpret_cast<TPart*>(w + off); off += align256(sizeof(TPart) * rows * ta.T);
    ta.w.zpart = reinterpret_cast<float*>(w + off); off += align256(sizeof(float) * rows * ta.T);
    ta.w.dpart = reinterpret_cast<TDraw*>(w + off);
    cudaError_t e = cudaMemsetAsync(w, 0, zero_bytes, stream);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(ta.fb_count, 0, sizeof(int), stream);
    if (e != cudaSuccess) return e;
    const long long ntasks = (long long)rows * ta.T;
    if (ntasks > 0x7fffffffLL - grid_max) return cudaSuccess;
    const int grid = (int)(ntasks < grid_max ? ntasks : grid_max);
    if (a.dt == 0) k_tile<0><<<grid, TT, 0, stream>>>(ta, (int)ntasks);
    else k_tile<1><<<grid, TT, 0, stream>>>(ta, (int)ntasks);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    k_tile_fixup<<<(a.B + 127) / 128, 128, 0, stream>>>(a, o, ta.stop, ta.wait_failed);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    *launched = true;
    return general_draw_list(a, p, u_final, o, ws, ta.fb_list, ta.fb_count, stream);
}

}  // namespace bebop
