// Fused verify kernel: one thread-block cluster walks the row pairs of a
// sequence in order, reads every logit from HBM exactly once and computes one
// exponential per logit.
//
//   - each CTA of the cluster owns a contiguous vocabulary slice; a bulk
//     asynchronous copy (TMA, no multicast) brings the slice of the target row
//     and of the draft row into a two-stage shared-memory ring two items ahead;
//   - every thread keeps the exponentials of its contiguous chunk in registers,
//     relative to a per-CTA power-of-two reference, so the cluster-wide merge
//     of the softmax normalisers is exact (integer exponents + fp64 sums) and
//     needs one exchange through distributed shared memory per row pair;
//   - with the normalisers known: accept test (fp32, re-done in fp64 near the
//     margin), TV = sum max(0, p - q) from the registers, and at the stop row
//     the residual prefix scan (fp64 across threads) with the inverse-CDF
//     crossing located by the thread that owns it;
//   - the draw is accepted only if the crossing clears an error bound derived
//     from the fp32 element error (see draw_bound); otherwise the sequence is
//     appended to a list and re-drawn by the fp64 kernels of the general path;
//   - sequences whose drafts are all accepted get their bonus row in a second
//     phase of the same kernel, through the same ring.
//
// Control flow is uniform across the cluster: every decision that changes the
// number of cluster barriers is computed from exchanged data by every CTA in
// the same way.  Waits on the copy barriers are bounded; an expired wait sets
// BEBOP_ROW_WAIT_EXPIRED and the kernel carries on (results undefined, flagged).
#include "bebop_kernels.h"
#include "bebop_ptx.cuh"

namespace bebop {

namespace {

constexpr int FT = 512;          // threads per CTA
constexpr int CS = 8;            // CTAs per cluster
constexpr int NWARP = FT / 32;
constexpr int E_EMPTY = INT_MIN / 2;   // exponent reference of a slice without finite logits
#ifndef BEBOP_TMA_CHUNK
#define BEBOP_TMA_CHUNK 4096
#endif
constexpr uint32_t kChunk = BEBOP_TMA_CHUNK;   // bytes per bulk copy (multiple of 16)
constexpr double kEClamp = 268435456.0;   // |max logit / tau * log2 e| beyond 2^28 saturates

// flags exchanged per CTA slice
constexpr int F_BAD = 1;         // NaN or +inf seen

// ----------------------------------------------------------------- shared state
struct __align__(16) Slot {      // per (parity, source rank): softmax partials of one item
    double sp, sq;               // sum 2^(x*c - E) over the slice (target, draft)
    int ep, eq;                  // integer exponent references E_c
    float zprev;                 // slice part of Z of the PREVIOUS item
    int flags;                   // F_BAD bits: bit0 target, bit1 draft
};
struct __align__(16) DSlot {     // per source rank: draw partials of the stop row
    double tot;                  // residual mass of the slice
    float sq;                    // sum p^2 + q^2 over the slice
    int pad;
};
struct __align__(8) RSlot {      // per source rank: result of the owner's walk
    int y;                       // token, or -1 when this CTA does not own the crossing
    int certified;
};

struct Shared {
    unsigned long long full[2];          // copy barriers of the two stages
    Slot slot[2][CS];
    DSlot dslot[CS];
    RSlot rslot[CS];
    int wmax[2][2];                      // [parity][row] block max (ordered-int), reset by thread 0
    double wsum[NWARP][2];               // warp sums (target, draft)
    double wscan[NWARP];                 // warp totals for the fp64 scan
    float wz[NWARP];
    float wsq[NWARP];
    // broadcast of the merged row state (written by thread 0 after the exchange)
    float a_c, b_c;                      // per-CTA scale: p = e * a_c, q = e * b_c
    int stop_here, bad;
    double cta_off, Ttarget, bound;
    int wait_failed;
};

struct FusedArgs {
    RowArgs r;
    const int32_t* draft_tokens;
    const float* u_accept;
    const float* u_final;
    VerifyOut o;
    int* stop;
    int* fb_count;
    int* fb_list;
    int vs;                              // vectors per CTA slice
    long long* trace;                    // BEBOP_TRACE builds only: clock stamps of cluster 0
};
#ifdef BEBOP_TRACE
#define TRACE(id) do { if (a.trace && cid == 0 && rank == 0 && tid == 0 && item < 60) a.trace[item * 16 + (id)] = clock64(); } while (0)
#else
#define TRACE(id) do {} while (0)
#endif

__device__ __forceinline__ float tau_of(const RowArgs& a, int b) { return a.temperature ? a.temperature[b] : a.temperature_all; }
__device__ __forceinline__ bool tau_ok(float t) { return t > 0.f && t < INFINITY; }
__device__ __forceinline__ int len_of(const RowArgs& a, int b) {
    int L = a.draft_len ? a.draft_len[b] : a.K;
    return max(0, min(L, a.K));
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

// One row of one item, per thread: raw -> exponentials relative to 2^E_c.
template <int DT, int NV>
struct RowRegs {
    float e[NV * Elem<DT>::VEC];
};

}  // namespace

// =============================================================================
template <int DT, int NV>
__global__ void __launch_bounds__(FT, 1) k_fused(const FusedArgs a) {
    constexpr int VEC = Elem<DT>::VEC;
    constexpr int NE = NV * VEC;
    constexpr int ROW_BYTES = FT * NV * 16;             // stage bytes per row slice (capacity)
    extern __shared__ __align__(128) unsigned char smem_raw[];
    unsigned char* stage = smem_raw;                    // [2 stages][2 rows][ROW_BYTES]
    Shared& S = *reinterpret_cast<Shared*>(smem_raw + 4 * ROW_BYTES);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rank = (int)cluster_rank();
    const int cid = (int)cluster_id(), ncl = (int)num_clusters();
    const RowArgs& R = a.r;
    const int K = R.K, V = R.V, B = R.B;

    // this CTA's slice of every row, in 16-byte vectors
    const int v_begin = min(rank * a.vs, R.nvec);
    const int nv_cta = min(a.vs, R.nvec - v_begin);
    const uint32_t slice_bytes = (uint32_t)nv_cta * 16u;
    const int64_t slice_off = (int64_t)v_begin * 16;
    const int lv0 = tid * NV;                            // first local vector of this thread

    if (tid == 0) {
        mbar_init(smem_u32(&S.full[0]), 1);
        mbar_init(smem_u32(&S.full[1]), 1);
        S.wmax[0][0] = S.wmax[0][1] = S.wmax[1][0] = S.wmax[1][1] = INT_MIN;
        S.wait_failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    __syncthreads();
    cluster_arrive();
    cluster_wait();

    // ---- item stream of this cluster: phase 1 = row pairs of sequences cid, cid+ncl, ...;
    //      phase 2 = bonus rows of those of them that accepted every draft.
    // A cursor enumerates phase-1 items; every thread advances identical cursors.
    struct Cursor { int b, k, L; };
    auto first_item = [&](Cursor& c) {
        c.b = cid; c.k = 0;
        while (c.b < B && (c.L = len_of(R, c.b)) == 0) c.b += ncl;
    };
    auto next_item = [&](Cursor& c) {
        if (c.b >= B) return;
        if (++c.k < c.L) return;
        c.k = 0; c.b += ncl;
        while (c.b < B && (c.L = len_of(R, c.b)) == 0) c.b += ncl;
    };
    // bonus list: kept in shared memory, identical in every CTA of the cluster
    __shared__ int bonus_list[1024];
    __shared__ int bonus_count;
    __shared__ int bonus_overflow;
    if (tid == 0) { bonus_count = 0; bonus_overflow = 0; }

    auto issue = [&](int st, const char* prow, const char* qrow) {
        // warp 0 only: lane 0 arms the barrier, then the lanes start the copies of this CTA's
        // slice in chunks of kChunk bytes (many small bulk copies keep more requests in flight
        // than one large one)
        if (nv_cta <= 0) return;
        const uint32_t bar = smem_u32(&S.full[st]);
        const uint32_t dst = smem_u32(stage + (size_t)st * 2 * ROW_BYTES);
        if (lane == 0) mbar_expect_tx(bar, qrow ? 2 * slice_bytes : slice_bytes);
        __syncwarp();
        const uint32_t nchunk = (slice_bytes + kChunk - 1) / kChunk;
        for (uint32_t cidx = lane; cidx < (qrow ? 2 * nchunk : nchunk); cidx += 32) {
            const uint32_t row = cidx >= nchunk ? 1u : 0u, cc = cidx - row * nchunk;
            const uint32_t off = cc * kChunk, len = min(kChunk, slice_bytes - off);
            bulk_g2s(dst + row * ROW_BYTES + off, (row ? qrow : prow) + slice_off + off, len, bar);
        }
    };
    auto trow = [&](int b, int k) { return R.target + ((int64_t)b * R.t_seq_rows + k) * R.t_row_bytes; };
    auto drow = [&](int b, int k) { return R.draft + ((int64_t)b * R.d_seq_rows + k) * R.d_row_bytes; };

    // sequences with no drafts go straight to the bonus list (all CTAs agree)
    if (tid == 0) {
        for (int b = cid; b < B; b += ncl) {
            if (len_of(R, b) == 0) {
                if (bonus_count < 1024) bonus_list[bonus_count++] = b; else bonus_overflow = 1;
            }
        }
    }
    __syncthreads();

    Cursor cur, ld;
    first_item(cur);
    ld = cur;
    // prologue: fill both stages
    uint32_t use[2] = {0, 0};                            // completed uses per stage (parity tracking)
    for (int s = 0; s < 2; ++s) {
        if (ld.b < B) { if (warp == 0) issue(s, trow(ld.b, ld.k), drow(ld.b, ld.k)); next_item(ld); }
    }

    // per-sequence state, identical in every thread of the cluster
    int seq_alive = 1, seq_n = 0, seq_st = 0;
    // deferred outputs of the previous item (its Z arrives with the next exchange)
    int prev_b = -1, prev_k = 0, prev_fatal = 0;
    float my_zprev = 0.f;                                // this CTA's Z part of the previous item (thread 0)
    int pend_draw_b = -1, pend_draw_n = 0;               // draw whose result sits in rslot

    int item = 0;
    int phase = 1;
    int bonus_pos = 0, bonus_ld = 0;

    for (;;) {
        // ------------------------------------------------ what is this item?
        int b, k, L;
        bool pair;
        if (phase == 1 && cur.b >= B) {
            // phase 1 is over for this cluster: both stages are free; start streaming bonus rows
            phase = 2;
            __syncthreads();
            if (warp == 0) {
                fence_proxy_async();
                for (int s = 0; s < 2 && s < bonus_count; ++s) {
                    int bb = bonus_list[s];
                    issue((item + s) & 1, trow(bb, len_of(R, bb)), nullptr);
                }
            }
            bonus_ld = min(2, bonus_count);
        }
        if (phase == 1) { b = cur.b; k = cur.k; L = cur.L; pair = true; }
        else if (bonus_pos < bonus_count) { b = bonus_list[bonus_pos]; L = len_of(R, b); k = L; pair = false; }
        else if (prev_b >= 0 || pend_draw_b >= 0) { b = -1; k = 0; L = 0; pair = false; }
        else break;
        const int st = item & 1;
        const bool have_rows = b >= 0;
        TRACE(0);

        float tau = 1.f;
        if (have_rows) tau = tau_of(R, b);
        const bool tok_tau_ok = tau_ok(tau);
        const float c = kLog2e / (tok_tau_ok ? tau : 1.f);
        const double c64 = 1.4426950408889634 / (double)(tok_tau_ok ? tau : 1.f);

        if (have_rows && pair && k == 0) {
            // a bad temperature, then a bad token id, pre-empt everything else
            seq_alive = 1; seq_n = L; seq_st = tok_tau_ok ? 0 : ST_BAD_TEMP;
            if (!seq_st)
                for (int j = 0; j < L; ++j) {
                    int t = a.draft_tokens[(int64_t)b * K + j];
                    if (t < 0 || t >= V) seq_st |= ST_BAD_TOKEN;
                }
        }
        if (have_rows && !pair) seq_st = tok_tau_ok ? 0 : ST_BAD_TEMP;

        // gathered logits of the drafted token (thread 0, consumed after the exchange)
        float zpx = 0.f, zqx = 0.f, u_acc = 0.5f;
        if (tid == 0 && have_rows && pair) {
            int tk = min(max(a.draft_tokens[(int64_t)b * K + k], 0), V - 1);
            zpx = DT == 0 ? load_one<0>(trow(b, k), tk) : load_one<1>(trow(b, k), tk);
            zqx = DT == 0 ? load_one<0>(drow(b, k), tk) : load_one<1>(drow(b, k), tk);
            u_acc = a.u_accept[(int64_t)b * K + k];
        }

        // ------------------------------------------------ ingest: stage -> registers
        float ep[NE], eq[NE];
        double sp_c = 0.0, sq_c = 0.0;
        int Ep = E_EMPTY, Eq = E_EMPTY, flags = 0;
        if (have_rows) {
            uint4 rp[NV], rq[NV];
            if (nv_cta > 0) {
                bool ok = mbar_wait(smem_u32(&S.full[st]), use[st] & 1);
                if (!ok) S.wait_failed = 1;
            }
            use[st]++;
            TRACE(1);
            const unsigned char* sp_ = stage + (size_t)st * 2 * ROW_BYTES;
#pragma unroll
            for (int j = 0; j < NV; ++j) {
                int lv = lv0 + j;
                if (lv < nv_cta) {
                    rp[j] = *reinterpret_cast<const uint4*>(sp_ + (size_t)lv * 16);
                    rq[j] = pair ? *reinterpret_cast<const uint4*>(sp_ + ROW_BYTES + (size_t)lv * 16) : neg_inf_vec<DT>();
                    int gbase = (v_begin + lv) * VEC;
                    if (gbase + VEC > V) { mask_tail<DT>(rp[j], V - gbase); mask_tail<DT>(rq[j], V - gbase); }
                } else {
                    rp[j] = neg_inf_vec<DT>(); rq[j] = neg_inf_vec<DT>();
                }
            }
            // thread max -> warp max -> block max (ordered ints, shared atomics)
            float mp = vec_max<DT>(rp[0]), mq = vec_max<DT>(rq[0]);
#pragma unroll
            for (int j = 1; j < NV; ++j) { mp = max_nan(mp, vec_max<DT>(rp[j])); mq = max_nan(mq, vec_max<DT>(rq[j])); }
            int op = redux_max(f2ord(mp)), oq = redux_max(f2ord(mq));
            if (lane == 0) { atomicMax(&S.wmax[st][0], op); atomicMax(&S.wmax[st][1], oq); }
            __syncthreads();                             // also: every read of the stage is done
            TRACE(2);
            if (warp == 0) {
                // refill this stage with the item two ahead
                fence_proxy_async();
                if (phase == 1) {
                    if (ld.b < B) { issue(st, trow(ld.b, ld.k), drow(ld.b, ld.k)); }
                } else if (bonus_ld < bonus_count) {
                    int bb = bonus_list[bonus_ld];
                    issue(st, trow(bb, len_of(R, bb)), nullptr);
                }
            }
            mp = ord2f(S.wmax[st][0]); mq = ord2f(S.wmax[st][1]);
            // exponent references: E = ceil(m * c) so that 2^(x*c - E) <= 1
            float fp_ = 0.f, fq_ = 0.f, mp_use = 0.f, mq_use = 0.f;
            if (mp != mp || mp == INFINITY) flags |= F_BAD;
            else if (mp != -INFINITY) { double t = fmin(fmax((double)mp * c64, -kEClamp), kEClamp); double E = ceil(t); Ep = (int)E; fp_ = (float)(E - t); mp_use = mp; }
            if (pair) {
                if (mq != mq || mq == INFINITY) flags |= 2 * F_BAD;
                else if (mq != -INFINITY) { double t = fmin(fmax((double)mq * c64, -kEClamp), kEClamp); double E = ceil(t); Eq = (int)E; fq_ = (float)(E - t); mq_use = mq; }
            }
            float s_p = 0.f, s_q = 0.f;
#pragma unroll
            for (int j = 0; j < NV; ++j) {
                float f[VEC];
                unpack<DT>(rp[j], f);
#pragma unroll
                for (int i = 0; i < VEC; ++i) {
                    float e = ex2f(fmaf(f[i] - mp_use, c, -fp_));
                    ep[j * VEC + i] = e; s_p += e;
                }
            }
            if (pair) {
#pragma unroll
                for (int j = 0; j < NV; ++j) {
                    float f[VEC];
                    unpack<DT>(rq[j], f);
#pragma unroll
                    for (int i = 0; i < VEC; ++i) {
                        float e = ex2f(fmaf(f[i] - mq_use, c, -fq_));
                        eq[j * VEC + i] = e; s_q += e;
                    }
                }
            } else {
#pragma unroll
                for (int i = 0; i < NE; ++i) eq[i] = 0.f;
            }
            TRACE(3);
            // block sums in double
            double dp = (double)s_p, dq = (double)s_q;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) { dp += shfl_xor_d(dp, o); dq += shfl_xor_d(dq, o); }
            if (lane == 0) { S.wsum[warp][0] = dp; S.wsum[warp][1] = dq; }
        } else {
#pragma unroll
            for (int i = 0; i < NE; ++i) { ep[i] = 0.f; eq[i] = 0.f; }
        }
        __syncthreads();
        if (tid == 0) {
            S.wmax[st][0] = INT_MIN; S.wmax[st][1] = INT_MIN;     // reset for the item after next
            for (int w = 0; w < NWARP; ++w) { sp_c += S.wsum[w][0]; sq_c += S.wsum[w][1]; }
            if (!have_rows) { sp_c = 0.0; sq_c = 0.0; }
        }
        if (phase == 1) { if (have_rows) next_item(ld); } else if (have_rows) { bonus_ld++; }
        // NOTE: in phase 2 the first two bonus items are issued when phase 2 begins (below).

        TRACE(4);
        // ------------------------------------------------ exchange through DSMEM
        if (tid < CS) {
            // thread `tid` delivers this CTA's partials to CTA `tid`
            double sp0 = __shfl_sync(0xffu, sp_c, 0), sq0 = __shfl_sync(0xffu, sq_c, 0);
            float z0 = __shfl_sync(0xffu, my_zprev, 0);
            uint32_t dst = mapa(smem_u32(&S.slot[st][rank]), (uint32_t)tid);
            uint4 w0, w1;
            w0.x = (uint32_t)__double2loint(sp0); w0.y = (uint32_t)__double2hiint(sp0);
            w0.z = (uint32_t)__double2loint(sq0); w0.w = (uint32_t)__double2hiint(sq0);
            w1.x = (uint32_t)Ep; w1.y = (uint32_t)Eq; w1.z = __float_as_uint(z0); w1.w = (uint32_t)flags;
            st_cluster_v4(dst, w0);
            st_cluster_v4(dst + 16, w1);
        }
        __syncwarp();
        cluster_arrive();
        cluster_wait();
        TRACE(5);

        // ------------------------------------------------ merge (warp 0), accept test (thread 0)
        if (warp == 0) {
            Slot sl;
            if (lane < CS) sl = S.slot[st][lane]; else { sl.sp = sl.sq = 0.0; sl.ep = sl.eq = E_EMPTY; sl.zprev = 0.f; sl.flags = 0; }
            int Em_p = redux_max(sl.ep), Em_q = redux_max(sl.eq);
            double tp = sl.ep > E_EMPTY ? sl.sp * pow2d(max(sl.ep - Em_p, -2000)) : 0.0;
            double tq = sl.eq > E_EMPTY ? sl.sq * pow2d(max(sl.eq - Em_q, -2000)) : 0.0;
            float zp = sl.zprev;
            int fl = sl.flags;
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) {
                tp += shfl_xor_d(tp, o); tq += shfl_xor_d(tq, o);
                zp += __shfl_xor_sync(0xffffffffu, zp, o);
                fl |= __shfl_xor_sync(0xffffffffu, fl, o);
            }
            if (lane == 0) {
                // ---- outputs of the previous item that were waiting for its Z
                if (rank == 0 && prev_b >= 0 && a.o.tv)
                    a.o.tv[(int64_t)prev_b * K + prev_k] = prev_fatal ? 0.f : fminf(fmaxf(zp, 0.f), 1.f);
                // ---- status of this item
                int bad = 0;
                if (have_rows) {
                    bad |= (fl & F_BAD) || !(tp == tp) ? ST_NONFINITE : (Em_p == E_EMPTY ? ST_EMPTY : 0);
                    if (pair) bad |= (fl & (2 * F_BAD)) || !(tq == tq) ? ST_NONFINITE : (Em_q == E_EMPTY ? ST_EMPTY : 0);
                }
                S.bad = bad;
                const double Sp = tp, Sq = tq;
                // this CTA's scale factors: p = e * 2^(Ep - Em_p) / Sp
                float ac = 0.f, bc = 0.f;
                if (have_rows && !bad) {
                    ac = Ep > E_EMPTY ? (float)(pow2d(max(Ep - Em_p, -2000)) * __drcp_rn(Sp)) : 0.f;
                    if (pair) bc = Eq > E_EMPTY ? (float)(pow2d(max(Eq - Em_q, -2000)) * __drcp_rn(Sq)) : 0.f;
                }
                S.a_c = ac; S.b_c = bc;
                int stop_here = 0;
                if (have_rows && pair && !bad && !(seq_st & ST_FATAL)) {
                    // p(x), q(x): fp32 first, fp64 when the test is close
                    float pxf = ex2f(zpx * c - (float)Em_p) / (float)Sp;
                    float qxf = ex2f(zqx * c - (float)Em_q) / (float)Sq;
                    float lhs = u_acc * qxf;
                    bool acc = lhs < pxf;
                    double pxd = pxf, qxd = qxf;
                    if (fabsf(lhs - pxf) <= 1e-3f * fmaxf(lhs, pxf)) {
                        pxd = exp2((double)zpx * c64 - (double)Em_p) / Sp;
                        qxd = exp2((double)zqx * c64 - (double)Em_q) / Sq;
                        acc = (double)u_acc * qxd < pxd;
                    }
                    if (rank == 0) {
                        if (a.o.p_draft) a.o.p_draft[(int64_t)b * K + k] = (float)pxd;
                        if (a.o.q_draft) a.o.q_draft[(int64_t)b * K + k] = (float)qxd;
                    }
                    if (seq_alive && !acc) stop_here = 1;
                }
                S.stop_here = stop_here;
            }
        }
        __syncthreads();
        TRACE(6);
        const int bad = S.bad;
        const int stop_here = S.stop_here;
        const float a_c = S.a_c, b_c = S.b_c;
        if (have_rows && !(seq_st & ST_FATAL)) seq_st |= bad;   // only the first bad row counts
        const bool do_draw = have_rows && !(seq_st & ST_FATAL) && (pair ? stop_here != 0 : true);

        // pending draw result of an earlier item (delivered by the exchange above)
        if (pend_draw_b >= 0 && rank == 0 && tid == 0) {
            int y = -1, cert = 0, owners = 0;
            for (int r = 0; r < CS; ++r) if (S.rslot[r].y >= 0) { y = S.rslot[r].y; cert = S.rslot[r].certified; owners++; }
            if (owners == 1 && cert) a.o.out_tokens[(int64_t)pend_draw_b * (K + 1) + pend_draw_n] = y;
            else { int idx = atomicAdd(a.fb_count, 1); a.fb_list[idx] = pend_draw_b; }
        }
        pend_draw_b = -1;

        // ------------------------------------------------ phase 2 of the item: TV (and draw sums)
        float z_t = 0.f;
        double zt64 = 0.0;
        float sq_t = 0.f;
        if (have_rows && !bad) {
            if (!do_draw) {
                float z0 = 0.f, z1 = 0.f;
#pragma unroll
                for (int i = 0; i < NE; i += 2) {
                    z0 += fmaxf(__fmul_rn(ep[i], a_c) - __fmul_rn(eq[i], b_c), 0.f);
                    z1 += fmaxf(__fmul_rn(ep[i + 1], a_c) - __fmul_rn(eq[i + 1], b_c), 0.f);
                }
                z_t = z0 + z1;
            } else {
#pragma unroll
                for (int j = 0; j < NV; ++j) {
                    float r[VEC];
#pragma unroll
                    for (int i = 0; i < VEC; ++i) {
                        float p = __fmul_rn(ep[j * VEC + i], a_c), q = __fmul_rn(eq[j * VEC + i], b_c);
                        r[i] = fmaxf(p - q, 0.f);
                        sq_t = fmaf(p, p, sq_t); sq_t = fmaf(q, q, sq_t);
                    }
                    // pairwise sum of the vector, then double across vectors
#pragma unroll
                    for (int w = 1; w < VEC; w <<= 1)
#pragma unroll
                        for (int i = 0; i + w < VEC; i += 2 * w) r[i] += r[i + w];
                    z_t += r[0];
                    zt64 += (double)r[0];
                }
            }
        }
        // block sum of z (fp32) for TV
        {
            float zw = warp_sum(z_t);
            if (lane == 0) S.wz[warp] = zw;
        }
        double incl = 0.0;
        if (do_draw) {
            // inclusive scan of the chunk sums within the warp (double)
            incl = zt64;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) { double t = shfl_up_d(incl, d); if (lane >= d) incl += t; }
            if (lane == 31) S.wscan[warp] = incl;
            float sw = warp_sum(sq_t);
            if (lane == 0) S.wsq[warp] = sw;
        }
        __syncthreads();
        if (tid == 0) {
            float z = 0.f;
            for (int w = 0; w < NWARP; ++w) z += S.wz[w];
            my_zprev = pair && have_rows ? z : 0.f;
        }

        TRACE(7);
        // record what the next exchange has to flush
        if (have_rows && pair) { prev_b = b; prev_k = k; prev_fatal = (seq_st & ST_FATAL) ? 1 : 0; }
        else prev_b = -1;

        if (do_draw) {     // uniform across the cluster
            // CTA total and warp offsets (serial, so that the partition of the line is consistent)
            double woff = 0.0, ctot = 0.0;
            for (int w = 0; w < NWARP; ++w) { if (w == warp) woff = ctot; ctot += S.wscan[w]; }
            if (tid < CS) {
                float sq = 0.f;
                for (int w = 0; w < NWARP; ++w) sq += S.wsq[w];
                uint32_t dst = mapa(smem_u32(&S.dslot[rank]), (uint32_t)tid);
                uint4 w0;
                w0.x = (uint32_t)__double2loint(ctot); w0.y = (uint32_t)__double2hiint(ctot);
                w0.z = __float_as_uint(sq); w0.w = 0;
                st_cluster_v4(dst, w0);
            }
            __syncwarp();
            cluster_arrive();
            cluster_wait();
            if (tid == 0) {
                double off = 0.0, Z = 0.0, sumsq = 0.0;
                for (int r = 0; r < CS; ++r) { if (r == rank) off = Z; Z += S.dslot[r].tot; sumsq += (double)S.dslot[r].sq; }
                S.cta_off = off;
                S.Ttarget = (double)a.u_final[b] * Z;
                S.bound = draw_bound(sumsq);
            }
            __syncthreads();
            const double T = S.Ttarget;
            const double base = S.cta_off + woff;
            double prev_incl = shfl_up_d(incl, 1);
            if (lane == 0) prev_incl = 0.0;
            const double lower = base + prev_incl, upper = base + incl;
            int my_y = -1, my_cert = 0;
            if (T > 0.0 && lower < T && T <= upper) {
                // this thread owns the crossing: walk its elements
                double C = lower, bound = S.bound;
                const int g0 = (v_begin + lv0) * VEC;
#pragma unroll
                for (int i = 0; i < NE; ++i) {
                    if (my_y < 0) {
                        float p = __fmul_rn(ep[i], a_c), q = __fmul_rn(eq[i], b_c);
                        double r = (double)fmaxf(p - q, 0.f);
                        double Cn = C + r;
                        if (r > 0.0 && Cn >= T) {
                            my_y = g0 + i;
                            my_cert = (T - C > bound) && (Cn - T >= bound);
                        }
                        C = Cn;
                    }
                }
            }
            // one owner at most per warp; deliver this CTA's result to rank 0
            unsigned own = __ballot_sync(0xffffffffu, my_y >= 0);
            if (own) {
                int src = __ffs(own) - 1;
                int y = __shfl_sync(0xffffffffu, my_y, src), ce = __shfl_sync(0xffffffffu, my_cert, src);
                if (lane == 0) { S.wz[warp] = __int_as_float(y); S.wsq[warp] = __int_as_float(ce); }
            } else if (lane == 0) { S.wz[warp] = __int_as_float(-1); S.wsq[warp] = __int_as_float(0); }
            __syncthreads();
            if (tid == 0) {
                int y = -1, ce = 0, cnt = 0;
                for (int w = 0; w < NWARP; ++w) { int yy = __float_as_int(S.wz[w]); if (yy >= 0) { y = yy; ce = __float_as_int(S.wsq[w]); cnt++; } }
                if (cnt > 1) ce = 0;
                uint32_t dst = mapa(smem_u32(&S.rslot[rank]), 0u);
                asm volatile("st.shared::cluster.v2.b32 [%0], {%1,%2};" :: "r"(dst), "r"(y), "r"(ce) : "memory");
            }
            pend_draw_b = b; pend_draw_n = pair ? k : L;
            __syncthreads();
        }

        // ------------------------------------------------ sequence bookkeeping
        if (have_rows && pair) {
            if (stop_here) { seq_alive = 0; seq_n = k; }
            if (k == L - 1) {
                // last pair of the sequence: integer outputs (rank 0), bonus list (every CTA)
                const bool fatal = (seq_st & ST_FATAL) != 0;
                if (rank == 0 && tid <= K) {
                    int n = fatal ? 0 : seq_n;
                    int t = (tid < n) ? a.draft_tokens[(int64_t)b * K + tid] : -1;
                    // position n belongs to the draw (already delivered, pending, or re-drawn later)
                    if (fatal || tid != n) a.o.out_tokens[(int64_t)b * (K + 1) + tid] = t;
                    if (tid == 0) {
                        a.o.accept_len[b] = n;
                        a.stop[b] = fatal ? -1 : n;
                        if (a.o.row_status) a.o.row_status[b] = seq_st;
                    }
                    if (fatal && tid < K) {
                        if (a.o.tv) a.o.tv[(int64_t)b * K + tid] = 0.f;
                        if (a.o.p_draft) a.o.p_draft[(int64_t)b * K + tid] = 0.f;
                        if (a.o.q_draft) a.o.q_draft[(int64_t)b * K + tid] = 0.f;
                    }
                }
                if (!fatal && seq_alive && tid == 0) {
                    if (bonus_count < 1024) bonus_list[bonus_count++] = b; else bonus_overflow = 1;
                }
                // zero padding of the ragged outputs
                if (rank == 0 && tid >= L && tid < K) {
                    if (a.o.tv) a.o.tv[(int64_t)b * K + tid] = 0.f;
                    if (a.o.p_draft) a.o.p_draft[(int64_t)b * K + tid] = 0.f;
                    if (a.o.q_draft) a.o.q_draft[(int64_t)b * K + tid] = 0.f;
                }
            }
            next_item(cur);
        } else if (have_rows && !pair) {
            // bonus item: L == 0 sequences get their integer outputs here
            const bool fatal = (seq_st & ST_FATAL) != 0;
            if (rank == 0 && tid <= K) {
                if (L == 0 || fatal) {
                    if (fatal || tid != 0) a.o.out_tokens[(int64_t)b * (K + 1) + tid] = -1;
                    if (tid < K) {
                        if (a.o.tv) a.o.tv[(int64_t)b * K + tid] = 0.f;
                        if (a.o.p_draft) a.o.p_draft[(int64_t)b * K + tid] = 0.f;
                        if (a.o.q_draft) a.o.q_draft[(int64_t)b * K + tid] = 0.f;
                    }
                    if (tid == 0) {
                        a.o.accept_len[b] = 0;
                        float tb = tau_of(R, b);
                        int stb = (tau_ok(tb) ? 0 : ST_BAD_TEMP) | seq_st;
                        if (L == 0) { a.stop[b] = (stb & ST_FATAL) ? -1 : 0; if (a.o.row_status) a.o.row_status[b] = stb; }
                        else { a.stop[b] = -1; if (a.o.row_status) a.o.row_status[b] |= stb; }
                    }
                }
            }
            bonus_pos++;
        }
        TRACE(8);
        ++item;
    }

    // make sure no CTA exits while a peer may still write into its shared memory
    cluster_arrive();
    cluster_wait();
    if (tid == 0 && S.wait_failed && a.o.row_status) {
        for (int b = cid; b < B; b += ncl) atomicOr(&a.o.row_status[b], ST_WAIT);
    }
}

// -----------------------------------------------------------------------------
namespace {

template <int DT, int NV>
cudaError_t launch_fused(const FusedArgs& fa, int num_clusters, cudaStream_t stream) {
    constexpr size_t smem = 4 * (size_t)FT * NV * 16 + sizeof(Shared) + 128;
    static bool configured[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(k_fused<DT, NV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(num_clusters * CS), 1, 1);
    cfg.blockDim = dim3(FT, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CS; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_fused<DT, NV>, fa);
}

template <int DT, int NV>
int max_clusters() {
    static int cached[64] = {0};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && cached[dev]) return cached[dev];
    constexpr size_t smem = 4 * (size_t)FT * NV * 16 + sizeof(Shared) + 128;
    cudaFuncSetAttribute(k_fused<DT, NV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(CS * 64, 1, 1);
    cfg.blockDim = dim3(FT, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CS; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, k_fused<DT, NV>, &cfg) != cudaSuccess || n < 1) { cudaGetLastError(); n = 0; }
    if (dev >= 0 && dev < 64) cached[dev] = n;
    return n;
}

}  // namespace

// Shapes the fused kernel takes: every CTA slice fits the per-thread register
// chunks (nvec <= CS * FT * NV) and is not degenerate, at most 1024 bonus rows
// per cluster.
bool fused_supported(const RowArgs& a) {
    constexpr int NV = 5;
    if (((((a.nvec + CS - 1) / CS) + 7) & ~7) > FT * NV) return false;
    if (a.nvec < 4 * CS) return false;
    return true;
}

long long* g_trace = nullptr;
void fused_set_trace(long long* p) { g_trace = p; }

int fused_max_clusters(int dt) { return dt == 0 ? max_clusters<0, 5>() : max_clusters<1, 5>(); }

cudaError_t fused_verify(const RowArgs& a, const Plan& p, const int32_t* draft_tokens,
                         const float* u_accept, const float* u_final, VerifyOut o, char* ws,
                         cudaStream_t stream, bool* launched) {
    constexpr int NV = 5;
    *launched = false;
    int ncl = a.dt == 0 ? max_clusters<0, NV>() : max_clusters<1, NV>();
    if (ncl < 1) return cudaSuccess;
    if (ncl > a.B) ncl = a.B;
    if ((a.B + ncl - 1) / ncl > 1024) return cudaSuccess;   // bonus list capacity
    FusedArgs fa;
    fa.r = a; fa.draft_tokens = draft_tokens; fa.u_accept = u_accept; fa.u_final = u_final; fa.o = o;
    fa.stop = reinterpret_cast<int*>(ws + p.off_stop);
    fa.fb_count = reinterpret_cast<int*>(ws + p.off_fb);
    fa.fb_list = fa.fb_count + 16;
    fa.vs = (((a.nvec + CS - 1) / CS) + 7) & ~7;   // slices start on 128-byte boundaries
    fa.trace = g_trace;
    cudaError_t e = cudaMemsetAsync(fa.fb_count, 0, sizeof(int), stream);
    if (e != cudaSuccess) return e;
    e = a.dt == 0 ? launch_fused<0, NV>(fa, ncl, stream) : launch_fused<1, NV>(fa, ncl, stream);
    if (e != cudaSuccess) return e;
    *launched = true;
    return general_draw_list(a, p, u_final, o, ws, fa.fb_list, fa.fb_count, stream);
}

}  // namespace bebop
