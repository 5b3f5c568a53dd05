// Streaming verify kernel: the single-read, one-exponential-per-logit hot path.
//
// A cluster of CS CTAs walks the row pairs of its sequences in order.  Each CTA
// owns a contiguous, 128-byte aligned vocabulary slice of every row; bulk
// asynchronous copies (TMA, no multicast) stream the slices of the target and
// the draft row into a two-stage shared-memory ring two items ahead.
//
// Warps run free: there is no block-wide or cluster-wide barrier in the steady
// state.  A warp reads its contiguous chunk of the stage, keeps one exponential
// per logit in registers relative to its own power-of-two reference 2^E_w, and
// publishes (E_w, fixed-point sum).  The last warp of a CTA to publish combines
// the sixteen partials exactly (integer exponents, integer sums) and sends the
// CTA partial to every CTA of the cluster through distributed shared memory,
// arriving on their mbarriers.  A warp that needs the row normalisers waits on
// its CTA's mbarrier, merges the CS partials (exact scaling, fp64 sums) and runs
// the accept test, TV = sum max(0, p - q) and, at the stop row, the residual
// prefix scan whose crossing is located by the thread that owns it.
//
// The draw is kept only if the crossing clears an error bound derived from the
// fp32 element error (draw_bound); otherwise the sequence is appended to a list
// that the fp64 kernels of the general path re-draw.  Sequences that accept
// every draft get their bonus row in a second phase through the same ring.
//
// Every decision that changes what a warp waits for is computed from the same
// exchanged data by every warp, so all warps of a cluster agree on the item
// stream.  Every wait is bounded; an expired wait raises BEBOP_ROW_WAIT_EXPIRED
// and the warp carries on (results undefined, flagged).
#include "bebop_kernels.h"
#include "bebop_ptx.cuh"

namespace bebop {

namespace {

constexpr int NT = 512;            // threads per CTA
constexpr int NW = NT / 32;        // warps per CTA
constexpr int CS = 8;              // CTAs per cluster
constexpr int RING = 4;            // depth of the exchange rings
constexpr int MAXSEQ = 128;        // sequences per cluster and launch (two 64-bit bonus masks)
constexpr int E_EMPTY = INT_MIN / 2;
constexpr double kEClamp = 268435456.0;   // |max logit / tau * log2 e| beyond 2^28 saturates
constexpr double kFix = 1099511627776.0;  // 2^40: fixed-point scale of the per-thread sums
#ifndef BEBOP_TMA_CHUNK
#define BEBOP_TMA_CHUNK 8192
#endif
constexpr uint32_t kChunk = BEBOP_TMA_CHUNK;

struct __align__(16) WPart { long long sp, sq; int ep, eq, flags, pad; };   // per-warp softmax partial
struct __align__(16) CPart { double sp, sq; int ep, eq, flags, pad; };      // per-CTA softmax partial
struct __align__(16) DPart { double tot; float sq; int pad; };              // residual mass and sum of squares
struct __align__(8) RPart { int y, cert; };                                  // result of an owner's walk

struct StreamShared {
    unsigned long long full[2];
    unsigned long long stats_bar[RING], draw_bar[RING], z_bar[RING], res_bar[RING];
    int relcnt[2];
    int wcnt[RING], zcnt[RING], dcnt[RING], rcnt[RING];
    WPart wpart[RING][NW];
    CPart cslot[RING][CS];
    float wz[RING][NW];
    float zslot[RING][CS];
    DPart wdraw[RING][NW];
    DPart dslot[RING][CS];
    RPart wres[RING][NW];
    RPart rslot[RING][CS];
    int wait_failed;
};

struct StreamArgs {
    RowArgs r;
    const int32_t* draft_tokens;
    const float* u_accept;
    const float* u_final;
    VerifyOut o;
    int* stop;
    int* fb_count;
    int* fb_list;
    int vs;          // vectors per CTA slice (multiple of 8)
    int b0, nb;      // this launch covers sequences b0 .. b0+nb-1
    long long* trace;
};

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

// exact warp sum of non-negative fixed-point values below 2^46
__device__ __forceinline__ long long warp_sum_fixed(long long v) {
    uint32_t lo = (uint32_t)(v & 0xFFFFF), hi = (uint32_t)(v >> 20);
    return ((long long)redux_add(hi) << 20) + (long long)redux_add(lo);
}

// status of one row from its merged partials
__device__ __forceinline__ int row_status(int flagbit, int E, double S) {
    if (flagbit || !(S == S)) return ST_NONFINITE;
    return E == E_EMPTY ? ST_EMPTY : 0;
}

}  // namespace

#ifdef BEBOP_TRACE
#ifndef BEBOP_TRACE_TID
#define BEBOP_TRACE_TID 0
#endif
#ifndef BEBOP_TRACE_RANK
#define BEBOP_TRACE_RANK 0
#endif
#define TRACE(id) do { if (a.trace && cid == 0 && rank == BEBOP_TRACE_RANK && tid == BEBOP_TRACE_TID && r < 60) a.trace[r * 16 + (id)] = clock64(); } while (0)
#else
#define TRACE(id) do {} while (0)
#endif

// =============================================================================
template <int DT, int NV>
__global__ void __launch_bounds__(NT, 1) k_stream(const StreamArgs a) {
    constexpr int VEC = Elem<DT>::VEC;
    constexpr int NE = NV * VEC;
    constexpr int ROW_BYTES = NT * NV * 16;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    unsigned char* stage = smem_raw;                     // [2 stages][2 rows][ROW_BYTES]
    StreamShared& S = *reinterpret_cast<StreamShared*>(smem_raw + 4 * ROW_BYTES);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rank = (int)cluster_rank();
    const int cid = (int)cluster_id(), ncl = (int)num_clusters();
    const RowArgs& R = a.r;
    const int K = R.K, V = R.V;

    const int v_begin = min(rank * a.vs, R.nvec);
    const int nv_cta = min(a.vs, R.nvec - v_begin);
    const uint32_t slice_bytes = (uint32_t)max(nv_cta, 0) * 16u;
    const int64_t slice_off = (int64_t)v_begin * 16;
    const int lv0 = tid * NV;

    if (tid == 0) {
        mbar_init(smem_u32(&S.full[0]), 1);
        mbar_init(smem_u32(&S.full[1]), 1);
        for (int i = 0; i < RING; ++i) {
            mbar_init(smem_u32(&S.stats_bar[i]), CS);
            mbar_init(smem_u32(&S.draw_bar[i]), CS);
            mbar_init(smem_u32(&S.z_bar[i]), CS);
            mbar_init(smem_u32(&S.res_bar[i]), CS);
            S.wcnt[i] = S.zcnt[i] = S.dcnt[i] = S.rcnt[i] = 0;
        }
        S.relcnt[0] = S.relcnt[1] = 0;
        S.wait_failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    __syncthreads();
    cluster_arrive();
    cluster_wait();

    // ---- sequences of this cluster: b = b0 + cid + j * ncl, j = 0 .. nseq-1 (nseq <= MAXSEQ)
    const int nseq = (a.nb - cid + ncl - 1) / ncl;
    auto seq_b = [&](int j) { return a.b0 + cid + j * ncl; };
    auto trow = [&](int b, int k) { return R.target + ((int64_t)b * R.t_seq_rows + k) * R.t_row_bytes; };
    auto drow = [&](int b, int k) { return R.draft + ((int64_t)b * R.d_seq_rows + k) * R.d_row_bytes; };

    // bonus mask: bit j set when sequence j needs its bonus row (L == 0 from the start)
    unsigned long long bm0 = 0, bm1 = 0;
    for (int j = 0; j < nseq; ++j)
        if (len_of(R, seq_b(j)) == 0) { if (j < 64) bm0 |= 1ull << j; else bm1 |= 1ull << (j - 64); }

    // ---- pair cursor
    struct PC { int j, k, L; };
    auto pc_skip = [&](PC& c) { while (c.j < nseq && (c.L = len_of(R, seq_b(c.j))) == 0) ++c.j; };
    auto pc_next = [&](PC& c) { if (c.j >= nseq) return; if (++c.k < c.L) return; c.k = 0; ++c.j; pc_skip(c); };
    // ---- bonus cursor over a mask copy
    struct BC { unsigned long long m0, m1; };
    auto bc_peek = [&](const BC& c) { return c.m0 ? __ffsll((long long)c.m0) - 1 : (c.m1 ? 63 + __ffsll((long long)c.m1) : -1); };
    auto bc_pop = [&](BC& c) { if (c.m0) c.m0 &= c.m0 - 1; else if (c.m1) c.m1 &= c.m1 - 1; };

    // ---- bulk copies of this CTA's slice (called by a whole warp)
    auto issue = [&](int st, const char* prow, const char* qrow) {
        if (nv_cta <= 0) return;
        const uint32_t bar = smem_u32(&S.full[st]);
        const uint32_t dst = smem_u32(stage + (size_t)st * 2 * ROW_BYTES);
        if (lane == 0) mbar_expect_tx(bar, qrow ? 2 * slice_bytes : slice_bytes);
        __syncwarp();
        const uint32_t nchunk = (slice_bytes + kChunk - 1) / kChunk;
        for (uint32_t ci = lane; ci < (qrow ? 2 * nchunk : nchunk); ci += 32) {
            const uint32_t row = ci >= nchunk ? 1u : 0u, cc = ci - row * nchunk;
            const uint32_t off = cc * kChunk, len = min(kChunk, slice_bytes - off);
            bulk_g2s(dst + row * ROW_BYTES + off, (row ? qrow : prow) + slice_off + off, len, bar);
        }
    };

    PC cur{0, 0, 0}, ld{0, 0, 0};
    pc_skip(cur);
    ld = cur;
    BC bcur{0, 0}, bld{0, 0};
    int phase = cur.j < nseq ? 1 : 2;
    if (phase == 2) { bcur.m0 = bm0; bcur.m1 = bm1; bld = bcur; }
    // prologue: warp 0 fills both stages
    for (int s = 0; s < 2; ++s) {
        if (phase == 1) {
            if (ld.j < nseq) { if (warp == 0) issue(s, trow(seq_b(ld.j), ld.k), drow(seq_b(ld.j), ld.k)); pc_next(ld); }
        } else {
            int j = bc_peek(bld);
            if (j >= 0) { int bb = seq_b(j); if (warp == 0) issue(s, trow(bb, len_of(R, bb)), nullptr); bc_pop(bld); }
        }
    }

    // ---- per-sequence state (identical in every warp of the cluster)
    int seq_alive = 1, seq_n = 0, seq_st = 0;
    float tau = 1.f, c = kLog2e;
    double c64 = 1.4426950408889634;
    int tokl = 0;                          // lane t holds draft token t of the current sequence
    float ufin = 0.5f;
    int ndraw = 0;                         // draws so far (index into the draw / result rings)
    // deferred outputs (used by warp 0 of rank 0 only): two rounds of history
    int h_r[2] = {0, 0}, h_b[2] = {-1, -1}, h_k[2] = {0, 0}, h_fatal[2] = {0, 0};
    int hd_b[2] = {-1, -1}, hd_n[2] = {0, 0}, hd_idx[2] = {0, 0};

    auto load_seq_scalars = [&](int b, int L) {
        tau = tau_of(R, b);
        tokl = lane < L ? a.draft_tokens[(int64_t)b * K + lane] : 0;
        ufin = a.u_final[b];
    };
    if (phase == 1) load_seq_scalars(seq_b(cur.j), cur.L);
    else { int j = bc_peek(bcur); if (j >= 0) load_seq_scalars(seq_b(j), 0); }

    auto flush_outputs = [&](int hi) {
        // rank 0, warp 0: outputs of the round recorded in history entry hi, once every CTA delivered them
        const int slot_r = h_r[hi];
        if (h_b[hi] >= 0) {
            if (!mbar_wait_cluster(smem_u32(&S.z_bar[slot_r & (RING - 1)]), (slot_r / RING) & 1)) S.wait_failed = 1;
            if (lane == 0 && a.o.tv) {
                float z = 0.f;
                for (int i = 0; i < CS; ++i) z += S.zslot[slot_r & (RING - 1)][i];
                a.o.tv[(int64_t)h_b[hi] * K + h_k[hi]] = h_fatal[hi] ? 0.f : fminf(fmaxf(z, 0.f), 1.f);
            }
            h_b[hi] = -1;
        }
        if (hd_b[hi] >= 0) {
            const int di = hd_idx[hi];
            if (!mbar_wait_cluster(smem_u32(&S.res_bar[di & (RING - 1)]), (di / RING) & 1)) S.wait_failed = 1;
            if (lane == 0) {
                int y = -1, cert = 0, owners = 0;
                for (int i = 0; i < CS; ++i) {
                    RPart p = S.rslot[di & (RING - 1)][i];
                    if (p.y >= 0) { y = p.y; cert = p.cert; owners++; }
                }
                if (owners == 1 && cert) a.o.out_tokens[(int64_t)hd_b[hi] * (K + 1) + hd_n[hi]] = y;
                else { int idx = atomicAdd(a.fb_count, 1); a.fb_list[idx] = hd_b[hi]; }
            }
            hd_b[hi] = -1;
        }
    };

    // =========================================================================
    for (int r = 0;; ++r) {
        // ------------------------------------------------ the item of this round
        int j, b, k, L;
        bool pair;
        if (phase == 1) { j = cur.j; k = cur.k; L = cur.L; pair = true; }
        else { j = bc_peek(bcur); if (j < 0) break; L = len_of(R, seq_b(j)); k = L; pair = false; }
        b = seq_b(j);
        const int st = r & 1, slot = r & (RING - 1);
        const uint32_t ring_par = (uint32_t)(r / RING) & 1u;
        TRACE(0);

        if (pair ? k == 0 : true) {
            // first item of a sequence (or a bonus item): scalars were loaded ahead
            const bool ok = tau_ok(tau);
            c64 = 1.4426950408889634 / (double)(ok ? tau : 1.f);
            c = (float)c64;
            if (pair) {
                seq_alive = 1; seq_n = L; seq_st = ok ? 0 : ST_BAD_TEMP;
                if (!seq_st && __ballot_sync(0xffffffffu, lane < L && (tokl < 0 || tokl >= V))) seq_st = ST_BAD_TOKEN;
            } else {
                seq_st = ok ? 0 : ST_BAD_TEMP;
            }
        }
        // gathered logits of the drafted token and its uniform (consumed after the exchange)
        float zpx = 0.f, zqx = 0.f, u_acc = 0.5f;
        if (pair) {
            int tk = min(max(__shfl_sync(0xffffffffu, tokl, k), 0), V - 1);
            zpx = DT == 0 ? load_one<0>(trow(b, k), tk) : load_one<1>(trow(b, k), tk);
            zqx = DT == 0 ? load_one<0>(drow(b, k), tk) : load_one<1>(drow(b, k), tk);
            u_acc = a.u_accept[(int64_t)b * K + k];
        }
        // scalars of the next sequence, if the next item starts one (consumed next round)
        PC nxt = cur;
        float tau_n = tau, ufin_n = ufin;
        int tokl_n = tokl;
        bool new_seq_next = false;
        if (phase == 1) {
            pc_next(nxt);
            if (nxt.j < nseq && nxt.k == 0) {
                int bn = seq_b(nxt.j);
                tau_n = tau_of(R, bn);
                tokl_n = lane < nxt.L ? a.draft_tokens[(int64_t)bn * K + lane] : 0;
                ufin_n = a.u_final[bn];
                new_seq_next = true;
            }
        } else {
            BC t = bcur; bc_pop(t);
            int jn = bc_peek(t);
            if (jn >= 0) { int bn = seq_b(jn); tau_n = tau_of(R, bn); ufin_n = a.u_final[bn]; tokl_n = 0; new_seq_next = true; }
        }

        // ------------------------------------------------ ingest: stage -> registers
        float ep[NE], eq[NE];
        int Ep = E_EMPTY, Eq = E_EMPTY, flags = 0;
        {
            uint4 rp[NV], rq[NV];
            TRACE(9);
            if (nv_cta > 0 && !mbar_wait(smem_u32(&S.full[st]), (uint32_t)(r >> 1) & 1u)) S.wait_failed = 1;
            TRACE(1);
            const unsigned char* sp_ = stage + (size_t)st * 2 * ROW_BYTES;
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                const int lv = lv0 + i;
                if (lv < nv_cta) {
                    rp[i] = *reinterpret_cast<const uint4*>(sp_ + (size_t)lv * 16);
                    rq[i] = pair ? *reinterpret_cast<const uint4*>(sp_ + ROW_BYTES + (size_t)lv * 16) : neg_inf_vec<DT>();
                    const int gbase = (v_begin + lv) * VEC;
                    if (gbase + VEC > V) { mask_tail<DT>(rp[i], V - gbase); mask_tail<DT>(rq[i], V - gbase); }
                } else {
                    rp[i] = neg_inf_vec<DT>(); rq[i] = neg_inf_vec<DT>();
                }
            }
            TRACE(10);
            float mp = vec_max<DT>(rp[0]), mq = vec_max<DT>(rq[0]);
#pragma unroll
            for (int i = 1; i < NV; ++i) { mp = max_nan(mp, vec_max<DT>(rp[i])); mq = max_nan(mq, vec_max<DT>(rq[i])); }
            mp = ord2f(redux_max(f2ord(mp)));
            mq = ord2f(redux_max(f2ord(mq)));
            TRACE(11);
            // this warp has consumed the stage: the last warp to say so refills it
            {
                int last = 0;
                if (lane == 0) last = atomicAdd(&S.relcnt[st], 1) == NW - 1;
                last = __shfl_sync(0xffffffffu, last, 0);
                if (last) {
                    if (lane == 0) S.relcnt[st] = 0;
                    fence_proxy_async();
                    if (phase == 1) {
                        if (ld.j < nseq) issue(st, trow(seq_b(ld.j), ld.k), drow(seq_b(ld.j), ld.k));
                    } else {
                        int jn = bc_peek(bld);
                        if (jn >= 0) { int bb = seq_b(jn); issue(st, trow(bb, len_of(R, bb)), nullptr); }
                    }
                }
                if (phase == 1) pc_next(ld); else bc_pop(bld);
            }
            TRACE(2);
            // exponent references of this warp: E = ceil(m * c), 2^(x*c - E) <= 1
            float fp_ = 0.f, fq_ = 0.f, mpu = 0.f, mqu = 0.f;
            if (mp != mp || mp == INFINITY) flags |= 1;
            else if (mp != -INFINITY) { double t = fmin(fmax((double)mp * c64, -kEClamp), kEClamp); double E = ceil(t); Ep = (int)E; fp_ = (float)(E - t); mpu = mp; }
            if (pair) {
                if (mq != mq || mq == INFINITY) flags |= 2;
                else if (mq != -INFINITY) { double t = fmin(fmax((double)mq * c64, -kEClamp), kEClamp); double E = ceil(t); Eq = (int)E; fq_ = (float)(E - t); mqu = mq; }
            }
            TRACE(12);
            float s_p = 0.f, s_q = 0.f;
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                float f[VEC];
                unpack<DT>(rp[i], f);
#pragma unroll
                for (int e = 0; e < VEC; ++e) { float x = ex2f(fmaf(f[e] - mpu, c, -fp_)); ep[i * VEC + e] = x; s_p += x; }
            }
            if (pair) {
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    float f[VEC];
                    unpack<DT>(rq[i], f);
#pragma unroll
                    for (int e = 0; e < VEC; ++e) { float x = ex2f(fmaf(f[e] - mqu, c, -fq_)); eq[i * VEC + e] = x; s_q += x; }
                }
            } else {
#pragma unroll
                for (int e = 0; e < NE; ++e) eq[e] = 0.f;
            }
            TRACE(3);
            // publish the warp partial; the last warp of the CTA combines and sends
            long long fs_p = warp_sum_fixed(__double2ll_rn((double)s_p * kFix));
            long long fs_q = warp_sum_fixed(__double2ll_rn((double)s_q * kFix));
            if (flags & 1) fs_p = 0;
            if (flags & 2) fs_q = 0;
            TRACE(13);
            int last = 0;
            if (lane == 0) {
                WPart w; w.sp = fs_p; w.sq = fs_q; w.ep = Ep; w.eq = Eq; w.flags = flags; w.pad = 0;
                S.wpart[slot][warp] = w;
                __threadfence_block();
                last = atomicAdd(&S.wcnt[slot], 1) == NW - 1;
            }
            last = __shfl_sync(0xffffffffu, last, 0);
            if (last) {
                __threadfence_block();
                if (lane == 0) S.wcnt[slot] = 0;
                WPart w;
                if (lane < NW) w = S.wpart[slot][lane]; else { w.sp = w.sq = 0; w.ep = w.eq = E_EMPTY; w.flags = 0; }
                const int Ecp = redux_max(w.ep), Ecq = redux_max(w.eq);
                double tp = w.ep > E_EMPTY ? (double)w.sp * pow2d(max(w.ep - Ecp, -1000) - 40) : 0.0;
                double tq = w.eq > E_EMPTY ? (double)w.sq * pow2d(max(w.eq - Ecq, -1000) - 40) : 0.0;
                int fl = w.flags;
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) {
                    tp += shfl_xor_d(tp, o); tq += shfl_xor_d(tq, o);
                    fl |= __shfl_xor_sync(0xffffffffu, fl, o);
                }
                if (lane < CS) {
                    const uint32_t dst = mapa(smem_u32(&S.cslot[slot][rank]), (uint32_t)lane);
                    uint4 w0, w1;
                    w0.x = (uint32_t)__double2loint(tp); w0.y = (uint32_t)__double2hiint(tp);
                    w0.z = (uint32_t)__double2loint(tq); w0.w = (uint32_t)__double2hiint(tq);
                    w1.x = (uint32_t)Ecp; w1.y = (uint32_t)Ecq; w1.z = (uint32_t)fl; w1.w = 0;
                    st_cluster_v4(dst, w0);
                    st_cluster_v4(dst + 16, w1);
                    mbar_arrive_remote(mapa(smem_u32(&S.stats_bar[slot]), (uint32_t)lane));
                }
                __syncwarp();
            }
        }
        TRACE(4);

        // ------------------------------------------------ deferred outputs of round r-2 (rank 0, warp 0)
        if (rank == 0 && warp == 0 && r >= 2) flush_outputs(r & 1);

        // ------------------------------------------------ merged normalisers, accept test
        if (!mbar_wait_cluster(smem_u32(&S.stats_bar[slot]), ring_par)) S.wait_failed = 1;
        TRACE(5);
        float a_w = 0.f, b_w = 0.f;
        int bad = 0, stop_here = 0;
        int Em_p, Em_q;
        double Sp, Sq;
        {
            CPart cp;
            if (lane < CS) cp = S.cslot[slot][lane]; else { cp.sp = cp.sq = 0.0; cp.ep = cp.eq = E_EMPTY; cp.flags = 0; }
            Em_p = redux_max(cp.ep); Em_q = redux_max(cp.eq);
            Sp = cp.ep > E_EMPTY ? cp.sp * pow2d(max(cp.ep - Em_p, -1000)) : 0.0;
            Sq = cp.eq > E_EMPTY ? cp.sq * pow2d(max(cp.eq - Em_q, -1000)) : 0.0;
            int fl = cp.flags;
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) {
                Sp += shfl_xor_d(Sp, o); Sq += shfl_xor_d(Sq, o);
                fl |= __shfl_xor_sync(0xffffffffu, fl, o);
            }
            Sp = __shfl_sync(0xffffffffu, Sp, 0); Sq = __shfl_sync(0xffffffffu, Sq, 0);
            fl = __shfl_sync(0xffffffffu, fl, 0);
            bad = row_status(fl & 1, Em_p, Sp);
            if (pair) bad |= row_status(fl & 2, Em_q, Sq);
            if (!bad) {
                a_w = Ep > E_EMPTY ? (float)(pow2d(max(Ep - Em_p, -1000)) * __drcp_rn(Sp)) : 0.f;
                if (pair) b_w = Eq > E_EMPTY ? (float)(pow2d(max(Eq - Em_q, -1000)) * __drcp_rn(Sq)) : 0.f;
            }
        }
        if (pair && !bad && !(seq_st & ST_FATAL)) {
            // p(x), q(x): fp32 first, fp64 when the test is close
            float pxf = ex2f(fmaf(zpx, c, -(float)Em_p)) * (float)__drcp_rn(Sp);
            float qxf = ex2f(fmaf(zqx, c, -(float)Em_q)) * (float)__drcp_rn(Sq);
            float lhs = u_acc * qxf;
            bool acc = lhs < pxf;
            double pxd = pxf, qxd = qxf;
            if (fabsf(lhs - pxf) <= 1e-3f * fmaxf(lhs, pxf)) {
                pxd = exp2((double)zpx * c64 - (double)Em_p) / Sp;
                qxd = exp2((double)zqx * c64 - (double)Em_q) / Sq;
                acc = (double)u_acc * qxd < pxd;
            }
            if (rank == 0 && warp == 0 && lane == 0) {
                if (a.o.p_draft) a.o.p_draft[(int64_t)b * K + k] = (float)pxd;
                if (a.o.q_draft) a.o.q_draft[(int64_t)b * K + k] = (float)qxd;
            }
            if (seq_alive && !acc) stop_here = 1;
        }
        if (!(seq_st & ST_FATAL)) seq_st |= bad;          // only the first bad row counts
        const bool do_draw = !(seq_st & ST_FATAL) && (pair ? stop_here != 0 : true);
        TRACE(6);

        // ------------------------------------------------ TV (and the chunk sums of a draw)
        float z_t = 0.f, sq_t = 0.f;
        double zt64 = 0.0;
        if (!bad) {
            if (!do_draw) {
                float z0 = 0.f, z1 = 0.f;
#pragma unroll
                for (int e = 0; e < NE; e += 2) {
                    z0 += fmaxf(fmaf(ep[e], a_w, -__fmul_rn(eq[e], b_w)), 0.f);
                    z1 += fmaxf(fmaf(ep[e + 1], a_w, -__fmul_rn(eq[e + 1], b_w)), 0.f);
                }
                z_t = z0 + z1;
            } else {
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    float rr[VEC];
#pragma unroll
                    for (int e = 0; e < VEC; ++e) {
                        float q = __fmul_rn(eq[i * VEC + e], b_w);
                        rr[e] = fmaxf(fmaf(ep[i * VEC + e], a_w, -q), 0.f);
                        float p = __fmul_rn(ep[i * VEC + e], a_w);
                        sq_t = fmaf(p, p, sq_t); sq_t = fmaf(q, q, sq_t);
                    }
#pragma unroll
                    for (int w = 1; w < VEC; w <<= 1)
#pragma unroll
                        for (int e = 0; e + w < VEC; e += 2 * w) rr[e] += rr[e + w];
                    z_t += rr[0];
                    zt64 += (double)rr[0];
                }
            }
        }
        {
            // Z of the slice: warp partial -> CTA partial (last warp, in warp order) -> rank 0
            float zw = warp_sum(z_t);
            int last = 0;
            if (lane == 0) {
                S.wz[slot][warp] = pair ? zw : 0.f;
                __threadfence_block();
                last = atomicAdd(&S.zcnt[slot], 1) == NW - 1;
            }
            last = __shfl_sync(0xffffffffu, last, 0);
            if (last) {
                __threadfence_block();
                if (lane == 0) {
                    S.zcnt[slot] = 0;
                    float z = 0.f;
                    for (int w = 0; w < NW; ++w) z += S.wz[slot][w];
                    st_cluster_b32(mapa(smem_u32(&S.zslot[slot][rank]), 0u), __float_as_uint(z));
                    mbar_arrive_remote(mapa(smem_u32(&S.z_bar[slot]), 0u));
                }
                __syncwarp();
            }
        }
        TRACE(7);
        if (rank == 0 && warp == 0) {
            h_r[r & 1] = r; h_b[r & 1] = pair ? b : -1; h_k[r & 1] = k; h_fatal[r & 1] = (seq_st & ST_FATAL) ? 1 : 0;
        }

        // ------------------------------------------------ the draw at the stop row / bonus row
        if (do_draw) {
            const int ds = ndraw & (RING - 1);
            const uint32_t dpar = (uint32_t)(ndraw / RING) & 1u;
            double incl = zt64;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) { double t = shfl_up_d(incl, d); if (lane >= d) incl += t; }
            const float sqw = warp_sum(sq_t);
            int last = 0;
            if (lane == 31) { DPart p; p.tot = incl; p.sq = sqw; p.pad = 0; S.wdraw[ds][warp] = p; __threadfence_block(); }
            __syncwarp();
            if (lane == 0) last = atomicAdd(&S.dcnt[ds], 1) == NW - 1;
            last = __shfl_sync(0xffffffffu, last, 0);
            if (last) {
                __threadfence_block();
                if (lane == 0) S.dcnt[ds] = 0;
                double tot = 0.0; float sq = 0.f;
                for (int w = 0; w < NW; ++w) { tot += S.wdraw[ds][w].tot; sq += S.wdraw[ds][w].sq; }
                if (lane < CS) {
                    const uint32_t dst = mapa(smem_u32(&S.dslot[ds][rank]), (uint32_t)lane);
                    uint4 w0;
                    w0.x = (uint32_t)__double2loint(tot); w0.y = (uint32_t)__double2hiint(tot);
                    w0.z = __float_as_uint(sq); w0.w = 0;
                    st_cluster_v4(dst, w0);
                    mbar_arrive_remote(mapa(smem_u32(&S.draw_bar[ds]), (uint32_t)lane));
                }
                __syncwarp();
            }
            if (!mbar_wait_cluster(smem_u32(&S.draw_bar[ds]), dpar)) S.wait_failed = 1;
            // offsets: CTA totals in rank order, then this CTA's warp totals in warp order
            double base = 0.0, Z = 0.0, sumsq = 0.0;
            for (int i = 0; i < CS; ++i) { if (i == rank) base = Z; Z += S.dslot[ds][i].tot; sumsq += (double)S.dslot[ds][i].sq; }
            for (int w = 0; w < warp; ++w) base += S.wdraw[ds][w].tot;
            const double T = (double)ufin * Z;
            const double bound = draw_bound(sumsq);
            double prev_incl = shfl_up_d(incl, 1);
            if (lane == 0) prev_incl = 0.0;
            const double lower = base + prev_incl, upper = base + incl;
            int my_y = -1, my_cert = 0;
            if (T > 0.0 && lower < T && T <= upper) {
                double C = lower;
                const int g0 = (v_begin + lv0) * VEC;
#pragma unroll
                for (int e = 0; e < NE; ++e) {
                    if (my_y < 0) {
                        double rr = (double)fmaxf(fmaf(ep[e], a_w, -__fmul_rn(eq[e], b_w)), 0.f);
                        double Cn = C + rr;
                        if (rr > 0.0 && Cn >= T) { my_y = g0 + e; my_cert = (T - C > bound) && (Cn - T >= bound); }
                        C = Cn;
                    }
                }
            }
            // this warp's result, then the CTA's (last warp), then to rank 0
            const unsigned own = __ballot_sync(0xffffffffu, my_y >= 0);
            int wy = -1, wc = 0;
            if (own) { const int src = __ffs(own) - 1; wy = __shfl_sync(0xffffffffu, my_y, src); wc = __shfl_sync(0xffffffffu, my_cert, src); if (__popc(own) > 1) wc = 0; }
            last = 0;
            if (lane == 0) {
                RPart p; p.y = wy; p.cert = wc; S.wres[ds][warp] = p;
                __threadfence_block();
                last = atomicAdd(&S.rcnt[ds], 1) == NW - 1;
            }
            last = __shfl_sync(0xffffffffu, last, 0);
            if (last) {
                __threadfence_block();
                if (lane == 0) {
                    S.rcnt[ds] = 0;
                    int y = -1, ce = 0, cnt = 0;
                    for (int w = 0; w < NW; ++w) { RPart p = S.wres[ds][w]; if (p.y >= 0) { y = p.y; ce = p.cert; cnt++; } }
                    if (cnt > 1) ce = 0;
                    st_cluster_v2(mapa(smem_u32(&S.rslot[ds][rank]), 0u), (uint32_t)y, (uint32_t)ce);
                    mbar_arrive_remote(mapa(smem_u32(&S.res_bar[ds]), 0u));
                }
                __syncwarp();
            }
            if (rank == 0 && warp == 0) { hd_b[r & 1] = b; hd_n[r & 1] = pair ? k : L; hd_idx[r & 1] = ndraw; }
            ndraw++;
        } else if (rank == 0 && warp == 0) hd_b[r & 1] = -1;
        TRACE(8);

        // ------------------------------------------------ sequence bookkeeping
        if (pair) {
            if (stop_here) { seq_alive = 0; seq_n = k; }
            if (k == L - 1) {
                const bool fatal = (seq_st & ST_FATAL) != 0;
                if (rank == 0 && warp == 0) {
                    // TV values of this sequence still waiting in the history must not survive a fatal status
                    if (fatal) { if (h_b[0] == b) h_fatal[0] = 1; if (h_b[1] == b) h_fatal[1] = 1; }
                    const int n = fatal ? 0 : seq_n;
                    for (int t = lane; t <= K; t += 32) {
                        // position n belongs to the draw (delivered later, or re-drawn in fp64)
                        if (fatal || t != n) a.o.out_tokens[(int64_t)b * (K + 1) + t] = t < n ? tokl : -1;   // t < n <= 32: t == lane
                    }
                    if (lane == 0) {
                        a.o.accept_len[b] = n;
                        a.stop[b] = fatal ? -1 : n;
                        if (a.o.row_status) a.o.row_status[b] = seq_st;
                    }
                    for (int t = lane; t < K; t += 32) {
                        if (fatal || t >= L) {
                            if (a.o.tv) a.o.tv[(int64_t)b * K + t] = 0.f;
                            if (a.o.p_draft) a.o.p_draft[(int64_t)b * K + t] = 0.f;
                            if (a.o.q_draft) a.o.q_draft[(int64_t)b * K + t] = 0.f;
                        }
                    }
                }
                if (!fatal && seq_alive) { if (j < 64) bm0 |= 1ull << j; else bm1 |= 1ull << (j - 64); }
            }
            cur = nxt;
            if (cur.j >= nseq) {
                // phase 1 is over: the bonus mask is final; warp 0 starts the bonus stream.  Stage
                // (r+1)&1 was never refilled; stage r&1 is free because every warp of the cluster
                // published its partial of this item after reading the stage.
                phase = 2;
                bcur.m0 = bm0; bcur.m1 = bm1; bld = bcur;
                for (int s = 0; s < 2; ++s) {
                    int jn = bc_peek(bld);
                    if (jn >= 0) {
                        int bb = seq_b(jn);
                        if (warp == 0) { fence_proxy_async(); issue((r + 1 + s) & 1, trow(bb, len_of(R, bb)), nullptr); }
                        bc_pop(bld);
                    }
                }
                int jn = bc_peek(bcur);
                if (jn >= 0) { int bn = seq_b(jn); tau_n = tau_of(R, bn); ufin_n = a.u_final[bn]; tokl_n = 0; new_seq_next = true; }
            }
        } else {
            const bool fatal = (seq_st & ST_FATAL) != 0;
            if (rank == 0 && warp == 0 && (L == 0 || fatal)) {
                for (int t = lane; t <= K; t += 32)
                    if (fatal || t != 0) a.o.out_tokens[(int64_t)b * (K + 1) + t] = -1;
                for (int t = lane; t < K; t += 32) {
                    if (a.o.tv) a.o.tv[(int64_t)b * K + t] = 0.f;
                    if (a.o.p_draft) a.o.p_draft[(int64_t)b * K + t] = 0.f;
                    if (a.o.q_draft) a.o.q_draft[(int64_t)b * K + t] = 0.f;
                }
                if (lane == 0) {
                    a.o.accept_len[b] = 0;
                    if (L == 0) { a.stop[b] = fatal ? -1 : 0; if (a.o.row_status) a.o.row_status[b] = seq_st; }
                    else { a.stop[b] = -1; if (a.o.row_status) a.o.row_status[b] |= seq_st; }
                }
            }
            bc_pop(bcur);
        }
        if (new_seq_next) { tau = tau_n; tokl = tokl_n; ufin = ufin_n; }
    }

    // ---- epilogue: the last two rounds of deferred outputs (older first), then leave together
    if (rank == 0 && warp == 0) {
        const int first = h_r[0] <= h_r[1] ? 0 : 1;
        flush_outputs(first);
        flush_outputs(first ^ 1);
    }
    __syncthreads();
    cluster_arrive();
    cluster_wait();
    if (tid == 0 && S.wait_failed && a.o.row_status) {
        for (int jj = 0; jj < nseq; ++jj) atomicOr(&a.o.row_status[seq_b(jj)], ST_WAIT);
    }
}

// -----------------------------------------------------------------------------
namespace {

constexpr int kNV = 5;

template <int DT>
constexpr size_t stream_smem() { return 4 * (size_t)NT * kNV * 16 + sizeof(StreamShared) + 128; }

template <int DT>
cudaLaunchConfig_t stream_config(int clusters, cudaStream_t stream, cudaLaunchAttribute* attr) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(clusters * CS), 1, 1);
    cfg.blockDim = dim3(NT, 1, 1);
    cfg.dynamicSmemBytes = stream_smem<DT>();
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CS; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cfg;
}

// Co-resident clusters on the current device (0: the kernel cannot run here), cached per device.
template <int DT>
int stream_clusters() {
    static int cached[64] = {0};
    static bool known[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (dev >= 0 && dev < 64 && known[dev]) return cached[dev];
    int n = 0;
    if (cudaFuncSetAttribute(k_stream<DT, kNV>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)stream_smem<DT>()) == cudaSuccess) {
        cudaLaunchAttribute attr[1];
        cudaLaunchConfig_t cfg = stream_config<DT>(64, nullptr, attr);
        if (cudaOccupancyMaxActiveClusters(&n, k_stream<DT, kNV>, &cfg) != cudaSuccess) n = 0;
    }
    cudaGetLastError();
    if (dev >= 0 && dev < 64) { cached[dev] = n; known[dev] = true; }
    return n;
}

long long* g_stream_trace = nullptr;

}  // namespace

void stream_set_trace(long long* p) { g_stream_trace = p; }
int stream_max_clusters(int dt) { return dt == 0 ? stream_clusters<0>() : stream_clusters<1>(); }

// Shapes the streaming kernel takes: every CTA slice (rounded up to 128 bytes) fits the
// per-thread register chunks, and no slice is degenerate.
bool stream_supported(const RowArgs& a) {
    const int vs = (((a.nvec + CS - 1) / CS) + 7) & ~7;
    return vs <= NT * kNV && a.nvec >= 4 * CS;
}

cudaError_t stream_verify(const RowArgs& a, const Plan& p, const int32_t* draft_tokens,
                          const float* u_accept, const float* u_final, VerifyOut o, char* ws,
                          cudaStream_t stream, bool* launched) {
    *launched = false;
    int ncl = stream_max_clusters(a.dt);
    if (ncl < 1) return cudaSuccess;
    StreamArgs sa;
    sa.r = a; sa.draft_tokens = draft_tokens; sa.u_accept = u_accept; sa.u_final = u_final; sa.o = o;
    sa.stop = reinterpret_cast<int*>(ws + p.off_stop);
    sa.fb_count = reinterpret_cast<int*>(ws + p.off_fb);
    sa.fb_list = sa.fb_count + 16;
    sa.vs = (((a.nvec + CS - 1) / CS) + 7) & ~7;
    sa.trace = g_stream_trace;
    cudaError_t e = cudaMemsetAsync(sa.fb_count, 0, sizeof(int), stream);
    if (e != cudaSuccess) return e;
    // at most MAXSEQ sequences per cluster and launch
    for (int b0 = 0; b0 < a.B; b0 += ncl * MAXSEQ) {
        sa.b0 = b0;
        sa.nb = a.B - b0 < ncl * MAXSEQ ? a.B - b0 : ncl * MAXSEQ;
        const int clusters = sa.nb < ncl ? sa.nb : ncl;
        cudaLaunchAttribute attr[1];
        if (a.dt == 0) {
            cudaLaunchConfig_t cfg = stream_config<0>(clusters, stream, attr);
            e = cudaLaunchKernelEx(&cfg, k_stream<0, kNV>, sa);
        } else {
            cudaLaunchConfig_t cfg = stream_config<1>(clusters, stream, attr);
            e = cudaLaunchKernelEx(&cfg, k_stream<1, kNV>, sa);
        }
        if (e != cudaSuccess) return e;
    }
    *launched = true;
    return general_draw_list(a, p, u_final, o, ws, sa.fb_list, sa.fb_count, stream);
}

}  // namespace bebop
