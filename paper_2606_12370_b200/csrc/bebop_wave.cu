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
#define BEBOP_CTA_SYNC() __syncthreads()
#include "bebop_wave.cuh"

namespace bebop {

template <int DT>
__global__ void __launch_bounds__(WT, 4) k_wave(const WaveArgs a) {
    __shared__ WaveShared S;
    __shared__ float vsum_buf[SLICE_VECS / 2];
    const int tid = threadIdx.x;
    if (tid == 0) S.vsum = vsum_buf;
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
    wa.rowcnt = nullptr;
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
    wave_flag_launch(wa.wait_failed, o.row_status, a.B, stream);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    *launched = true;
    return redraw_launch(a, u_final, o, wa.fb_count, wa.fb_list, w, wp, stream);
}

void wave_flag_launch(const int* wait_failed, int32_t* row_status, int B, cudaStream_t stream) {
    k_wave_flag<<<(B + 255) / 256, 256, 0, stream>>>(wait_failed, row_status, B);
}

// fp64 re-draw of the listed sequences (usually a few per cent of the batch; the count stays on the device)
cudaError_t redraw_launch(const RowArgs& a, const float* u_final, VerifyOut o, const int* fb_count,
                          const int* fb_list, char* w, const WavePlan& wp, cudaStream_t stream) {
    RedrawArgs ra;
    ra.r = a; ra.u_final = u_final; ra.o = o;
    ra.fb_count = fb_count; ra.fb_list = fb_list;
    ra.sinfo = reinterpret_cast<const SeqInfo*>(w + wp.off_sinfo);
    ra.rstat = reinterpret_cast<const RowStat*>(w + wp.off_rstat);
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
