// The fp64 re-draw of the sequences whose fast draw did not clear its error bound, the kernel that turns
// an expired device-side wait into a status bit, and the hooks that time and trace the main kernel.
#define BEBOP_CTA_SYNC() __syncthreads()
#include "bebop_pipe.cuh"

namespace bebop {

namespace {

// ------------------------------------------------------------------ fp64 re-draw of the listed sequences
// Two small kernels behind the pipelined kernel, for the few sequences whose fast draw did not clear its
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

__global__ void k_wait_flag(const int* __restrict__ wait_failed, int32_t* row_status, int B) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B && *wait_failed && row_status) row_status[b] |= ST_WAIT;
}

long long* g_wave_trace = nullptr;
void wave_set_trace(long long* p) { g_wave_trace = p; }
cudaEvent_t g_ev_start = nullptr, g_ev_stop = nullptr;
void wave_set_events(cudaEvent_t start, cudaEvent_t stop) { g_ev_start = start; g_ev_stop = stop; }

void wave_flag_launch(const int* wait_failed, int32_t* row_status, int B, cudaStream_t stream) {
    k_wait_flag<<<(B + 255) / 256, 256, 0, stream>>>(wait_failed, row_status, B);
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
