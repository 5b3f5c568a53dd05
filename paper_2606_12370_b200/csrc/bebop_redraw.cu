// The fp64 re-draw of the sequences whose fast draw did not clear its error bound (its first kernel also turns
// an expired device-side wait into a status bit), and the hook that times the main kernel.
#include "bebop_pipe.cuh"

namespace bebop {

namespace {

// ------------------------------------------------------------------ fp64 re-draw of the listed sequences
// One small kernel beside the pipelined kernel, for the few sequences whose fast draw did not clear its
// error bound.  Every row is cut into XT = 4T quarter slices; the work items (listed sequence, quarter
// slice) are taken from a counter by a grid that fits the device at once.  Everything is evaluated in double
// around the row exponents that phase A left (any common reference cancels in p = a / sum a).  An item is
//   sum    exact normalisers: sum of exponentials of its quarter slice of the draw rows; then, once
//          the sums of all quarter slices of the sequence are there (a counter per listed sequence),
//   mass   residual mass of the quarter slice, one sum per warp (warp w owns the contiguous vectors
//          [w*cw, (w+1)*cw)); the CTA that completes a sequence picks its token at once: quarter slice
//          and warp chunk from the stored sums, then the few hundred tokens of that chunk are evaluated
//          once more, one or two per thread, and scanned.
// The kernel is a programmatic dependent of the pipelined kernel that does NOT wait for that grid: its
// CTAs move in as CTAs of the main kernel leave, and work through the list while it still grows (records
// carry a mark; one word counts the listed sequences and the sequences whose draw is decided, which tells the
// end of the list).  The sequences
// listed early are finished before the main kernel ends.
struct RedrawArgs {
    RowArgs r;
    const float* u_final;
    VerifyOut o;
    const unsigned long long* fb_count;   // low half: listed sequences so far; high half: sequences whose draw is decided
    const FbRec* fb_list;    // records, valid once their b1 is non-zero
    int expect;              // sequences that get decided: the list is complete when the high half reaches it
    int* wait_failed;        // set by a device-side wait that gave up
    double2* xsum;           // [B][XT] sums of exponentials (target row, draft row) per quarter slice
    double* xmass;           // [B][XT][WW] residual mass per quarter slice and warp chunk
    int* xsdone;             // [B] per listed sequence: sum tasks finished
    int* xdone;              // [B] per listed sequence: mass tasks finished
    int expire;              // test hook: the wait for the list gives up at once
    unsigned* xticket;       // [1] next work item
    int T, slice_vecs;
};

// 2^t in double for t <= about 0: t = n/64 + f with |f| <= 1/128, 2^t = 2^(n >> 6) * tab[n & 63] * 2^f,
// 2^f by its series to the fifth power (the next term is below 4e-17 of the result).  About a dozen
// double-precision instructions, a third of the library routine; the result is within 2 ulp.
// `tab` holds 2^(j/64), j = 0..63, in shared memory.  Arguments below -1000 (and -inf) give 0.
constexpr int XTAB = 64;
__device__ __forceinline__ void x_exp2_table(double* tab) {
    if (threadIdx.x < XTAB) tab[threadIdx.x] = exp2((double)threadIdx.x * (1.0 / XTAB));
}
__device__ __forceinline__ double x_exp2(double t, const double* tab) {
    const double magic = 6755399441055744.0;                 // 1.5 * 2^52: adding it rounds to an integer
    const double tm = fma(t, (double)XTAB, magic);
    const int n = __double2loint(tm);
    const double f = fma(tm - magic, -1.0 / XTAB, t);         // exact
    double p = fma(f, 0.0013333558146428443, 0.009618129107628477);     // ln2^5/120, ln2^4/24
    p = fma(f, p, 0.05550410866482158);                                 // ln2^3/6
    p = fma(f, p, 0.2402265069591007);                                  // ln2^2/2
    p = fma(f, p, 0.6931471805599453);                                  // ln2
    const double s = tab[n & (XTAB - 1)];
    const double r = fma(s * f, p, s);
    // branch-free: an argument of -inf runs through as NaN and is replaced here
    return t > -1000.0 ? __hiloint2double(__double2hiint(r) + ((n >> 6) << 20), __double2loint(r)) : 0.0;
}

struct XRow {
    const char* prow; const char* qrow;
    double c, ep, eq, ip, iq;      // p = exp2(x * c - ep) * ip
    int b, k;
    bool pair;
};
__device__ __forceinline__ double x_resid(const XRow& d, float zp, float zq, const double* tab) {
    // explicit roundings: a contracted p * ip - q would leave rounding dust when p == q
    const double p = __dmul_rn(x_exp2(fma((double)zp, d.c, -d.ep), tab), d.ip);
    if (!d.pair) return p;
    const double q = __dmul_rn(x_exp2(fma((double)zq, d.c, -d.eq), tab), d.iq);
    const double df = p - q;
    return df > 0.0 ? df : 0.0;
}
__device__ __forceinline__ void x_row(const RedrawArgs& a, int slot, XRow* d) {
    const RowArgs& R = a.r;
    bool there;
    const FbRec rec = ld_fb(a.fb_list + slot, &there);          // (x_wait_slot has seen the record valid)
    const int b = rec.b1 - 1, k = rec.kp >> 1;
    d->b = b; d->k = k;
    d->pair = rec.kp & 1;
    d->prow = row_ptr(R, b, k);
    d->qrow = d->pair ? row_ptr(R, b, R.K + 1 + k) : d->prow;
    d->c = 1.4426950408889634 / (double)tau_of(R, b);
    d->ep = (double)rec.ep;
    d->eq = (double)rec.eq;
    d->ip = 1.0; d->iq = 1.0;
}
constexpr int XNU = (kPipeSliceVecs / kRedrawCut + WT - 1) / WT;     // vectors per thread and row in a work item
static_assert(kPipeSliceVecs % (kRedrawCut * 2) == 0 && XNU >= 1 && XNU <= 2, "work items of the fp64 re-draw");

// this thread's vectors of quarter slice s: warp chunk [warp*cw, warp*cw + cw), lanes interleaved
template <int DT>
__device__ __forceinline__ void x_load(const RedrawArgs& a, const XRow& d, int s, float (*fp)[Elem<DT>::VEC],
                                       float (*fq)[Elem<DT>::VEC]) {
    constexpr int VEC = Elem<DT>::VEC;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int qv = a.slice_vecs / kRedrawCut, cw = (qv + WW - 1) / WW;
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

struct PickShared {
    double part[kRedrawCut * MAX_SLICES];     // slice masses of the sequence, later the warp masses of one slice
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

__device__ __forceinline__ unsigned long long x_ld_count(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
// 1: slot is listed and its record is valid; 0: the list is complete and ends before it; -1: a wait gave up
__device__ __forceinline__ int x_wait_slot(const RedrawArgs& a, int slot) {
    if (a.expire) return -1;                             // test hook: this wait's bound has run out already
    uint32_t i = 0;
    for (; i < kSpin; ++i) {
        const unsigned long long w = x_ld_count(a.fb_count);
        if (slot < (int)(w & 0xffffffffull)) break;
        if ((int)(w >> 32) >= a.expect) return 0;
        __nanosleep(256);
    }
    if (i == kSpin) return -1;
    for (i = 0; i < kSpin; ++i) {                       // a place in the list is taken before its record is written
        if (rec_valid(ld_cg(a.fb_list + slot))) return 1;
        __nanosleep(64);
    }
    return -1;
}

template <int DT>
__global__ void __launch_bounds__(WT) k_redraw(const RedrawArgs a) {
    constexpr int VEC = Elem<DT>::VEC;
    __shared__ PickShared S;
    __shared__ double sh[2][WW];
    __shared__ double tab[XTAB];
    __shared__ int go;
    __shared__ unsigned item_sh;
    extern __shared__ double xe[];       // [2][XNU * VEC][WT] exponentials of this item's elements (target row, draft row)
    const RowArgs& R = a.r;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    x_exp2_table(tab);
    const int K = R.K, XT = kRedrawCut * a.T;
    const int qv = a.slice_vecs / kRedrawCut, cw = (qv + WW - 1) / WW;
    const long items_max = (long)R.B * XT;
    __syncthreads();
    // Work items are taken in order from a ticket counter, so the CTAs that are on the device work on the oldest
    // listed sequence; whoever holds an item is running, so the wait for a sequence's other items cannot
    // depend on a CTA that has not started.
    for (;;) {
        if (tid == 0) {
            const unsigned item = atomicAdd(a.xticket, 1u);
            item_sh = item;
            go = item < (unsigned long)items_max ? x_wait_slot(a, (int)(item / (unsigned)XT)) : 0;
        }
        __syncthreads();
        const int g = go;
        const int slot = (int)(item_sh / (unsigned)XT), s = (int)(item_sh - (unsigned)slot * (unsigned)XT);
        __syncthreads();
        if (g <= 0) {                                   // slots come in rising order: nothing behind this one either
            if (g < 0 && tid == 0) atomicExch(a.wait_failed, 1);
            break;
        }
        XRow d;
        x_row(a, slot, &d);
        const int b = d.b;
        // ---- sum of exponentials of this quarter slice
        {
            float fp[XNU][VEC], fq[XNU][VEC];
            x_load<DT>(a, d, s, fp, fq);
            double sa = 0.0, sb = 0.0;
#pragma unroll
            for (int u = 0; u < XNU; ++u) {
#pragma unroll
                for (int i = 0; i < VEC; ++i) {
                    const double ea = x_exp2(fma((double)fp[u][i], d.c, -d.ep), tab);
                    sa += ea;
                    if (d.pair) {
                        const double eb = x_exp2(fma((double)fq[u][i], d.c, -d.eq), tab);
                        sb += eb;
                        // kept for the mass pass, which then needs neither the rows nor the exponentials again
                        xe[(u * VEC + i) * WT + tid] = ea;
                        xe[((XNU + u) * VEC + i) * WT + tid] = eb;
                    }
                }
            }
            sa = warp_sum(sa); sb = warp_sum(sb);
            if (lane == 0) { sh[0][warp] = sa; sh[1][warp] = sb; }
            __syncthreads();
            if (tid == 0) {
                double ta = 0.0, tb = 0.0;
                for (int w = 0; w < WW; ++w) { ta += sh[0][w]; tb += sh[1][w]; }
                a.xsum[(int64_t)b * XT + s] = make_double2(ta, tb);
                __threadfence();
                atomicAdd(a.xsdone + slot, 1);
                // ... and wait (bounded) for the other quarter slices of the sequence
                go = spin_ge(a.xsdone + slot, XT) ? 1 : 0;
            }
            __syncthreads();
            const int ok = go;
            __syncthreads();
            if (!ok) {
                if (tid == 0) { atomicExch(a.wait_failed, 1); if (a.o.row_status) atomicOr(a.o.row_status + b, ST_WAIT); }
                continue;
            }
        }
        // exact normalisers: every warp adds the quarter-slice sums in the same order (lane t takes sums t,
        // t + 32, ...; the butterfly leaves the same bits in every lane), so every CTA gets the same value
        double Sa = 0.0, Sb = 0.0;
        for (int t = lane; t < XT; t += 32) { const double2 x = __ldcg(a.xsum + (int64_t)b * XT + t); Sa += x.x; Sb += x.y; }
        Sa = warp_sum(Sa); Sb = warp_sum(Sb);
        d.ip = 1.0 / Sa; d.iq = d.pair ? 1.0 / Sb : 0.0;
        if (d.pair) {     // a bonus row needs no mass pass: its masses are sums of exponentials over Sa
            double m = 0.0;
#pragma unroll
            for (int j = 0; j < XNU * VEC; ++j) {
                // as x_resid, from the stored exponentials (explicit roundings: see there)
                const double p = __dmul_rn(xe[j * WT + tid], d.ip);
                const double q = __dmul_rn(xe[(XNU * VEC + j) * WT + tid], d.iq);
                const double df = p - q;
                m += df > 0.0 ? df : 0.0;
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
                else m = __ldcg(a.xsum + (int64_t)b * XT + t).x * d.ip;
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
            if (zero_resid && a.o.row_status) {
                // the main kernel writes this row's status word once, with a plain store: add the bit only when
                // that grid is through (rare, and then a wait of some microseconds at most)
                asm volatile("griddepcontrol.wait;" ::: "memory");
                atomicOr(a.o.row_status + b, ST_ZERO_RESID);
            }
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
                    for (int i = 0; i < VEC; ++i) wm += x_resid(d, f[i], 0.f, tab);
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
                r[i] = x_resid(d, zp, zq, tab);
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
    // Every CTA waits here for the main grid, whatever the caller asked for: a dependent of a grid that lets its
    // dependents start early has to, or work enqueued behind this kernel (a copy of the results, the next call's
    // clearing of this workspace) would not be ordered behind that grid.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // a wait that gave up, in the main kernel or here: every row's status says so
    if (a.o.row_status && ld_acquire(a.wait_failed) != 0)
        for (int b = blockIdx.x * WT + tid; b < R.B; b += gridDim.x * WT) atomicOr(a.o.row_status + b, ST_WAIT);
}

}  // namespace

cudaEvent_t g_ev_start = nullptr, g_ev_stop = nullptr;
void pipe_set_events(cudaEvent_t start, cudaEvent_t stop) { g_ev_start = start; g_ev_stop = stop; }

namespace {
template <int DT>
constexpr size_t redraw_smem() { return sizeof(double) * 2 * XNU * Elem<DT>::VEC * WT; }
template <int DT>
int redraw_grid() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (dev >= 0 && dev < 64 && cached[dev]) return cached[dev];
    int per_sm = 0, sms = 0;
    if (cudaFuncSetAttribute(k_redraw<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)redraw_smem<DT>()) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_redraw<DT>, WT, redraw_smem<DT>()) != cudaSuccess) per_sm = 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaGetLastError();
    const int n = per_sm * sms;
    if (dev >= 0 && dev < 64) cached[dev] = n;
    return n;
}
}  // namespace

// fp64 re-draw of the listed sequences (usually a few per cent of the batch; the count stays on the device).
// `expect` sequences get their draw decided by the main kernel (0: none, nothing is listed).
cudaError_t redraw_launch(const RowArgs& a, const float* u_final, VerifyOut o, const unsigned long long* fb_count,
                          const FbRec* fb_list, int expect, int* wait_failed, char* w,
                          const PipePlan& wp, cudaStream_t stream, bool expire_list_wait) {
    RedrawArgs ra;
    ra.expire = expire_list_wait ? 1 : 0;
    ra.r = a; ra.u_final = u_final; ra.o = o;
    ra.fb_count = fb_count; ra.fb_list = fb_list; ra.expect = expect;
    ra.wait_failed = wait_failed;
    ra.xsum = reinterpret_cast<double2*>(w + wp.off_xsum);
    ra.xmass = reinterpret_cast<double*>(w + wp.off_xmass);
    ra.xsdone = reinterpret_cast<int*>(w + wp.off_xsdone);
    ra.xdone = reinterpret_cast<int*>(w + wp.off_xdone);
    ra.xticket = reinterpret_cast<unsigned*>(w + kRedrawTicketOffset);
    ra.T = wp.T; ra.slice_vecs = wp.slice_vecs;
    // CTAs of this grid wait for one another (the sums of a sequence come from kRedrawCut * T of them), so
    // the grid is at most what fits the device at once; a CTA takes work items from a counter.
    const int cap = a.dt == 0 ? redraw_grid<0>() : redraw_grid<1>();
    if (cap < 1) return cudaErrorLaunchOutOfResources;
    const long items_max = (long)a.B * kRedrawCut * wp.T;
    const int grid = (int)(items_max < cap ? items_max : cap);
    // scheduled as soon as the main kernel lets go of SMs; it does not wait for that grid as a whole
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(WT); cfg.stream = stream;
    cfg.dynamicSmemBytes = a.dt == 0 ? redraw_smem<0>() : redraw_smem<1>();
    cfg.attrs = attr; cfg.numAttrs = 1;
    return a.dt == 0 ? cudaLaunchKernelEx(&cfg, k_redraw<0>, ra) : cudaLaunchKernelEx(&cfg, k_redraw<1>, ra);
}

}  // namespace bebop
