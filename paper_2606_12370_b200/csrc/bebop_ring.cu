// Ring kernel: the single-read, one-exponential-per-logit hot path of bebop_verify.
//
// A cluster of CS CTAs walks the row pairs of its sequences in order.  Each CTA
// owns a contiguous, 128-byte aligned vocabulary slice of every row; bulk
// asynchronous copies (TMA, no multicast) stream the slices of the target and the
// draft row into a two-stage shared-memory ring two items ahead.
//
// Warps run free (no block- or cluster-wide barrier in the steady state) and work
// in chunks of 32 vectors (256 bf16 logits per row).  Producing a chunk means:
// read it from the stage, take its maximum, compute one exponential per logit
// relative to the chunk's own power-of-two reference 2^E, and park the
// exponentials in TENSOR MEMORY (each warp owns an 8-slot ring there).  When all
// chunks of an item are parked the warp publishes its (E, sum); the last warp of
// the CTA combines the partials and sends them to every CTA of the cluster through
// distributed shared memory, arriving on their mbarriers.  Consuming a chunk, once
// the row normalisers are merged, means: load it back from tensor memory, scale by
// an exact power of two times 1/S, and accumulate TV = sum max(0, p - q); at the
// stop row the residuals also stay in registers for the inverse-CDF walk.
//
// Because the exponentials of item t wait in tensor memory, a warp produces the
// chunks of item t+1 (exponential pipe) while the normalisers of item t are still
// being exchanged, and interleaves the consumption of item t (FMA pipe) with the
// rest of item t+1: the exchange latency and the TV arithmetic hide behind the
// exponentials of the next item.
//
// The draw is kept only if the crossing clears an error bound derived from the
// fp32 element error (draw_bound); otherwise the sequence is appended to a list that
// the fp64 kernels of the general path re-draw.  Sequences that accept every draft
// get their bonus row in a second phase through the same rings.
//
// All warps of a cluster derive the item stream from the same exchanged data, so
// they agree on what to wait for.  Every wait is bounded; an expired wait raises
// BEBOP_ROW_WAIT_EXPIRED and the warp carries on (results undefined, flagged).
#include "bebop_kernels.h"
#include "bebop_ptx.cuh"

namespace bebop {

namespace {

constexpr int NT = 512;            // threads per CTA
constexpr int NW = NT / 32;        // warps per CTA
constexpr int CS = 8;              // CTAs per cluster
constexpr int RING = 4;            // depth of the exchange rings
constexpr int NSLOT = 8;           // tensor-memory slots (chunks) per warp
constexpr int NCH = 5;             // chunks per warp and item, at most
constexpr int MAXCH = NW * NCH;    // chunks per CTA slice, at most
constexpr int MAXSEQ = 128;        // sequences per cluster and launch (two 64-bit bonus masks)
constexpr int E_EMPTY = INT_MIN / 2;
#ifndef BEBOP_TMA_CHUNK
#define BEBOP_TMA_CHUNK 8192
#endif
constexpr uint32_t kChunk = BEBOP_TMA_CHUNK;

struct __align__(16) WPart { float sp, sq; int ep, eq; };                  // per-warp softmax partial
struct __align__(16) CPart { double sp, sq; int ep, eq, flags, pad; };     // per-CTA softmax partial
struct __align__(16) DPart { double tot; float sq; int pad; };             // residual mass, sum of squares
struct __align__(8) RPart { int y, cert; };                                 // result of an owner's walk

struct RingShared {
    unsigned long long full[2];
    unsigned long long stats_bar[RING], draw_bar[RING], z_bar[RING], res_bar[RING];
    int relcnt[2];
    int wcnt[RING], zcnt[RING], dcnt[RING], rcnt[RING];
    int wflags[RING];
    WPart wpart[RING][NW];
    CPart cslot[RING][CS];
    float wz[RING][NW];
    float zslot[RING][CS];
    double csum[RING][MAXCH];        // residual mass of every chunk of the slice (draw items)
    float wsq[RING][NW];
    DPart dslot[RING][CS];
    RPart wres[RING][NW];
    RPart rslot[RING][CS];
    uint32_t tmem_base;
    int wait_failed;
};

struct RingArgs {
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

__device__ __forceinline__ int row_status(int flagbit, int E, double S) {
    if (flagbit || !(S == S)) return ST_NONFINITE;
    return E == E_EMPTY ? ST_EMPTY : 0;
}

// Reference exponent of a chunk with maximum m: E = ceil(m * c) and frac = E - m * c in [0, 1],
// evaluated without rounding loss (the product's rounding error is recovered with an FMA), so
// that 2^((x - m) * c - frac) equals 2^(x * c - E) for every chunk alike.
__device__ __forceinline__ void chunk_reference(float m, float c, int* E, float* frac) {
    float th = fminf(fmaxf(m * c, -4.0e6f), 4.0e6f);
    float te = fmaf(m, c, -th);
    if (th != m * c) te = 0.f;                    // saturated: absurd range, keep it finite
    float Ef;
    int Ei = ceil_alu(th, &Ef);
    float f = (Ef - th) - te;
    if (f < 0.f) { f += 1.f; Ei += 1; }
    *E = Ei; *frac = f;
}

}  // namespace

#ifdef BEBOP_TRACE
#ifndef BEBOP_TRACE_TID
#define BEBOP_TRACE_TID 0
#endif
#ifndef BEBOP_TRACE_RANK
#define BEBOP_TRACE_RANK 0
#endif
#define TRACE(id) do { if (a.trace && cid == 0 && rank == BEBOP_TRACE_RANK && tid == BEBOP_TRACE_TID && t < 60) a.trace[t * 16 + (id)] = clock64(); } while (0)
#else
#define TRACE(id) do {} while (0)
#endif

// =============================================================================
template <int DT>
__global__ void __launch_bounds__(NT, 1) k_ring(const RingArgs a) {
    constexpr int VEC = Elem<DT>::VEC;
    constexpr int ROW_BYTES = NW * NCH * 32 * 16;        // stage bytes per row slice (capacity)
    extern __shared__ __align__(128) unsigned char smem_raw[];
    unsigned char* stage = smem_raw;                     // [2 stages][2 rows][ROW_BYTES]
    RingShared& S = *reinterpret_cast<RingShared*>(smem_raw + 4 * ROW_BYTES);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rank = (int)cluster_rank();
    const int cid = (int)cluster_id(), ncl = (int)num_clusters();
    const RowArgs& R = a.r;
    const int K = R.K, V = R.V;

    const int v_begin = min(rank * a.vs, R.nvec);
    const int nv_cta = max(min(a.vs, R.nvec - v_begin), 0);
    const uint32_t slice_bytes = (uint32_t)nv_cta * 16u;
    const int64_t slice_off = (int64_t)v_begin * 16;
    const int nchunks = (nv_cta + 31) >> 5;              // chunks of this CTA's slice
    const int nc = nchunks > warp ? (nchunks - warp + NW - 1) / NW : 0;   // chunks of this warp per item

    if (tid == 0) {
        mbar_init(smem_u32(&S.full[0]), 1);
        mbar_init(smem_u32(&S.full[1]), 1);
        for (int i = 0; i < RING; ++i) {
            mbar_init(smem_u32(&S.stats_bar[i]), CS);
            mbar_init(smem_u32(&S.draw_bar[i]), CS);
            mbar_init(smem_u32(&S.z_bar[i]), CS);
            mbar_init(smem_u32(&S.res_bar[i]), CS);
            S.wcnt[i] = S.zcnt[i] = S.dcnt[i] = S.rcnt[i] = 0;
            S.wflags[i] = 0;
        }
        S.relcnt[0] = S.relcnt[1] = 0;
        S.wait_failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    if (warp == 0) tmem_alloc512(smem_u32(&S.tmem_base));
    tmem_fence_before_sync();
    __syncthreads();
    tmem_fence_after_sync();
    cluster_arrive();
    cluster_wait();
    // this warp's ring in tensor memory: lanes 32*(warp%4).., columns 128*(warp/4) .. +127
    const uint32_t tm_warp = S.tmem_base + (((uint32_t)(warp & 3) * 32u) << 16) + (uint32_t)(warp >> 2) * 128u;

    // ---- sequences of this cluster: b = b0 + cid + j * ncl, j = 0 .. nseq-1 (nseq <= MAXSEQ)
    const int nseq = (a.nb - cid + ncl - 1) / ncl;
    auto seq_b = [&](int j) { return a.b0 + cid + j * ncl; };
    auto trow = [&](int b, int k) { return R.target + ((int64_t)b * R.t_seq_rows + k) * R.t_row_bytes; };
    auto drow = [&](int b, int k) { return R.draft + ((int64_t)b * R.d_seq_rows + k) * R.d_row_bytes; };

    unsigned long long bm0 = 0, bm1 = 0;   // bonus mask: bit j set when sequence j needs its bonus row
    for (int j = 0; j < nseq; ++j)
        if (len_of(R, seq_b(j)) == 0) { if (j < 64) bm0 |= 1ull << j; else bm1 |= 1ull << (j - 64); }

    // ---- item descriptors.  An item is a row pair (b, k) or a bonus row (k == L).
    struct Item { int j, k, L; bool pair; bool valid; };
    struct PC { int j, k, L; };
    auto pc_skip = [&](PC& c) { while (c.j < nseq && (c.L = len_of(R, seq_b(c.j))) == 0) ++c.j; };
    auto pc_next = [&](PC& c) { if (c.j >= nseq) return; if (++c.k < c.L) return; c.k = 0; ++c.j; pc_skip(c); };
    struct BC { unsigned long long m0, m1; };
    auto bc_peek = [&](const BC& c) { return c.m0 ? __ffsll((long long)c.m0) - 1 : (c.m1 ? 63 + __ffsll((long long)c.m1) : -1); };
    auto bc_pop = [&](BC& c) { if (c.m0) c.m0 &= c.m0 - 1; else if (c.m1) c.m1 &= c.m1 - 1; };

    auto issue = [&](int st, const char* prow, const char* qrow) {   // by a whole warp
        if (nv_cta <= 0) return;
        const uint32_t bar = smem_u32(&S.full[st]);
        const uint32_t dst = smem_u32(stage + (size_t)st * 2 * ROW_BYTES);
        if (lane == 0) mbar_expect_tx(bar, qrow ? 2 * slice_bytes : slice_bytes);
        __syncwarp();
        const uint32_t nck = (slice_bytes + kChunk - 1) / kChunk;
        for (uint32_t ci = lane; ci < (qrow ? 2 * nck : nck); ci += 32) {
            const uint32_t row = ci >= nck ? 1u : 0u, cc = ci - row * nck;
            const uint32_t off = cc * kChunk, len = min(kChunk, slice_bytes - off);
            bulk_g2s(dst + row * ROW_BYTES + off, (row ? qrow : prow) + slice_off + off, len, bar);
        }
    };
    auto issue_item = [&](int st, const Item& it) {
        const int b = seq_b(it.j);
        issue(st, trow(b, it.k), it.pair ? drow(b, it.k) : nullptr);
    };

    // Item streams: `pc`/`bc` enumerate what is PRODUCED next; `ld*` run two items ahead for the copies.
    int phase = 1;                      // phase of the producer cursor: 1 pairs, 2 bonus rows
    PC pc{0, 0, 0}, ldc{0, 0, 0};
    pc_skip(pc);
    ldc = pc;
    BC bc{0, 0}, ldb{0, 0};
    if (pc.j >= nseq) { phase = 2; bc.m0 = bm0; bc.m1 = bm1; ldb = bc; }
    auto prod_item = [&]() {
        Item it; it.valid = false; it.j = 0; it.k = 0; it.L = 0; it.pair = true;
        if (phase == 1) { if (pc.j < nseq) { it.j = pc.j; it.k = pc.k; it.L = pc.L; it.pair = true; it.valid = true; } }
        else { int j = bc_peek(bc); if (j >= 0) { it.j = j; it.L = len_of(R, seq_b(j)); it.k = it.L; it.pair = false; it.valid = true; } }
        return it;
    };
    auto ld_item_pop = [&]() {          // next item to copy, advancing the copy cursor
        Item it; it.valid = false; it.j = 0; it.k = 0; it.L = 0; it.pair = true;
        if (phase == 1) { if (ldc.j < nseq) { it.j = ldc.j; it.k = ldc.k; it.L = ldc.L; it.valid = true; pc_next(ldc); } }
        else { int j = bc_peek(ldb); if (j >= 0) { it.j = j; it.L = len_of(R, seq_b(j)); it.k = it.L; it.pair = false; it.valid = true; bc_pop(ldb); } }
        return it;
    };
    // prologue: warp 0 starts the copies of the first two items
    for (int s = 0; s < 2; ++s) { Item it = ld_item_pop(); if (it.valid && warp == 0) issue_item(s, it); }

    // ---- per-warp ring state
    int nprod = 0, ncons = 0;           // chunks produced / consumed so far (slot = count % NSLOT)
    int meta_ep = E_EMPTY, meta_eq = E_EMPTY;   // lane s holds the chunk references of slot s
    int pitem = 0;                      // index of the item being produced (stage = pitem & 1)

    // running softmax partial of the item being produced
    int Ewp = E_EMPTY, Ewq = E_EMPTY, pflags = 0;
    float slp = 0.f, slq = 0.f;
    int pchunk = 0;                     // chunks of the current item produced so far by this warp
    float pc_c = kLog2e;                // log2(e) / tau of the item being produced

    // Produce chunk `pchunk` of the current item (it) into the ring.
    auto produce = [&](const Item& it) {
        const int st = pitem & 1;
        const int cidx = warp + pchunk * NW;                 // chunk of the CTA slice
        const int lv = (cidx << 5) + lane;                   // vector of the slice
        const unsigned char* sp_ = stage + (size_t)st * 2 * ROW_BYTES;
        uint4 rp = neg_inf_vec<DT>(), rq = neg_inf_vec<DT>();
        if (lv < nv_cta) {
            rp = *reinterpret_cast<const uint4*>(sp_ + (size_t)lv * 16);
            if (it.pair) rq = *reinterpret_cast<const uint4*>(sp_ + ROW_BYTES + (size_t)lv * 16);
            const int gbase = (v_begin + lv) * VEC;
            if (gbase + VEC > V) { mask_tail<DT>(rp, V - gbase); mask_tail<DT>(rq, V - gbase); }
        }
        float mp = ord2f(redux_max(f2ord(vec_max<DT>(rp))));
        float mq = ord2f(redux_max(f2ord(vec_max<DT>(rq))));
        int Ep = E_EMPTY, Eq = E_EMPTY;
        float fp_ = 0.f, fq_ = 0.f, mpu = 0.f, mqu = 0.f;
        if (mp != mp || mp == INFINITY) pflags |= 1;
        else if (mp != -INFINITY) { chunk_reference(mp, pc_c, &Ep, &fp_); mpu = mp; }
        if (it.pair) {
            if (mq != mq || mq == INFINITY) pflags |= 2;
            else if (mq != -INFINITY) { chunk_reference(mq, pc_c, &Eq, &fq_); mqu = mq; }
        }
        const int slot = nprod & (NSLOT - 1);
        const uint32_t taddr = tm_warp + (uint32_t)slot * 16u;
        float f[VEC], e[8];
        float cs_p = 0.f, cs_q = 0.f;
        // target row
        unpack<DT>(rp, f);
#pragma unroll
        for (int i = 0; i < VEC; ++i) { e[i] = ex2f(fmaf(f[i] - mpu, pc_c, -fp_)); cs_p += e[i]; }
#pragma unroll
        for (int i = VEC; i < 8; ++i) e[i] = 0.f;
        tmem_st8(taddr, e);
        if (it.pair) {
            unpack<DT>(rq, f);
#pragma unroll
            for (int i = 0; i < VEC; ++i) { e[i] = ex2f(fmaf(f[i] - mqu, pc_c, -fq_)); cs_q += e[i]; }
            tmem_st8(taddr + 8, e);
        }
        if (lane == slot) { meta_ep = Ep; meta_eq = Eq; }
        // running sums of this lane, relative to the running references of the warp
        if (Ep > E_EMPTY) {
            const int En = max(Ewp, Ep);
            slp = slp * pow2f(Ewp > E_EMPTY ? Ewp - En : -200) + cs_p * pow2f(Ep - En);
            Ewp = En;
        }
        if (Eq > E_EMPTY) {
            const int En = max(Ewq, Eq);
            slq = slq * pow2f(Ewq > E_EMPTY ? Ewq - En : -200) + cs_q * pow2f(Eq - En);
            Ewq = En;
        }
        tmem_wait_st();
        nprod++; pchunk++;
    };

    // After the last chunk of an item: release the stage (the last warp refills it) and publish.
    auto finish_item = [&](int slot_r) {
        const int st = pitem & 1;
        {
            int last = 0;
            if (lane == 0) last = atomicAdd(&S.relcnt[st], 1) == NW - 1;
            last = __shfl_sync(0xffffffffu, last, 0);
            Item nx = ld_item_pop();              // every warp advances the copy cursor
            if (last) {
                if (lane == 0) S.relcnt[st] = 0;
                fence_proxy_async();
                if (nx.valid) issue_item(st, nx);
            }
        }
        // warp partial: sums of the lanes in a fixed order
        float sp = slp, sq = slq;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { sp += __shfl_xor_sync(0xffffffffu, sp, o); sq += __shfl_xor_sync(0xffffffffu, sq, o); }
        int last = 0;
        if (lane == 0) {
            WPart w; w.sp = sp; w.sq = sq; w.ep = Ewp; w.eq = Ewq;
            S.wpart[slot_r][warp] = w;
            if (pflags) atomicOr(&S.wflags[slot_r], pflags);
            __threadfence_block();
            last = atomicAdd(&S.wcnt[slot_r], 1) == NW - 1;
        }
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {
            __threadfence_block();
            WPart w;
            if (lane < NW) w = S.wpart[slot_r][lane]; else { w.sp = w.sq = 0.f; w.ep = w.eq = E_EMPTY; }
            const int fl = S.wflags[slot_r];
            __syncwarp();
            if (lane == 0) { S.wcnt[slot_r] = 0; S.wflags[slot_r] = 0; }
            const int Ecp = redux_max(w.ep), Ecq = redux_max(w.eq);
            double tp = w.ep > E_EMPTY ? (double)(w.sp * pow2f(max(w.ep - Ecp, -200))) : 0.0;
            double tq = w.eq > E_EMPTY ? (double)(w.sq * pow2f(max(w.eq - Ecq, -200))) : 0.0;
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) { tp += shfl_xor_d(tp, o); tq += shfl_xor_d(tq, o); }
            if (lane < CS) {
                const uint32_t dst = mapa(smem_u32(&S.cslot[slot_r][rank]), (uint32_t)lane);
                uint4 w0, w1;
                w0.x = (uint32_t)__double2loint(tp); w0.y = (uint32_t)__double2hiint(tp);
                w0.z = (uint32_t)__double2loint(tq); w0.w = (uint32_t)__double2hiint(tq);
                w1.x = (uint32_t)Ecp; w1.y = (uint32_t)Ecq; w1.z = (uint32_t)fl; w1.w = 0;
                st_cluster_v4(dst, w0);
                st_cluster_v4(dst + 16, w1);
                mbar_arrive_remote(mapa(smem_u32(&S.stats_bar[slot_r]), (uint32_t)lane));
            }
            __syncwarp();
        }
        Ewp = E_EMPTY; Ewq = E_EMPTY; pflags = 0; slp = 0.f; slq = 0.f; pchunk = 0;
        pitem++;
    };

    // Begin producing item `it`: wait for its stage, set the scale.
    auto begin_item = [&](const Item& it, float tau_it) {
        if (nv_cta > 0 && !mbar_wait(smem_u32(&S.full[pitem & 1]), (uint32_t)(pitem >> 1) & 1u)) S.wait_failed = 1;
        pc_c = kLog2e / (tau_ok(tau_it) ? tau_it : 1.f);
    };

    // ---- consumer-side state: scalars of the sequence being consumed, history for deferred outputs
    int seq_alive = 1, seq_n = 0, seq_st = 0;
    int tokl = 0;
    float c_tau = 1.f, c_ufin = 0.5f;
    int ndraw = 0;
    int h_r[2] = {0, 0}, h_b[2] = {-1, -1}, h_k[2] = {0, 0}, h_fatal[2] = {0, 0};
    int hd_b[2] = {-1, -1}, hd_n[2] = {0, 0}, hd_idx[2] = {0, 0};
    // pending draw (resolved one step later): residuals of this lane's elements, per chunk
    float rr[NCH][8];
    float rls[NCH];
    int pd_valid = 0, pd_idx = 0, pd_b = 0, pd_n = 0, pd_step = 0, pd_cancel = 0;
    float pd_ufin = 0.5f;
#pragma unroll
    for (int i = 0; i < NCH; ++i) { rls[i] = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) rr[i][e] = 0.f; }

    auto flush_outputs = [&](int hi) {      // rank 0, warp 0
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

    // Second half of a draw: locate the crossing among this CTA's chunks, walk it, report to rank 0.
    auto resolve_draw = [&]() {
        const int ds = pd_idx & (RING - 1);
        if (!mbar_wait_cluster(smem_u32(&S.draw_bar[ds]), (uint32_t)(pd_idx / RING) & 1u)) S.wait_failed = 1;
        double base = 0.0, Z = 0.0, sumsq = 0.0, mytot = 0.0;
        for (int i = 0; i < CS; ++i) {
            if (i == rank) { base = Z; mytot = S.dslot[ds][i].tot; }
            Z += S.dslot[ds][i].tot; sumsq += (double)S.dslot[ds][i].sq;
        }
        const double T = (double)pd_ufin * Z;
        const double bound = draw_bound(sumsq);
        int wy = -1, wc = 0;
        if (T > base && T <= base + mytot) {
            // prefix over this CTA's chunk totals, identical in every warp
            double run = base;
            int cstar = -1; double cbase = 0.0;
            for (int c = 0; c < nchunks; ++c) {
                const double nx = run + S.csum[ds][c];
                if (cstar < 0 && T > run && T <= nx) { cstar = c; cbase = run; }
                run = nx;
            }
            if (cstar >= 0 && (cstar & (NW - 1)) == warp) {
                const int istar = cstar / NW;
                float ls = 0.f;
#pragma unroll
                for (int i = 0; i < NCH; ++i) if (i == istar) ls = rls[i];
                double incl = (double)ls;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) { double tt = shfl_up_d(incl, d); if (lane >= d) incl += tt; }
                double prev = shfl_up_d(incl, 1);
                if (lane == 0) prev = 0.0;
                const double lower = cbase + prev, upper = cbase + incl;
                int my_y = -1, my_cert = 0;
                if (lower < T && T <= upper) {
                    double C = lower;
                    const int g0 = (v_begin + (cstar << 5) + lane) * VEC;
#pragma unroll
                    for (int i = 0; i < NCH; ++i) {
                        if (i == istar) {
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                if (my_y < 0) {
                                    const double r1 = (double)rr[i][e];
                                    const double Cn = C + r1;
                                    if (r1 > 0.0 && Cn >= T) { my_y = g0 + e; my_cert = (T - C > bound) && (Cn - T >= bound); }
                                    C = Cn;
                                }
                            }
                        }
                    }
                }
                const unsigned own = __ballot_sync(0xffffffffu, my_y >= 0);
                if (own) {
                    const int src = __ffs(own) - 1;
                    wy = __shfl_sync(0xffffffffu, my_y, src); wc = __shfl_sync(0xffffffffu, my_cert, src);
                    if (__popc(own) > 1) wc = 0;
                }
            }
        }
        int last = 0;
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
        if (rank == 0 && warp == 0) { const int hi = pd_step & 1; hd_b[hi] = pd_cancel ? -1 : pd_b; hd_n[hi] = pd_n; hd_idx[hi] = pd_idx; }
        pd_valid = 0;
    };

    // =========================================================================
    // prologue: produce every chunk of the first item
    Item cur_it = prod_item();                      // item t (to be consumed at step t)
    float tau_cur = 1.f;
    if (cur_it.valid) {
        const int b = seq_b(cur_it.j);
        tau_cur = tau_of(R, b);
        tokl = lane < cur_it.L ? a.draft_tokens[(int64_t)b * K + lane] : 0;
        c_ufin = a.u_final[b];
        begin_item(cur_it, tau_cur);
        for (int i = 0; i < nc; ++i) produce(cur_it);
        finish_item(0);
        if (phase == 1) pc_next(pc); else bc_pop(bc);
    }
    c_tau = tau_cur;

    for (int t = 0; cur_it.valid; ++t) {
        const int slot = t & (RING - 1);
        const uint32_t ring_par = (uint32_t)(t / RING) & 1u;
        const bool pair = cur_it.pair;
        const int j = cur_it.j, k = cur_it.k, L = cur_it.L;
        const int b = seq_b(j);
        TRACE(0);

        // ------------------------------------------------ the next item (produced during this step)
        Item nx = prod_item();
        float tau_nx = c_tau, ufin_nx = c_ufin;
        int tokl_nx = tokl;
        const bool nx_new_seq = nx.valid && (nx.pair ? nx.k == 0 : true);
        if (nx_new_seq) {
            const int bn = seq_b(nx.j);
            tau_nx = tau_of(R, bn);
            tokl_nx = lane < nx.L && nx.pair ? a.draft_tokens[(int64_t)bn * K + lane] : 0;
            ufin_nx = a.u_final[bn];
        }
        // scalars of the item consumed now
        if (pair ? k == 0 : true) {
            const bool ok = tau_ok(c_tau);
            if (pair) {
                seq_alive = 1; seq_n = L; seq_st = ok ? 0 : ST_BAD_TEMP;
                if (!seq_st && __ballot_sync(0xffffffffu, lane < L && (tokl < 0 || tokl >= V))) seq_st = ST_BAD_TOKEN;
            } else seq_st = ok ? 0 : ST_BAD_TEMP;
        }
        const float c = kLog2e / (tau_ok(c_tau) ? c_tau : 1.f);
        float zpx = 0.f, zqx = 0.f, u_acc = 0.5f;
        if (pair) {
            int tk = min(max(__shfl_sync(0xffffffffu, tokl, k), 0), V - 1);
            zpx = DT == 0 ? load_one<0>(trow(b, k), tk) : load_one<1>(trow(b, k), tk);
            zqx = DT == 0 ? load_one<0>(drow(b, k), tk) : load_one<1>(drow(b, k), tk);
            u_acc = a.u_accept[(int64_t)b * K + k];
        }

        // ------------------------------------------------ part 1 of the next item: fill the free slots
        int n1 = 0;
        if (nx.valid) {
            begin_item(nx, tau_nx);
            n1 = min(nc, NSLOT - (nprod - ncons));
            for (int i = 0; i < n1; ++i) produce(nx);
        }
        TRACE(1);
        if (pd_valid) resolve_draw();
        if (rank == 0 && warp == 0 && t >= 2) flush_outputs(t & 1);
        TRACE(2);

        // ------------------------------------------------ merged normalisers of item t, accept test
        if (!mbar_wait_cluster(smem_u32(&S.stats_bar[slot]), ring_par)) S.wait_failed = 1;
        TRACE(3);
        int bad = 0, stop_here = 0, Em_p, Em_q;
        double Sp, Sq, iSp = 0.0, iSq = 0.0;
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
            if (!bad) { iSp = __drcp_rn(Sp); if (pair) iSq = __drcp_rn(Sq); }
        }
        const float iSp_hi = (float)iSp, iSp_lo = (float)(iSp - (double)iSp_hi);
        const float iSq_hi = (float)iSq, iSq_lo = (float)(iSq - (double)iSq_hi);
        if (pair && !bad && !(seq_st & ST_FATAL)) {
            float pxf = ex2f(fmaf(zpx, c, -(float)Em_p)) * iSp_hi;
            float qxf = ex2f(fmaf(zqx, c, -(float)Em_q)) * iSq_hi;
            float lhs = u_acc * qxf;
            bool acc = lhs < pxf;
            double pxd = pxf, qxd = qxf;
            if (fabsf(lhs - pxf) <= 1e-3f * fmaxf(lhs, pxf)) {
                const double cd = (double)c;
                pxd = exp2((double)zpx * cd - (double)Em_p) * iSp;
                qxd = exp2((double)zqx * cd - (double)Em_q) * iSq;
                acc = (double)u_acc * qxd < pxd;
            }
            if (rank == 0 && warp == 0 && lane == 0) {
                if (a.o.p_draft) a.o.p_draft[(int64_t)b * K + k] = (float)pxd;
                if (a.o.q_draft) a.o.q_draft[(int64_t)b * K + k] = (float)qxd;
            }
            if (seq_alive && !acc) stop_here = 1;
        }
        if (!(seq_st & ST_FATAL)) seq_st |= bad;
        const bool do_draw = !(seq_st & ST_FATAL) && (pair ? stop_here != 0 : true);
        TRACE(4);

        // ------------------------------------------------ consume item t, produce the rest of item t+1
        float z_l = 0.f, sq_l = 0.f;
        const int ds = ndraw & (RING - 1);
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            if (i < nc) {
                const int cslot_ = ncons & (NSLOT - 1);
                const uint32_t taddr = tm_warp + (uint32_t)cslot_ * 16u;
                float ep[8], eq[8];
                tmem_ld8(taddr, ep);
                if (pair) tmem_ld8(taddr + 8, eq);
                const int Ecp = __shfl_sync(0xffffffffu, meta_ep, cslot_);
                const int Ecq = __shfl_sync(0xffffffffu, meta_eq, cslot_);
                const float sa = Ecp > E_EMPTY ? pow2f(max(Ecp - Em_p, -126)) : 0.f;
                const float sb = Ecq > E_EMPTY ? pow2f(max(Ecq - Em_q, -126)) : 0.f;
                tmem_wait_ld();
                if (!pair) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) eq[e] = 0.f;
                }
                if (!bad) {
                    if (!do_draw) {
                        const float aa = sa * iSp_hi, bb = sb * iSq_hi;
#pragma unroll
                        for (int e = 0; e < 8; ++e) z_l += fmaxf(fmaf(ep[e], aa, -__fmul_rn(eq[e], bb)), 0.f);
                    } else {
                        const float ah = sa * iSp_hi, al = sa * iSp_lo, bh = sb * iSq_hi, bl = sb * iSq_lo;
                        float v[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const float p = fmaf(ep[e], al, __fmul_rn(ep[e], ah));
                            const float q = fmaf(eq[e], bl, __fmul_rn(eq[e], bh));
                            v[e] = fmaxf(p - q, 0.f);
                            rr[i][e] = v[e];
                            sq_l = fmaf(p, p, sq_l); sq_l = fmaf(q, q, sq_l);
                        }
                        const float ls = ((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7]));
                        rls[i] = ls;
                        z_l += ls;
                        double ct = (double)ls;
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) ct += shfl_xor_d(ct, o);
                        if (lane == 0) S.csum[ds][warp + i * NW] = ct;
                    }
                }
                ncons++;
                // the slot just freed takes the next chunk of item t+1
                if (nx.valid && n1 + i < nc) produce(nx);
            }
        }
        if (nx.valid) finish_item((t + 1) & (RING - 1));
        TRACE(5);

        // ------------------------------------------------ Z of the slice -> rank 0
        {
            float zw = warp_sum(z_l);
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
        if (rank == 0 && warp == 0) {
            h_r[t & 1] = t; h_b[t & 1] = pair ? b : -1; h_k[t & 1] = k; h_fatal[t & 1] = (seq_st & ST_FATAL) ? 1 : 0;
        }

        // ------------------------------------------------ first half of the draw: chunk totals -> cluster
        if (do_draw) {
            const float sqw = warp_sum(sq_l);
            int last = 0;
            if (lane == 0) {
                S.wsq[ds][warp] = sqw;
                __threadfence_block();
                last = atomicAdd(&S.dcnt[ds], 1) == NW - 1;
            }
            last = __shfl_sync(0xffffffffu, last, 0);
            if (last) {
                __threadfence_block();
                if (lane == 0) S.dcnt[ds] = 0;
                double tot = 0.0;
                for (int cidx = 0; cidx < nchunks; ++cidx) tot += S.csum[ds][cidx];   // same order as the resolver
                float sq = 0.f;
                for (int w = 0; w < NW; ++w) sq += S.wsq[ds][w];
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
            pd_valid = 1; pd_cancel = 0; pd_idx = ndraw; pd_b = b; pd_n = pair ? k : L; pd_ufin = c_ufin; pd_step = t;
            ndraw++;
        }
        TRACE(6);

        // ------------------------------------------------ sequence bookkeeping
        bool transition = false;
        if (pair) {
            if (stop_here) { seq_alive = 0; seq_n = k; }
            if (k == L - 1) {
                const bool fatal = (seq_st & ST_FATAL) != 0;
                if (rank == 0 && warp == 0) {
                    if (fatal) { if (h_b[0] == b) h_fatal[0] = 1; if (h_b[1] == b) h_fatal[1] = 1; }
                    const int n = fatal ? 0 : seq_n;
                    for (int q = lane; q <= K; q += 32)
                        if (fatal || q != n) a.o.out_tokens[(int64_t)b * (K + 1) + q] = q < n ? tokl : -1;   // q < n <= 32: q == lane
                    if (lane == 0) {
                        a.o.accept_len[b] = n;
                        a.stop[b] = fatal ? -1 : n;
                        if (a.o.row_status) a.o.row_status[b] = seq_st;
                    }
                    for (int q = lane; q < K; q += 32) {
                        if (fatal || q >= L) {
                            if (a.o.tv) a.o.tv[(int64_t)b * K + q] = 0.f;
                            if (a.o.p_draft) a.o.p_draft[(int64_t)b * K + q] = 0.f;
                            if (a.o.q_draft) a.o.q_draft[(int64_t)b * K + q] = 0.f;
                        }
                    }
                }
                // a draw of this sequence that is still on its way must not survive a fatal status
                if (fatal) {
                    if (pd_valid && pd_b == b) pd_cancel = 1;
                    if (hd_b[0] == b) hd_b[0] = -1;
                    if (hd_b[1] == b) hd_b[1] = -1;
                }
                if (!fatal && seq_alive) { if (j < 64) bm0 |= 1ull << j; else bm1 |= 1ull << (j - 64); }
            }
            if (!nx.valid) transition = true;      // the last pair item was just consumed
        } else {
            const bool fatal = (seq_st & ST_FATAL) != 0;
            if (rank == 0 && warp == 0 && (L == 0 || fatal)) {
                for (int q = lane; q <= K; q += 32)
                    if (fatal || q != 0) a.o.out_tokens[(int64_t)b * (K + 1) + q] = -1;
                for (int q = lane; q < K; q += 32) {
                    if (a.o.tv) a.o.tv[(int64_t)b * K + q] = 0.f;
                    if (a.o.p_draft) a.o.p_draft[(int64_t)b * K + q] = 0.f;
                    if (a.o.q_draft) a.o.q_draft[(int64_t)b * K + q] = 0.f;
                }
                if (lane == 0) {
                    a.o.accept_len[b] = 0;
                    if (L == 0) { a.stop[b] = fatal ? -1 : 0; if (a.o.row_status) a.o.row_status[b] = seq_st; }
                    else { a.stop[b] = -1; if (a.o.row_status) a.o.row_status[b] |= seq_st; }
                }
            }
        }

        // ------------------------------------------------ advance
        if (nx.valid) {
            if (phase == 1) pc_next(pc); else bc_pop(bc);
            cur_it = nx;
            if (nx_new_seq) { c_tau = tau_nx; tokl = tokl_nx; c_ufin = ufin_nx; }
        } else if (transition && phase == 1) {
            // The bonus mask is final.  Both stages are free: stage (pitem & 1) was never refilled and the
            // other one was read by every warp of the cluster before the normalisers of this item merged.
            phase = 2;
            bc.m0 = bm0; bc.m1 = bm1; ldb = bc;
            for (int s = 0; s < 2; ++s) {
                Item it = ld_item_pop();
                if (it.valid && warp == 0) { fence_proxy_async(); issue_item((pitem + s) & 1, it); }
            }
            cur_it = prod_item();
            if (cur_it.valid) {
                const int bn = seq_b(cur_it.j);
                c_tau = tau_of(R, bn); c_ufin = a.u_final[bn]; tokl = 0;
                begin_item(cur_it, c_tau);
                for (int i = 0; i < nc; ++i) produce(cur_it);
                finish_item((t + 1) & (RING - 1));
                bc_pop(bc);
            }
        } else {
            cur_it.valid = false;
        }
        TRACE(7);
    }

    // ---- epilogue
    if (pd_valid) resolve_draw();
    if (rank == 0 && warp == 0) {
        const int first = h_r[0] <= h_r[1] ? 0 : 1;
        flush_outputs(first);
        flush_outputs(first ^ 1);
    }
    tmem_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc512(S.tmem_base);
    cluster_arrive();
    cluster_wait();
    if (tid == 0 && S.wait_failed && a.o.row_status) {
        for (int jj = 0; jj < nseq; ++jj) atomicOr(&a.o.row_status[seq_b(jj)], ST_WAIT);
    }
}

// -----------------------------------------------------------------------------
namespace {

template <int DT>
constexpr size_t ring_smem() { return 4 * (size_t)NW * NCH * 32 * 16 + sizeof(RingShared) + 128; }

template <int DT>
cudaLaunchConfig_t ring_config(int clusters, cudaStream_t stream, cudaLaunchAttribute* attr) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(clusters * CS), 1, 1);
    cfg.blockDim = dim3(NT, 1, 1);
    cfg.dynamicSmemBytes = ring_smem<DT>();
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CS; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cfg;
}

template <int DT>
int ring_clusters() {
    static int cached[64] = {0};
    static bool known[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (dev >= 0 && dev < 64 && known[dev]) return cached[dev];
    int n = 0;
    if (cudaFuncSetAttribute(k_ring<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ring_smem<DT>()) == cudaSuccess) {
        cudaLaunchAttribute attr[1];
        cudaLaunchConfig_t cfg = ring_config<DT>(64, nullptr, attr);
        if (cudaOccupancyMaxActiveClusters(&n, k_ring<DT>, &cfg) != cudaSuccess) n = 0;
    }
    cudaGetLastError();
    if (dev >= 0 && dev < 64) { cached[dev] = n; known[dev] = true; }
    return n;
}

long long* g_ring_trace = nullptr;

}  // namespace

void ring_set_trace(long long* p) { g_ring_trace = p; }
int ring_max_clusters(int dt) { return dt == 0 ? ring_clusters<0>() : ring_clusters<1>(); }

// Shapes the ring kernel takes: every CTA slice (rounded up to 128 bytes) fits NW * NCH chunks
// of 32 vectors, and no slice is degenerate.
bool ring_supported(const RowArgs& a) {
    const int vs = (((a.nvec + CS - 1) / CS) + 7) & ~7;
    return vs <= MAXCH * 32 && a.nvec >= 4 * CS;
}

cudaError_t ring_verify(const RowArgs& a, const Plan& p, const int32_t* draft_tokens,
                        const float* u_accept, const float* u_final, VerifyOut o, char* ws,
                        cudaStream_t stream, bool* launched) {
    *launched = false;
    int ncl = ring_max_clusters(a.dt);
    if (ncl < 1) return cudaSuccess;
    RingArgs ra;
    ra.r = a; ra.draft_tokens = draft_tokens; ra.u_accept = u_accept; ra.u_final = u_final; ra.o = o;
    ra.stop = reinterpret_cast<int*>(ws + p.off_stop);
    ra.fb_count = reinterpret_cast<int*>(ws + p.off_fb);
    ra.fb_list = ra.fb_count + 16;
    ra.vs = (((a.nvec + CS - 1) / CS) + 7) & ~7;
    ra.trace = g_ring_trace;
    cudaError_t e = cudaMemsetAsync(ra.fb_count, 0, sizeof(int), stream);
    if (e != cudaSuccess) return e;
    for (int b0 = 0; b0 < a.B; b0 += ncl * MAXSEQ) {
        ra.b0 = b0;
        ra.nb = a.B - b0 < ncl * MAXSEQ ? a.B - b0 : ncl * MAXSEQ;
        const int clusters = ra.nb < ncl ? ra.nb : ncl;
        cudaLaunchAttribute attr[1];
        if (a.dt == 0) {
            cudaLaunchConfig_t cfg = ring_config<0>(clusters, stream, attr);
            e = cudaLaunchKernelEx(&cfg, k_ring<0>, ra);
        } else {
            cudaLaunchConfig_t cfg = ring_config<1>(clusters, stream, attr);
            e = cudaLaunchKernelEx(&cfg, k_ring<1>, ra);
        }
        if (e != cudaSuccess) return e;
    }
    *launched = true;
    return general_draw_list(a, p, u_final, o, ws, ra.fb_list, ra.fb_count, stream);
}

}  // namespace bebop
