// bebop_verify, row kernel: every logit is read from HBM once.
//
// A group of G CTAs (any SMs; all CTAs of the persistent grid are resident) takes one row pair (target row k and
// draft row k of a sequence, or the bonus row alone) at a time and keeps it in shared memory, CTA `rank` the
// vectors [rank * SV, rank * SV + SV) of both rows, in chunks of kRowChunkVecs vectors:
//   pass 1   as the chunks arrive (bulk copies issued by a producer thread): online softmax partials (E, S) of
//            both rows; the G partials meet in global memory (16-byte records that carry their own validity
//            mark) and every CTA merges them in rank order: the row normalisers.  p(x), q(x) of the drafted
//            token and the accept decision u * q(x) < p(x) follow at once (Eq. reject_sample);
//   pass 2   from shared memory: TV(p, q) = sum max(0, p - q); on a rejected position, whose residual may be the
//            one a token is drawn from, also the residual mass and the sum of squares of every chunk.  A chunk
//            is handed back to the producer as soon as the eight consumer warps are through with it.
// Row tasks do not depend on each other.  The publisher warp of the CTA that delivers a sequence's last partial
// finishes the sequence: accept length, tokens, TV, and the inverse-CDF draw from the chunk masses (Algorithm 3),
// kept when it clears the error bound, else listed for the fp64 re-draw kernels.
//
// Every wait is bounded; a wait that gives up sets the wait flag (status bit 32 of every row).
// No multicast, no cluster: each CTA copies from this GPU's own memory.
#define BEBOP_CTA_SYNC() asm volatile("bar.sync 1, 256;" ::: "memory")
#include "bebop_pipe.cuh"

namespace bebop {

extern cudaEvent_t g_ev_start, g_ev_stop;

namespace {

constexpr int RC = WT;                        // consumer threads (8 warps)
constexpr int RT = RC + 64;                   // + producer warp + publisher warp
constexpr int CV = kRowChunkVecs;             // vectors per chunk and row
constexpr int NCHM = kRowMaxChunks;
constexpr int NVC = CV / RC;                  // vectors per consumer thread, chunk and row
constexpr int ROW_CTAS = 3;                   // CTAs per SM the kernel is built for
constexpr double kFixTvR = 1099511627776.0;            // 2^40: fixed point of TV parts and sums of squares
constexpr double kFixMassR = 288230376151711744.0;     // 2^58: fixed point of chunk masses
constexpr uint32_t kBarSpinR = 1u << 17;

// a position's accept record, written by rank 0 of the group that had the row pair
struct __align__(16) ARec { float px, qx; int acc; int mark; };

struct RowKArgs {
    RowArgs r;
    const int32_t* draft_tokens;
    const float* u_accept;
    const float* u_final;
    VerifyOut o;
    int* fb_count;
    FbRec* fb_list;
    int* wait_failed;
    P1Part* grec;                  // [tasks][G][2]
    RowStat* rstat;                // [B][2K+1]
    ARec* arec;                    // [B][K]
    unsigned long long* tvacc;     // [B][K]   TV in 2^-40 units << 16 | parts added
    unsigned long long* cacc;      // [B][K+1][G*NCH][2]  chunk mass (2^-58) and sum of squares (2^-40), each << 4 | 1
    int* seqcnt;                   // [B]
    int G, NG, SV, NCH, ntasks;
};

struct RowShared {
    unsigned long long full[NCHM], empty[NCHM];   // mbarriers per chunk: data there / chunk free again
    unsigned long long pdone, pfree;              // consumer partials of a task there / taken by the publisher
    float p1s[2][WW]; int p1e[2][WW]; float p1m[2][WW];      // pass 1: per warp (S, E, max) of both rows
    RowScale P, Q;                                // pass 2: the rows' scales
    double sinv[2]; int se[2];                    // the rows' normalisers as merged (for the bonus chunk masses)
    int rejected, pub_masses;
    float tvw[WW];                                // pass 2 partials per warp
    double cm[NCHM][WW]; float csq[NCHM][WW];
    double f_tot[kRowMaxGroup * NCHM]; float f_sq[kRowMaxGroup * NCHM];   // finisher: chunk masses of a row
};

__device__ __forceinline__ uint32_t smem_u32r(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void rbar_init(unsigned long long* b, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32r(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void rbar_arrive(unsigned long long* b) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(smem_u32r(b)) : "memory");
}
__device__ __forceinline__ void rbar_arrive_expect(unsigned long long* b, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(smem_u32r(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool rbar_wait(unsigned long long* b, uint32_t parity) {
    const uint32_t addr = smem_u32r(b);
    for (uint32_t i = 0; i < kBarSpinR; ++i) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}
// contiguous copy global -> shared of this CTA; 16-byte aligned on both sides, size a multiple of 16
__device__ __forceinline__ void rbulk_load(void* dst, const void* src, uint32_t bytes, unsigned long long* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(smem_u32r(dst)), "l"(src), "r"(bytes), "r"(smem_u32r(bar)) : "memory");
}
__device__ __forceinline__ uint4 rlds16(const unsigned char* p) { return *reinterpret_cast<const uint4*>(p); }
__device__ __forceinline__ void red_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" :: "l"(p), "l"(v) : "memory");
}

// task t of the launch: sequence, position, and what kind of task it is for that sequence
struct RowTask { int b, k, L; bool skip, pair; };
__device__ __forceinline__ RowTask row_task(const RowKArgs& a, int t) {
    RowTask x;
    x.b = t / (a.r.K + 1); x.k = t - x.b * (a.r.K + 1);
    x.L = len_of(a.r, x.b);
    x.skip = x.k > x.L;
    x.pair = x.k < x.L;
    return x;
}
// vectors of chunk c of this CTA's slice of a row
__device__ __forceinline__ int chunk_vecs(const RowKArgs& a, int rank, int c) {
    const int nvs = max(min(a.SV, a.r.nvec - rank * a.SV), 0);
    return max(min(CV, nvs - c * CV), 0);
}

// ------------------------------------------------------------------ producer
// One thread: for every task of the group, chunk by chunk as the consumers hand the chunks back, the bulk copies
// of this CTA's slice of the target row (first half of the buffer) and of the draft row (second half).
__device__ __forceinline__ void row_producer(const RowKArgs& a, RowShared& S, unsigned char* data, int group, int rank) {
    const RowArgs& R = a.r;
    const size_t half = (size_t)a.SV * 16;
    uint32_t use = 0;                                   // tasks staged so far: the chunks' barrier phase
    for (int t = group; t < a.ntasks; t += a.NG) {
        const RowTask x = row_task(a, t);
        if (x.skip) continue;
        const char* prow = row_ptr(R, x.b, x.k);
        const char* qrow = x.pair ? row_ptr(R, x.b, R.K + 1 + x.k) : nullptr;
        for (int c = 0; c < a.NCH; ++c) {
            if (!rbar_wait(&S.empty[c], (use & 1u) ^ 1u)) atomicExch(a.wait_failed, 1);
            const uint32_t bytes = (uint32_t)chunk_vecs(a, rank, c) * 16u;
            if (bytes) {
                const int64_t off = ((int64_t)rank * a.SV + (int64_t)c * CV) * 16;
                rbar_arrive_expect(&S.full[c], qrow ? 2u * bytes : bytes);
                rbulk_load(data + (size_t)c * CV * 16, prow + off, bytes, &S.full[c]);
                if (qrow) rbulk_load(data + half + (size_t)c * CV * 16, qrow + off, bytes, &S.full[c]);
            } else {
                rbar_arrive(&S.full[c]);
            }
        }
        ++use;
    }
}

// ------------------------------------------------------------------ consumers, pass 1
// A thread's running softmax partial of one row: S = sum 2^(x * c - E) around the integer exponent E.
struct Run1 { int E; float Ef, s; bool bad; };
__device__ __forceinline__ Run1 run1_init() { Run1 r; r.E = E_EMPTY; r.Ef = 0.f; r.s = 0.f; r.bad = false; return r; }

// takes the thread's vectors of one chunk into the running partial; returns the chunk's own sum (around the
// exponent the partial has afterwards) and, if asked, its sum of squares
template <int DT, bool SQ>
__device__ __forceinline__ float p1_chunk(Run1& st, const uint4* raw, const TempScale& ts, float* sq) {
    constexpr int VEC = Elem<DT>::VEC;
    float m = vec_max<DT>(raw[0]);
#pragma unroll
    for (int u = 1; u < NVC; ++u) m = max_nan(m, vec_max<DT>(raw[u]));
    if (m != m || m == INFINITY) { st.bad = true; return 0.f; }
    if (m == -INFINITY) return 0.f;
    float Ef;
    const int E = ref_exponent(m, ts, &Ef);
    if (E > st.E) {          // exact power-of-two rescaling of what was summed around the smaller exponent
        st.s = st.E > E_EMPTY ? st.s * pow2f(max(st.E - E, -126)) : 0.f;
        st.E = E; st.Ef = Ef;
    }
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f, q0 = 0.f, q1 = 0.f;
#pragma unroll
    for (int u = 0; u < NVC; ++u) {
        float f[VEC];
        unpack<DT>(raw[u], f);
#pragma unroll
        for (int i = 0; i < VEC; i += 4) {
            const float e0 = exp2_scaled(f[i], ts, st.Ef), e1 = exp2_scaled(f[i + 1], ts, st.Ef);
            const float e2 = exp2_scaled(f[i + 2], ts, st.Ef), e3 = exp2_scaled(f[i + 3], ts, st.Ef);
            s0 += e0; s1 += e1; s2 += e2; s3 += e3;
            if (SQ) { q0 = fmaf(e0, e0, q0); q1 = fmaf(e1, e1, q1); q0 = fmaf(e2, e2, q0); q1 = fmaf(e3, e3, q1); }
        }
    }
    const float cs = (s0 + s1) + (s2 + s3);
    st.s += cs;
    if (SQ) *sq = q0 + q1;
    return cs;
}

// thread -> warp: exact power-of-two rescaling, sums in a fixed order; lane 0 leaves the warp's partial
__device__ __forceinline__ void p1_warp(RowShared& S, int row, const Run1& st) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int Ew = redux_max(st.E);
    float sw = st.E > E_EMPTY ? st.s * pow2f(max(st.E - Ew, -126)) : 0.f;
    sw = warp_sum(sw);
    const unsigned anybad = __ballot_sync(0xffffffffu, st.bad);
    if (lane == 0) { S.p1s[row][warp] = sw; S.p1e[row][warp] = Ew; S.p1m[row][warp] = anybad ? __int_as_float(0x7fc00000) : 0.f; }
}

// Warp 0 of the consumers: this CTA's partial of a row (the eight warp partials, warp order) goes to the group's
// records; the G partials are merged in rank order once they are all there.  Every CTA of the group gets the
// same bits.
__device__ __forceinline__ RowStat row_gather(const RowKArgs& a, RowShared& S, int t, int rank, int row) {
    const int lane = threadIdx.x & 31;
    const int w = lane & (WW - 1);
    const int ii = S.p1e[row][w];
    const float f0 = S.p1s[row][w], mm = S.p1m[row][w];
    int Ec = ii;
#pragma unroll
    for (int o = 4; o > 0; o >>= 1) Ec = max(Ec, __shfl_xor_sync(0xffffffffu, Ec, o));
    const double mine = ii > E_EMPTY ? (double)(f0 * pow2f(max(ii - Ec, -126))) : 0.0;
    double sum = 0.0; float mc = 0.f;
#pragma unroll
    for (int k = 0; k < WW; ++k) { sum += __shfl_sync(0xffffffffu, mine, k); mc = max_nan(mc, __shfl_sync(0xffffffffu, mm, k)); }
    P1Part* recs = a.grec + ((int64_t)t * a.G) * 2;
    if (lane == 0) {
        // the record's exponent is stored as 2e + 1: zero means "not there yet"
        P1Part p; p.s = (mc != mc) ? 0.0 : sum; p.e = 2 * Ec + 1; p.m = mc;
        st16(recs + rank * 2 + row, p);
    }
    P1Part rec; rec.s = 0.0; rec.e = 2 * E_EMPTY + 1; rec.m = 0.f;
    if (lane < a.G) {
        rec = ld_cg(recs + lane * 2 + row);
        for (uint32_t i = 0; rec.e == 0 && i < kSpin; ++i) { __nanosleep(32); rec = ld_cg(recs + lane * 2 + row); }
        if (rec.e == 0) { atomicExch(a.wait_failed, 1); rec.e = 2 * E_EMPTY + 1; }
    }
    const int e_l = (rec.e - 1) >> 1;
    const int Em = redux_max(e_l);
    double s_l = e_l > E_EMPTY ? rec.s * pow2d(max(e_l - Em, -1000)) : 0.0;
    int f_l = rec.m != rec.m;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { s_l += shfl_xor_d(s_l, o); f_l |= __shfl_xor_sync(0xffffffffu, f_l, o); }
    int st = 0;
    if (f_l || !(s_l == s_l)) st = ST_NONFINITE; else if (Em == E_EMPTY) st = ST_EMPTY;
    RowStat rs; rs.inv_s = (!st && s_l > 0.0) ? 1.0 / s_l : 0.0; rs.e = Em; rs.st = st | kRowValid;
    return rs;
}

// ------------------------------------------------------------------ consumers
template <int DT>
__device__ __forceinline__ void row_consumers(const RowKArgs& a, RowShared& S, const unsigned char* data, int group, int rank) {
    constexpr int VEC = Elem<DT>::VEC;
    const RowArgs& R = a.r;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = R.K;
    const unsigned char* qdata = data + (size_t)a.SV * 16;
    uint32_t use = 0;
    for (int t = group; t < a.ntasks; t += a.NG) {
        const RowTask x = row_task(a, t);
        if (x.skip) continue;
        const int b = x.b, k = x.k;
        const float tau = tau_of(R, b);
        const TempScale ts = temp_scale(tau);
        // thread 0: the drafted token's logits and its uniform, asked for now, used after the merge
        int tk = 0; bool tok_ok = false; float zpx = 0.f, zqx = 0.f, u = 0.f;
        if (x.pair && tid == 0) {
            tk = a.draft_tokens[(int64_t)b * K + k];
            tok_ok = tk >= 0 && tk < R.V;
            if (tok_ok) { zpx = load_one<DT>(row_ptr(R, b, k), tk); zqx = load_one<DT>(row_ptr(R, b, K + 1 + k), tk); }
            u = a.u_accept[(int64_t)b * K + k];
        }
        // ---- pass 1, chunk by chunk as the data arrives
        Run1 sp = run1_init(), sq = run1_init();
        float bsc[NCHM], bsq[NCHM]; int bec[NCHM];        // bonus row: the chunks' own sums
#pragma unroll
        for (int c = 0; c < NCHM; ++c) { bsc[c] = 0.f; bsq[c] = 0.f; bec[c] = E_EMPTY; }
#pragma unroll
        for (int c = 0; c < NCHM; ++c) {
            if (c < a.NCH) {
                if (!rbar_wait(&S.full[c], use & 1u)) { if (tid == 0) atomicExch(a.wait_failed, 1); }
                const int nvc = chunk_vecs(a, rank, c);
                const int gv0 = rank * a.SV + c * CV;                 // first vector of the chunk in the row
                uint4 rp[NVC], rq[NVC];
#pragma unroll
                for (int j = 0; j < NVC; ++j) {
                    const int v = tid + j * RC;
                    rp[j] = neg_inf_vec<DT>(); rq[j] = neg_inf_vec<DT>();
                    if (v < nvc) {
                        rp[j] = rlds16(data + (size_t)(c * CV + v) * 16);
                        if (x.pair) rq[j] = rlds16(qdata + (size_t)(c * CV + v) * 16);
                    }
                }
                if ((gv0 + nvc) * VEC > R.V) {                        // the row's last vector is in this chunk and is partial
#pragma unroll
                    for (int j = 0; j < NVC; ++j) {
                        const int gbase = (gv0 + tid + j * RC) * VEC;
                        if (tid + j * RC < nvc && gbase + VEC > R.V) { mask_tail<DT>(rp[j], R.V - gbase); mask_tail<DT>(rq[j], R.V - gbase); }
                    }
                }
                if (x.pair) {
                    p1_chunk<DT, false>(sp, rp, ts, nullptr);
                    p1_chunk<DT, false>(sq, rq, ts, nullptr);
                } else {
                    bsc[c] = p1_chunk<DT, true>(sp, rp, ts, &bsq[c]);
                    bec[c] = sp.E;
                    __syncwarp();
                    if (lane == 0) rbar_arrive(&S.empty[c]);          // a bonus row has no second pass
                }
            }
        }
        p1_warp(S, 0, sp);
        if (x.pair) p1_warp(S, 1, sq);
        BEBOP_CTA_SYNC();
        // ---- the group's partials -> normalisers, accept decision
        if (warp == 0) {
            const RowStat rsP = row_gather(a, S, t, rank, 0);
            RowStat rsQ; rsQ.inv_s = 0.0; rsQ.e = 0; rsQ.st = kRowValid;
            if (x.pair) rsQ = row_gather(a, S, t, rank, 1);
            if (lane == 0) {
                S.P = row_scale(rsP); S.Q = x.pair ? row_scale(rsQ) : no_row();
                S.sinv[0] = rsP.inv_s; S.se[0] = rsP.e;
                double px = 0.0, qx = 0.0; bool acc = false;
                if (x.pair && tok_ok && tau_ok(tau) && !(rsP.st & 0xff) && !(rsQ.st & 0xff)) {
                    const double cd = (double)ts.hi;
                    px = exp2((double)zpx * cd - (double)rsP.e) * rsP.inv_s;
                    qx = exp2((double)zqx * cd - (double)rsQ.e) * rsQ.inv_s;
                    acc = (double)u * qx < px;
                }
                S.rejected = !acc;
                if (rank == 0) {
                    st16(a.rstat + (int64_t)b * (2 * K + 1) + k, rsP);
                    if (x.pair) {
                        st16(a.rstat + (int64_t)b * (2 * K + 1) + K + 1 + k, rsQ);
                        ARec ar; ar.px = (float)px; ar.qx = (float)qx; ar.acc = acc ? 1 : 0; ar.mark = 1;
                        st16(a.arec + (int64_t)b * K + k, ar);
                    }
                }
            }
        }
        BEBOP_CTA_SYNC();
        // ---- pass 2 (row pairs) or the chunk masses of a bonus row
        float z0 = 0.f, z1 = 0.f;
        double cmass[NCHM]; float csq[NCHM];
#pragma unroll
        for (int c = 0; c < NCHM; ++c) { cmass[c] = 0.0; csq[c] = 0.f; }
        const bool rejected = S.rejected != 0;
        if (x.pair) {
            TempScale cc; cc.hi = ts.hi;
            const RowScale SP = S.P, SQ = S.Q;
#pragma unroll
            for (int c = 0; c < NCHM; ++c) {
                if (c < a.NCH) {
                    const int nvc = chunk_vecs(a, rank, c);
                    const int gv0 = rank * a.SV + c * CV;
                    uint4 rp[NVC], rq[NVC];
#pragma unroll
                    for (int j = 0; j < NVC; ++j) {
                        const int v = tid + j * RC;
                        rp[j] = neg_inf_vec<DT>(); rq[j] = neg_inf_vec<DT>();
                        if (v < nvc) { rp[j] = rlds16(data + (size_t)(c * CV + v) * 16); rq[j] = rlds16(qdata + (size_t)(c * CV + v) * 16); }
                    }
                    if ((gv0 + nvc) * VEC > R.V) {
#pragma unroll
                        for (int j = 0; j < NVC; ++j) {
                            const int gbase = (gv0 + tid + j * RC) * VEC;
                            if (tid + j * RC < nvc && gbase + VEC > R.V) { mask_tail<DT>(rp[j], R.V - gbase); mask_tail<DT>(rq[j], R.V - gbase); }
                        }
                    }
                    if (!rejected) {
#pragma unroll
                        for (int j = 0; j < NVC; ++j) {
                            float r[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) r[i] = 0.f;
                            residual_vec<DT, false>(rp[j], rq[j], cc, SP, SQ, r, nullptr);
                            const float vs = ((r[0] + r[1]) + (r[2] + r[3])) + ((r[4] + r[5]) + (r[6] + r[7]));
                            if (j & 1) z1 += vs; else z0 += vs;
                        }
                    } else {
                        // a rejected position: its residual may be the one a token is drawn from
                        float sqs = 0.f; double zd = 0.0;
#pragma unroll
                        for (int j = 0; j < NVC; ++j) {
                            float r[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) r[i] = 0.f;
                            residual_vec<DT, true>(rp[j], rq[j], cc, SP, SQ, r, &sqs);
                            const float vs = ((r[0] + r[1]) + (r[2] + r[3])) + ((r[4] + r[5]) + (r[6] + r[7]));
                            z0 += vs; zd += (double)vs;
                        }
                        cmass[c] = zd; csq[c] = sqs;
                    }
                    __syncwarp();
                    if (lane == 0) rbar_arrive(&S.empty[c]);
                }
            }
        } else {
            // bonus row: the chunks' masses are their sums of exponentials over the row's sum
            const int Er = S.se[0];
            const double inv = S.sinv[0];
#pragma unroll
            for (int c = 0; c < NCHM; ++c) {
                if (c < a.NCH && bec[c] > E_EMPTY) {
                    const float sc = pow2f(max(bec[c] - Er, -126));
                    cmass[c] = (double)(bsc[c] * sc) * inv;
                    csq[c] = (float)((double)(bsq[c] * sc * sc) * inv * inv);
                }
            }
        }
        const float z = warp_sum(z0 + z1);
        const bool masses = !x.pair || rejected;
        if (masses) {
#pragma unroll
            for (int c = 0; c < NCHM; ++c) if (c < a.NCH) { cmass[c] = warp_sum(cmass[c]); csq[c] = warp_sum(csq[c]); }
        }
        // the warp's partials, once the publisher has taken the previous task's
        if (!rbar_wait(&S.pfree, (use & 1u) ^ 1u)) { if (tid == 0) atomicExch(a.wait_failed, 1); }
        if (lane == 0) {
            S.tvw[warp] = z;
#pragma unroll
            for (int c = 0; c < NCHM; ++c) { S.cm[c][warp] = cmass[c]; S.csq[c][warp] = csq[c]; }
            if (warp == 0) S.pub_masses = masses ? 1 : 0;
        }
        __syncwarp();
        if (lane == 0) rbar_arrive(&S.pdone);
        ++use;
    }
}

// ------------------------------------------------------------------ finishing a sequence
// residual mass of vector v of a row pair (or of the bonus row), same arithmetic as pass 2 on a rejected position
template <int DT>
__device__ __forceinline__ void vec_resid(const RowArgs& R, const char* prow, const char* qrow, int v, const TempScale& c,
                                          const RowScale& SP, const RowScale& SQ, float* r) {
    constexpr int VEC = Elem<DT>::VEC;
    uint4 rp = ldg16(prow + (size_t)v * 16), rq = neg_inf_vec<DT>();
    if (qrow) rq = ldg16(qrow + (size_t)v * 16);
    const int gbase = v * VEC;
    if (gbase + VEC > R.V) { mask_tail<DT>(rp, R.V - gbase); mask_tail<DT>(rq, R.V - gbase); }
#pragma unroll
    for (int i = 0; i < 8; ++i) r[i] = 0.f;
    residual_vec<DT, true>(rp, rq, c, SP, SQ, r, nullptr);
}

// One warp, once every row task of the sequence has delivered its partials: the accept scan over the positions'
// records (first rejected position, status), the outputs, TV, and the draw: the chunk that owns u * Z from the
// chunk masses, then the token inside it from the logits (a few KB, read again).
template <int DT>
__device__ __noinline__ void finish_warp(const RowKArgs& a, RowShared& S, int b) {
    constexpr int VEC = Elem<DT>::VEC;
    const RowArgs& R = a.r;
    const int lane = threadIdx.x & 31;
    const int K = R.K, V = R.V, L = len_of(R, b), NR = 2 * K + 1;
    const float tau = tau_of(R, b);
    const bool ok = tau_ok(tau);
    const TempScale ts = temp_scale(tau);
    const bool active = lane < L;
    const int tk = active ? a.draft_tokens[(int64_t)b * K + lane] : 0;
    auto row = [&](int r) {                                            // a row's record (waits, bounded, for its mark)
        RowStat x = ld_cg(a.rstat + (int64_t)b * NR + r);
        for (uint32_t i = 0; x.st == 0 && i < kSpin; ++i) { __nanosleep(64); x = ld_cg(a.rstat + (int64_t)b * NR + r); }
        if (x.st == 0) atomicExch(a.wait_failed, 1);
        x.st &= 0xff;
        return x;
    };
    RowStat sp, sq;
    sp.inv_s = 0.0; sp.e = E_EMPTY; sp.st = 0; sq = sp;
    ARec ar; ar.px = 0.f; ar.qx = 0.f; ar.acc = 0; ar.mark = 1;
    if (active) {
        sp = row(lane); sq = row(K + 1 + lane);
        ar = ld_cg(a.arec + (int64_t)b * K + lane);
        for (uint32_t i = 0; ar.mark == 0 && i < kSpin; ++i) { __nanosleep(64); ar = ld_cg(a.arec + (int64_t)b * K + lane); }
        if (ar.mark == 0) atomicExch(a.wait_failed, 1);
    }
    const RowStat sb = row(L);                                         // bonus row
    int seq_st = ok ? 0 : ST_BAD_TEMP;
    const bool tok_ok = tk >= 0 && tk < V;
    if (!seq_st && __ballot_sync(0xffffffffu, active && !tok_ok)) seq_st = ST_BAD_TOKEN;
    // the first bad row pair decides the status; rows after it do not count
    const int rs = active ? (sp.st | sq.st) : 0;
    const unsigned badrows = __ballot_sync(0xffffffffu, rs != 0);
    const int first_bad = badrows ? __ffs(badrows) - 1 : 32;
    const int rs_first = __shfl_sync(0xffffffffu, rs, first_bad & 31);
    if (!seq_st && badrows) seq_st = rs_first;
    const bool acc = active && !(seq_st & ST_FATAL) && lane < first_bad && ar.acc != 0;
    const unsigned rej = __ballot_sync(0xffffffffu, active && !acc);
    const int n = rej ? __ffs(rej) - 1 : L;
    if (!(seq_st & ST_FATAL) && n == L && sb.st) seq_st |= sb.st;   // bonus row, counted only now
    const bool fatal = (seq_st & ST_FATAL) != 0;
    const int nn = fatal ? 0 : n;
    // outputs: lane q writes position q (position nn is filled by the draw)
    for (int q = lane; q <= K; q += 32)
        if (fatal || q != nn) a.o.out_tokens[(int64_t)b * (K + 1) + q] = q < nn ? tk : -1;   // q < nn <= 32: q == lane
    if (lane < K) {
        const bool zero = fatal || lane >= L;
        if (a.o.p_draft) a.o.p_draft[(int64_t)b * K + lane] = zero ? 0.f : ar.px;
        if (a.o.q_draft) a.o.q_draft[(int64_t)b * K + lane] = zero ? 0.f : ar.qx;
        if (a.o.tv) {
            float z = 0.f;
            if (!zero) {
                // the position's TV parts were added in fixed point, with a count of one each in the low 16 bits
                unsigned long long w = 0;
                for (uint32_t i = 0; i < kSpin; ++i) {
                    w = __ldcg(a.tvacc + (int64_t)b * K + lane);
                    if ((int)(w & 0xffffull) >= a.G) break;
                    __nanosleep(64);
                }
                if ((int)(w & 0xffffull) < a.G) atomicExch(a.wait_failed, 1);
                z = fminf(fmaxf((float)((double)(w >> 16) * 9.094947017729282e-13), 0.f), 1.f);      // 2^-40
            }
            a.o.tv[(int64_t)b * K + lane] = z;
        }
    }
    if (lane == 0) {
        a.o.accept_len[b] = nn;
        if (a.o.row_status) a.o.row_status[b] = seq_st;
    }
    if (fatal) return;
    // ---- the draw, from position nn (the residual of a rejected position, or the bonus row)
    const int k = nn;
    const bool pair = k < L;
    const RowStat rsP = row(k);
    RowStat rsQ; rsQ.inv_s = 0.0; rsQ.e = 0; rsQ.st = 0;
    if (pair) rsQ = row(K + 1 + k);
    const int nchunks = a.G * a.NCH;
    const unsigned long long* words = a.cacc + (((int64_t)b * (K + 1) + k) * nchunks) * 2;
    for (int i = lane; i < nchunks; i += 32) {
        unsigned long long w0 = 0, w1 = 0;
        for (uint32_t j = 0; j < kSpin; ++j) {
            w0 = __ldcg(words + 2 * i); w1 = __ldcg(words + 2 * i + 1);
            if ((w0 & 15ull) != 0 && (w1 & 15ull) != 0) break;
            __nanosleep(64);
        }
        if ((w0 & 15ull) == 0 || (w1 & 15ull) == 0) atomicExch(a.wait_failed, 1);
        S.f_tot[i] = (double)(w0 >> 4) * 3.469446951953614e-18;            // 2^-58
        S.f_sq[i] = (float)((double)(w1 >> 4) * 9.094947017729282e-13);    // 2^-40
    }
    __syncwarp();
    double Tt = 0.0, base = 0.0, bound = 0.0; int owner = -1;
    if (lane == 0) {
        double Z = 0.0, sumsq = 0.0;
        for (int s = 0; s < nchunks; ++s) { Z += S.f_tot[s]; sumsq += (double)S.f_sq[s]; }
        Tt = (double)a.u_final[b] * Z;
        double run = 0.0;
        for (int s = 0; s < nchunks; ++s) {
            const double nx = run + S.f_tot[s];
            if (owner < 0 && Tt > run && Tt <= nx) { owner = s; base = run; }
            run = nx;
        }
        if (!(Tt > 0.0)) owner = -1;
        bound = draw_bound(sumsq);
    }
    __syncwarp();
    owner = __shfl_sync(0xffffffffu, owner, 0);
    Tt = __shfl_sync(0xffffffffu, Tt, 0); base = __shfl_sync(0xffffffffu, base, 0); bound = __shfl_sync(0xffffffffu, bound, 0);
    int found_y = -1, found_cert = 0;
    if (owner >= 0) {
        const int rank_o = owner / a.NCH, c_o = owner - rank_o * a.NCH;
        const int v_first = rank_o * a.SV + c_o * CV;                    // the chunk's first vector in the row
        const int nvc = chunk_vecs(a, rank_o, c_o);
        const char* prow = row_ptr(R, b, k);
        const char* qrow = pair ? row_ptr(R, b, K + 1 + k) : nullptr;
        const RowScale SP = row_scale(rsP), SQ = pair ? row_scale(rsQ) : no_row();
        constexpr int VPL = CV / 32;                                     // consecutive vectors per lane
        const int vb = min(lane * VPL, nvc), ve = min(vb + VPL, nvc);
        double mine = 0.0;
        for (int v = vb; v < ve; ++v) {
            float r[8];
            vec_resid<DT>(R, prow, qrow, v_first + v, ts, SP, SQ, r);
            mine += (double)(((r[0] + r[1]) + (r[2] + r[3])) + ((r[4] + r[5]) + (r[6] + r[7])));
        }
        double incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const double t2 = shfl_up_d(incl, o); if (lane >= o) incl += t2; }
        const double lower = base + (incl - mine), upper = base + incl;
        if (lower < Tt && Tt <= upper) {
            double C = lower;
            for (int v = vb; v < ve && found_y < 0; ++v) {
                float r[8];
                vec_resid<DT>(R, prow, qrow, v_first + v, ts, SP, SQ, r);
                const double nxt = C + (double)(((r[0] + r[1]) + (r[2] + r[3])) + ((r[4] + r[5]) + (r[6] + r[7])));
                if (Tt <= nxt) {
                    double Cw = C;
#pragma unroll
                    for (int i = 0; i < VEC; ++i) {
                        if (found_y < 0) {
                            const double r1 = (double)r[i];
                            const double Cn = Cw + r1;
                            if (r1 > 0.0 && Cn >= Tt) { found_y = (v_first + v) * VEC + i; found_cert = (Tt - Cw > bound) && (Cn - Tt >= bound); }
                            Cw = Cn;
                        }
                    }
                    break;
                }
                C = nxt;
            }
        }
    }
    // at most one lane should have found the token
    const unsigned own = __ballot_sync(0xffffffffu, found_y >= 0);
    const int src = own ? __ffs(own) - 1 : 0;
    const int y = __shfl_sync(0xffffffffu, found_y, src), cert = __shfl_sync(0xffffffffu, found_cert, src);
    if (lane == 0) {
        if (__popc(own) == 1 && cert && y >= 0) a.o.out_tokens[(int64_t)b * (K + 1) + k] = y;
        else {
            FbRec rec;
            rec.b = b; rec.kp = 2 * k + (pair ? 1 : 0); rec.ep = rsP.e; rec.eq = pair ? rsQ.e : 0;
            st16(a.fb_list + atomicAdd(a.fb_count, 1), rec);
        }
    }
    __syncwarp();
}

// ------------------------------------------------------------------ publisher
// One warp.  For every task: wait for the eight warp partials, take them, hand the slots back, then publish:
// the position's TV part and, where a token may be drawn, the chunk masses, in fixed point with a count in the
// low bits (one relaxed add publishes value and count, and integer sums do not depend on the order of arrival);
// then the sequence's counter, whose last increment finishes the sequence.
template <int DT>
__device__ __forceinline__ void row_publisher(const RowKArgs& a, RowShared& S, int group, int rank) {
    const RowArgs& R = a.r;
    const int lane = threadIdx.x & 31;
    const int K = R.K;
    uint32_t use = 0;
    for (int t = group; t < a.ntasks; t += a.NG) {
        const RowTask x = row_task(a, t);
        if (x.skip) continue;
        if (!rbar_wait(&S.pdone, use & 1u)) { if (lane == 0) atomicExch(a.wait_failed, 1); return; }
        const float tv = S.tvw[lane & (WW - 1)];
        const int masses = S.pub_masses;
        double tot = 0.0; float sq = 0.f;
        if (lane < a.NCH) {
#pragma unroll
            for (int w = 0; w < WW; ++w) { tot += S.cm[lane][w]; sq += S.csq[lane][w]; }
        }
        __syncwarp();
        if (lane == 0) rbar_arrive(&S.pfree);
        float zz = 0.f;
#pragma unroll
        for (int w = 0; w < WW; ++w) zz += __shfl_sync(0xffffffffu, tv, w);
        if (x.pair && lane == 0)
            red_u64(a.tvacc + (int64_t)x.b * K + x.k, ((unsigned long long)__double2ll_rn((double)zz * kFixTvR) << 16) | 1ull);
        if (masses && lane < a.NCH) {
            unsigned long long* wd = a.cacc + ((((int64_t)x.b * (K + 1) + x.k) * a.G + rank) * a.NCH + lane) * 2;
            red_u64(wd, ((unsigned long long)__double2ll_rn(tot * kFixMassR) << 4) | 1ull);
            red_u64(wd + 1, ((unsigned long long)__double2ll_rn((double)sq * kFixTvR) << 4) | 1ull);
        }
        __syncwarp();
        int fin = 0;
        if (lane == 0) fin = atomicAdd(a.seqcnt + x.b, 1) == a.G * (x.L + 1) - 1;
        if (__shfl_sync(0xffffffffu, fin, 0)) finish_warp<DT>(a, S, x.b);
        ++use;
    }
}

}  // namespace

template <int DT>
__global__ void __launch_bounds__(RT, ROW_CTAS) k_row(const __grid_constant__ RowKArgs a) {
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* data = smem;
    RowShared& S = *reinterpret_cast<RowShared*>(smem + (size_t)a.SV * 32);
    const int tid = threadIdx.x;
    const int group = blockIdx.x / a.G, rank = blockIdx.x - group * a.G;
    // the re-draw kernel behind this one may be scheduled as CTAs of this one leave; it waits for this grid's
    // completion before it reads anything (programmatic dependent launch)
    if (tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) {
        for (int c = 0; c < NCHM; ++c) { rbar_init(&S.full[c], 1); rbar_init(&S.empty[c], WW); }
        rbar_init(&S.pdone, WW); rbar_init(&S.pfree, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (tid >= RC) {
        if (tid == RC) row_producer(a, S, data, group, rank);
        else if (tid >= RC + 32) row_publisher<DT>(a, S, group, rank);
        return;
    }
    row_consumers<DT>(a, S, data, group, rank);
}

// -----------------------------------------------------------------------------
namespace {

size_t row_smem(const RowPlan& rp) { return (size_t)rp.SV * 32 + sizeof(RowShared); }

// CTAs of the kernel that are resident at once on this device with `smem` bytes each (0: the kernel cannot run)
template <int DT>
int row_resident(size_t smem) {
    if (cudaFuncSetAttribute(k_row<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    int dev = 0, per_sm = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_row<DT>, RT, smem) != cudaSuccess) per_sm = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) sms = 0;
    return per_sm * sms;
}

}  // namespace

bool row_supported(const RowArgs& a) {
    const RowPlan rp = make_row_plan(a.B, a.K, a.nvec);
    return rp.G >= 1 && rp.NCH <= kRowMaxChunks && a.K <= 32 && row_smem(rp) <= 100 * 1024;
}

cudaError_t row_verify(const RowArgs& a, const Plan& p, const int32_t* draft_tokens,
                       const float* u_accept, const float* u_final, VerifyOut o, char* ws,
                       cudaStream_t stream, bool* launched) {
    *launched = false;
    const RowPlan rp = make_row_plan(a.B, a.K, a.nvec);
    const size_t smem = row_smem(rp);
    const int resident = a.dt == 0 ? row_resident<0>(smem) : row_resident<1>(smem);
    const long long ntasks = (long long)a.B * (a.K + 1);
    if (resident < rp.G || ntasks > 0x7fff0000LL) return cudaSuccess;
    const WavePlan wp = make_wave_plan(a.B, a.K, a.nvec, a.dt);
    char* w = ws + p.off_wave;
    char* rw = ws + p.off_row;
    RowKArgs ka;
    ka.r = a; ka.draft_tokens = draft_tokens; ka.u_accept = u_accept; ka.u_final = u_final; ka.o = o;
    ka.fb_count = reinterpret_cast<int*>(w + kFbCountOffset);
    ka.fb_list = reinterpret_cast<FbRec*>(ws + p.off_fb);
    ka.wait_failed = reinterpret_cast<int*>(w) + 1;
    ka.rstat = reinterpret_cast<RowStat*>(w + wp.off_rstat);
    ka.tvacc = reinterpret_cast<unsigned long long*>(w + wp.off_tvacc);
    ka.grec = reinterpret_cast<P1Part*>(rw + rp.off_grec);
    ka.arec = reinterpret_cast<ARec*>(rw + rp.off_arec);
    ka.cacc = reinterpret_cast<unsigned long long*>(rw + rp.off_cacc);
    ka.seqcnt = reinterpret_cast<int*>(rw + rp.off_seqcnt);
    ka.G = rp.G; ka.SV = rp.SV; ka.NCH = rp.NCH; ka.ntasks = (int)ntasks;
    int NG = resident / rp.G;
    if ((long long)NG > ntasks) NG = (int)ntasks;
    ka.NG = NG;
    cudaError_t e = cudaMemsetAsync(w, 0, wp.zero_bytes, stream);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(rw, 0, rp.total, stream);
    if (e != cudaSuccess) return e;
    if (g_ev_start) cudaEventRecord(g_ev_start, stream);
    if (a.dt == 0) k_row<0><<<NG * rp.G, RT, smem, stream>>>(ka);
    else k_row<1><<<NG * rp.G, RT, smem, stream>>>(ka);
    e = cudaGetLastError();
    if (g_ev_stop) cudaEventRecord(g_ev_stop, stream);
    if (e != cudaSuccess) return e;
    *launched = true;
    return redraw_launch(a, u_final, o, ka.fb_count, ka.fb_list, ka.wait_failed, w, wp, stream);
}

}  // namespace bebop
