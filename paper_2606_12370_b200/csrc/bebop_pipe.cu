// Pipelined kernel: the hot path of bebop_verify as one persistent, ticket-scheduled kernel with the
// data movement and the bookkeeping taken off the compute warps.
//
// The work is a queue of tickets in three blocks, sequences ascending in each: P1 (softmax partial of one
// slice of one row) for every row; then P2 (TV part and residual mass of one half slice of a row pair) for the
// row each sequence's token is drawn from; then P2 for the other positions, which only TV needs.  Phase A --
// merging a row's partials, and the accept scan of a sequence -- has no tickets: it runs in the publisher warp
// that completes the row / the sequence, long before the second sweep asks for its results.  Nor has the draw:
// the publisher warp that completes a sequence's draw row sets the draw up and hands it to its own CTA as a
// task D (the fast draw with its certificate); the one that completes all the sequence's rows writes its TV.
// A sequence whose fast draw is not certified is listed for the fp64 re-draw kernel, which runs beside the end
// of this one.
//
// A CTA is eight consumer warps, a producer warp and a publisher warp around a ring of shared-memory
// stages.  The producer's first lane claims tickets, decodes them into runs of consecutive slices,
// fetches the few per-row numbers (length, temperature, row normalisers), checks that the sequence is
// ready for the phase (a run that is not is set aside while later tickets go ahead) and, once a stage
// is free, describes the task there and starts bulk copies (cp.async.bulk, completion counted on the
// stage's mbarrier) of the logits the task reads.  The consumers wait on the stage's barrier, compute
// from shared memory, leave one partial per warp and signal a second barrier; the publisher takes the
// eight partials, hands the stage back, merges them in warp order and publishes.  No CTA-wide barrier
// sits on the streaming path.
//
// What CTAs pass to each other through global memory needs no fence: records of two 64-bit words, both
// non-zero once written (the memory starts at zero), which a reader takes only when it sees both; and
// fixed-point sums with a count of contributions in the low bits of the same word, added by relaxed atomics.
// Counters only say when to look; whoever looks checks the record and waits (bounded) for one that is not
// there yet.
//
// Every wait is bounded; a wait that gives up sets the wait flag (status bit 32 of every row).
// No multicast, no cluster: each CTA copies from this GPU's own memory.
#include "bebop_pipe.cuh"

namespace bebop {

namespace {

// what the kernel is compiled for: bebop_verify; bebop_tv (row pairs, no accept test, no draw); the greedy mode
// (one sweep over the target rows for their argmax)
constexpr int kModeVerify = 0, kModeTv = 1, kModeGreedy = 2;
constexpr int NST = 2;                            // stages of the ring
constexpr int PIPE_CTAS = 3;                      // CTAs per SM the kernel is built for
constexpr int PC = WT;                            // consumer threads (8 warps); thread PC is the producer
constexpr int PT = PC + 64;                       // + producer warp + publisher warp
constexpr int PSLICE = kPipeSliceVecs;            // vectors per stage
constexpr int STAGE_BYTES = PSLICE * 16;
constexpr int kPend = 4;                          // runs a producer may set aside
constexpr int kTailZone = 8;                      // the last kTailZone tickets per CTA are claimed kBatchTail at a time
constexpr int kBatchTail = 2;
constexpr int kBatch = 5;                         // tickets claimed at a time (measured: 4 to 6 alike, 2 and 8 slower)
constexpr double kFixTv = 1099511627776.0;             // 2^40: fixed point of TV parts and sums of squares
constexpr double kFixMass = 288230376151711744.0;      // 2^58: fixed point of the draw-row mass
constexpr uint32_t kBarSpin = 1u << 20;           // tries of one barrier wait (each try itself waits a while)

struct __align__(16) TaskDesc {
    int phase;        // 0 P1, 2 P2, 3 D, -1: no more tasks
    int b, r;         // sequence; row (P1) or draft position (P2, D)
    int s, v0, nv;    // slice, its first vector, its vectors
    int flags;        // bit 0: row pair (else bonus row alone), bit 1: the pair a token is drawn from,
                      // bit 2 (D): no half slice owns the target, the draw goes to the fp64 re-draw
    float tau;        // temperature, and c = log2(e) / tau computed once per row
    float c;
    RowScale P, Q;
    int need;         // P2: partials the sequence's second sweep delivers in all (the last one starts the draw's set-up)
    float bound;      // D: the error bound the draw must clear,
    double tt, base;  //    the target of the inverse CDF and the mass before the half slice in the stage
};

// A draw the publisher warp hands to the producer of its CTA: sequence, draw row, the half slice that owns the
// target of the inverse CDF, and the numbers the task needs.
struct DrawTask {
    double tt, base;
    float bound, c;
    int b, k, owner, pair;
    RowScale P, Q;
};
constexpr int kMbox = 16;                    // mailbox entries: more than the tasks a CTA can have unpublished
static_assert(kMbox >= kBatch + NST + 1, "a run's tasks plus the ring may each complete a sequence before the producer looks");

struct Run { int ph, wv, off, cnt; };       // cnt consecutive tasks of sequence wv in phase ph, from offset off

struct PipeShared {
    DrawShared W;                               // scratch of phases A and D
    TaskDesc desc[NST];
    unsigned long long full[NST], empty[NST];   // mbarriers: data and description there / stage free again
    unsigned long long pdone[NST];              // mbarrier: the eight warp partials of the stage's task are there
    unsigned long long dsync;                   // mbarrier: the consumer warps meet here inside a draw task (bounded wait)
    float wf[NST][2][WW];                       // per-warp partials of the task in the stage
    double wd[NST][WW];
    int wi[NST][WW];
    Run pend[kPend];                            // producer: runs set aside
    DrawTask mbox[kMbox];                       // publisher -> producer: draws to stage
    int mb_tail, mb_head;                       // entries written (publisher) and taken (producer)
    int pub_count;                              // streaming tasks the publisher has dealt with
    float vsum[PSLICE / 2];                     // D: residual mass per vector of the half slice
    double d1_tot[2 * MAX_SLICES];              // publisher: half-slice masses and sums of squares of a sequence
    float d1_sq[2 * MAX_SLICES];
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned long long* b, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* b) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect(unsigned long long* b, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_wait(unsigned long long* b, uint32_t parity) {
    const uint32_t addr = smem_u32(b);
    for (uint32_t i = 0; i < kBarSpin; ++i) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}
// contiguous copy global -> shared of this CTA; 16-byte aligned on both sides, size a multiple of 16
// `policy`: an L2 eviction policy (first sweep: keep, the second sweep comes back for these lines; second sweep: drop)
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, unsigned long long* bar,
                                          unsigned long long policy) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 :: "r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy) : "memory");
}
__device__ __forceinline__ unsigned long long l2_policy(bool keep) {
    unsigned long long p;
    if (keep) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    else asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
// n / d for 0 <= n < 2^31, 0 < d, with inv = 1.0 / d: a multiplication and a correction instead of the
// forty-odd instructions of an integer division (the producer is one thread: its instructions are its time)
__device__ __forceinline__ int div_by(int n, int d, double inv) {
    int q = __double2int_rz((double)n * inv);
    const int r = n - q * d;
    if (r >= d) ++q; else if (r < 0) --q;
    return q;
}
__device__ __forceinline__ uint4 lds16(const unsigned char* p) { return *reinterpret_cast<const uint4*>(p); }
// The consumer warps of a CTA meet (inside a draw task).  A counted barrier with a bounded wait, not bar.sync: should
// a warp have left the loop after a wait of its own gave up, the others still return, with the wait flag set.
// `phase` is the warp's count of such meetings so far (every consumer warp sees the same draw tasks).
__device__ __forceinline__ void consumers_meet(int* wait_failed, unsigned long long* bar, uint32_t& phase) {
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
    if (!mbar_wait(bar, phase & 1u)) atomicExch(wait_failed, 1);
    ++phase;
}


// ------------------------------------------------------------------ producer
// One thread.  Tickets are claimed kBatch at a time; consecutive tickets of one (phase, sequence) block are
// consecutive slices of a row, then the next row, then the next sequence, so a batch decodes once and
// then steps, and the per-row numbers (length, temperature, normalisers, row addresses) are fetched
// once per row.  Draw tasks have no tickets: the publisher warp of this CTA leaves one in the CTA's mailbox
// when it has delivered the last partial of a sequence's second sweep, and the producer stages it ahead of
// the next ticket.  Returns when the stop description has been handed to the consumers.
template <int DT, int MODE>
__device__ __forceinline__ void producer(const PipeArgs& a, PipeShared& S, unsigned char* data) {
    constexpr bool TVO = MODE == kModeTv, GRD = MODE == kModeGreedy;
    const RowArgs& R = a.r;
    const int K = R.K, T = a.T, T2 = 2 * a.T, NR = 2 * K + 1;
    const int B = R.B;
    // (a caller that asks for no TV needs the second sweep over one row per sequence only: the one a token is drawn from)
    // (and bebop_tv has the K row pairs and no bonus row)
    // (the greedy mode sweeps the K + 1 target rows once)
    // The second sweep comes in two passes: first the row each sequence's token is drawn from (so that every draw,
    // and the list of the sequences that go to the fp64 re-draw, is done early in the sweep), then the other
    // rows, which only TV needs.  bebop_tv has the K row pairs and no draw; the greedy mode sweeps the K + 1 target
    // rows once.
    const int c0 = (GRD ? K + 1 : NR) * T;
    const int c2a = (GRD || TVO) ? 0 : T2, c2b = GRD ? 0 : ((TVO || a.o.tv) ? K * T2 : 0);
    const double inv_c0 = 1.0 / c0, inv_c2a = c2a ? 1.0 / c2a : 0.0, inv_c2b = c2b ? 1.0 / c2b : 0.0;
    const double inv_T = 1.0 / T, inv_T2 = 1.0 / T2;
    const int sv1 = a.slice_vecs, sv2 = a.slice_vecs >> 1;
    // Ticket order: blocks 0 .. B-1 hold the first sweep of sequence i, blocks B .. 2B-1 the first pass of the
    // second sweep, blocks 2B .. 3B-1 its second pass: full sweeps, sequences ascending, so that a sequence's
    // accept scan is long done when the second sweep reaches it.  (Pairing the sweeps so that the second finds
    // its logits in L2 was measured and dropped: it waited for accept scans more than the L2 hits saved.)
    const unsigned long long pol_keep = l2_policy(true), pol_drop = l2_policy(false);
    auto clampB = [&](int x) { return x < 0 ? 0 : (x > B ? B : x); };
    auto before = [&](int i) { return c0 * clampB(i) + c2a * clampB(i - B) + c2b * clampB(i - 2 * B); };   // tickets before block i
    int blk = 0, f_here = 0, f_next = before(1);      // tickets of this CTA only grow: the block is tracked, not searched
    // the run of consecutive tasks of one sequence and phase that starts at ticket t, at most `want` tasks;
    // Run.wv is the sequence, Run.off the offset inside the sequence's tasks of that phase (second sweep: the draw row
    // is row 0, the other rows follow)
    const int t1 = B * c0, t2 = t1 + B * c2a;
    auto decode = [&](int t, int want) {
        if (f_next <= t) {
            // the block follows from one division (a CTA's next tickets are some thirty blocks on: stepping there
            // one block at a time was most of what the producer did between two runs)
            blk = (GRD || t < t1) ? div_by(t, c0, inv_c0)
                                  : (t < t2 ? B + div_by(t - t1, c2a, inv_c2a) : 2 * B + div_by(t - t2, c2b, inv_c2b));
            f_here = before(blk); f_next = before(blk + 1);
        }
        while (f_next <= t) { ++blk; f_here = f_next; f_next = before(blk + 1); }
        Run r;
        const int o = t - f_here;
        if (blk < B) { r.ph = 0; r.wv = blk; r.off = o; }
        else if (blk < 2 * B) { r.ph = 2; r.wv = blk - B; r.off = o; }
        else { r.ph = 2; r.wv = blk - 2 * B; r.off = o + c2a; }
        r.cnt = min(want, f_next - t);
        return r;
    };
    // Is sequence b ready for the phase?  P2 needs its accept scan.  A run that is not ready is set aside (up to
    // kPend of them) while later tickets go ahead; the oldest one is looked at again before every new run and
    // waited for only when the shelf is full or no tickets are left.
    // the sequence's record of the accept scan, valid once its mark is set (waits, bounded, if asked to)
    auto seq_info = [&](int b, bool wait) {
        SeqInfo si = ld_seq(a.sinfo + b);
        if (a.expire) { if (wait) si.pad = 0; return si; }          // test hook: this wait's bound has run out already
        if (wait) for (uint32_t i = 0; si.pad == 0 && i < kSpin; ++i) { __nanosleep(64); si = ld_seq(a.sinfo + b); }
        return si;
    };
    SeqInfo seen; seen.n = 0; seen.draw_row = 0; seen.pad0 = 0; seen.pad = 0;     // the record `ready` last saw valid,
    int seen_b = -1;                                                              // and whose it is
    auto ready = [&](int ph, int b, bool wait) {
        if (ph != 2) return true;
        if (seen_b == b) return true;
        if (a.expire && !wait) return false;                        // test hook: every second-sweep run goes through the wait
        const SeqInfo si = seq_info(b, wait);
        if (si.pad == 0) return false;
        seen = si; seen_b = b;
        return true;
    };
    int it = 0, n_stream = 0, mb_head = 0;
    // hand one task to the consumers: its description, and its logits on their way into the stage
    auto issue = [&](const TaskDesc& d, const char* row0, const char* row1, unsigned long long pol) {
        const int stage = it % NST;
        if (!mbar_wait(&S.empty[stage], ((uint32_t)(it / NST) & 1u) ^ 1u)) atomicExch(a.wait_failed, 1);
        S.desc[stage] = d;
        const uint32_t bytes = (uint32_t)d.nv * 16u;
        if (row0 && bytes) {
            mbar_arrive_expect(&S.full[stage], row1 ? 2u * bytes : bytes);
            bulk_load(data + (size_t)stage * STAGE_BYTES, row0 + (int64_t)d.v0 * 16, bytes, &S.full[stage], pol);
            if (row1) bulk_load(data + (size_t)stage * STAGE_BYTES + STAGE_BYTES / 2, row1 + (int64_t)d.v0 * 16, bytes, &S.full[stage], pol);
        } else {
            mbar_arrive(&S.full[stage]);
        }
        ++it;
    };
    // the draw tasks the publisher left in the mailbox: the half slice that owns the target, staged like a P2 task
    auto drain = [&]() {
        while (mb_head != *(volatile int*)&S.mb_tail) {
            const DrawTask t = S.mbox[mb_head % kMbox];
            ++mb_head;
            *(volatile int*)&S.mb_head = mb_head;
            TaskDesc d;
            d.phase = 3; d.b = t.b; d.r = t.k; d.s = t.owner; d.flags = (t.pair ? 1 : 0) | 2;
            d.v0 = t.owner * sv2; d.nv = max(min(sv2, R.nvec - d.v0), 0);
            d.tau = 1.f; d.c = t.c; d.P = t.P; d.Q = t.Q; d.need = 0;
            d.bound = t.bound; d.tt = t.tt; d.base = t.base;
            issue(d, row_ptr(R, t.b, t.k), t.pair ? row_ptr(R, t.b, K + 1 + t.k) : nullptr, pol_drop);
        }
    };
    const int tail_zone = (int)gridDim.x * kTailZone;
    int npend = 0;
    bool exhausted = false;
    int bt = 0, bleft = 0;                         // tickets of the claimed batch not yet turned into runs
    int last_seen = 0;                             // the latest ticket this CTA has seen handed out
    for (;;) {
        drain();
        // ---- next run
        Run run;
        if (npend > 0 && (ready(S.pend[0].ph, S.pend[0].wv, false) || npend == kPend || (exhausted && bleft == 0))) {
            run = S.pend[0];
            if (!ready(run.ph, run.wv, true)) atomicExch(a.wait_failed, 1);
            --npend;
            for (int i = 0; i < npend; ++i) S.pend[i] = S.pend[i + 1];
        } else {
            if (bleft == 0 && !exhausted) {
                // (claiming a batch ahead of need gained nothing and made the CTAs finish further apart)
                const int cnt = (a.ntickets - last_seen <= tail_zone) ? kBatchTail : kBatch;
                bt = atomicAdd(a.ticket, cnt); bleft = min(cnt, a.ntickets - bt);
                last_seen = bt;
                if (bleft <= 0) { bleft = 0; exhausted = true; }
            }
            if (bleft == 0) {
                if (npend > 0) continue;
                // no tickets left: stay until the publisher has dealt with every streaming task of this CTA (it
                // may still leave draw tasks), then stop the consumers
                bool done = false;
                for (uint32_t i = 0; i < kSpin && !done; ++i) {
                    done = *(volatile int*)&S.pub_count == n_stream;      // read before the mailbox: its entries come first
                    drain();
                    if (!done) __nanosleep(100);
                }
                if (!done) atomicExch(a.wait_failed, 1);
                const int stage = it % NST;
                if (!mbar_wait(&S.empty[stage], ((uint32_t)(it / NST) & 1u) ^ 1u)) atomicExch(a.wait_failed, 1);
                S.desc[stage].phase = -1;
                mbar_arrive(&S.full[stage]);
                return;
            }
            run = decode(bt, bleft);
            bt += run.cnt; bleft -= run.cnt;
            if (!ready(run.ph, run.wv, false)) { S.pend[npend++] = run; continue; }
        }
        // ---- the tasks of the run
        const int ph = run.ph;
        const int per_row = ph == 0 ? T : T2;
        // a run starts inside its sequence's block of the phase: row and slice from the offset (rows * per_row tasks)
        int r = div_by(run.off, per_row, ph == 0 ? inv_T : inv_T2);
        int s = run.off - r * per_row;
        const int b = run.wv;                      // a run stays within one sequence
        int left = run.cnt;
        while (left > 0) {
            // the row's numbers
            TaskDesc d;
            d.phase = ph; d.b = b; d.r = r; d.s = 0; d.v0 = 0; d.nv = 0; d.flags = 0; d.tau = 1.f; d.c = 0.f;
            d.P = no_row(); d.Q = no_row();
            d.need = 0; d.bound = 0.f; d.tt = 0.0; d.base = 0.0;
            const char* row0 = nullptr; const char* row1 = nullptr;
            bool skip = false;
            if (ph == 0) {
                const int L = len_of(R, b);
                const bool is_target = r <= K;
                const int k = is_target ? r : r - (K + 1);
                if (!GRD) { d.tau = tau_of(R, b); d.c = temp_scale(d.tau).hi; }
                skip = is_target ? (TVO ? k >= L : k > L) : k >= L;     // (bebop_tv has no bonus row)
                row0 = row_ptr(R, b, r);
            } else {
                // everything the row needs is requested at once (the sequence was seen ready: its records are there)
                const SeqInfo si = seen_b == b ? seen : ld_seq(a.sinfo + b);
                // row 0 of the sequence's second sweep is the row its token is drawn from; the others follow in order
                const bool drawrow = !TVO && r == 0;
                const int rp = TVO ? r : r - 1;
                const int k = drawrow ? max(si.draw_row, 0) : (TVO ? rp : rp + (rp >= si.draw_row ? 1 : 0));
                d.r = k;
                RowStat sp = ld_cg(a.rstat + (int64_t)b * NR + k);
                RowStat sq = ld_cg(a.rstat + (int64_t)b * NR + K + 1 + min(k, K - 1));
                const int L = len_of(R, b);
                // (the accept scan saw these row records before it set the sequence's mark; should a load have
                // overtaken that all the same, ask again)
                const bool no_row_k = TVO && k >= L;      // bebop_tv has no bonus row: nothing was merged for it
                if (k <= L && !no_row_k) for (uint32_t i = 0; !rec_valid(sp) && i < kSpin; ++i) sp = ld_cg(a.rstat + (int64_t)b * NR + k);
                if (k < L) for (uint32_t i = 0; !rec_valid(sq) && i < kSpin; ++i) sq = ld_cg(a.rstat + (int64_t)b * NR + K + 1 + k);
                d.c = __int_as_float(si.pad0);
                const bool pair = k < L;
                skip = k > L || si.n < 0 || (!pair && !(drawrow && si.draw_row == L)) || no_row_k;
                // the sequence's second sweep: every half slice of the L row pairs, and of the bonus row if drawn from
                d.need = T2 * (L + (si.draw_row == L ? 1 : 0));
                if (!a.o.tv) d.need = T2;
                if (!skip) {
                    d.flags = (pair ? 1 : 0) | (drawrow ? 2 : 0);
                    d.P = row_scale(sp);
                    if (pair) d.Q = row_scale(sq);
                    row0 = row_ptr(R, b, k);
                    if (pair) row1 = row_ptr(R, b, K + 1 + k);
                }
            }
            const int n_row = min(left, per_row - s);         // tasks of this run in this row
            if (!skip) {
                const int sv = ph == 0 ? sv1 : sv2;
                for (int i = 0; i < n_row; ++i) {
                    d.s = s + i; d.v0 = d.s * sv; d.nv = max(min(sv, R.nvec - d.v0), 0);
                    issue(d, row0, row1, ph == 0 ? pol_keep : pol_drop);
                    ++n_stream;
                }
            }
            left -= n_row;
            s = 0;
            ++r;
        }
    }
}

// a merged row's record (it has been seen by the sequence's accept scan; should this thread's load run ahead of that
// all the same, it asks again)
__device__ __forceinline__ RowStat ld_row(const PipeArgs& a, int64_t i) {
    RowStat x = ld_cg(a.rstat + i);
    for (uint32_t k = 0; !rec_valid(x) && k < kSpin; ++k) { __nanosleep(64); x = ld_cg(a.rstat + i); }
    return x;
}

// ------------------------------------------------------------------ phase A without tickets
// The warp that delivers the last softmax partial of a ROW merges that row's partials (exactly:
// integer exponents, fp64 sums in a fixed tree) and leaves the row's normaliser; the warp that merges
// the last row of a SEQUENCE runs the accept scan at once and writes accept_len, the accepted tokens,
// p(x), q(x), the status and the stop position.  No ticket, no CTA barrier, and the work is done
// long before the second sweep of the sequence is handed out.
__device__ __forceinline__ void merge_row_warp(const PipeArgs& a, int b, int r) {
    const int lane = threadIdx.x & 31;
    const int NR = 2 * a.r.K + 1, T = a.T;
    const P1Part* pp = a.part + ((int64_t)b * NR + r) * T;
    // lanes take slices in order; exponent first, then the scaled sum in a fixed tree
    int e_l = E_EMPTY; double s_l = 0.0; int f_l = 0;
    P1Part mine[2];
    int cnt = 0;
    for (int s = lane; s < T && cnt < 2; s += 32) {
        // (the record's exponent is stored as 2e + 1, its sum with non-zero bits: a record is there when both words are)
        P1Part rec = ld_cg(pp + s);
        for (uint32_t i = 0; !rec_valid(rec) && i < kSpin; ++i) { __nanosleep(64); rec = ld_cg(pp + s); }
        if (!rec_valid(rec)) { atomicExch(a.wait_failed, 1); rec.e = 2 * E_EMPTY + 1; rec.s = 0.0; rec.m = 0.f; }
        rec.e = (rec.e - 1) >> 1;
        mine[cnt] = rec; e_l = max(e_l, rec.e);
        if (rec.m != rec.m) f_l = 1;
        cnt++;
    }
    const int Em = redux_max(e_l);
    for (int i = 0; i < cnt; ++i) if (mine[i].e > E_EMPTY) s_l += mine[i].s * pow2d(max(mine[i].e - Em, -1000));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { s_l += shfl_xor_d(s_l, o); f_l |= __shfl_xor_sync(0xffffffffu, f_l, o); }
    if (lane == 0) {
        int st = 0;
        if (f_l || !(s_l == s_l)) st = ST_NONFINITE; else if (Em == E_EMPTY) st = ST_EMPTY;
        RowStat rs; rs.inv_s = nonzero_bits((!st && s_l > 0.0) ? 1.0 / s_l : 0.0); rs.e = Em; rs.st = st | kRowValid;
        st16(a.rstat + (int64_t)b * NR + r, rs);
    }
}

template <int DT, bool TVO>
__device__ __noinline__ void accept_warp(const PipeArgs& a, int b) {
    const RowArgs& R = a.r;
    const int lane = threadIdx.x & 31;
    const int K = R.K, V = R.V, L = len_of(R, b), NR = 2 * K + 1;
    const float tau = tau_of(R, b);
    const bool ok = tau_ok(tau);
    const TempScale ts = temp_scale(tau);
    // lane k owns draft position k (K <= 32): everything it needs is requested before anything is used
    const bool active = lane < L;
    const bool tvo = TVO;              // row pairs only: no tokens, no accept test, no bonus row
    const int tk = (active && !tvo) ? a.draft_tokens[(int64_t)b * K + lane] : 0;
    const float u = (active && !tvo) ? a.u_accept[(int64_t)b * K + lane] : 0.f;
    RowStat sp, sq, sb;
    sp.inv_s = 0.0; sp.e = E_EMPTY; sp.st = 0;
    sq = sp;
    auto row = [&](int r) {                                            // a merged row's record (waits, bounded, for its mark)
        RowStat x = ld_cg(a.rstat + (int64_t)b * NR + r);
        for (uint32_t i = 0; !rec_valid(x) && i < kSpin; ++i) { __nanosleep(64); x = ld_cg(a.rstat + (int64_t)b * NR + r); }
        if (!rec_valid(x)) { atomicExch(a.wait_failed, 1); x.inv_s = 0.0; x.e = E_EMPTY; x.st = ST_WAIT; }
        x.st &= 0xff;
        return x;
    };
    if (active) { sp = row(lane); sq = row(K + 1 + lane); }
    if (tvo) { sb = sp; sb.st = 0; } else sb = row(L);                  // bonus row (row L <= K: always merged)
    int seq_st = ok ? 0 : ST_BAD_TEMP;
    const bool tok_ok = tvo || (tk >= 0 && tk < V);
    float zpx = 0.f, zqx = 0.f;
    if (active && tok_ok && !tvo) { zpx = load_one<DT>(row_ptr(R, b, lane), tk); zqx = load_one<DT>(row_ptr(R, b, K + 1 + lane), tk); }
    if (!seq_st && __ballot_sync(0xffffffffu, active && !tok_ok)) seq_st = ST_BAD_TOKEN;
    // the first bad row pair decides the status; rows after it do not count
    const int rs = active ? (sp.st | sq.st) : 0;
    const unsigned badrows = __ballot_sync(0xffffffffu, rs != 0);
    const int first_bad = badrows ? __ffs(badrows) - 1 : 32;
    const int rs_first = __shfl_sync(0xffffffffu, rs, first_bad & 31);
    if (!seq_st && badrows) seq_st = rs_first;
    double px = 0.0, qx = 0.0;
    bool acc = false;
    if (active && !tvo && !(seq_st & ST_FATAL) && lane < first_bad) {
        const double cd = (double)ts.hi;
        px = exp2((double)zpx * cd - (double)sp.e) * sp.inv_s;
        qx = exp2((double)zqx * cd - (double)sq.e) * sq.inv_s;
        acc = (double)u * qx < px;
    }
    const unsigned rej = __ballot_sync(0xffffffffu, active && !acc);
    const int n = rej ? __ffs(rej) - 1 : L;
    if (!(seq_st & ST_FATAL) && n == L && sb.st) seq_st |= sb.st;   // bonus row, counted only now
    const bool fatal = (seq_st & ST_FATAL) != 0;
    const int nn = fatal ? 0 : n;
    // outputs: lane q writes position q (position nn is filled by the draw)
    if (!tvo) for (int q = lane; q <= K; q += 32)
        if (fatal || q != nn) a.o.out_tokens[(int64_t)b * (K + 1) + q] = q < nn ? tk : -1;   // q < nn <= 32: q == lane
    if (lane < K) {
        const bool zero = fatal || lane >= L;
        if (a.o.p_draft) a.o.p_draft[(int64_t)b * K + lane] = zero ? 0.f : (float)px;
        if (a.o.q_draft) a.o.q_draft[(int64_t)b * K + lane] = zero ? 0.f : (float)qx;
        if (zero && a.o.tv) a.o.tv[(int64_t)b * K + lane] = 0.f;
        if (TVO && zero && a.s_aux) a.s_aux[(int64_t)b * K + lane] = 0.f;
    }
    if (lane == 0) {
        if (!tvo) { a.o.accept_len[b] = nn; a.stop[b] = fatal ? -1 : nn; }
        if (a.o.row_status) a.o.row_status[b] = seq_st;
        // the record's mark makes it (and, through the row records it was computed from, the sequence) ready
        // (pad0 carries c = log2(e) / tau of the sequence: the second sweep's producer need not divide again)
        SeqInfo si; si.n = fatal ? -1 : nn; si.draw_row = (fatal || tvo) ? -1 : nn; si.pad0 = __float_as_int(ts.hi); si.pad = 1;
        st_seq(a.sinfo + b, si);
        if (fatal && !tvo) draw_decided(a.fb_count);     // no draw will come
    }
}

// ------------------------------------------------------------------ consumers
// Each consumer warp leaves its partial of a task in shared memory and signals the stage's `pdone` barrier;
// the publisher warp merges the eight partials in warp order and publishes the result, off the consumers'
// path.
__device__ __forceinline__ void red_add_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" :: "l"(p), "l"(v) : "memory");
}

// P1: softmax partial (E, S) of one slice of one row, from shared memory.
template <int DT>
__device__ __forceinline__ void pipe_p1(const PipeArgs& a, PipeShared& S, const TaskDesc& d, const unsigned char* data,
                                        int stage) {
    constexpr int VEC = Elem<DT>::VEC, NV = PSLICE / PC;
    const RowArgs& R = a.r;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    TempScale ts; ts.hi = d.c;
    const int nv = d.nv;
    uint4 raw[NV];
    if (nv >= (NV - 1) * PC) {                   // the usual case: only a thread's last vector may lie beyond the slice
#pragma unroll
        for (int u = 0; u < NV - 1; ++u) raw[u] = lds16(data + (size_t)(tid + u * PC) * 16);
        raw[NV - 1] = neg_inf_vec<DT>();
        if (tid + (NV - 1) * PC < nv) raw[NV - 1] = lds16(data + (size_t)(tid + (NV - 1) * PC) * 16);
    } else {
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            const int v = tid + u * PC;
            raw[u] = neg_inf_vec<DT>();
            if (v < nv) raw[u] = lds16(data + (size_t)v * 16);
        }
    }
    if ((d.v0 + nv) * VEC > R.V) {               // the row's last vector is in this slice and is partial
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            const int gbase = (d.v0 + tid + u * PC) * VEC;
            if (tid + u * PC < nv && gbase + VEC > R.V) mask_tail<DT>(raw[u], R.V - gbase);
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
    // thread -> warp, exact power-of-two rescaling, sums in a fixed order
    float st = (s0 + s1) + (s2 + s3);
    const int Ew = redux_max(E);
    st = E > E_EMPTY ? st * pow2f(max(E - Ew, -126)) : 0.f;
    st = warp_sum(st);
    const unsigned anybad = __ballot_sync(0xffffffffu, bad);
    float mw = ord2f(redux_max(f2ord(bad ? -INFINITY : m)));
    if (anybad) mw = __int_as_float(0x7fc00000);
    if (lane == 0) { S.wf[stage][0][warp] = st; S.wi[stage][warp] = Ew; S.wf[stage][1][warp] = mw; }
    __syncwarp();
    if (lane == 0) mbar_arrive(&S.pdone[stage]);
}

// Greedy mode: maximum and lowest index of the maximum over one slice of a target row (no exponentials).
template <int DT>
__device__ __forceinline__ void pipe_g(const PipeArgs& a, PipeShared& S, const TaskDesc& d, const unsigned char* data,
                                       int stage) {
    constexpr int VEC = Elem<DT>::VEC, NV = PSLICE / PC;
    const RowArgs& R = a.r;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nv = d.nv;
    uint4 raw[NV];
#pragma unroll
    for (int u = 0; u < NV; ++u) {
        const int v = tid + u * PC;
        raw[u] = neg_inf_vec<DT>();
        if (v < nv) raw[u] = lds16(data + (size_t)v * 16);
    }
    if ((d.v0 + nv) * VEC > R.V) {               // the row's last vector is in this slice and is partial
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            const int gbase = (d.v0 + tid + u * PC) * VEC;
            if (tid + u * PC < nv && gbase + VEC > R.V) mask_tail<DT>(raw[u], R.V - gbase);
        }
    }
    float m = vec_max<DT>(raw[0]);
#pragma unroll
    for (int u = 1; u < NV; ++u) m = max_nan(m, vec_max<DT>(raw[u]));
    if (!(m < INFINITY)) m = __int_as_float(0x7fc00000);      // NaN or +inf poisons the row
    m += 0.f;                                                 // -0 becomes +0: the ordered-integer maximum below must not tell them apart
    // the thread's lowest token with that value (its vectors ascend with u)
    int idx = INT_MAX;
    if (m == m && m > -INFINITY) {
#pragma unroll
        for (int u = NV - 1; u >= 0; --u) {
            float f[VEC];
            unpack<DT>(raw[u], f);
#pragma unroll
            for (int j = VEC - 1; j >= 0; --j) if (f[j] == m) idx = (d.v0 + tid + u * PC) * VEC + j;
        }
    }
    // warp: the maximum (NaN sorts above +inf), then the lowest index among the lanes that hold it
    const int om = f2ord(m);
    const int ow = redux_max(om);
    int iw;
    { const int mine = om == ow ? idx : INT_MAX; asm volatile("redux.sync.min.s32 %0, %1, 0xffffffff;" : "=r"(iw) : "r"(mine)); }
    if (lane == 0) { S.wi[stage][warp] = ow; S.wf[stage][0][warp] = __int_as_float(iw); }
    __syncwarp();
    if (lane == 0) mbar_arrive(&S.pdone[stage]);
}

// P2: TV partial of one half slice of a row pair; on the pair (or bonus row) a token is drawn from,
// also the mass in double and the sum of squares.  Target row in the first half of the stage, draft
// row in the second.
template <int DT, bool TVO>
__device__ __forceinline__ void pipe_p2(const PipeArgs& a, PipeShared& S, const TaskDesc& d, const unsigned char* data,
                                        int stage) {
    constexpr int VEC = Elem<DT>::VEC, NV = PSLICE / (2 * PC);
    const RowArgs& R = a.r;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool pair = (d.flags & 1) != 0, draw = (d.flags & 2) != 0;
    const int nv = d.nv;
    const unsigned char* qdata = data + STAGE_BYTES / 2;
    // Vectors beyond the slice, and the draft row of a bonus task, read as -inf: they give p = q = 0 and add
    // nothing, so the arithmetic below runs unguarded.
    uint4 rp[NV], rq[NV];
    if (nv >= (NV - 1) * PC && pair) {           // the usual case: only a thread's last vector may lie beyond the slice
#pragma unroll
        for (int u = 0; u < NV - 1; ++u) { rp[u] = lds16(data + (size_t)(tid + u * PC) * 16); rq[u] = lds16(qdata + (size_t)(tid + u * PC) * 16); }
        rp[NV - 1] = neg_inf_vec<DT>(); rq[NV - 1] = neg_inf_vec<DT>();
        if (tid + (NV - 1) * PC < nv) { rp[NV - 1] = lds16(data + (size_t)(tid + (NV - 1) * PC) * 16); rq[NV - 1] = lds16(qdata + (size_t)(tid + (NV - 1) * PC) * 16); }
    } else {
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            const int v = tid + u * PC;
            rp[u] = neg_inf_vec<DT>(); rq[u] = neg_inf_vec<DT>();
            if (v < nv) { rp[u] = lds16(data + (size_t)v * 16); if (pair) rq[u] = lds16(qdata + (size_t)v * 16); }
        }
    }
    TempScale c; c.hi = d.c;
    const RowScale SP = d.P, SQ = d.Q;
    if ((d.v0 + nv) * VEC > R.V) {
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            const int gbase = (d.v0 + tid + u * PC) * VEC;
            if (tid + u * PC < nv && gbase + VEC > R.V) { mask_tail<DT>(rp[u], R.V - gbase); mask_tail<DT>(rq[u], R.V - gbase); }
        }
    }
    float z0 = 0.f, z1 = 0.f, sqs = 0.f;
    double zd = 0.0;
    if (TVO && a.sacc) {
        // bebop_tv with the auxiliary sum: TV and S = sum of q over the tokens with q <= p (Eq. tv_grad)
        float sx = 0.f;
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            float fp[VEC], fq[VEC];
            unpack<DT>(rp[u], fp);
            unpack<DT>(rq[u], fq);
#pragma unroll
            for (int i = 0; i < VEC; ++i) {
                const float p = __fmul_rn(exp2_scaled(fp[i], c, SP.ef), SP.inv);
                const float q = __fmul_rn(exp2_scaled(fq[i], c, SQ.ef), SQ.inv);
                z0 += fmaxf(p - q, 0.f);
                sx += q <= p ? q : 0.f;
            }
        }
        zd = (double)warp_sum(sx);
    } else if (!draw) {
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            float r[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) r[i] = 0.f;
            residual_vec<DT, false>(rp[u], rq[u], c, SP, SQ, r, nullptr);
            const float vs = ((r[0] + r[1]) + (r[2] + r[3])) + ((r[4] + r[5]) + (r[6] + r[7]));
            if (u & 1) z1 += vs; else z0 += vs;
        }
    } else {
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            float r[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) r[i] = 0.f;
            residual_vec<DT, true>(rp[u], rq[u], c, SP, SQ, r, &sqs);
            const float vs = ((r[0] + r[1]) + (r[2] + r[3])) + ((r[4] + r[5]) + (r[6] + r[7]));
            z0 += vs;
            zd += (double)vs;
        }
    }
    const float z = warp_sum(z0 + z1);
    if (draw && !(TVO && a.sacc)) { zd = warp_sum(zd); sqs = warp_sum(sqs); }
    if (lane == 0) { S.wf[stage][0][warp] = z; S.wd[stage][warp] = zd; S.wf[stage][1][warp] = sqs; }
    __syncwarp();
    if (lane == 0) mbar_arrive(&S.pdone[stage]);
}

// ------------------------------------------------------------------ the draw
// mass and sum of squares of half slice i of a sequence's draw rows (waits, bounded, for a part not there yet)
__device__ __forceinline__ DPart load_dpart(const PipeArgs& a, int64_t i) {
    unsigned long long w0 = 0, w1 = 0;
    for (uint32_t k = 0; k < kSpin; ++k) {
        w0 = __ldcg(a.dacc + 2 * i); w1 = __ldcg(a.dacc + 2 * i + 1);
        if ((w0 & 15ull) != 0 && (w1 & 15ull) != 0) break;
        __nanosleep(64);
    }
    if ((w0 & 15ull) == 0 || (w1 & 15ull) == 0) atomicExch(a.wait_failed, 1);
    DPart d;
    d.tot = (double)(w0 >> 4) * 3.469446951953614e-18;            // 2^-58
    d.sq = (float)((double)(w1 >> 4) * 9.094947017729282e-13);    // 2^-40
    d.pad = 1;
    return d;
}

// Set-up of a sequence's draw, by the publisher warp that delivered the last partial of the sequence's second
// sweep: TV of every draft position from the fixed-point sums, then the residual mass Z of the draw rows, the
// target u * Z of the inverse CDF and the half slice that owns it.  The draw task goes into the CTA's mailbox:
// the producer stages that half slice and the consumers find the token.
template <bool TVO>
__device__ __noinline__ void draw_setup_warp(const PipeArgs& a, PipeShared& S, int b, int what) {
    const RowArgs& R = a.r;
    const int lane = threadIdx.x & 31;
    const int K = R.K, NR = 2 * K + 1, L = len_of(R, b), T2 = 2 * a.T;
    const SeqInfo si = ld_seq(a.sinfo + b);
    if (si.n < 0) return;
    const int k = si.draw_row;
    const bool pair = k >= 0 && k < L;
    // lane 0 will need the draw rows' records: asked for now, with everything else
    RowStat sp, sq;
    sp.inv_s = 0.0; sp.e = 0; sp.st = 0; sq = sp;
    if (lane == 0 && k >= 0 && (what & 2)) { sp = ld_row(a, (int64_t)b * NR + k); if (pair) sq = ld_row(a, (int64_t)b * NR + K + 1 + k); }
    if ((what & 1) && lane < L && a.o.tv) {
        // the position's TV parts were added in fixed point, with a count of one each in the low 16 bits
        unsigned long long w = 0;
        for (uint32_t i = 0; i < kSpin; ++i) {
            w = __ldcg(a.tvacc + (int64_t)b * K + lane);
            if ((int)(w & 0xffffull) >= T2) break;
            __nanosleep(64);
        }
        if ((int)(w & 0xffffull) < T2) atomicExch(a.wait_failed, 1);
        const float z = (float)((double)(w >> 16) * 9.094947017729282e-13);      // 2^-40
        a.o.tv[(int64_t)b * K + lane] = fminf(fmaxf(z, 0.f), 1.f);
    }
    if (TVO && (what & 1) && lane < L && a.s_aux) {
        unsigned long long w = 0;
        for (uint32_t i = 0; i < kSpin; ++i) {
            w = __ldcg(a.sacc + (int64_t)b * K + lane);
            if ((int)(w & 0xffffull) >= T2) break;
            __nanosleep(64);
        }
        if ((int)(w & 0xffffull) < T2) atomicExch(a.wait_failed, 1);
        a.s_aux[(int64_t)b * K + lane] = (float)((double)(w >> 16) * 9.094947017729282e-13);
    }
    if (k < 0 || !(what & 2)) return;
    // the half slices' masses: lanes fetch them in parallel, lane 0 scans them in slice order
    for (int s = lane; s < T2; s += 32) { const DPart dp = load_dpart(a, (int64_t)b * T2 + s); S.d1_tot[s] = dp.tot; S.d1_sq[s] = dp.sq; }
    __syncwarp();
    if (lane == 0) {
        double Z = 0.0, sumsq = 0.0;
        for (int s = 0; s < T2; ++s) { Z += S.d1_tot[s]; sumsq += (double)S.d1_sq[s]; }
        const double Tt = (double)a.u_final[b] * Z;
        double run = 0.0; int owner = -1; double base = 0.0;
        for (int s = 0; s < T2; ++s) {
            const double nx = run + S.d1_tot[s];
            if (owner < 0 && Tt > run && Tt <= nx) { owner = s; base = run; }
            run = nx;
        }
        if (!(Tt > 0.0)) owner = -1;
        if (owner < 0) {
            // no half slice owns the target (no residual mass, or u = 0): the fp64 re-draw decides
            st_fb(a.fb_list + draw_listed(a.fb_count), b, 2 * k + (pair ? 1 : 0), sp.e, pair ? sq.e : 0);
        } else {
            // the mailbox has room for more draws than this CTA's unpublished tasks can bring; should it be full
            // all the same, wait (bounded) for the producer
            const int tail = S.mb_tail;
            bool room = false;
            for (uint32_t i = 0; i < kSpin && !room; ++i) {
                room = tail - *(volatile int*)&S.mb_head < kMbox;
                if (!room) __nanosleep(100);
            }
            if (!room) atomicExch(a.wait_failed, 1);
            else {
                DrawTask t;
                t.tt = Tt; t.base = base; t.bound = (float)draw_bound(sumsq, (double)a.kappa); t.c = __int_as_float(si.pad0);
                t.b = b; t.k = k; t.owner = owner; t.pair = pair ? 1 : 0;
                t.P = row_scale(sp); t.Q = pair ? row_scale(sq) : no_row();
                S.mbox[tail % kMbox] = t;
                __threadfence_block();
                *(volatile int*)&S.mb_tail = tail + 1;
            }
        }
    }
    __syncwarp();
}

// D: the token of a sequence from the half slice that owns the target of the inverse CDF (target row in the
// first half of the stage, draft row in the second, like a P2 task).  The fp32 draw is kept when target and
// running sum are further apart than the error bound on both sides of the token; else the sequence is listed
// for the fp64 re-draw.
template <int DT>
__device__ __forceinline__ void pipe_d(const PipeArgs& a, PipeShared& PS, const TaskDesc& d, const unsigned char* data, uint32_t& meet) {
    constexpr int VEC = Elem<DT>::VEC;
    const RowArgs& R = a.r;
    DrawShared& S = PS.W;
    float* vsum = PS.vsum;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = R.K, NR = 2 * K + 1, b = d.b, k = d.r;
    const bool pair = (d.flags & 1) != 0;
    const unsigned char* qdata = data + STAGE_BYTES / 2;
    int found_y = -1, found_cert = 0;
    if (!(d.flags & 4)) {
        TempScale c; c.hi = d.c;
        const RowScale SP = d.P, SQ = d.Q;
        const int v0 = d.v0, nv = d.nv;
        // per-vector residual mass, same arithmetic as phase P2
        for (int v = tid; v < nv; v += PC) {
            uint4 rp = lds16(data + (size_t)v * 16), rq = neg_inf_vec<DT>();
            if (pair) rq = lds16(qdata + (size_t)v * 16);
            const int gbase = (v0 + v) * VEC;
            if (gbase + VEC > R.V) { mask_tail<DT>(rp, R.V - gbase); mask_tail<DT>(rq, R.V - gbase); }
            float r[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) r[i] = 0.f;
            residual_vec<DT, true>(rp, rq, c, SP, SQ, r, nullptr);
            vsum[v] = ((r[0] + r[1]) + (r[2] + r[3])) + ((r[4] + r[5]) + (r[6] + r[7]));
        }
        consumers_meet(a.wait_failed, &PS.dsync, meet);
        // contiguous ranges of vectors per thread, inclusive scan over threads
        const int per = (nv + PC - 1) / PC;
        const int vb = min(tid * per, nv), ve = min(vb + per, nv);
        double mine = 0.0;
        for (int v = vb; v < ve; ++v) mine += (double)vsum[v];
        double incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { double t2 = shfl_up_d(incl, o); if (lane >= o) incl += t2; }
        if (lane == 31) S.redd[warp] = incl;
        consumers_meet(a.wait_failed, &PS.dsync, meet);
        double woff = 0.0;
        for (int w = 0; w < warp; ++w) woff += S.redd[w];
        double prev = shfl_up_d(incl, 1);
        if (lane == 0) prev = 0.0;
        const double Tt = d.tt, bound = (double)d.bound;
        const double lower = d.base + woff + prev, upper = d.base + woff + incl;
        if (lower < Tt && Tt <= upper) {
            double C = lower;
            for (int v = vb; v < ve && found_y < 0; ++v) {
                const double nxt = C + (double)vsum[v];
                if (Tt <= nxt) {
                    uint4 rp = lds16(data + (size_t)v * 16), rq = neg_inf_vec<DT>();
                    if (pair) rq = lds16(qdata + (size_t)v * 16);
                    const int gbase = (v0 + v) * VEC;
                    if (gbase + VEC > R.V) { mask_tail<DT>(rp, R.V - gbase); mask_tail<DT>(rq, R.V - gbase); }
                    float r[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) r[i] = 0.f;
                    residual_vec<DT, true>(rp, rq, c, SP, SQ, r, nullptr);
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
    consumers_meet(a.wait_failed, &PS.dsync, meet);
    if (own && lane == (__ffs(own) - 1)) S.redi[warp] = (__popc(own) == 1 && found_cert) ? found_y : -2;
    consumers_meet(a.wait_failed, &PS.dsync, meet);
    if (tid == 0) {
        int y = -1, cnt = 0;
        for (int w = 0; w < WW; ++w) if (S.redi[w] != -1) { y = S.redi[w]; cnt++; }
        if (cnt == 1 && y >= 0) { a.o.out_tokens[(int64_t)b * (K + 1) + k] = y; draw_decided(a.fb_count); }
        else {
            st_fb(a.fb_list + draw_listed(a.fb_count), b, 2 * k + (pair ? 1 : 0), ld_row(a, (int64_t)b * NR + k).e,
                  pair ? ld_row(a, (int64_t)b * NR + K + 1 + k).e : 0);
        }
    }
}

// ------------------------------------------------------------------ publisher
// One warp.  For every streaming task: wait for the eight warp partials, take them into registers,
// hand the stage back, then merge (warp order, so the result does not depend on timing) and publish:
// P1 -- the slice's (E, S) partial and the row's counter, whose last increment starts the merge of the
// row, whose last merged row starts the accept scan of the sequence; P2 -- the TV part (and the
// draw-row mass) and the sequence's counter.
template <int DT, int MODE>
__device__ __forceinline__ void publisher(const PipeArgs& a, PipeShared& S) {
    constexpr bool TVO = MODE == kModeTv, GRD = MODE == kModeGreedy;
    const RowArgs& R = a.r;
    const int lane = threadIdx.x & 31;
    const int K = R.K, T2 = 2 * a.T;
    uint32_t pd_par = 0;                                      // per stage: parity of the next `pdone` phase
    for (int it = 0;; ++it) {
        const int stage = it % NST;
        const uint32_t par = (uint32_t)(it / NST) & 1u;
        if (!mbar_wait(&S.full[stage], par)) { if (lane == 0) atomicExch(a.wait_failed, 1); return; }
        const int phase = S.desc[stage].phase;
        if (phase < 0) return;
        if (phase != 0 && phase != 2) {                       // D: nothing to publish
            __syncwarp();
            if (lane == 0) mbar_arrive(&S.empty[stage]);
            continue;
        }
        // `pdone` only advances on streaming tasks (a D task leaves no partials), so its phase is tracked per
        // stage rather than derived from the task number
        if (!mbar_wait(&S.pdone[stage], (pd_par >> stage) & 1u)) { if (lane == 0) atomicExch(a.wait_failed, 1); return; }
        pd_par ^= 1u << stage;
        const int b = S.desc[stage].b, r = S.desc[stage].r, sl = S.desc[stage].s, flags = S.desc[stage].flags;
        const int need = S.desc[stage].need;
        const int w = lane & (WW - 1);
        const float f0 = S.wf[stage][0][w], f1 = S.wf[stage][1][w];
        const double dd = S.wd[stage][w];
        const int ii = S.wi[stage][w];
        __syncwarp();
        if (lane == 0) mbar_arrive(&S.empty[stage]);
        if (GRD) {
            // lanes 0..7 hold the warps' (maximum, lowest index): the slice's record, read by the kernel that finishes
            const int iw = __float_as_int(f0);
            int om = ii;
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) om = max(om, __shfl_xor_sync(0xffffffffu, om, o));
            int im = ii == om ? iw : INT_MAX;
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) im = min(im, __shfl_xor_sync(0xffffffffu, im, o));
            if (lane == 0) {
                P1Part p; p.s = nonzero_bits((double)im); p.e = 1; p.m = ord2f(om);
                st16(a.part + ((int64_t)b * (2 * K + 1) + r) * a.T + sl, p);
            }
        } else if (phase == 0) {
            // lanes 0..7 hold the warps' (sum, exponent, max); merge in warp order
            const int Ec = max(max(max(__shfl_sync(0xffffffffu, ii, 0), __shfl_sync(0xffffffffu, ii, 1)),
                                   max(__shfl_sync(0xffffffffu, ii, 2), __shfl_sync(0xffffffffu, ii, 3))),
                               max(max(__shfl_sync(0xffffffffu, ii, 4), __shfl_sync(0xffffffffu, ii, 5)),
                                   max(__shfl_sync(0xffffffffu, ii, 6), __shfl_sync(0xffffffffu, ii, 7))));
            const double mine = ii > E_EMPTY ? (double)(f0 * pow2f(max(ii - Ec, -126))) : 0.0;
            double sum = 0.0; float mc = -INFINITY;
#pragma unroll
            for (int k = 0; k < WW; ++k) { sum += __shfl_sync(0xffffffffu, mine, k); mc = max_nan(mc, __shfl_sync(0xffffffffu, f1, k)); }
            int run_a = 0;
            if (lane == 0) {
                // the slice's record (exponent stored as 2e + 1: zero means "not there yet"), then the row's counter.
                // No fence: whoever the counter wakes checks that both words of every record are there before using it.
                P1Part p; p.s = nonzero_bits((mc != mc) ? 0.0 : sum); p.e = 2 * Ec + 1; p.m = mc;
                st16(a.part + ((int64_t)b * (2 * K + 1) + r) * a.T + sl, p);
                run_a = atomicAdd(&a.rowcnt[(int64_t)b * (2 * K + 1) + r], 1) == a.T - 1;
            }
            if (__shfl_sync(0xffffffffu, run_a, 0)) {
                merge_row_warp(a, b, r);
                // the last merged row of the sequence (2L+1 rows are in use, 2L without a bonus row) starts the accept scan
                int last_row = 0;
                if (lane == 0) last_row = atomicAdd(&a.p1done[b], 1) == 2 * len_of(R, b) - (TVO ? 1 : 0);
                if (__shfl_sync(0xffffffffu, last_row, 0)) accept_warp<DT, TVO>(a, b);
            }
        } else {
            float zz = 0.f, sq = 0.f; double tot = 0.0;
            int run_d = 0;
#pragma unroll
            for (int k = 0; k < WW; ++k) {
                zz += __shfl_sync(0xffffffffu, f0, k); sq += __shfl_sync(0xffffffffu, f1, k); tot += __shfl_sync(0xffffffffu, dd, k);
            }
            if (lane == 0) {
                // Fixed point with a count of one in the low bits of the same word: one relaxed add publishes value
                // and count together, and integer sums do not depend on the order of arrival.
                if (flags & 1) red_add_u64(a.tvacc + (int64_t)b * K + r, ((unsigned long long)__double2ll_rn((double)zz * kFixTv) << 16) | 1ull);
                if (TVO && a.sacc) red_add_u64(a.sacc + (int64_t)b * K + r, ((unsigned long long)__double2ll_rn(tot * kFixTv) << 16) | 1ull);
                if (flags & 2) {
                    unsigned long long* wd = a.dacc + ((int64_t)b * T2 + sl) * 2;
                    red_add_u64(wd, ((unsigned long long)__double2ll_rn(tot * kFixMass) << 4) | 1ull);
                    red_add_u64(wd + 1, ((unsigned long long)__double2ll_rn((double)sq * kFixTv) << 4) | 1ull);
                }
                // the last partial of the sequence's draw row starts the set-up of its draw, the last partial of all its rows
                // finishes its TV
                // (without a TV output the draw row is the sequence's whole second sweep: one counter)
                const bool all_rows = TVO || a.o.tv != nullptr;
                if ((flags & 2) && atomicAdd(a.ddone + b, 1) == T2 - 1) run_d |= all_rows ? 2 : 3;
                if (all_rows && atomicAdd(a.p2done + b, 1) == need - 1) run_d |= 1;
            }
            run_d = __shfl_sync(0xffffffffu, run_d, 0);
            if (run_d) draw_setup_warp<TVO>(a, S, b, run_d);
        }
        // the producer stays until every streaming task has been dealt with here (mailbox entries come first)
        __syncwarp();
        if (lane == 0) { __threadfence_block(); *(volatile int*)&S.pub_count = *(volatile int*)&S.pub_count + 1; }
    }
}

}  // namespace

template <int DT, int MODE>
__global__ void __launch_bounds__(PT, PIPE_CTAS) k_pipe(const __grid_constant__ PipeArgs a) {
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* data = smem;
    PipeShared& S = *reinterpret_cast<PipeShared*>(smem + (size_t)NST * STAGE_BYTES);
    const int tid = threadIdx.x;
    // the re-draw kernel behind this one may be scheduled as CTAs of this one leave (programmatic dependent
    // launch); it follows the list of sequences as it grows (`fb_count` tells it when the list is complete)
    if (tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) {
        for (int i = 0; i < NST; ++i) { mbar_init(&S.full[i], 1); mbar_init(&S.empty[i], WW + 1); mbar_init(&S.pdone[i], WW); }
        mbar_init(&S.dsync, WW);
        S.mb_tail = 0; S.mb_head = 0; S.pub_count = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (tid >= PC) {
        if (tid == PC) producer<DT, MODE>(a, S, data);
        else if (tid >= PC + 32) publisher<DT, MODE>(a, S);
        return;
    }
    const int lane = tid & 31;
    uint32_t meet = 0;
    for (int it = 0;; ++it) {
        const int stage = it % NST;
        const uint32_t par = (uint32_t)(it / NST) & 1u;
        if (!mbar_wait(&S.full[stage], par)) { if (tid == 0) atomicExch(a.wait_failed, 1); break; }
        const TaskDesc d = S.desc[stage];
        if (d.phase < 0) break;
        const unsigned char* sd = data + (size_t)stage * STAGE_BYTES;
        if (MODE == kModeGreedy) pipe_g<DT>(a, S, d, sd, stage);
        else if (d.phase == 0) pipe_p1<DT>(a, S, d, sd, stage);
        else if (d.phase == 2) pipe_p2<DT, MODE == kModeTv>(a, S, d, sd, stage);
        else {
            pipe_d<DT>(a, S, d, sd, meet);
            consumers_meet(a.wait_failed, &S.dsync, meet);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&S.empty[stage]);
    }
}

// -----------------------------------------------------------------------------
namespace {

constexpr size_t kPipeSmem = (size_t)NST * STAGE_BYTES + sizeof(PipeShared);

template <int DT, int MODE>
int pipe_grid() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (dev >= 0 && dev < 64 && cached[dev]) return cached[dev];
    if (cudaFuncSetAttribute(k_pipe<DT, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPipeSmem) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    int per_sm = 0, sms = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_pipe<DT, MODE>, PT, kPipeSmem) != cudaSuccess) per_sm = 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaGetLastError();
    const int n = per_sm * sms;
    if (dev >= 0 && dev < 64) cached[dev] = n;
    return n;
}

}  // namespace

extern cudaEvent_t g_ev_start, g_ev_stop;

bool pipe_supported(const RowArgs& a) {
    const int T = (a.nvec + PSLICE - 1) / PSLICE;
    return T >= 1 && T <= MAX_SLICES && a.K <= BEBOP_MAX_K_INT;
}

cudaError_t pipe_verify(const RowArgs& a, const Plan& p, const int32_t* draft_tokens,
                        const float* u_accept, const float* u_final, VerifyOut o, char* ws,
                        cudaStream_t stream, bool* launched, bool tv_only, float* s_aux) {
    *launched = false;
    const int grid_max = tv_only ? (a.dt == 0 ? pipe_grid<0, kModeTv>() : pipe_grid<1, kModeTv>())
                                 : (a.dt == 0 ? pipe_grid<0, kModeVerify>() : pipe_grid<1, kModeVerify>());
    if (grid_max < 1) return cudaSuccess;
    const PipePlan wp = make_pipe_plan(a.B, a.K, a.nvec, a.dt, PSLICE);
    PipeArgs wa;
    wa.r = a; wa.draft_tokens = draft_tokens; wa.u_accept = u_accept; wa.u_final = u_final; wa.o = o;
    wa.stop = reinterpret_cast<int*>(ws + p.off_stop);
    char* w = ws + p.off_pipe;
    wa.fb_count = reinterpret_cast<unsigned long long*>(w + kFbCountOffset);
    wa.fb_list = reinterpret_cast<FbRec*>(w + wp.off_fbrec);
    wa.ticket = reinterpret_cast<int*>(w);
    wa.wait_failed = wa.ticket + 1;
    wa.p1done = reinterpret_cast<int*>(w + wp.off_p1done);
    wa.p2done = reinterpret_cast<int*>(w + wp.off_p2done);
    wa.ddone = reinterpret_cast<int*>(w + wp.off_ddone);
    wa.rowcnt = reinterpret_cast<int*>(w + wp.off_rowcnt);
    wa.part = reinterpret_cast<P1Part*>(w + wp.off_part);
    wa.rstat = reinterpret_cast<RowStat*>(w + wp.off_rstat);
    wa.dacc = reinterpret_cast<unsigned long long*>(w + wp.off_dpart);
    wa.tvacc = reinterpret_cast<unsigned long long*>(w + wp.off_tvacc);
    wa.sinfo = reinterpret_cast<SeqInfo*>(w + wp.off_sinfo);
    const int expire = take_expire_wait();
    wa.expire = expire == 2 ? 1 : 0;
    wa.kappa = draw_kappa();
    wa.tv_only = tv_only ? 1 : 0;
    wa.s_aux = tv_only ? s_aux : nullptr;
    wa.sacc = (tv_only && s_aux) ? reinterpret_cast<unsigned long long*>(w + wp.off_sacc) : nullptr;
    wa.T = wp.T; wa.slice_vecs = wp.slice_vecs;
    {
        const long long NR = 2 * a.K + 1;
        const long long total = (long long)a.B * (NR * wp.T + (long long)(tv_only ? a.K : (o.tv ? a.K + 1 : 1)) * 2 * wp.T);
        if (total > 0x7fff0000LL) return cudaSuccess;
        wa.ntickets = (int)total;
    }
    cudaError_t e = cudaMemsetAsync(w, 0, wp.zero_bytes, stream);
    if (e != cudaSuccess) return e;
    const int grid = wa.ntickets < grid_max ? wa.ntickets : grid_max;
    if (g_ev_start) cudaEventRecord(g_ev_start, stream);
    if (tv_only) {
        if (a.dt == 0) k_pipe<0, kModeTv><<<grid, PT, kPipeSmem, stream>>>(wa);
        else k_pipe<1, kModeTv><<<grid, PT, kPipeSmem, stream>>>(wa);
    } else {
        if (a.dt == 0) k_pipe<0, kModeVerify><<<grid, PT, kPipeSmem, stream>>>(wa);
        else k_pipe<1, kModeVerify><<<grid, PT, kPipeSmem, stream>>>(wa);
    }
    e = cudaGetLastError();
    if (g_ev_stop) cudaEventRecord(g_ev_stop, stream);
    if (e != cudaSuccess) return e;
    *launched = true;
    return redraw_launch(a, u_final, o, wa.fb_count, wa.fb_list, tv_only ? 0 : a.B, wa.wait_failed, w, wp, stream, expire == 1);
}

// ------------------------------------------------------------------ greedy mode
namespace {

// One warp per sequence, behind the sweep: lane k merges the slice records of target row k (maximum, lowest
// index), then the argmax match x_k == g_k runs down the drafts; the argmax of the stop position is emitted.
__global__ void __launch_bounds__(128) k_greedy_finish(PipeArgs a, int32_t* __restrict__ accept_len,
                                                        int32_t* __restrict__ out_tokens, int32_t* __restrict__ row_status) {
    asm volatile("griddepcontrol.wait;" ::: "memory");       // programmatic dependent of the sweep
    const RowArgs& R = a.r;
    const int b = (int)((blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5);
    const int lane = threadIdx.x & 31;
    if (b >= R.B) return;
    const int K = R.K, L = len_of(R, b), NR = 2 * K + 1;
    int st = *a.wait_failed ? ST_WAIT : 0;
    const int tok = lane < L ? a.draft_tokens[(int64_t)b * K + lane] : -1;
    if (lane < L && (tok < 0 || tok >= R.V)) st |= ST_BAD_TOKEN;
    // lanes 0..L merge the target rows 0..L (two rounds when L + 1 > 32)
    int g = -1, g_bonus = -1;
    for (int round = 0; round < 2; ++round) {
        const int k = round == 0 ? lane : 32 + lane;
        if (k <= L && k <= K) {
            const P1Part* pp = a.part + ((int64_t)b * NR + k) * a.T;
            float best = -INFINITY; int bidx = INT_MAX;
            for (int s = 0; s < a.T; ++s) {
                const P1Part rec = pp[s];
                if (rec.m != rec.m) { best = rec.m; break; }
                if (rec.m > best) { best = rec.m; bidx = (int)rec.s; }        // slices ascend: the lowest index wins a tie
            }
            if (best != best) st |= ST_NONFINITE;
            else if (best == -INFINITY) st |= ST_EMPTY;
            if (round == 0) g = bidx; else g_bonus = bidx;
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) st |= __shfl_xor_sync(0xffffffffu, st, off);
    if (st & ST_FATAL) {
        if (lane <= K) out_tokens[(int64_t)b * (K + 1) + lane] = -1;
        if (K == 32 && lane == 0) out_tokens[(int64_t)b * (K + 1) + 32] = -1;
        if (lane == 0) { accept_len[b] = 0; if (row_status) row_status[b] = st; }
        return;
    }
    const unsigned mis = __ballot_sync(0xffffffffu, lane < L && tok != g);
    const int n = mis ? (__ffs(mis) - 1) : L;
    const int y = n < 32 ? __shfl_sync(0xffffffffu, g, n & 31) : __shfl_sync(0xffffffffu, g_bonus, 0);
    if (lane <= K && lane < 32) out_tokens[(int64_t)b * (K + 1) + lane] = lane < n ? tok : (lane == n ? y : -1);
    if (K == 32 && lane == 0) out_tokens[(int64_t)b * (K + 1) + 32] = (n == 32) ? y : -1;
    if (lane == 0) { accept_len[b] = n; if (row_status) row_status[b] = st; }
}

}  // namespace

cudaError_t pipe_greedy(const RowArgs& a, const Plan& p, const int32_t* draft_tokens, int32_t* accept_len,
                        int32_t* out_tokens, int32_t* row_status, char* ws, cudaStream_t stream, bool* launched) {
    *launched = false;
    const int grid_max = a.dt == 0 ? pipe_grid<0, kModeGreedy>() : pipe_grid<1, kModeGreedy>();
    if (grid_max < 1) return cudaSuccess;
    const PipePlan wp = make_pipe_plan(a.B, a.K, a.nvec, a.dt, PSLICE);
    const long long total = (long long)a.B * (a.K + 1) * wp.T;
    if (total > 0x7fff0000LL) return cudaSuccess;
    char* w = ws + p.off_pipe;
    PipeArgs wa = {};
    wa.r = a; wa.draft_tokens = draft_tokens;
    wa.ticket = reinterpret_cast<int*>(w);
    wa.wait_failed = wa.ticket + 1;
    wa.part = reinterpret_cast<P1Part*>(w + wp.off_part);
    wa.T = wp.T; wa.slice_vecs = wp.slice_vecs;
    wa.ntickets = (int)total;
    cudaError_t e = cudaMemsetAsync(w, 0, 256, stream);       // ticket counter and wait flag
    if (e != cudaSuccess) return e;
    const int grid = wa.ntickets < grid_max ? wa.ntickets : grid_max;
    if (a.dt == 0) k_pipe<0, kModeGreedy><<<grid, PT, kPipeSmem, stream>>>(wa);
    else k_pipe<1, kModeGreedy><<<grid, PT, kPipeSmem, stream>>>(wa);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    *launched = true;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((a.B + 3) / 4); cfg.blockDim = dim3(128); cfg.dynamicSmemBytes = 0; cfg.stream = stream;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_greedy_finish, wa, accept_len, out_tokens, row_status);
}

}  // namespace bebop
