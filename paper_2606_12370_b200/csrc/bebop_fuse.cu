// Fused kernel: bebop_verify and bebop_tv with every logit row read from memory once and exponentiated once.
//
// A row (pair) is cut into T slices of at most FSV 16-byte vectors; a task is one slice of a row pair (target row
// k, draft row k of a sequence: a "unit") or two slices of a sequence's bonus row.  Tasks are dealt round robin
// over a grid that is resident as a whole (one CTA per SM), so the T slices of a unit are in the hands of T
// different CTAs at about the same time.  Per task, a CTA
//   pass 1  takes the slice from shared memory (bulk copies, a ring of stages), forms e = 2^(x c - E) around an
//           integer reference exponent E per warp, parks the e of both rows in TENSOR MEMORY (this path has no
//           contraction, so the 256 KB of TMEM per SM are free to serve as a store), and publishes the
//           slice's softmax partial (E, sum e) as a record in global memory;
//   stats   (a few tasks later) finds the T records of the unit, merges them -- exact power-of-two scalings,
//           one fixed order, so every CTA gets the same bits -- and so knows both normalisers S_p, S_q;
//   pass 2  (three tasks behind pass 1: the depth of the TMEM ring hides the exchange) takes its e back from
//           TMEM and forms r' = max(0, e_p - rho e_q), rho = S_p / S_q as two floats scaled to the warp's
//           exponents: the residual p - q up to the factor 1 / S_p, which is applied once per warp chunk, in
//           double.  The chunk and slice masses give TV (their sum) and the inverse CDF of the draw (it walks
//           them); for bebop_tv the auxiliary sum of Eq. tv_grad goes with them.
// The consumer warps neither shuffle nor wait for each other: a thread leaves its partial sums in shared
// memory and publisher warps add them up.  When a CTA has run out of tasks, its consumer warps complete
// sequences, one warp each: run the accept scan (Algorithm 3) on the merged rows, write TV, locate the slice and
// the warp chunk that own the target u Z of the inverse CDF, evaluate that chunk's tokens again and keep the
// token if the crossing clears the error bound; else the sequence is listed for the fp64 re-draw kernel.
//
// Warps: 16 consumers, producer, publisher of the softmax partials, two publishers of the masses, four stats
// warps (stats warp j serves the tasks n = j mod 4, so that the latency of one merge does not bound the task rate).
// What CTAs pass to each other: records of two 8-byte words, each word valid by itself once non-zero (the memory
// is zeroed per call), written and read by relaxed 64-bit accesses; and the per-sequence count of delivered
// parts, added after a fence and read with acquire.  Every wait is bounded and sleeps between looks (a waiting
// warp that spins takes issue slots from the warp it waits for); one that gives up sets the wait flag and lets
// the CTA run out without further waits.  No cluster, no multicast.
#include "bebop_pipe.cuh"

namespace bebop {

namespace {

constexpr int FV = BEBOP_FUSE_VPT;            // vectors per thread, row and task
constexpr int FCW = kFuseWarps;               // consumer warps = warp chunks of a slice
constexpr int FCT = FCW * 32;
constexpr int FSV = kFuseSliceVecs;           // vectors per slice, at most
static_assert(FSV == FCT * FV && FCW == 16 && FV == 2, "slice size, consumer threads, TMEM columns per warp");
constexpr int FSTAGE = 2 * FSV * 16;          // bytes of one stage: target slice, draft slice
constexpr int FNS = 4;                        // stages of the shared-memory ring
constexpr int FRING = 16;                     // task descriptions in flight
constexpr int FND = 4;                        // tasks whose exponentials TMEM holds (32 columns per warp and task)
constexpr int FLAG = FND - 1;                 // pass 2 runs this many tasks behind pass 1
constexpr int FNSW = 4;                       // stats warps
constexpr int FR8 = 8;                        // ring of what lives from a task's pass 1 to the publication of its pass 2
constexpr int FNPB = 2;                       // publishers of the masses (the fence before a sequence's count takes a while)
constexpr int W_PROD = FCW, W_PUBA = FCW + 1, W_PUBB = FCW + 2, W_STAT0 = W_PUBB + FNPB;
constexpr int FT = (W_STAT0 + FNSW) * 32;     // threads per CTA
static_assert(FNPB <= FNSW, "the end is marked in FNSW descriptions");
constexpr int FTCOLS = 512;                   // TMEM columns of a CTA
constexpr int FEPL = FCT / 32;                // thread partials a publisher lane adds up
constexpr int FLPC = 32 / FCW;                // publisher lanes per warp chunk
static_assert(FLPC == 2, "publisher lanes and warp chunks");

constexpr int FPAD = FCT + FCT / FEPL;        // partial-sum arrays: one entry of padding per publisher lane (bank conflicts)
constexpr int kPair = 0, kBonus = 1, kStop = -1;
constexpr uint32_t kFBarSpin = 1u << 20;
constexpr unsigned kFSleep = 1024;            // ns between two looks of a consumer's wait
constexpr unsigned kFSleepHelper = 100;       // ... of a helper warp's wait

template <int DT> struct FuseDims {
    static constexpr int VEC = Elem<DT>::VEC;
    static constexpr int NVAL = FV * 2 * VEC;         // exponentials per thread and task = TMEM columns used
    static_assert(NVAL == 16 || NVAL == 32, "TMEM access shapes");
};

// A pair task is slice s of target row k and draft row k.  A bonus task is TWO slices, s and s + 1, of the bonus row
// (the stage's second half, the draft row's place, takes the second slice), so that the bonus row costs per byte
// what the row pairs cost: nv then holds both slices' vector counts (low and high 16 bits), and the ragged vector's
// place counts on through both slices (FSV + i: vector i of the second).
struct __align__(16) FTask {
    int kind, nv, tailv;                    // tailv: the slice's vector that holds the row's ragged end (-1: none)
    float c;                                // log2(e) / tau of the sequence
    int b, k, s, unit;
};
// what the publication of a task's pass 2 needs: the rows' exponents and normalisers
struct __align__(16) FScale { double inv_p, inv_q; int ep, eq; float rho_h, rho_l; int stp, stq, pad0, pad1; };
struct __align__(16) FWarpE { int ep, eq, flags, pad; };               // a consumer warp's exponents of a task
// Softmax partial of one slice of one row; each 8-byte word is valid by itself once non-zero.  `flags`: bit 0 says
// that the slice holds a NaN or +inf; the other bits are those of a float u, with which the slice's sum of e^2
// (around the slice's exponent) is at most sqrt(2) u: u = sum over the warp chunks of 4^(E_w - E_s) times the
// chunk's sum of e, as the e of a chunk are at most sqrt(2) around the chunk's own exponent.
struct __align__(16) FRec { double s; int ecode; int flags; };
__device__ __forceinline__ float rec_ub(const FRec& r) { return __int_as_float(r.flags & ~1); }
struct __align__(16) FRow { double inv_s; int e; int st; };           // a merged row: 1/S, exponent, status bits
struct FRho { float h, l; };

struct FuseArgs {
    RowArgs r;
    const int32_t* draft_tokens;
    const float* u_accept;
    const float* u_final;
    VerifyOut o;
    float* s_aux;
    int tv_mode;
    int ups;                 // units per sequence: K + 1 (row pairs, bonus row), or 1 for bebop_tv
    int tps;                 // tasks per sequence: K T for the row pairs and (T + 1) / 2 for the bonus row, or T for bebop_tv
    int T, slice_vecs;
    int expire;              // test hook: the stats warps' wait for a unit's records counts as run out
    float kappa;             // factor of the fast draw's error bound
    int* wait_failed;
    unsigned long long* fb_count;
    FbRec* fb_list;
    int* seqcnt;             // [B] parts of the sequence delivered
    FRec* rec;               // [units][T][2]
    double* mass;            // [units][T][FCW] residual mass per warp chunk (bonus row: sum of e around the warp's exponent)
    int2* wexp;              // [units][T][FCW] the warps' reference exponents (target row, draft row)
    double* sauxp;           // [units][T] bebop_tv: sum of q over the tokens with q <= p
    double* smass;           // [units][T] residual mass of the slice (row pairs)
    FRow* rows;              // [units][2] the merged rows of a row pair (written with its slice 0)
};

struct FShared {
    unsigned long long full[FNS], empty[FNS];
    unsigned long long dready[FRING];
    unsigned long long iter[4];              // one phase per iteration of the consumers: the threads' sums are in place
    unsigned long long sfree[4];             // ... both publishers have read them
    unsigned long long stats[4];             // one phase per task: rho of the task is in place
    unsigned long long bdone[FR8];           // one phase per task: the publisher of the softmax partials is through with it
    float2 bsum[FR8][FCW];                   // bonus task: the chunks' sums of e (around the warps' exponents), both slices
    FTask task[FRING];
    FScale scale[FR8];
    FRho rho[FR8][FCW];
    FWarpE we[FR8][FCW];
    float2 p1t[4][FPAD];                     // per thread: sums of e (target row, draft row)
    float2 p2t[4][FPAD];                     // per thread: sum r', sum of e_q where q <= p
    uint32_t tmem_base;
    int abort;
};

// ------------------------------------------------------------------ PTX helpers
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
__device__ __forceinline__ bool mbar_try(uint32_t addr, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
    return ok != 0;
}
// bounded; gives up at once when the CTA has already given up somewhere
__device__ __noinline__ bool mbar_wait_slow(FShared& S, uint32_t addr, uint32_t parity) {
    for (uint32_t i = 0; i < kFBarSpin; ++i) {
        if (*(volatile int*)&S.abort) return false;
        __nanosleep(kFSleep);
        if (mbar_try(addr, parity)) return true;
    }
    return false;
}
// the first look is inline (a barrier that is already complete costs one instruction); the wait itself is a call
__device__ __forceinline__ bool mbar_wait(FShared& S, unsigned long long* b, uint32_t parity) {
    const uint32_t addr = smem_u32(b);
    if (mbar_try(addr, parity)) return true;
    return mbar_wait_slow(S, addr, parity);
}
// the helper warps' wait: they are few, and what they wait for is what the consumers wait for next, so they look often
__device__ __noinline__ bool mbar_wait_helper_slow(FShared& S, uint32_t addr, uint32_t parity) {
    for (uint32_t i = 0; i < 4u * kFBarSpin; ++i) {
        if (*(volatile int*)&S.abort) return false;
        __nanosleep(kFSleepHelper);
        if (mbar_try(addr, parity)) return true;
    }
    return false;
}
__device__ __forceinline__ bool mbar_wait_helper(FShared& S, unsigned long long* b, uint32_t parity) {
    const uint32_t addr = smem_u32(b);
    if (mbar_try(addr, parity)) return true;
    return mbar_wait_helper_slow(S, addr, parity);
}
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, unsigned long long* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ uint4 lds16(const unsigned char* p) { return *reinterpret_cast<const uint4*>(p); }
__device__ __forceinline__ float set_ge0(float d) {          // 1.0 where d >= 0, else 0.0
    float m; asm("set.ge.f32.f32 %0, %1, 0f00000000;" : "=f"(m) : "f"(d)); return m;
}

__device__ __forceinline__ void tmem_alloc(uint32_t* dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(dst)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(taddr), "r"(ncols) : "memory");
}
// N consecutive 32-bit columns of this thread's TMEM lane
template <int N> __device__ __forceinline__ void tmem_st(uint32_t t, const float* v) {
    static_assert(N == 16 || N == 32, "shape");
#pragma unroll
    for (int h = 0; h < N; h += 16)
        asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
                     :: "r"(t + h), "r"(__float_as_uint(v[h + 0])), "r"(__float_as_uint(v[h + 1])), "r"(__float_as_uint(v[h + 2])),
                        "r"(__float_as_uint(v[h + 3])), "r"(__float_as_uint(v[h + 4])), "r"(__float_as_uint(v[h + 5])),
                        "r"(__float_as_uint(v[h + 6])), "r"(__float_as_uint(v[h + 7])), "r"(__float_as_uint(v[h + 8])),
                        "r"(__float_as_uint(v[h + 9])), "r"(__float_as_uint(v[h + 10])), "r"(__float_as_uint(v[h + 11])),
                        "r"(__float_as_uint(v[h + 12])), "r"(__float_as_uint(v[h + 13])), "r"(__float_as_uint(v[h + 14])),
                        "r"(__float_as_uint(v[h + 15])) : "memory");
}
template <int N> __device__ __forceinline__ void tmem_ld(uint32_t t, float* v) {
    static_assert(N == 16 || N == 32, "shape");
    uint32_t r[N];
#pragma unroll
    for (int h = 0; h < N; h += 16)
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                     : "=r"(r[h + 0]), "=r"(r[h + 1]), "=r"(r[h + 2]), "=r"(r[h + 3]), "=r"(r[h + 4]), "=r"(r[h + 5]), "=r"(r[h + 6]),
                       "=r"(r[h + 7]), "=r"(r[h + 8]), "=r"(r[h + 9]), "=r"(r[h + 10]), "=r"(r[h + 11]), "=r"(r[h + 12]), "=r"(r[h + 13]),
                       "=r"(r[h + 14]), "=r"(r[h + 15]) : "r"(t + h) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < N; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// a record as it stands now; valid once both words are non-zero
__device__ __forceinline__ bool ld_rec(const FRec* p, FRec* v) {
    unsigned long long w0, w1;
    asm volatile("ld.relaxed.gpu.global.v2.b64 {%0, %1}, [%2];" : "=l"(w0), "=l"(w1) : "l"(p) : "memory");
    v->s = __longlong_as_double((long long)w0);
    v->ecode = (int)(unsigned)(w1 & 0xffffffffull);
    v->flags = (int)(unsigned)(w1 >> 32);
    return w0 != 0ull && w1 != 0ull;
}
__device__ __forceinline__ int ld_relaxed(const int* p) {
    int v; asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory"); return v;
}
__device__ __forceinline__ void give_up(const FuseArgs& a, FShared& S) {
    atomicExch(a.wait_failed, 1);
    *(volatile int*)&S.abort = 1;
}
__device__ __forceinline__ bool aborted(const FShared& S) { return *(volatile const int*)&S.abort != 0; }

// ------------------------------------------------------------------ merged rows
// Merge the T slice records of the rows of `unit` (a full warp; lane l takes slices l, l + 32, ...).  The records'
// sums are scaled to the largest exponent by powers of two (exactly) and added in one fixed order, so every
// warp that merges the same records gets the same bits.  Waits (bounded) for records not there yet.
template <int SPL>
__device__ __forceinline__ void merge_rows_n(const FuseArgs& a, FShared& S, int unit, int rows, FRow* out_p, FRow* out_q) {
    const int lane = threadIdx.x & 31, T = a.T;
    const FRec* base = a.rec + ((int64_t)unit * T) * 2;
    // every record this lane needs is asked for at once, and asked for again (all that are still missing, together)
    // until it is there
    FRec r[SPL][2];
    unsigned missing = 0;
#pragma unroll
    for (int i = 0; i < SPL; ++i)
#pragma unroll
        for (int w = 0; w < 2; ++w) {
            r[i][w].s = 0.0; r[i][w].ecode = 2 * E_EMPTY + 1; r[i][w].flags = 0;
            if (lane + 32 * i < T && w < rows) missing |= 1u << (2 * i + w);
        }
    for (uint32_t it = 0; it < kSpin; ++it) {
#pragma unroll
        for (int i = 0; i < SPL; ++i)
#pragma unroll
            for (int w = 0; w < 2; ++w)
                if (missing & (1u << (2 * i + w))) { if (ld_rec(base + 2 * (lane + 32 * i) + w, &r[i][w])) missing &= ~(1u << (2 * i + w)); }
        if (!__any_sync(0xffffffffu, missing != 0)) break;
        if ((it & 63u) == 63u && (aborted(S) || ld_relaxed(a.wait_failed))) break;
        __nanosleep(200);
    }
    if (__any_sync(0xffffffffu, missing != 0)) {
        give_up(a, S);
#pragma unroll
        for (int i = 0; i < SPL; ++i)
#pragma unroll
            for (int w = 0; w < 2; ++w) if (missing & (1u << (2 * i + w))) { r[i][w].s = 0.0; r[i][w].ecode = 2 * E_EMPTY + 1; r[i][w].flags = 0; }
    }
    int el[2] = {E_EMPTY, E_EMPTY}, fl = 0;
#pragma unroll
    for (int i = 0; i < SPL; ++i)
#pragma unroll
        for (int w = 0; w < 2; ++w) { el[w] = max(el[w], (r[i][w].ecode - 1) >> 1); fl |= (r[i][w].flags & 1) << w; }
    const int Em[2] = {redux_max(el[0]), redux_max(el[1])};
    fl = __reduce_or_sync(0xffffffffu, fl);
    double v[2] = {0.0, 0.0};
#pragma unroll
    for (int i = 0; i < SPL; ++i)
#pragma unroll
        for (int w = 0; w < 2; ++w) {
            const int e = (r[i][w].ecode - 1) >> 1;
            if (e > E_EMPTY) v[w] += r[i][w].s * pow2d(max(e - Em[w], -1000));
        }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { v[0] += shfl_xor_d(v[0], o); v[1] += shfl_xor_d(v[1], o); }
#pragma unroll
    for (int w = 0; w < 2; ++w) {
        FRow x;
        int st = 0;
        if (((fl >> w) & 1) || !(v[w] == v[w])) st = ST_NONFINITE; else if (Em[w] == E_EMPTY) st = ST_EMPTY;
        x.inv_s = (!st && v[w] > 0.0) ? 1.0 / v[w] : 0.0; x.e = Em[w]; x.st = st;
        if (w == 0) *out_p = x; else if (rows > 1) *out_q = x;
    }
}
__device__ __noinline__ void merge_rows(const FuseArgs& a, FShared& S, int unit, int rows, FRow* out_p, FRow* out_q) {
    if (a.T <= 32) merge_rows_n<1>(a, S, unit, rows, out_p, out_q);
    else if (a.T <= 64) merge_rows_n<2>(a, S, unit, rows, out_p, out_q);
    else merge_rows_n<kFuseMaxSlices / 32>(a, S, unit, rows, out_p, out_q);
}

// rho = S_p / S_q as two floats; pass 2 forms r' = max(0, e_p - rho e_q) = (p - q) S_p 2^(E_p - E_wp)
__device__ __forceinline__ FScale scale_of(const FRow& rp, const FRow& rq) {
    FScale sc;
    sc.inv_p = rp.inv_s; sc.inv_q = rq.inv_s; sc.ep = rp.e; sc.eq = rq.e; sc.stp = rp.st; sc.stq = rq.st; sc.pad0 = 0; sc.pad1 = 0;
    const double rho = rp.inv_s > 0.0 ? rq.inv_s / rp.inv_s : 0.0;
    sc.rho_h = (float)rho; sc.rho_l = (float)(rho - (double)sc.rho_h);
    return sc;
}
// the warp's rho: e_p sits around E_wp, e_q around E_wq, so rho takes the factor 2^((E_wq - E_rq) - (E_wp - E_rp))
// (exact; a chunk whose target or draft part is empty has no such factor: its e are all zero)
__device__ __forceinline__ FRho warp_rho(const FScale& sc, int ewp, int ewq) {
    int k = 0;
    if (ewp > E_EMPTY && ewq > E_EMPTY && sc.ep > E_EMPTY && sc.eq > E_EMPTY) k = (ewq - sc.eq) - (ewp - sc.ep);
    k = max(min(k, 126), -126);
    const float f = pow2f(k);
    FRho r; r.h = sc.rho_h * f; r.l = sc.rho_l * f;
    return r;
}
// the factor that turns the chunk's sum of r' (or of e) into probability mass: 2^(E_wp - E_rp) / S_p
__device__ __forceinline__ double chunk_scale(double inv_s, int e_row, int e_warp) {
    return e_warp > E_EMPTY && e_row > E_EMPTY ? pow2d(max(e_warp - e_row, -1000)) * inv_s : 0.0;
}

// ------------------------------------------------------------------ producer
// One thread.  A sequence has `tps` tasks: slice s of row pair k for k = 0 .. K - 1, s = 0 .. T - 1, then the bonus
// row two slices at a time; CTA i takes the tasks i, i + grid, ... and skips those of positions past the sequence's
// draft length.  What the next task needs from memory (draft length, temperature) is asked for one task ahead.
struct FNext { int t, b, k, s, L, bonus; float tau; };
__device__ __forceinline__ FNext f_fetch(const FuseArgs& a, int t) {
    const RowArgs& R = a.r;
    FNext x;
    x.t = t;
    x.b = t / a.tps;
    const int r = t - x.b * a.tps;
    x.L = a.tv_mode ? 1 : len_of(R, x.b);
    x.tau = tau_of(R, x.b);
    const int npair = a.tv_mode ? a.tps : R.K * a.T;
    if (r < npair) { x.k = r / a.T; x.s = r - x.k * a.T; x.bonus = 0; }
    else { x.k = x.L; x.s = 2 * (r - npair); x.bonus = 1; }
    return x;
}
template <int DT>
__device__ __forceinline__ void f_producer(const FuseArgs& a, FShared& S, unsigned char* data, int total) {
    constexpr int VEC = Elem<DT>::VEC;
    const RowArgs& R = a.r;
    const int K = R.K, grid = (int)gridDim.x;
    const int tail_tokens = R.V - (R.nvec - 1) * VEC;            // tokens of the row's last vector
    const int tail_vec = tail_tokens < VEC ? R.nvec - 1 : -1;    // the row's ragged vector, if any
    int n = 0;
    long long t = (long long)blockIdx.x;
    FNext nx;
    nx.t = -1;
    if (t < total) nx = f_fetch(a, (int)t);
    while (nx.t >= 0 && !aborted(S)) {
        const FNext cur = nx;
        t += grid;
        if (t < total) nx = f_fetch(a, (int)t); else nx.t = -1;
        if (!cur.bonus && !a.tv_mode && cur.k >= cur.L) continue;     // a position past the sequence's draft length
        const int slot = n % FRING, stage = n % FNS;
        if (!mbar_wait_helper(S, &S.empty[stage], (((uint32_t)(n / FNS)) & 1u) ^ 1u)) { give_up(a, S); break; }
        const int kind = cur.bonus ? kBonus : kPair;
        const int v0 = cur.s * a.slice_vecs, nv = max(min(a.slice_vecs, R.nvec - v0), 0);
        const int v1 = v0 + a.slice_vecs, nv1 = (cur.bonus && cur.s + 1 < a.T) ? max(min(a.slice_vecs, R.nvec - v1), 0) : 0;
        int tv = tail_vec - v0;
        if (tv < 0 || tv >= nv) { tv = tail_vec - v1; tv = (tv >= 0 && tv < nv1) ? FSV + tv : -1; }
        int4* d = reinterpret_cast<int4*>(&S.task[slot]);
        d[0] = make_int4(kind, cur.bonus ? (nv | (nv1 << 16)) : nv, tv, __float_as_int(temp_scale(cur.tau).hi));
        d[1] = make_int4(cur.b, cur.k, cur.s, cur.b * a.ups + cur.k);
        mbar_arrive(&S.dready[slot]);
        const uint32_t bytes = (uint32_t)nv * 16u, bytes1 = (uint32_t)nv1 * 16u;
        if (bytes) {
            unsigned char* dst = data + (size_t)stage * FSTAGE;
            const char* row = row_ptr(R, cur.b, cur.k);
            mbar_arrive_expect(&S.full[stage], kind == kPair ? 2u * bytes : bytes + bytes1);
            bulk_load(dst, row + (int64_t)v0 * 16, bytes, &S.full[stage]);
            if (kind == kPair) bulk_load(dst + FSTAGE / 2, row_ptr(R, cur.b, K + 1 + cur.k) + (int64_t)v0 * 16, bytes, &S.full[stage]);
            else if (bytes1) bulk_load(dst + FSTAGE / 2, row + (int64_t)v1 * 16, bytes1, &S.full[stage]);
        } else mbar_arrive(&S.full[stage]);
        ++n;
    }
    // the end: every stats warp must meet it (stats warp j looks at the tasks j mod 4), the consumers once
    for (int i = 0; i < FNSW; ++i) {
        const int slot = (n + i) % FRING;
        reinterpret_cast<int4*>(&S.task[slot])[0] = make_int4(kStop, 0, 0, 0);
        mbar_arrive(&S.dready[slot]);
    }
    if (mbar_wait_helper(S, &S.empty[n % FNS], (((uint32_t)(n / FNS)) & 1u) ^ 1u)) mbar_arrive(&S.full[n % FNS]);
}

// ------------------------------------------------------------------ consumers
// Reference exponent of a warp chunk from its maximum m: the integer nearest to m c (any integer near it serves),
// found by adding 1.5 * 2^23.  The sum y = m c + 1.5 * 2^23 of a finite m with |m c| < 2^22 lies in [2^23, 2^24):
// a positive float whose bit pattern grows with its value, so the warp's maximum is one integer reduction, and
// everything that is not the usual case -- NaN or +inf (bits above the range), -inf in every lane (negative),
// huge logits -- shows as a result outside [kYLo, kYHi] and takes the slow way.
constexpr float kMagic = 12582912.f;                  // 1.5 * 2^23
constexpr int kMagicBits = 0x4B400000;
constexpr int kYLo = 0x4B000000, kYHi = 0x4B7FFFFF;   // bit patterns of 2^23 and of the float below 2^24
struct FExp { int e; float ef; int bad; };
__device__ __noinline__ FExp warp_exponent_slow(float m, float c) {
    // m: this lane's maximum (the warp's is found here, in the order-preserving integer map that puts NaN on top)
    const float mw = ord2f(redux_max(f2ord(m)));
    FExp x;
    x.bad = !(mw < INFINITY);
    x.ef = 0.f; x.e = E_EMPTY;
    if (x.bad || mw == -INFINITY) return x;            // around 0 the chunk's -inf logits give e = 0
    const float th = fminf(fmaxf(mw * c, -4.0e6f), 4.0e6f);
    const float y = th + kMagic;
    x.ef = y - kMagic;
    x.e = __float_as_int(y) - kMagicBits;
    return x;
}
__device__ __forceinline__ FExp warp_exponent(float m, float c) {
    const int yi = redux_max(__float_as_int(fmaf(m, c, kMagic)));
    if (yi < kYLo || yi > kYHi) return warp_exponent_slow(m, c);
    FExp x;
    x.e = yi - kMagicBits; x.ef = __int_as_float(yi) - kMagic; x.bad = 0;
    return x;
}

// the exponentials of one vector around exponent Ef, two at a time
template <int DT>
__device__ __forceinline__ void exp_vec(const uint4& raw, float c, float Ef, float* e) {
    constexpr int VEC = Elem<DT>::VEC;
    float f[VEC];
    unpack<DT>(raw, f);
    const float2 c2 = make_float2(c, c), m2 = make_float2(-Ef, -Ef);
#pragma unroll
    for (int i = 0; i < VEC; i += 2) {
        const float2 t = __ffma2_rn(make_float2(f[i], f[i + 1]), c2, m2);
        e[i] = ex2f(t.x);
        e[i + 1] = ex2f(t.y);
    }
}
// sum of N floats, two at a time (one fixed order)
template <int N> __device__ __forceinline__ float sum_fixed(const float* e) {
    float2 acc = make_float2(e[0], e[1]);
#pragma unroll
    for (int i = 2; i < N; i += 2) acc = __fadd2_rn(acc, make_float2(e[i], e[i + 1]));
    return acc.x + acc.y;
}
// Residuals of N token pairs from their exponentials: d = e_p - rho e_q, rho as two floats, each product entering
// one fused multiply-add (equal rows give rho = 1 and d = 0 exactly); r' = max(0, d) = d * [d >= 0].  Adds the sum of
// the r' to *tm and, with AUX, the sum of e_q over the pairs with d >= 0 (q <= p) to *sx; with R, leaves the r'.
template <int N, bool AUX, bool R>
__device__ __forceinline__ void resid_n(const float* ep, const float* eq, const FRho& rho, float2* tm, float2* sx, float* r) {
    const float2 nh = make_float2(-rho.h, -rho.h), nl = make_float2(-rho.l, -rho.l);
#pragma unroll
    for (int i = 0; i < N; i += 2) {
        const float2 q2 = make_float2(eq[i], eq[i + 1]);
        const float2 d = __ffma2_rn(nl, q2, __ffma2_rn(nh, q2, make_float2(ep[i], ep[i + 1])));
        const float2 mk = make_float2(set_ge0(d.x), set_ge0(d.y));
        if (R) { r[i] = d.x * mk.x; r[i + 1] = d.y * mk.y; }
        *tm = __ffma2_rn(d, mk, *tm);
        if (AUX) *sx = __ffma2_rn(q2, mk, *sx);
    }
}

// What is not a full pair of vectors inside the slice(s): vectors beyond a slice read as -inf, the row's ragged last
// vector loses the lanes beyond the vocabulary.  Out of line and by value: the
// vectors of the usual case never leave the registers.
struct FVecs { uint4 p[FV], q[FV]; };
template <int DT>
__device__ __noinline__ FVecs mask_cold(FVecs v, int vi0, int nv, int nv2, int tailv, int tailkeep, bool pair) {
#pragma unroll
    for (int j = 0; j < FV; ++j) {
        const int vi = vi0 + j * 32;
        if (vi >= nv) v.p[j] = neg_inf_vec<DT>();
        if (vi >= nv2) v.q[j] = neg_inf_vec<DT>();
        if (vi == tailv) { mask_tail<DT>(v.p[j], tailkeep); if (pair) mask_tail<DT>(v.q[j], tailkeep); }
        if (!pair && FSV + vi == tailv) mask_tail<DT>(v.q[j], tailkeep);
    }
    return v;
}
template <int DT> __device__ __forceinline__ float vecs_max(const uint4* v) {
    float m = vec_max<DT>(v[0]);
#pragma unroll
    for (int j = 1; j < FV; ++j) m = max_nan(m, vec_max<DT>(v[j]));
    return m;
}
template <> __device__ __forceinline__ float vecs_max<1>(const uint4* v) {
    uint32_t m = max_nan_bf16x2(max_nan_bf16x2(v[0].x, v[0].y), max_nan_bf16x2(v[0].z, v[0].w));
#pragma unroll
    for (int j = 1; j < FV; ++j) m = max_nan_bf16x2(m, max_nan_bf16x2(max_nan_bf16x2(v[j].x, v[j].y), max_nan_bf16x2(v[j].z, v[j].w)));
    return max_nan(__uint_as_float(m << 16), __uint_as_float(m & 0xffff0000u));
}

// A consumer warp: per iteration n, pass 1 of its chunk of task n, then pass 2 of its chunk of task n - FLAG.
// The warps do not wait for each other: each takes its share of a stage when the stage is full and moves on.
template <int DT, bool TVM>
__device__ __forceinline__ void f_consumer(const FuseArgs& a, FShared& S, const unsigned char* data, int tid) {
    constexpr int VEC = Elem<DT>::VEC, NVAL = FuseDims<DT>::NVAL, NH = FV * VEC;
    const int lane = tid & 31, w = tid >> 5;
    // the warp's 128 columns of its quarter of the lanes
    const uint32_t tbase = S.tmem_base + ((uint32_t)(32 * (w & 3)) << 16) + (uint32_t)((w >> 2) * 128);
    const int tailkeep = a.r.V - (a.r.nvec - 1) * VEC;
    const int vi0 = w * (32 * FV) + lane;
    const int wfull = (w + 1) * (32 * FV);            // the slice holds this warp's vectors in full if it has this many
    float2* const p1t = &S.p1t[0][tid + tid / FEPL];
    float2* const p2t = &S.p2t[0][tid + tid / FEPL];
    const unsigned char* const mydata = data + (size_t)vi0 * 16;
    uint32_t n_end = 0x3fffffffu;
#pragma unroll 1
    for (uint32_t n = 0; n < n_end + FLAG; ++n) {
        const uint32_t slot4 = n & 3u;
        float2 o1 = make_float2(0.f, 0.f), o2 = make_float2(0.f, 0.f);
        int e_p = E_EMPTY, e_q = E_EMPTY, e_fl = 0;
        bool stored = false;
        if (aborted(S)) n_end = min(n_end, n);
        if (n < n_end) {
            if (!mbar_wait(S, &S.full[slot4], (n >> 2) & 1u)) { if (lane == 0) give_up(a, S); }
            // the stage's vectors are asked for at once; what the description says about them is applied afterwards
            const unsigned char* pd = mydata + (size_t)slot4 * FSTAGE;
            FVecs x;
#pragma unroll
            for (int j = 0; j < FV; ++j) { x.p[j] = lds16(pd + (size_t)j * 512); x.q[j] = lds16(pd + FSTAGE / 2 + (size_t)j * 512); }
            const int4 d0 = *reinterpret_cast<const int4*>(&S.task[n & (FRING - 1)]);
            __syncwarp();
            if (lane == 0) mbar_arrive(&S.empty[slot4]);
            if (d0.x == kStop) n_end = n;
            else {
                const int tailv = d0.z;
                const float c = __int_as_float(d0.w);
                const bool pair = d0.x == kPair;
                const int nv = pair ? d0.y : (d0.y & 0xffff), nv2 = pair ? d0.y : (d0.y >> 16);
                if (wfull > nv2 || tailv >= 0) x = mask_cold<DT>(x, vi0, nv, nv2, tailv, tailkeep, pair);
                // ---- pass 1: the warp's reference exponents, the exponentials, the thread's sums (a bonus task's second
                // slice stands where the draft row stands; its exponentials are summed and not kept)
                const FExp xp = warp_exponent(vecs_max<DT>(x.p), c);
                const FExp xq = warp_exponent(vecs_max<DT>(x.q), c);
                e_p = xp.e; e_q = xq.e; e_fl = xp.bad | (xq.bad << 1);
                float e[NVAL];
#pragma unroll
                for (int j = 0; j < FV; ++j) { exp_vec<DT>(x.p[j], c, xp.ef, e + j * VEC); exp_vec<DT>(x.q[j], c, xq.ef, e + NH + j * VEC); }
                if (pair) { tmem_st<NVAL>(tbase + slot4 * 32u, e); stored = true; }
                o1 = make_float2(sum_fixed<NH>(e), sum_fixed<NH>(e + NH));
            }
        }
        // ---- pass 2 of the task FLAG back: r' = max(0, e_p - rho e_q) from the exponentials in TMEM
        const uint32_t m = n - FLAG;
        if (n >= FLAG && m < n_end) {
            if (!mbar_wait(S, &S.stats[m & 3u], (m >> 2) & 1u)) { if (lane == 0) give_up(a, S); }
            if (S.task[m & (FRING - 1)].kind == kPair) {
                const FRho rho = S.rho[m & (FR8 - 1)][w];
                float e[NVAL];
                tmem_ld<NVAL>(tbase + (m & 3u) * 32u, e);
                float2 tm = make_float2(0.f, 0.f), sx = make_float2(0.f, 0.f);
                resid_n<NH, TVM, false>(e, e + NH, rho, &tm, &sx, nullptr);
                o2 = make_float2(tm.x + tm.y, sx.x + sx.y);
            }
        }
        // ---- the thread's sums, once both publishers have read those of four iterations ago
        if (n >= 4 && !mbar_wait(S, &S.sfree[slot4], ((n >> 2) & 1u) ^ 1u)) { if (lane == 0) give_up(a, S); }
        p1t[slot4 * FPAD] = o1;
        p2t[((n + 4 - FLAG) & 3u) * FPAD] = o2;
        if (lane == 0) { FWarpE we; we.ep = e_p; we.eq = e_q; we.flags = e_fl; we.pad = 0; S.we[n & (FR8 - 1)][w] = we; }
        if (stored) tmem_wait_st();
        __syncwarp();
        if (lane == 0) mbar_arrive(&S.iter[slot4]);
        __syncwarp();      // (no lane goes ahead into the next wait while lane 0 has not arrived: see the publisher's store)
    }
}

// ------------------------------------------------------------------ publisher of the softmax partials
// Lane l adds up half of warp chunk l / 2 (16 threads' sums); a shuffle joins the halves; the chunks
// are scaled (exactly) to the slice's largest exponent and joined.  Pair: one record per row.  Bonus row: its
// records (two slices), and -- since it has no pass 2 -- its chunk sums for the draw.
__device__ __forceinline__ void f_puba(const FuseArgs& a, FShared& S) {
    const int lane = threadIdx.x & 31;
    const int chunk = lane / FLPC, role = lane % FLPC;        // role 0 carries the target row, role 1 the draft row
#pragma unroll 1
    for (int n = 0;; ++n) {
        const int slot = n % FRING, slot4 = n & 3;
        if (!mbar_wait_helper(S, &S.iter[slot4], ((uint32_t)(n >> 2)) & 1u)) { if (lane == 0) give_up(a, S); }
        if (aborted(S)) return;
        const FTask d = S.task[slot];
        if (d.kind == kStop) return;
        const float2* src = &S.p1t[slot4][lane * (FEPL + 1)];
        float2 s0 = make_float2(0.f, 0.f), s1 = make_float2(0.f, 0.f);
#pragma unroll
        for (int i = 0; i < FEPL; i += 2) { s0 = __fadd2_rn(s0, src[i]); s1 = __fadd2_rn(s1, src[i + 1]); }
        const FWarpE we = S.we[n & (FR8 - 1)][chunk];
        __syncwarp();
        if (lane == 0) mbar_arrive(&S.sfree[slot4]);
        __syncwarp();
        float2 sc2 = __fadd2_rn(s0, s1);
        sc2.x += __shfl_xor_sync(0xffffffffu, sc2.x, 1); sc2.y += __shfl_xor_sync(0xffffffffu, sc2.y, 1);    // the chunk's sums, in both its lanes
        const bool pair = d.kind == kPair;
        const int64_t us = (int64_t)d.unit * a.T + d.s;
        const int emp = redux_max(we.ep), emq = redux_max(we.eq), fl = __reduce_or_sync(0xffffffffu, we.flags);
        // role 0: the target row; role 1: the draft row.  A chunk's sum is below 2^11, its scaling a power of two.
        const bool second = role == 1;
        const int ew = second ? we.eq : we.ep, em = second ? emq : emp;
        const double f = ew > E_EMPTY ? pow2d(max(ew - em, -500)) : 0.0;
        double v = (double)(second ? sc2.y : sc2.x) * f;
        double ub = v * f;                                  // 4^(E_w - E_s) times the chunk's sum of e
#pragma unroll
        for (int o = 16; o >= FLPC; o >>= 1) { v += shfl_xor_d(v, o); ub += shfl_xor_d(ub, o); }
        {
            // Every lane forms the record; lanes 0 and (for a pair) 1 store it, by predicate.  As a branch for those two
            // lanes the store came about a microsecond late: nothing makes a warp that has split reconverge before
            // its next __syncwarp(), and the other thirty lanes had gone ahead into the wait of the next iteration.
            const int bad = fl & (second ? 2 : 1);
            double rs = em > E_EMPTY && !bad ? v : 0.0;
            if (rs == 0.0) rs = -0.0;
            const unsigned long long w0 = (unsigned long long)__double_as_longlong(rs);
            // (the bound rounded up, and up again to an even bit pattern: bit 0 of the word is the flag)
            const unsigned ubits = ((unsigned)__float_as_int(__double2float_ru((em > E_EMPTY && !bad) ? ub : 0.0)) + 1u) & ~1u;
            const unsigned long long w1 = (unsigned long long)(unsigned)(2 * em + 1) | ((unsigned long long)(ubits | (bad ? 1u : 0u)) << 32);
            const bool two = pair || d.s + 1 < a.T;            // a second record: the draft row's, or the bonus row's second slice's
            const unsigned doit = (lane == 0 || (lane == 1 && two)) ? 1u : 0u;
            asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %3, 0;\n\t@p st.relaxed.gpu.global.v2.b64 [%0], {%1, %2};\n\t}"
                         :: "l"(a.rec + (second ? (pair ? us * 2 + 1 : us * 2 + 2) : us * 2)), "l"(w0), "l"(w1), "r"(doit) : "memory");
        }
        // a bonus row has no pass 2: its chunk sums go to the publisher of the masses, which writes them out with the
        // sequence's count (the fence before the count would hold up the next task's record here)
        if (!pair && role == 0) S.bsum[n & (FR8 - 1)][chunk] = sc2;
        __syncwarp();
        if (lane == 0) mbar_arrive(&S.bdone[n & (FR8 - 1)]);
        __syncwarp();
    }
}

// ------------------------------------------------------------------ publisher of the masses
// Publisher j serves the iterations n = j mod FNPB.  Pair tasks: the chunks' sums of r' times 2^(E_wp - E_p) / S_p
// are the chunks' residual masses; with them go the warps' exponents, the slice's mass and auxiliary sum and, with
// slice 0, the unit's merged rows.  Bonus tasks: the chunk sums the other publisher left.  Then one count for the
// sequence, behind a fence: who sees the count sees the parts.  Pass 2 of task m is in place after iteration
// m + FLAG.
template <bool TVM>
__device__ __forceinline__ void f_pubb(const FuseArgs& a, FShared& S, int j) {
    const int lane = threadIdx.x & 31;
    const int chunk = lane / FLPC, role = lane % FLPC;
    int stop_n = 0x3fffffff;
#pragma unroll 1
    for (int n = j; n < stop_n + FLAG; n += FNPB) {
        const int slot4 = n & 3;
        if (!mbar_wait_helper(S, &S.iter[slot4], ((uint32_t)(n >> 2)) & 1u)) { if (lane == 0) give_up(a, S); }
        if (aborted(S)) return;
        // the end is marked in FNSW consecutive descriptions: the first of them is the one that counts
        if (n < stop_n && S.task[n % FRING].kind == kStop) {
            stop_n = n;
            for (int i = 1; i < FNPB && stop_n > 0 && S.task[(stop_n - 1) % FRING].kind == kStop; ++i) --stop_n;
            if (n >= stop_n + FLAG) break;
        }
        const int m = n - FLAG;
        bool done = false;
        if (m >= 0 && m < stop_n) {
            const FTask d = S.task[m % FRING];
            if (d.kind == kPair) {
                const int ps = m & 3;
                const int64_t us = (int64_t)d.unit * a.T + d.s;
                const float2* src = &S.p2t[ps][lane * (FEPL + 1)];
                float2 s0 = make_float2(0.f, 0.f), s1 = make_float2(0.f, 0.f);
#pragma unroll
                for (int i = 0; i < FEPL; i += 2) { s0 = __fadd2_rn(s0, src[i]); s1 = __fadd2_rn(s1, src[i + 1]); }
                const FWarpE we = S.we[m % FR8][chunk];
                const FScale sc = S.scale[m % FR8];
                __syncwarp();
                if (lane == 0) mbar_arrive(&S.sfree[slot4]);
                __syncwarp();
                done = true;
                float2 sc2 = __fadd2_rn(s0, s1);
                sc2.x += __shfl_xor_sync(0xffffffffu, sc2.x, 1); sc2.y += __shfl_xor_sync(0xffffffffu, sc2.y, 1);
                const double mass = (double)sc2.x * chunk_scale(sc.inv_p, sc.ep, we.ep);
                if (role == 0) { a.mass[us * FCW + chunk] = mass; a.wexp[us * FCW + chunk] = make_int2(we.ep, we.eq); }
                double sm = role == 0 ? mass : 0.0;
#pragma unroll
                for (int o = 16; o >= FLPC; o >>= 1) sm += shfl_xor_d(sm, o);
                if (lane == 0) {
                    a.smass[us] = sm;
                    if (d.s == 0) {
                        FRow x; x.inv_s = sc.inv_p; x.e = sc.ep; x.st = sc.stp; a.rows[2 * (int64_t)d.unit] = x;
                        x.inv_s = sc.inv_q; x.e = sc.eq; x.st = sc.stq; a.rows[2 * (int64_t)d.unit + 1] = x;
                    }
                }
                if (TVM && a.sauxp) {
                    double sxx = role == 0 ? (double)sc2.y * chunk_scale(sc.inv_q, sc.eq, we.eq) : 0.0;   // sum of q over the chunk's tokens with q <= p
#pragma unroll
                    for (int o = 16; o >= FLPC; o >>= 1) sxx += shfl_xor_d(sxx, o);
                    if (lane == 0) a.sauxp[us] = sxx;
                }
                __syncwarp();
                if (lane == 0) { __threadfence(); atomicAdd(a.seqcnt + d.b, 1); }
            } else if (d.kind == kBonus) {
                if (!mbar_wait_helper(S, &S.bdone[m & (FR8 - 1)], ((uint32_t)(m >> 3)) & 1u)) { if (lane == 0) give_up(a, S); }
                const int64_t us = (int64_t)d.unit * a.T + d.s;
                if (role == 0) {
                    const float2 bs = S.bsum[m & (FR8 - 1)][chunk];
                    const FWarpE we = S.we[m & (FR8 - 1)][chunk];
                    a.mass[us * FCW + chunk] = (double)bs.x;
                    a.wexp[us * FCW + chunk] = make_int2(we.ep, E_EMPTY);
                    if (d.s + 1 < a.T) { a.mass[(us + 1) * FCW + chunk] = (double)bs.y; a.wexp[(us + 1) * FCW + chunk] = make_int2(we.eq, E_EMPTY); }
                }
                __syncwarp();
                if (lane == 0) { __threadfence(); atomicAdd(a.seqcnt + d.b, 1); }
            }
        }
        if (!done) { __syncwarp(); if (lane == 0) mbar_arrive(&S.sfree[slot4]); }
        __syncwarp();
    }
}

// ------------------------------------------------------------------ stats warps
// Stats warp j serves the tasks n = j, j + FNSW, ...: it finds the T records of the task's unit, merges both
// rows and leaves each consumer warp's rho, and the normalisers for the publisher of the masses.
__device__ __forceinline__ void f_stats(const FuseArgs& a, FShared& S, int j) {
    const int lane = threadIdx.x & 31;
#pragma unroll 1
    for (int n = j;; n += FNSW) {
        const int slot = n % FRING;
        if (!mbar_wait_helper(S, &S.dready[slot], ((uint32_t)(n / FRING)) & 1u)) { if (lane == 0) give_up(a, S); }
        if (aborted(S)) return;
        const int kind = S.task[slot].kind;
        if (kind == kStop) return;
        // The stats barrier of a slot completes one phase per task, and a barrier must not get two phases ahead of the
        // warps that wait on it: so every task, with or without statistics, is held until the consumers' iteration n
        // is over (they waited for task n - 4 on this barrier in iteration n - 1).  For a row pair this is also when to
        // start looking: the records of the other slices come from CTAs that run in step with this one, so they are
        // not there before this CTA's own pass 1 of the task is over; and the consumers' exponents are in place.
        if (!mbar_wait_helper(S, &S.iter[n & 3], ((uint32_t)(n >> 2)) & 1u)) { if (lane == 0) give_up(a, S); }
        if (kind == kPair) {
            FRow rp, rq;
            if (a.expire) give_up(a, S);                    // test hook: this wait's bound has run out already
            merge_rows(a, S, S.task[slot].unit, 2, &rp, &rq);
            const FScale sc = scale_of(rp, rq);
            if (lane < FCW) { const FWarpE we = S.we[n % FR8][lane]; S.rho[n % FR8][lane] = warp_rho(sc, we.ep, we.eq); }
            if (lane == 0) S.scale[n % FR8] = sc;
            __syncwarp();
        }
        if (lane == 0) mbar_arrive(&S.stats[n & 3]);
        __syncwarp();
    }
}

// ------------------------------------------------------------------ completing sequences
__device__ __noinline__ bool wait_parts(const FuseArgs& a, FShared& S, int b, int need) {
    int ok = 0;
    if ((threadIdx.x & 31) == 0) {
        for (uint32_t i = 0; i < kSpin && !ok; ++i) {
            if (ld_acquire(a.seqcnt + b) >= need) ok = 1;
            else if ((i & 63u) == 63u && ld_relaxed(a.wait_failed)) break;
            else __nanosleep(200);
        }
    }
    ok = __shfl_sync(0xffffffffu, ok, 0);
    if (ok) __threadfence();      // the other lanes read the parts after lane 0 saw the count
    return ok != 0;
}

// bebop_tv: row pair b is complete when its T parts are in
__device__ __noinline__ void f_finish_tv(const FuseArgs& a, FShared& S, int b) {
    const RowArgs& R = a.r;
    const int lane = threadIdx.x & 31, T = a.T;
    const bool ok = wait_parts(a, S, b, T);
    if (!ok && lane == 0) atomicExch(a.wait_failed, 1);
    int st = tau_ok(tau_of(R, b)) ? 0 : ST_BAD_TEMP;
    if (ok && !st) {
        FRow rp, rq;
        merge_rows(a, S, b, 2, &rp, &rq);
        st = rp.st | rq.st;
    }
    double z = 0.0, sx = 0.0;
    if (ok && !st) {
        for (int i = lane; i < T * FCW; i += 32) z += __ldcg(a.mass + (int64_t)b * T * FCW + i);
        if (a.s_aux) for (int i = lane; i < T; i += 32) sx += __ldcg(a.sauxp + (int64_t)b * T + i);
        z = warp_sum(z); sx = warp_sum(sx);
    }
    if (lane == 0) {
        a.o.tv[b] = (float)fmin(fmax(z, 0.0), 1.0);
        if (a.s_aux) a.s_aux[b] = (float)sx;
        if (a.o.row_status) a.o.row_status[b] = st | ((ok && !ld_relaxed(a.wait_failed)) ? 0 : ST_WAIT);
    }
}

// a merged row as its publisher left it (two 8-byte loads past the first level of cache)
__device__ __forceinline__ FRow ld_row(const FRow* p) {
    const double2 v = __ldcg(reinterpret_cast<const double2*>(p));
    FRow x; x.inv_s = v.x; x.e = __double2loint(v.y); x.st = __double2hiint(v.y);
    return x;
}
__device__ __forceinline__ FRow shfl_row(const FRow& x, int src) {
    FRow y;
    y.inv_s = __shfl_sync(0xffffffffu, x.inv_s, src); y.e = __shfl_sync(0xffffffffu, x.e, src); y.st = __shfl_sync(0xffffffffu, x.st, src);
    return y;
}
// Which of a warp's values owns the target t of an inverse CDF: the values are laid out lane-major (lane l holds
// v[0..N) for the indices l * N + i), `below` is what lies before index 0.  Returns the owner's index (-1: none) in
// all lanes and leaves the running sum before it in *base and the total in *total (a target below zero finds no owner:
// that call is for the total).
template <int N>
__device__ __forceinline__ int owner_of(const double (&v)[N], double below, double t, double* base, double* total) {
    const int lane = threadIdx.x & 31;
    double mine = 0.0;
#pragma unroll
    for (int i = 0; i < N; ++i) mine += v[i];
    double incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const double t2 = shfl_up_d(incl, o); if (lane >= o) incl += t2; }
    *total = below + __shfl_sync(0xffffffffu, incl, 31);
    int idx = -1; double b0 = 0.0;
    double run = below + (incl - mine);
#pragma unroll
    for (int i = 0; i < N; ++i) {
        const double nx = run + v[i];
        if (idx < 0 && t > run && t <= nx) { idx = lane * N + i; b0 = run; }
        run = nx;
    }
    const unsigned own = __ballot_sync(0xffffffffu, idx >= 0);
    if (!own) { *base = 0.0; return -1; }
    const int src = __ffs(own) - 1;
    *base = __shfl_sync(0xffffffffu, b0, src);
    return __shfl_sync(0xffffffffu, idx, src);
}

// bebop_verify: sequence b is complete when the T parts of each of its L row pairs and of its bonus row are in.
// One warp; everything it reads was published before the sequence's count reached its final value.  The loads that
// do not depend on each other are asked for together: the chain is rows and tokens -> the tokens' logits -> accept
// scan -> slice masses of the draw unit -> chunk masses of the owning slice -> the owning chunk's vectors.
template <int DT, int SPL>                         // SPL: slices per lane, at most
__device__ __noinline__ void f_finish_seq(const FuseArgs& a, FShared& S, int b, int need) {
    constexpr int VEC = Elem<DT>::VEC;
    const RowArgs& R = a.r;
    const int lane = threadIdx.x & 31;
    const int K = R.K, V = R.V, T = a.T, L = len_of(R, b);
    const float tau = tau_of(R, b);
    const TempScale ts = temp_scale(tau);
    int seq_st = tau_ok(tau) ? 0 : ST_BAD_TEMP;
    const int unit0 = b * (K + 1);
    const int per = (T + 31) >> 5;                 // a lane's run of slices: [lane * per, lane * per + per)
    // ---- lane k owns draft position k: its token, uniform and the token's logits are the call's inputs, asked for
    // before the wait for the sequence's parts
    const bool active = lane < L;
    const int tk = active ? a.draft_tokens[(int64_t)b * K + lane] : 0;
    const float u = active ? a.u_accept[(int64_t)b * K + lane] : 0.f;
    const float uf = a.u_final[b];
    const bool tok_ok = tk >= 0 && tk < V;
    float zpx = 0.f, zqx = 0.f;
    if (active && tok_ok) { zpx = load_one<DT>(row_ptr(R, b, lane), tk); zqx = load_one<DT>(row_ptr(R, b, K + 1 + lane), tk); }
    if (!wait_parts(a, S, b, need)) {
        // the parts never came: the sequence gets no draw (the re-draw kernel must not wait for it) and says so
        if (lane == 0) {
            atomicExch(a.wait_failed, 1);
            a.o.accept_len[b] = 0;
            for (int q = 0; q <= K; ++q) a.o.out_tokens[(int64_t)b * (K + 1) + q] = -1;
            if (a.o.row_status) a.o.row_status[b] = ST_WAIT;
            draw_decided(a.fb_count);
        }
        return;
    }
    // ---- its rows
    FRow sp, sq;
    sp.inv_s = 0.0; sp.e = E_EMPTY; sp.st = 0; sq = sp;
    if (active) { sp = ld_row(a.rows + 2 * (int64_t)(unit0 + lane)); sq = ld_row(a.rows + 2 * (int64_t)(unit0 + lane) + 1); }
    // ---- TV of every position: the slices' masses, asked for now four positions at a time, summed after the scan
    constexpr int TVG = 4;
    double tvz[TVG];
#pragma unroll
    for (int g = 0; g < TVG; ++g) {
        tvz[g] = 0.0;
        if (a.o.tv && g < L) {
            const double* m = a.smass + (int64_t)(unit0 + g) * T + lane * per;
#pragma unroll
            for (int i = 0; i < SPL; ++i) if (i < per && lane * per + i < T) tvz[g] += __ldcg(m + i);
        }
    }
    if (!seq_st && __ballot_sync(0xffffffffu, active && !tok_ok)) seq_st = ST_BAD_TOKEN;
    const int rs = active ? (sp.st | sq.st) : 0;
    const unsigned badrows = __ballot_sync(0xffffffffu, rs != 0);
    const int first_bad = badrows ? __ffs(badrows) - 1 : 32;
    const int rs_first = __shfl_sync(0xffffffffu, rs, first_bad & 31);
    if (!seq_st && badrows) seq_st = rs_first;
    double px = 0.0, qx = 0.0;
    bool acc = false;
    if (active && !(seq_st & ST_FATAL) && lane < first_bad) {
        const double cd = (double)ts.hi;
        px = exp2((double)zpx * cd - (double)sp.e) * sp.inv_s;
        qx = exp2((double)zqx * cd - (double)sq.e) * sq.inv_s;
        acc = (double)u * qx < px;
    }
    const unsigned rej = __ballot_sync(0xffffffffu, active && !acc);
    const int n = rej ? __ffs(rej) - 1 : L;
    // ---- the bonus row, when every draft was accepted: merged here from its slices' records (kept: they are its masses)
    FRow rb; rb.inv_s = 0.0; rb.e = E_EMPTY; rb.st = 0;
    double bs[SPL], bu[SPL]; int be[SPL];
#pragma unroll
    for (int i = 0; i < SPL; ++i) { bs[i] = 0.0; bu[i] = 0.0; be[i] = E_EMPTY; }
    if (!(seq_st & ST_FATAL) && n == L) {
        const FRec* base = a.rec + ((int64_t)(unit0 + L) * T) * 2;
        int fl = 0, el = E_EMPTY;
#pragma unroll
        for (int i = 0; i < SPL; ++i) {
            const int si = lane * per + i;
            if (i < per && si < T) {
                FRec r;
                bool ok = ld_rec(base + 2 * si, &r);
                for (uint32_t it = 0; !ok && it < kSpin; ++it) { __nanosleep(200); ok = ld_rec(base + 2 * si, &r); }
                if (!ok) { atomicExch(a.wait_failed, 1); r.s = 0.0; r.ecode = 2 * E_EMPTY + 1; r.flags = 0; }
                bs[i] = r.s; be[i] = (r.ecode - 1) >> 1; bu[i] = (double)rec_ub(r); fl |= r.flags & 1; el = max(el, be[i]);
            }
        }
        const int Em = redux_max(el);
        fl = __reduce_or_sync(0xffffffffu, fl);
        // the slices' sums around the row's exponent, added in slice order
        double v = 0.0;
#pragma unroll
        for (int i = 0; i < SPL; ++i) {
            const double f = be[i] > E_EMPTY ? pow2d(max(be[i] - Em, -500)) : 0.0;
            bs[i] *= f; bu[i] *= f * f; v += bs[i];
        }
        double incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const double t2 = shfl_up_d(incl, o); if (lane >= o) incl += t2; }
        const double Sb = __shfl_sync(0xffffffffu, incl, 31);
        if (fl || !(Sb == Sb)) rb.st = ST_NONFINITE; else if (Em == E_EMPTY) rb.st = ST_EMPTY;
        rb.inv_s = (!rb.st && Sb > 0.0) ? 1.0 / Sb : 0.0; rb.e = Em;
        seq_st |= rb.st;
    }
    const bool fatal = (seq_st & ST_FATAL) != 0;
    const int nn = fatal ? 0 : n;
    for (int q = lane; q <= K; q += 32)
        if (fatal || q != nn) a.o.out_tokens[(int64_t)b * (K + 1) + q] = q < nn ? tk : -1;
    if (lane < K) {
        const bool zero = fatal || lane >= L;
        if (a.o.p_draft) a.o.p_draft[(int64_t)b * K + lane] = zero ? 0.f : (float)px;
        if (a.o.q_draft) a.o.q_draft[(int64_t)b * K + lane] = zero ? 0.f : (float)qx;
        if (zero && a.o.tv) a.o.tv[(int64_t)b * K + lane] = 0.f;
    }
    if (lane == 0) {
        a.o.accept_len[b] = nn;
        if (a.o.row_status) a.o.row_status[b] = seq_st;
    }
    if (fatal) { if (lane == 0) draw_decided(a.fb_count); return; }
    // ---- TV of every position: the sum of its slices' masses (slice order within a lane, lanes in a fixed tree)
    if (a.o.tv) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
#pragma unroll
            for (int g = 0; g < TVG; ++g) tvz[g] += shfl_xor_d(tvz[g], o);
#pragma unroll
        for (int g = 0; g < TVG; ++g)
            if (g < L && lane == 0) a.o.tv[(int64_t)b * K + g] = (float)fmin(fmax(tvz[g], 0.0), 1.0);
        for (int k = TVG; k < L; ++k) {
            const double* m = a.smass + (int64_t)(unit0 + k) * T + lane * per;
            double z = 0.0;
#pragma unroll
            for (int i = 0; i < SPL; ++i) if (i < per && lane * per + i < T) z += __ldcg(m + i);
            z = warp_sum(z);
            if (lane == 0) a.o.tv[(int64_t)b * K + k] = (float)fmin(fmax(z, 0.0), 1.0);
        }
    }
    // ---- the draw: position nn (row pair), or the bonus row when every draft was accepted
    const bool pair = nn < L;
    const int du = unit0 + nn;
    const FRow rp = pair ? shfl_row(sp, nn) : rb;
    FRow rq = shfl_row(sq, pair ? nn : 0);
    if (!pair) { rq.inv_s = 0.0; rq.e = E_EMPTY; rq.st = 0; }
    // The draw's error bound wants sum p^2 + q^2 over the row pair, for which the records carry an upper bound per slice
    // (a chunk's e are at most sqrt(2) around its own exponent, so its sum of e^2 is at most sqrt(2) times its sum of e:
    // chunks far below the row's largest logit count next to nothing, and a peaked row gets a bound close to the sum).
    double s2 = 0.0;
    if (pair) {
        const FRec* base = a.rec + ((int64_t)du * T) * 2;
#pragma unroll
        for (int i = 0; i < SPL; ++i) {
            const int si = lane * per + i;
            if (i < per && si < T) {
                FRec r0, r1;
                ld_rec(base + 2 * si, &r0); ld_rec(base + 2 * si + 1, &r1);
                const int e0 = (r0.ecode - 1) >> 1, e1 = (r1.ecode - 1) >> 1;
                if (e0 > E_EMPTY && rp.e > E_EMPTY) { const double f = pow2d(max(e0 - rp.e, -500)) * rp.inv_s; s2 += (double)rec_ub(r0) * f * f; }
                if (e1 > E_EMPTY && rq.e > E_EMPTY) { const double f = pow2d(max(e1 - rq.e, -500)) * rq.inv_s; s2 += (double)rec_ub(r1) * f * f; }
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < SPL; ++i) s2 += bu[i] * rp.inv_s * rp.inv_s;
    }
    s2 = warp_sum(s2);
    const double bound = draw_bound(1.4142135623730951 * s2, (double)a.kappa);
    // the slices' masses (bonus row: sums of e around the row's exponent -> probabilities); the slice that owns u Z
    double sm[SPL];
#pragma unroll
    for (int i = 0; i < SPL; ++i) {
        sm[i] = 0.0;
        if (pair) { if (i < per && lane * per + i < T) sm[i] = __ldcg(a.smass + (int64_t)du * T + lane * per + i); }
        else sm[i] = bs[i] * rp.inv_s;
    }
    // the total as the scan below adds it up, so that u = 1 lands inside the last slice
    double sbase, Zs;
    owner_of<SPL>(sm, 0.0, -1.0, &sbase, &Zs);
    const double Tt = (double)uf * Zs;
    int y = -1, cert = 0;
    const int lane_s = Tt > 0.0 ? owner_of<SPL>(sm, 0.0, Tt, &sbase, &Zs) : -1;      // lane-major index -> slice
    if (lane_s >= 0) {
        const int s = (lane_s / SPL) * per + (lane_s % SPL);
        // the 16 chunks of that slice: lane c < 16 holds chunk c
        const int64_t us = (int64_t)du * T + s;
        double cm[1] = {0.0};
        int2 we = make_int2(E_EMPTY, E_EMPTY);
        if (lane < FCW) {
            cm[0] = __ldcg(a.mass + us * FCW + lane);
            we = __ldcg(a.wexp + us * FCW + lane);
            if (!pair) cm[0] *= chunk_scale(rp.inv_s, rp.e, we.x);
        }
        double cbase, ctot;
        const int w = owner_of<1>(cm, sbase, Tt, &cbase, &ctot);
        if (w >= 0) {
            we.x = __shfl_sync(0xffffffffu, we.x, w); we.y = __shfl_sync(0xffffffffu, we.y, w);
            const FScale sc = scale_of(rp, rq);
            FRho rho; rho.h = 0.f; rho.l = 0.f;
            if (pair) rho = warp_rho(sc, we.x, we.y);
            const double fp = chunk_scale(rp.inv_s, rp.e, we.x);          // r' (or e) -> probability mass
            const float Efp = we.x > E_EMPTY ? (float)we.x : 0.f, Efq = we.y > E_EMPTY ? (float)we.y : 0.f;
            const int v0 = s * a.slice_vecs, nv = max(min(a.slice_vecs, R.nvec - v0), 0);
            const char* prow = row_ptr(R, b, nn);
            const char* qrow = pair ? row_ptr(R, b, K + 1 + nn) : prow;
            uint4 xp[FV], xq[FV];
#pragma unroll
            for (int j = 0; j < FV; ++j) {
                const int vi = w * (32 * FV) + j * 32 + lane;
                xp[j] = neg_inf_vec<DT>(); xq[j] = neg_inf_vec<DT>();
                if (vi < nv) {
                    xp[j] = ldg16(prow + (int64_t)(v0 + vi) * 16);
                    if (pair) xq[j] = ldg16(qrow + (int64_t)(v0 + vi) * 16);
                }
            }
            double base = cbase;
#pragma unroll
            for (int j = 0; j < FV; ++j) {
                const int vi = w * (32 * FV) + j * 32 + lane;
                const int gbase = (v0 + vi) * VEC;
                if (vi < nv && gbase + VEC > V) { mask_tail<DT>(xp[j], V - gbase); mask_tail<DT>(xq[j], V - gbase); }
                float ep[VEC], eq[VEC], r[VEC];
                exp_vec<DT>(xp[j], ts.hi, Efp, ep);
                exp_vec<DT>(xq[j], ts.hi, Efq, eq);
                if (pair) {
                    float2 tm = make_float2(0.f, 0.f), sx = make_float2(0.f, 0.f);
                    resid_n<VEC, false, true>(ep, eq, rho, &tm, &sx, r);
                } else {
#pragma unroll
                    for (int i = 0; i < VEC; ++i) r[i] = ep[i];
                }
                const double dv = (double)sum_fixed<VEC>(r) * fp;
                double vin = dv;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) { const double t2 = shfl_up_d(vin, o); if (lane >= o) vin += t2; }
                const double lo = base + (vin - dv), hi = base + vin;
                if (y < 0 && lo < Tt && Tt <= hi) {
                    double C = lo;
#pragma unroll
                    for (int i = 0; i < VEC; ++i) {
                        if (y < 0) {
                            const double r1 = (double)r[i] * fp, Cn = C + r1;
                            if (r1 > 0.0 && Cn >= Tt) { y = (v0 + vi) * VEC + i; cert = (Tt - C > bound) && (Cn - Tt >= bound); }
                            C = Cn;
                        }
                    }
                }
                base += __shfl_sync(0xffffffffu, vin, 31);
            }
        }
    }
    const unsigned found = __ballot_sync(0xffffffffu, y >= 0);
    const bool keep = __popc(found) == 1 && __shfl_sync(0xffffffffu, cert, (__ffs(found) - 1) & 31);
    if (keep) {
        if (y >= 0) { a.o.out_tokens[(int64_t)b * (K + 1) + nn] = y; draw_decided(a.fb_count); }
    } else if (lane == 0) {
        st_fb(a.fb_list + draw_listed(a.fb_count), b, 2 * nn + (pair ? 1 : 0), rp.e, pair ? rq.e : 0);
    }
}

// consumer warp w of CTA i completes the sequences w * grid + i, then every 16 * grid further on
template <int DT, bool TVM>
__device__ __forceinline__ void f_finish(const FuseArgs& a, FShared& S, int w) {
    const RowArgs& R = a.r;
    for (int b = w * (int)gridDim.x + (int)blockIdx.x; b < R.B; b += FCW * (int)gridDim.x) {
        if (TVM) { f_finish_tv(a, S, b); continue; }
        const int need = len_of(R, b) * a.T + (a.T + 1) / 2;
        if (a.T <= 32) f_finish_seq<DT, 1>(a, S, b, need);
        else if (a.T <= 64) f_finish_seq<DT, 2>(a, S, b, need);
        else f_finish_seq<DT, kFuseMaxSlices / 32>(a, S, b, need);
        __syncwarp();
    }
}

}  // namespace

template <int DT, bool TVM>
__global__ void __launch_bounds__(FT, 1) k_fuse(const __grid_constant__ FuseArgs a, int total) {
    extern __shared__ __align__(128) unsigned char smem[];
    FShared& S = *reinterpret_cast<FShared*>(smem + (size_t)FNS * FSTAGE);
    const int tid = threadIdx.x, warp = tid >> 5;
    if (tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0) {
        for (int i = 0; i < FNS; ++i) { mbar_init(&S.full[i], 1); mbar_init(&S.empty[i], FCW); }
        for (int i = 0; i < FRING; ++i) mbar_init(&S.dready[i], 1);
        for (int i = 0; i < 4; ++i) { mbar_init(&S.iter[i], FCW); mbar_init(&S.sfree[i], 2); mbar_init(&S.stats[i], 1); }
        for (int i = 0; i < FR8; ++i) mbar_init(&S.bdone[i], 1);
        S.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) tmem_alloc(&S.tmem_base, FTCOLS);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem0 = S.tmem_base;
    if (warp < FCW) {
        f_consumer<DT, TVM>(a, S, smem, tid);
        f_finish<DT, TVM>(a, S, warp);
    }
    else if (warp == W_PROD) { if ((tid & 31) == 0) f_producer<DT>(a, S, smem, total); __syncwarp(); }
    else if (warp == W_PUBA) f_puba(a, S);
    else if (warp < W_STAT0) f_pubb<TVM>(a, S, warp - W_PUBB);
    else f_stats(a, S, warp - W_STAT0);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem0, FTCOLS);
}

// -----------------------------------------------------------------------------
namespace {

constexpr size_t kFuseSmem = (size_t)FNS * FSTAGE + sizeof(FShared);

template <int DT, bool TVM>
int fuse_grid() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (dev >= 0 && dev < 64 && cached[dev]) return cached[dev];
    if (cudaFuncSetAttribute(k_fuse<DT, TVM>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFuseSmem) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    int per_sm = 0, sms = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_fuse<DT, TVM>, FT, kFuseSmem) != cudaSuccess) per_sm = 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaGetLastError();
    const int n = per_sm >= 1 ? sms : 0;      // the grid must be resident as a whole: one CTA per SM
    if (dev >= 0 && dev < 64) cached[dev] = n;
    return n;
}

}  // namespace

extern cudaEvent_t g_ev_start, g_ev_stop;

bool fuse_supported(const RowArgs& a) {
    const FusePlan fp = make_fuse_plan(a.B, a.K, a.nvec, a.K + 1);
    return fp.T >= 1 && fp.T <= kFuseMaxSlices && a.K <= BEBOP_MAX_K_INT;
}

// Measured on a B200 against the pipelined kernel (about 0.4 GB of logits per call unless said otherwise):
// bebop_tv is faster through the fused kernel at every shape tried with at most 32 slices per row (3 to 12 per cent
// from 32,768 to 262,144 bf16 logits per row, twice as fast at 8,192 and below; fp32 alike), and slower with more
// (the merge of a unit's records then takes several records per lane).  bebop_verify is faster up to eleven slices
// per row (5 per cent at 90,112 bf16 logits, 7 at 65,536, 15 at 32,768, twice as fast at 16,384 and below) and 2
// to 6 per cent slower from 100,000 on, where the pipelined kernel streams at close to the copy rate -- except with
// one draft position per sequence, where half of the rows are bonus rows (5 to 13 per cent faster at 100,000 to
// 262,144); small calls (a few dozen tasks per CTA) are faster fused at any row length, tiny ones (fewer than two
// tasks per SM) through the pipelined kernel.
bool fuse_preferred(const RowArgs& a, bool tv_only) {
    const int T = make_fuse_plan(a.B, a.K, a.nvec, 1).T;
    int sms = 0, dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { cudaGetLastError(); return false; }
    const long long tasks = (long long)a.B * (tv_only ? 1 : a.K + 1) * T;
    if (T > 32 || tasks < 2LL * sms) return false;       // (a call of a few tasks is all start-up: 0.038 against 0.031 ms)
    if (tv_only || T <= 11 || a.K == 1) return true;
    return tasks <= 40LL * sms;
}

cudaError_t fuse_verify(const RowArgs& a, const Plan& p, const int32_t* draft_tokens, const float* u_accept,
                        const float* u_final, VerifyOut o, char* ws, cudaStream_t stream, bool* launched, bool tv_only,
                        float* s_aux) {
    *launched = false;
    const int grid_max = tv_only ? (a.dt == 0 ? fuse_grid<0, true>() : fuse_grid<1, true>())
                                 : (a.dt == 0 ? fuse_grid<0, false>() : fuse_grid<1, false>());
    const int ups = tv_only ? 1 : a.K + 1;
    const FusePlan fp = make_fuse_plan(a.B, a.K, a.nvec, ups);
    // the T slices of a unit must be in flight together: T <= grid; and all tasks counted in an int
    if (grid_max < 1 || fp.T > grid_max) return cudaSuccess;
    const int tps = tv_only ? fp.T : a.K * fp.T + (fp.T + 1) / 2;
    const long long total = (long long)a.B * tps;
    if (total > 0x7fff0000LL) return cudaSuccess;
    char* w = ws + p.off_fuse;
    FuseArgs fa;
    fa.r = a; fa.draft_tokens = draft_tokens; fa.u_accept = u_accept; fa.u_final = u_final; fa.o = o;
    fa.s_aux = tv_only ? s_aux : nullptr; fa.tv_mode = tv_only ? 1 : 0; fa.ups = ups; fa.tps = tps;
    fa.T = fp.T; fa.slice_vecs = fp.slice_vecs;
    const int expire = take_expire_wait();
    fa.expire = expire == 2 ? 1 : 0;
    fa.kappa = draw_kappa();
    fa.wait_failed = reinterpret_cast<int*>(w) + 1;
    fa.fb_count = reinterpret_cast<unsigned long long*>(w + kFbCountOffset);
    fa.fb_list = reinterpret_cast<FbRec*>(w + fp.off_fbrec);
    fa.seqcnt = reinterpret_cast<int*>(w + fp.off_seqcnt);
    fa.rec = reinterpret_cast<FRec*>(w + fp.off_rec);
    fa.mass = reinterpret_cast<double*>(w + fp.off_mass);
    fa.wexp = reinterpret_cast<int2*>(w + fp.off_wexp);
    fa.sauxp = (tv_only && s_aux) ? reinterpret_cast<double*>(w + fp.off_saux) : nullptr;
    fa.smass = reinterpret_cast<double*>(w + fp.off_smass);
    fa.rows = reinterpret_cast<FRow*>(w + fp.off_rows);
    cudaError_t e = cudaMemsetAsync(w, 0, fp.zero_bytes, stream);
    if (e != cudaSuccess) return e;
    const int grid = (int)(total < grid_max ? total : grid_max);
    if (grid < fp.T) return cudaSuccess;
    if (g_ev_start) cudaEventRecord(g_ev_start, stream);
    {
        // A cooperative launch: the device takes the grid only as a whole, so CTAs of two such grids (two streams) cannot
        // end up holding SMs while each waits for partners that found no room.
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeCooperative;
        attr[0].val.cooperative = 1;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid); cfg.blockDim = dim3(FT); cfg.dynamicSmemBytes = kFuseSmem; cfg.stream = stream;
        cfg.attrs = attr; cfg.numAttrs = 1;
        const int tot = (int)total;
        if (tv_only) e = a.dt == 0 ? cudaLaunchKernelEx(&cfg, k_fuse<0, true>, fa, tot) : cudaLaunchKernelEx(&cfg, k_fuse<1, true>, fa, tot);
        else e = a.dt == 0 ? cudaLaunchKernelEx(&cfg, k_fuse<0, false>, fa, tot) : cudaLaunchKernelEx(&cfg, k_fuse<1, false>, fa, tot);
        if (e == cudaErrorCooperativeLaunchTooLarge) { cudaGetLastError(); return cudaSuccess; }     // no room for the whole grid: the caller takes the pipelined kernel
        if (e != cudaSuccess) return e;
    }
    e = cudaGetLastError();
    if (g_ev_stop) cudaEventRecord(g_ev_stop, stream);
    if (e != cudaSuccess) return e;
    *launched = true;
    if (tv_only) return cudaSuccess;
    // the fp64 re-draw of the listed sequences, on the same workspace head and list
    PipePlan wp = make_pipe_plan(a.B, a.K, a.nvec, a.dt);
    wp.off_xsdone = fp.off_xsdone; wp.off_xdone = fp.off_xdone; wp.off_xsum = fp.off_xsum; wp.off_xmass = fp.off_xmass;
    return redraw_launch(a, u_final, o, fa.fb_count, fa.fb_list, a.B, fa.wait_failed, w, wp, stream, expire == 1);
}

}  // namespace bebop
