// Device code shared by the pipelined kernel and the re-draw kernels: workspace records, small helpers,
// the residual arithmetic and the draw bound.
#pragma once
#include "bebop_kernels.h"
#include "bebop_ptx.cuh"

namespace bebop {

namespace {

constexpr int WT = 256;               // threads per CTA
constexpr int WW = WT / 32;
constexpr int SLICE_VECS = kPipeSliceVecs;   // vectors per row slice, at most
constexpr int BEBOP_MAX_K_INT = 32;
constexpr int MAX_SLICES = 64;
constexpr int E_EMPTY = INT_MIN / 2;
constexpr uint32_t kSpin = 1u << 22;

struct __align__(16) P1Part { double s; int e; float m; };             // per (row, slice); m = NaN marks a non-finite logit
struct __align__(16) RowStat { double inv_s; int e; int st; };   // per row, after the merge: 1/S, exponent E, status bits | kRowValid
constexpr int kRowValid = 0x100;
// Records that CTAs pass to each other through global memory (the memory starts at zero).  A record is two
// 8-byte words, written by one store of two 64-bit elements and read by one such load.  The PTX memory model
// treats a vector access as its elements accessed in no particular order, each 64-bit element being a single
// copy; so every record is laid out with BOTH words non-zero once written (a zero sum is stored as -0.0, counts
// and exponents carry an offset or a low mark bit), and a reader takes a record only when both words are
// non-zero: each word then is the written one.  No fence is needed for that, and none is used.
template <typename T> __device__ __forceinline__ void rec_words(const T& v, unsigned long long* w) {
    static_assert(sizeof(T) == 16, "16-byte record");
    memcpy(w, &v, 16);
}
template <typename T> __device__ __forceinline__ void st16(T* p, const T& v) {
    unsigned long long w[2];
    rec_words(v, w);
    asm volatile("st.relaxed.gpu.global.v2.b64 [%0], {%1, %2};" :: "l"(p), "l"(w[0]), "l"(w[1]) : "memory");
}
template <typename T> __device__ __forceinline__ bool rec_valid(const T& v) {
    unsigned long long w[2];
    rec_words(v, w);
    return w[0] != 0ull && w[1] != 0ull;
}
// a sum that may be exactly zero, made non-zero in its bits
__device__ __forceinline__ double nonzero_bits(double x) { return x == 0.0 ? -0.0 : x; }
struct __align__(16) DPart { double tot; float sq; int pad; };        // per (sequence, slice)
struct __align__(16) SeqInfo {          // per sequence, written by phase A
    int n;                              // accept count (stop position); -1: fatal
    int draw_row;                       // row whose residual is drawn from (n, or L for the bonus row); -1 none
    int pad0;
    int pad;
};

struct PipeArgs {
    RowArgs r;
    const int32_t* draft_tokens;
    const float* u_accept;
    const float* u_final;
    VerifyOut o;
    int* stop;
    unsigned long long* fb_count;   // [1] low half: sequences listed for the fp64 re-draw; high half: sequences whose
                                    // draw is decided (token written, listed, or none to come); zeroed with the workspace
    FbRec* fb_list;       // [B] (zeroed with the workspace: a record is valid once its b1 is non-zero)
    // workspace
    int* ticket;          // [1]
    int* wait_failed;     // [1]
    int* p1done;          // [B] rows of the sequence merged
    int* p2done;          // [B] partials of the sequence's second sweep delivered
    int* ddone;           // [B] ... of them, partials of the row the sequence's token is drawn from
    int* rowcnt;          // [B][2K+1] pipelined kernel: softmax partials delivered per row
    P1Part* part;         // [B][2K+1][T]
    RowStat* rstat;       // [B][2K+1]
    unsigned long long* dacc;    // [B][2T][2] draw-row mass (2^-58) and sum of squares (2^-40), each << 4 | parts added
    unsigned long long* tvacc;   // [B][K] TV sum in 2^-40 units << 16 | parts added
    SeqInfo* sinfo;       // [B]
    int ntickets;
    int expire;                      // test hook: the producers' wait for a sequence's accept scan gives up at once
    float kappa;                     // factor of the fast draw's error bound (kDrawKappa; a test hook can change it)
    int tv_only;                     // bebop_tv: row pairs only (no bonus row, no accept test, no draw)
    float* s_aux;                    // tv_only: [B] sum of q over the tokens with q <= p, or nullptr
    unsigned long long* sacc;        // [B][K] that sum in 2^-40 units << 16 | parts added
    int T, slice_vecs;
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
// The draw of a sequence is decided: count it (high half), and when it goes to the fp64 re-draw take its place in
// the list (low half).  One word, so that a reader who sees all sequences decided also sees the final list length.
__device__ __forceinline__ void draw_decided(unsigned long long* w) {
    asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(w), "l"(1ull << 32) : "memory");
}
__device__ __forceinline__ int draw_listed(unsigned long long* w) {
    return (int)(atomicAdd(w, (1ull << 32) | 1ull) & 0xffffffffull);
}
// Workspace records written by other CTAs of this launch: one load of two 64-bit elements, at GPU scope (the L1 of
// this SM may hold an older copy of the line).  Use the record only if rec_valid() says both words are there.
template <typename T> __device__ __forceinline__ T ld_cg(const T* p) {
    static_assert(sizeof(T) == 16, "16-byte record");
    unsigned long long w[2];
    asm volatile("ld.relaxed.gpu.global.v2.b64 {%0, %1}, [%2];" : "=l"(w[0]), "=l"(w[1]) : "l"(p) : "memory");
    T r;
    memcpy(&r, w, 16);
    return r;
}
// SeqInfo in memory: n and draw_row (both >= -1) are stored plus 2 and pad as 1, so that both words are non-zero (pad0 is
// the bit pattern of a positive float).  In registers the fields are plain again and pad says whether the record was there.
__device__ __forceinline__ void st_seq(SeqInfo* p, const SeqInfo& s) {
    SeqInfo m; m.n = s.n + 2; m.draw_row = s.draw_row + 2; m.pad0 = s.pad0; m.pad = 1;
    st16(p, m);
}
__device__ __forceinline__ SeqInfo ld_seq(const SeqInfo* p) {
    const SeqInfo m = ld_cg(p);
    SeqInfo s; s.n = m.n - 2; s.draw_row = m.draw_row - 2; s.pad0 = m.pad0; s.pad = rec_valid(m) ? 1 : 0;
    return s;
}
// FbRec in memory: the exponents as 2 e + 1 (b1 = sequence + 1 is non-zero already)
__device__ __forceinline__ void st_fb(FbRec* p, int b, int kp, int ep, int eq) {
    FbRec r; r.b1 = b + 1; r.kp = kp; r.ep = 2 * ep + 1; r.eq = 2 * eq + 1;
    st16(p, r);
}
__device__ __forceinline__ FbRec ld_fb(const FbRec* p, bool* valid) {
    const FbRec m = ld_cg(p);
    *valid = rec_valid(m);
    FbRec r; r.b1 = m.b1; r.kp = m.kp; r.ep = m.ep >> 1; r.eq = m.eq >> 1;      // (2 e + 1) >> 1 = e, for negative e too
    return r;
}
__device__ __forceinline__ bool spin_ge(const int* p, int want) {
    for (uint32_t i = 0; i < kSpin; ++i) {
        if (ld_acquire(p) >= want) return true;
        __nanosleep(64);
    }
    return false;
}

// The error bound a draw must clear.  The residual is formed from fp32 exponentials (ex2.approx:
// 2 ulp), an fp32 argument (half an ulp of a number below 64, times 2^arg) and one fp32 rounding of
// the product with the two-float normaliser, so each p, q carries a relative error below
// delta = 2^-22; the errors of different tokens are independent, hence the error of a prefix sum is
// of the order delta * sqrt(sum p^2 + q^2), and so is the part common to all tokens, the error of the
// fp32-summed normalisers.  Measured on 40 000 draws with the certification switched off, the largest
// error that changed a token was 0.1 * delta * sqrt(sum p^2 + q^2); kappa = 4 leaves a factor 40 over
// that.
constexpr double kDrawKappa = 4.0;
__device__ __forceinline__ double draw_bound(double sumsq, double kappa = kDrawKappa) {
    const double delta = 2.384185791015625e-07;   // 2^-22
    return kappa * delta * sqrt(sumsq) + 1e-300;
}

// c = log2(e) / tau in fp32, and 2^(x * c - E): the product is exact inside the fma, so the argument
// carries one rounding of half an ulp of itself.  The rounding of c itself acts like a temperature
// changed by at most 2^-24 relative; over a prefix of the vocabulary its effect, 2^-24 * sum p (z - zbar) / tau,
// is a sum of zero-mean terms of the size draw_bound() already allows per token.
struct TempScale { float hi; };
__device__ __forceinline__ TempScale temp_scale(float tau) {
    TempScale r; r.hi = kLog2e / (tau_ok(tau) ? tau : 1.f);
    return r;
}
__device__ __forceinline__ float exp2_scaled(float x, const TempScale& t, float Ef) {
    return ex2f(fmaf(x, t.hi, -Ef));
}
// E = ceil(m * c) of a maximum m, as int and float: any integer near m * c serves as the reference, and
// integer references make every merge of partial sums an exact power-of-two scaling.
__device__ __forceinline__ int ref_exponent(float m, const TempScale& t, float* Ef) {
    const float th = fminf(fmaxf(m * t.hi, -4.0e6f), 4.0e6f);
    return ceil_alu(th, Ef);
}

struct DrawShared {
    double redd[WW];
    float redf[2][WW];
    int redi[WW];
    int ticket, phase, index;
    // D-phase broadcast
    double base, Ttarget, bound;
    int owner_slice;
};

__device__ __forceinline__ const char* row_ptr(const RowArgs& R, int b, int r) {
    // r in [0, K]: target row r; r in [K+1, 2K]: draft row r - (K+1)
    const int K = R.K;
    return r <= K ? R.target + ((int64_t)b * R.t_seq_rows + r) * R.t_row_bytes
                  : R.draft + ((int64_t)b * R.d_seq_rows + (r - K - 1)) * R.d_row_bytes;
}

// residuals of one vector pair: p = 2^(x*c - E_p) / S_p, q likewise
struct RowScale { float ef, inv, inv_lo; };     // exponent E; 1/S = inv + inv_lo to about 2^-48
__device__ __forceinline__ RowScale row_scale(const RowStat& s) {
    RowScale r; r.ef = (float)s.e; r.inv = (float)s.inv_s; r.inv_lo = (float)(s.inv_s - (double)r.inv);
    return r;
}
__device__ __forceinline__ RowScale no_row() { RowScale r; r.ef = 0.f; r.inv = 0.f; r.inv_lo = 0.f; return r; }

// FINE (the rows a token is drawn from): the normaliser enters as two floats, so that its rounding to fp32
// is not an error common to all tokens of the row; what is left is one rounding per token.
// A row that is not there (the draft row of a bonus task, vectors beyond the slice) is passed as -inf logits
// with a zero normaliser: it gives q = 0 without a branch.
template <int DT, bool FINE>
__device__ __forceinline__ void residual_vec(const uint4& rp, const uint4& rq, const TempScale& c, const RowScale& P,
                                             const RowScale& Q, float* r, float* sq) {
    constexpr int VEC = Elem<DT>::VEC;
    float fp[VEC], fq[VEC];
    unpack<DT>(rp, fp);
    unpack<DT>(rq, fq);
#pragma unroll
    for (int i = 0; i < VEC; ++i) {
        const float ap = exp2_scaled(fp[i], c, P.ef);
        const float aq = exp2_scaled(fq[i], c, Q.ef);
        // explicit roundings: a contracted p - a*inv would leave rounding dust when the rows are equal
        const float p = FINE ? __fmaf_rn(ap, P.inv_lo, __fmul_rn(ap, P.inv)) : __fmul_rn(ap, P.inv);
        const float q = FINE ? __fmaf_rn(aq, Q.inv_lo, __fmul_rn(aq, Q.inv)) : __fmul_rn(aq, Q.inv);
        r[i] = fmaxf(p - q, 0.f);
        if (sq) { *sq = fmaf(p, p, *sq); *sq = fmaf(q, q, *sq); }
    }
}

}  // namespace

}  // namespace bebop
