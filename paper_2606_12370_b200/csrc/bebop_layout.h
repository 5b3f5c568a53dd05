// Workspace layout and launch-shape decisions shared by the host entry points
// and the kernels.  Plain host/device code, no CUDA calls.
#pragma once
#include <stddef.h>
#include <stdint.h>

namespace bebop {

// Workspace of the pipelined kernel and of the fp64 re-draw kernels.
constexpr int kPipeSliceVecs = 2048;   // 16-byte vectors per row slice, at most: one stage of the kernel's ring
// A sequence whose draw goes to the fp64 re-draw: all the re-draw kernels need to find its rows.
struct alignas(16) FbRec {
    int b1;                             // sequence + 1 (0: the record is not written yet)
    int kp;                             // 2 * draw row + (1 if the row is a residual of a target / draft pair)
    int ep, eq;                         // reference exponents of the target row and of the draft row
};
constexpr int kRedrawCut = 4;   // the fp64 re-draw cuts every row slice into so many work items
constexpr size_t kRedrawTicketOffset = 192;   // unsigned: next work item of the fp64 re-draw (zeroed head of the workspace)
constexpr size_t kFbCountOffset = 128;   // 8 bytes inside the zeroed head of the workspace: low int, sequences listed for the fp64
                                         // re-draw; high int, sequences whose draw is decided
struct PipePlan {
    int T, slice_vecs;     // slices per row, vectors per slice (multiple of 16)
    size_t off_p1done, off_p2done, off_ddone, off_xdone, off_xsdone, off_fbrec, off_rowcnt, zero_bytes;
    size_t off_xsum, off_xmass;   // fp64 re-draw: per listed sequence done counter; sums and masses per quarter slice
    size_t off_part, off_rstat, off_dpart, off_tvacc, off_sacc, off_sinfo, total;
};

static inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }
struct Plan {
    int B, K, V, dt;
    int nvec;        // 16-byte vectors per row (last one possibly ragged)
    int nsplit;      // CTAs per row in the fp32 sweeps
    int nsplit_d;    // CTAs per sequence in the fp64 draw
    int nsplit_l;    // CTAs per sequence in the list-driven fp64 draw (few sequences)
    // byte offsets into the workspace (all 256-byte aligned)
    size_t off_stats;   // float2 [B][K][2][nsplit]      (m, S) partials, fp32 sweep
    size_t off_zpart;   // float2 [B][K][nsplit]         (Z, S_aux) partials
    size_t off_stop;    // int    [B]                    stop position n, or -1 (fatal)
    size_t off_dstats;  // double2[B][2][nsplit_d]       (m, S) partials, fp64
    size_t off_dmass;   // double [B][nsplit_d]          residual / bonus mass partials
    size_t off_amax;    // float,int [B][K+1][nsplit]    argmax partials (greedy)
    size_t off_pipe;    // workspace of the pipelined kernel
    size_t off_fuse;    // workspace of the fused kernel (the same bytes)
    size_t total;
};

// Workspace of the fused kernel (bebop_fuse.cu).  A unit is a row pair or a bonus row; a sequence owns
// `ups` consecutive units (K + 1 for bebop_verify, 1 for bebop_tv); every unit is cut into T slices.
#ifndef BEBOP_FUSE_WARPS
#define BEBOP_FUSE_WARPS 16
#endif
constexpr int kFuseWarps = BEBOP_FUSE_WARPS;   // consumer warps of a group = warp chunks of a slice
#ifndef BEBOP_FUSE_VPT
#define BEBOP_FUSE_VPT 2
#endif
constexpr int kFuseSliceVecs = kFuseWarps * 32 * BEBOP_FUSE_VPT;   // 16-byte vectors per slice, at most
constexpr int kFuseMaxSlices = 128;
struct FusePlan {
    int T, slice_vecs;
    size_t units;
    // zeroed per call: head (ticket, wait flag, re-draw counters), the re-draw's per-sequence counters, its list, the
    // per-sequence count of delivered parts, the slice records
    size_t off_xdone, off_xsdone, off_fbrec, off_seqcnt, off_rec, zero_bytes;
    size_t off_mass, off_wexp, off_saux, off_smass, off_rows, off_xsum, off_xmass, total;
};


static inline PipePlan make_pipe_plan(int B, int K, int nvec, int dt, int slice_cap = kPipeSliceVecs) {
    (void)dt;
    PipePlan w;
    w.T = (nvec + slice_cap - 1) / slice_cap; if (w.T < 1) w.T = 1;
    w.slice_vecs = (((nvec + w.T - 1) / w.T) + 15) & ~15;   // halves (phase P2) stay 128-byte aligned
    const size_t NR = (size_t)(2 * K + 1);
    size_t o = 256;                                           // ticket, wait flag; at kFbCountOffset the re-draw count
    w.off_p1done = o; o += align256(sizeof(int) * (size_t)B);      // per sequence: rows merged
    w.off_p2done = o; o += align256(sizeof(int) * (size_t)B);
    w.off_ddone = o;  o += align256(sizeof(int) * (size_t)B);      // per sequence: partials of the draw row
    w.off_xdone = o;  o += align256(sizeof(int) * (size_t)B);
    w.off_xsdone = o; o += align256(sizeof(int) * (size_t)B);
    w.off_fbrec = o;  o += align256(16 * (size_t)B);          // records of the sequences whose draw goes to fp64
    w.off_rowcnt = o; o += align256(sizeof(int) * (size_t)B * NR);
    // records that readers validate by a mark inside them, and sums that start from zero
    w.off_part = o;   o += align256(16 * (size_t)B * NR * w.T);
    w.off_rstat = o;  o += align256(16 * (size_t)B * NR);
    w.off_dpart = o;  o += align256(16 * (size_t)B * 2 * w.T);
    w.off_tvacc = o;  o += align256(8 * (size_t)B * (K > 0 ? K : 1));
    w.off_sacc = o;   o += align256(8 * (size_t)B * (K > 0 ? K : 1));
    w.off_sinfo = o;  o += align256(16 * (size_t)B);
    w.zero_bytes = o;
    w.off_xsum = o;   o += align256(16 * (size_t)B * kRedrawCut * w.T);
    w.off_xmass = o;  o += align256(8 * (size_t)B * kRedrawCut * w.T * 8);
    w.total = o;
    return w;
}

static inline FusePlan make_fuse_plan(int B, int K, int nvec, int ups) {
    FusePlan f;
    f.T = (nvec + kFuseSliceVecs - 1) / kFuseSliceVecs; if (f.T < 1) f.T = 1;
    f.slice_vecs = (nvec + f.T - 1) / f.T;
    f.units = (size_t)B * (size_t)ups;
    const PipePlan wv = make_pipe_plan(B, K, nvec, 0);          // the fp64 re-draw cuts rows its own way
    size_t o = 256;
    f.off_xdone = o;  o += align256(sizeof(int) * (size_t)B);
    f.off_xsdone = o; o += align256(sizeof(int) * (size_t)B);
    f.off_fbrec = o;  o += align256(16 * (size_t)B);
    f.off_seqcnt = o; o += align256(sizeof(int) * (size_t)B);
    f.off_rec = o;    o += align256(16 * f.units * f.T * 2);
    f.zero_bytes = o;
    f.off_mass = o;   o += align256(8 * f.units * f.T * kFuseWarps);
    f.off_wexp = o;   o += align256(8 * f.units * f.T * kFuseWarps);
    f.off_saux = o;   o += align256(8 * f.units * f.T);
    f.off_smass = o;  o += align256(8 * f.units * f.T);
    f.off_rows = o;   o += align256(32 * f.units);
    f.off_xsum = o;   o += align256(16 * (size_t)B * kRedrawCut * wv.T);
    f.off_xmass = o;  o += align256(8 * (size_t)B * kRedrawCut * wv.T * 8);
    f.total = o;
    return f;
}

static inline Plan make_plan(int B, int K, int V, int dt) {
    Plan p;
    p.B = B; p.K = K; p.V = V; p.dt = dt;
    const int vec = dt == 0 ? 4 : 8;
    p.nvec = (V + vec - 1) / vec;
    // fp32 sweeps: aim at >= 4 CTAs per SM over 2*B*K rows, slices of >= 256 vectors
    long rows = (long)B * (K > 0 ? 2 * K : 1);
    long want = (4L * 148 * 8 + rows - 1) / rows;   // about four full waves of 8 CTAs per SM
    int cap = p.nvec / 256; if (cap < 1) cap = 1;
    p.nsplit = (int)(want < 1 ? 1 : want);
    if (p.nsplit > 32) p.nsplit = 32;
    if (p.nsplit > cap) p.nsplit = cap;
    long wantd = (8L * 148 + B - 1) / B;
    p.nsplit_d = (int)(wantd < 1 ? 1 : wantd);
    if (p.nsplit_d > 32) p.nsplit_d = 32;
    if (p.nsplit_d > cap) p.nsplit_d = cap;
    p.nsplit_l = 32 < cap ? 32 : cap;
    const int nsd = p.nsplit_d > p.nsplit_l ? p.nsplit_d : p.nsplit_l;
    size_t o = 0;
    const size_t Kk = (size_t)(K > 0 ? K : 1);
    p.off_stats = o;  o = align256(o + sizeof(float) * 2 * (size_t)B * Kk * 2 * p.nsplit);
    p.off_zpart = o;  o = align256(o + sizeof(float) * 2 * (size_t)B * Kk * p.nsplit);
    p.off_stop = o;   o = align256(o + sizeof(int) * (size_t)B);
    p.off_dstats = o; o = align256(o + sizeof(double) * 2 * (size_t)B * 2 * nsd);
    p.off_dmass = o;  o = align256(o + sizeof(double) * (size_t)B * nsd);
    p.off_amax = o;   o = align256(o + 8 * (size_t)B * (K + 1) * p.nsplit);
    {
        // one region for the pipelined and the fused kernel: a call runs one of them, and both keep the wait flag
        // and the re-draw's counters at the same place in its head
        const size_t wp = make_pipe_plan(B, K, p.nvec, dt).total, wf = make_fuse_plan(B, K, p.nvec, K + 1).total;
        p.off_pipe = o;
        p.off_fuse = o;   o = align256(o + (wp > wf ? wp : wf));
    }
    p.total = o;
    return p;
}

}  // namespace bebop
