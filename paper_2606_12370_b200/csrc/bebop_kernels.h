// Internal interface between the C-ABI entry points and the kernel launchers.
#pragma once
#include <climits>
#include <cmath>
#include <cuda_runtime.h>
#include <stdint.h>

#include "bebop_common.cuh"
#include "bebop_layout.h"

namespace bebop {

// Addressing of the logit rows of a batch.  Verify: t_seq_rows = K+1,
// d_seq_rows = K.  TV of N row pairs: B = N, K = 1, both = 1.
struct RowArgs {
    const char* target;
    const char* draft;
    int64_t t_row_bytes, d_row_bytes;   // ld * sizeof(element)
    int64_t t_seq_rows, d_seq_rows;
    const int32_t* draft_len;           // [B] or nullptr (= K)
    const float* temperature;           // [B] or nullptr (= temperature_all)
    float temperature_all;
    int B, K, V, dt, nvec, nsplit;
};

struct VerifyOut {
    int32_t* accept_len;   // [B]
    int32_t* out_tokens;   // [B, K+1]
    float* tv;             // [B, K] or nullptr
    float* p_draft;        // [B, K] or nullptr
    float* q_draft;        // [B, K] or nullptr
    int32_t* row_status;   // [B] or nullptr
};

cudaError_t general_verify(const RowArgs& a, const Plan& p, const int32_t* draft_tokens,
                           const float* u_accept, const float* u_final, VerifyOut o, char* ws,
                           cudaStream_t stream);
cudaError_t general_tv(const RowArgs& a, const Plan& p, float* tv, float* s_aux, int32_t* row_status,
                       char* ws, cudaStream_t stream);
cudaError_t general_greedy(const RowArgs& a, const Plan& p, const int32_t* draft_tokens,
                           int32_t* accept_len, int32_t* out_tokens, int32_t* row_status, char* ws,
                           cudaStream_t stream);

// Test hook: the number of the device-side wait that the next call lets give up at once (0: none); reading it clears it.
int take_expire_wait();
// Test hook: the factor of the fast draw's error bound (4 unless a test has set another value).
float draw_kappa();
void pipe_set_events(cudaEvent_t start, cudaEvent_t stop);   // bracket the main kernel of the next calls (nullptr: off)

// fp64 re-draw of the sequences a kernel listed (bebop_redraw.cu); `w` is the pipelined kernel's workspace laid out by `wp`.
// Launched behind the pipelined kernel, it follows the list while that kernel still runs: the low half of
// `fb_count` is the number of listed sequences so far, the high half the number of sequences whose draw is
// decided, `expect` of them in all.  It also turns a device-side wait that gave up (`wait_failed`) into status
// bit ST_WAIT of every row.
cudaError_t redraw_launch(const RowArgs& a, const float* u_final, VerifyOut o, const unsigned long long* fb_count,
                          const FbRec* fb_list, int expect, int* wait_failed, char* w,
                          const PipePlan& wp, cudaStream_t stream, bool expire_list_wait = false);

// Pipelined kernel (bebop_pipe.cu): a ticket schedule with a producer warp that stages every task's
// logits in shared memory by bulk copies while the other warps compute; same contract.  With `tv_only` it is
// bebop_tv: B row pairs (K = 1), o.tv and s_aux the outputs, no tokens, no uniforms, no draw.
bool pipe_supported(const RowArgs& a);
cudaError_t pipe_verify(const RowArgs& a, const Plan& p, const int32_t* draft_tokens,
                        const float* u_accept, const float* u_final, VerifyOut o, char* ws,
                        cudaStream_t stream, bool* launched, bool tv_only = false, float* s_aux = nullptr);

// Fused kernel (bebop_fuse.cu): every row read and exponentiated once, the exponentials parked in tensor memory
// between the softmax statistics and the residuals; same contract as pipe_verify.  fuse_preferred says whether,
// by measurement, it is the faster of the two for the shape.
bool fuse_supported(const RowArgs& a);
bool fuse_preferred(const RowArgs& a, bool tv_only);
cudaError_t fuse_verify(const RowArgs& a, const Plan& p, const int32_t* draft_tokens,
                        const float* u_accept, const float* u_final, VerifyOut o, char* ws,
                        cudaStream_t stream, bool* launched, bool tv_only = false, float* s_aux = nullptr);

// The greedy mode through the pipelined kernel: one sweep over the target rows (maximum and lowest index per
// slice), then a small kernel that merges the slices and runs the argmax match.
cudaError_t pipe_greedy(const RowArgs& a, const Plan& p, const int32_t* draft_tokens, int32_t* accept_len,
                        int32_t* out_tokens, int32_t* row_status, char* ws, cudaStream_t stream, bool* launched);

}  // namespace bebop
