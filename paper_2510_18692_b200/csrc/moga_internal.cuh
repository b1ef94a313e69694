// Internal declarations shared by the kernels of libmoga.so (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/moga.h"

namespace moga {

// ---------------------------------------------------------------------------
// Workspace layout.  The first 256 bytes are the header every stage shares:
//   word 0: device status (moga_status), word 1: detail, word 2: attention work
//   counter.  Scratch for the sort and the attention scheduler follows, then
//   (moga_forward only) the intermediate tensors.
// ---------------------------------------------------------------------------
constexpr size_t kWsAlign = 256;
constexpr int kSortChunk = 4096;   // assignments handled by one sort block
constexpr int kMaxM = 64;
constexpr int kMaxK = 8;

struct WsLayout {
  size_t header;      // 256 B
  size_t sort_hist;   // int32 [B, nblk, M]   per-block histograms, then bases
  size_t sched;       // int32 [B, 3, M+1]    attention schedule (order, tile prefix, ...)
  size_t wsplit;      // bf16 [3, MP, C]      router weight split into three bf16 parts (MP <= 64)
  size_t stats;       // int32 + float [B, nblk, M] per-block counts and gate sums (Eq. 6-8)
  size_t redo;        // int32 [4 + 2 * items]  work items the CTA-pair attention kernel hands to the exact path
  size_t scratch_end; // == moga_scratch_bytes
  size_t gid, gate, perm, inv, offsets, asg;  // routing results (asg: assignment index per sorted position)
  size_t Qp, Kp, Vp, Op;                 // permuted tensors
  size_t total;       // == moga_workspace_bytes
  int nblk;           // sort blocks per batch item
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline size_t elem_size(int dtype) { return dtype == MOGA_BF16 ? 2 : 4; }

inline WsLayout ws_layout(const moga_shape& s) {
  WsLayout L{};
  size_t T = (size_t)s.N * s.k;
  L.nblk = (int)((T + kSortChunk - 1) / kSortChunk);
  if (L.nblk < 1) L.nblk = 1;
  size_t off = 0;
  L.header = off;      off = align_up(off + 256, kWsAlign);
  L.sort_hist = off;   off = align_up(off + sizeof(int32_t) * (size_t)s.B * L.nblk * s.M, kWsAlign);
  L.sched = off;       off = align_up(off + sizeof(int32_t) * (size_t)s.B * 4 * (s.M + 1) + 64, kWsAlign);
  L.wsplit = off;      off = align_up(off + sizeof(uint16_t) * 3 * (size_t)kMaxM * s.C, kWsAlign);
  L.stats = off;       off = align_up(off + 2 * sizeof(int32_t) * (size_t)s.B * L.nblk * s.M, kWsAlign);
  {
    const size_t items = ((T + 255) / 256 + (size_t)s.M) * (size_t)s.B * (size_t)s.H;
    L.redo = off;      off = align_up(off + sizeof(int32_t) * (4 + 2 * items), kWsAlign);
  }
  L.scratch_end = off;
  L.gid = off;         off = align_up(off + sizeof(int32_t) * (size_t)s.B * T, kWsAlign);
  L.gate = off;        off = align_up(off + sizeof(float) * (size_t)s.B * T, kWsAlign);
  L.perm = off;        off = align_up(off + sizeof(int32_t) * (size_t)s.B * T, kWsAlign);
  L.inv = off;         off = align_up(off + sizeof(int32_t) * (size_t)s.B * T, kWsAlign);
  L.offsets = off;     off = align_up(off + sizeof(int32_t) * (size_t)s.B * (s.M + 1), kWsAlign);
  L.asg = off;         off = align_up(off + sizeof(int32_t) * (size_t)s.B * T, kWsAlign);
  size_t row = (size_t)s.B * s.H * T * s.D * elem_size(s.dtype);
  L.Qp = off;          off = align_up(off + row, kWsAlign);
  L.Kp = off;          off = align_up(off + row, kWsAlign);
  L.Vp = off;          off = align_up(off + row, kWsAlign);
  L.Op = off;          off = align_up(off + row, kWsAlign);
  L.total = off;
  return L;
}

struct Strides { long long b, h, n; };
inline Strides qkv_strides(const moga_shape& s) {
  if (s.q_stride_b == 0 && s.q_stride_h == 0 && s.q_stride_n == 0)
    return {(long long)s.H * s.N * s.D, (long long)s.N * s.D, (long long)s.D};
  return {s.q_stride_b, s.q_stride_h, s.q_stride_n};
}

// Device status word: the first non-zero code wins.
__device__ __forceinline__ void report_status(uint32_t* header, uint32_t code, uint32_t detail) {
  if (atomicCAS(header, 0u, code) == 0u) header[1] = detail;
}

// Stage launchers (each returns MOGA_OK or MOGA_ERR_CUDA; arguments already validated).
moga_status launch_route(const moga_shape& s, const void* X, const float* Wr, const float* bias,
                         int32_t* gid, float* gate, float* logits, cudaStream_t st);
moga_status launch_route_mma(const moga_shape& s, const WsLayout& L, const void* X, const float* Wr,
                             const float* bias, int32_t* gid, float* gate, float* logits, char* ws,
                             cudaStream_t st);
moga_status launch_balance_stats(const moga_shape& s, const WsLayout& L, const int32_t* gid, const float* gate,
                                 float alpha, float* F, float* P, float* loss, char* ws, cudaStream_t st);
// asg (optional, [B, T]): the assignment index n*k + j that sits at each sorted position
moga_status launch_sort(const moga_shape& s, const WsLayout& L, const int32_t* gid, int32_t* perm,
                        int32_t* inv, int32_t* offsets, char* ws, cudaStream_t st, int32_t* asg = nullptr);
// inv (optional): with it and 2 <= k <= 4 the copy runs token by token (each row read once, written k times)
moga_status launch_gather(const moga_shape& s, const int32_t* perm, const void* Q, const void* K,
                          const void* V, void* Qp, void* Kp, void* Vp, cudaStream_t st,
                          const int32_t* inv = nullptr);
moga_status launch_unpermute(const moga_shape& s, const void* Op, const int32_t* inv,
                             const float* gate, void* O, cudaStream_t st);
moga_status launch_attn_f32(const moga_shape& s, const float* Qp, const float* Kp, const float* Vp,
                            const int32_t* offsets, float* Op, float* lse, cudaStream_t st);
moga_status launch_attn_bf16(const moga_shape& s, const WsLayout& L, const void* Qp, const void* Kp,
                             const void* Vp, const int32_t* offsets, void* Op, float* lse, char* ws,
                             cudaStream_t st);

// Top-1 routing only: the attention epilogue writes gate * row straight to token order in O
// (the gated inverse permutation of Eq. 5), so no permuted output and no unpermute pass.
moga_status launch_attn_bf16_scatter(const moga_shape& s, const WsLayout& L, const void* Qp, const void* Kp,
                                     const void* Vp, const int32_t* offsets, const int32_t* perm,
                                     const float* gate, void* O, char* ws, cudaStream_t st);

// Top-2 routing: the attention epilogue adds gate * row into a zeroed O in token order (Eq. 5's
// sum over the two assignments as two commutative additions), so there is no permuted output and
// no unpermute pass.  asg: assignment index per sorted position; gate: [B, N, k].
moga_status launch_attn_bf16_add(const moga_shape& s, const WsLayout& L, const void* Qp, const void* Kp,
                                 const void* Vp, const int32_t* offsets, const int32_t* asg, const float* gate,
                                 void* O, char* ws, cudaStream_t st);
// Gradients of the bf16 group attention in sorted order (d_head = 128); see csrc/attn_bwd.cu.
moga_status launch_attn_backward(const moga_shape& s, const WsLayout& L, const void* Qp, const void* Kp,
                                 const void* Vp, const void* Op, const float* lse, const float* gate,
                                 const int32_t* perm, const int32_t* inv, const int32_t* offsets, const void* dO,
                                 void* dOp, float* delta, void* dQp, void* dKp, void* dVp, float* dgate, char* ws,
                                 cudaStream_t st);
// The same gradients for fp32 tensors on the fp32 ALUs (d_head 64 or 128); see csrc/attn_bwd_f32.cu.
moga_status launch_attn_backward_f32(const moga_shape& s, const float* Qp, const float* Kp, const float* Vp,
                                     const float* Op, const float* lse, const float* gate, const int32_t* perm,
                                     const int32_t* inv, const int32_t* offsets, const float* dO, float* dOp,
                                     float* delta, float* dQp, float* dKp, float* dVp, float* dgate,
                                     cudaStream_t st);
// Router backward (csrc/route_bwd.cu): scratch bytes and the launches.
size_t route_backward_bytes(const moga_shape& s);
moga_status launch_route_backward(const moga_shape& s, const void* X, const float* Wr, const float* logits,
                                  const int32_t* gid, const float* dgate, void* dX, float* dWr, float* dbias, char* ws,
                                  cudaStream_t st);
void set_fused_topk(int on);
bool fused_topk();

// Static groups (Sec. 3.2): attention with caller-given query / key ranges per group, shared by
// all batch items.  header: the device status word the kernel reports into (not cleared here);
// sched: 2*B*G + 1 int32 of schedule scratch.  The epilogue either stores the rows in the order
// of the query list (both pointers null), sends row p to token token_list[p] of a contiguous
// [B, H, N, D] output, or (rows already in token order) stores the mean of the row and the rows
// of mean_a and mean_b at the same place.  The last two need d_head = 128.
struct StaticEpilogue {
  const int32_t* token_list;
  const void* mean_a;
  const void* mean_b;
};
moga_status launch_attn_bf16_static(const moga_shape& s, int G, long long Tq, long long Tkv, const void* Qs,
                                    const void* Ks, const void* Vs, const int32_t* q_offsets,
                                    const int32_t* kv_offsets, void* Os, float* lse, uint32_t* header, char* sched,
                                    const StaticEpilogue& epi, cudaStream_t st);
moga_status launch_attn_f32_groups(int B, int H, int D, float scale, int G, int Tq, int Tkv, const float* Qp,
                                   const float* Kp, const float* Vp, const int32_t* q_offsets,
                                   const int32_t* kv_offsets, int off_stride, float* Op, float* lse,
                                   cudaStream_t st);
void set_attn_kernel(int mode);
moga_status launch_gather_list(const moga_shape& s, const int32_t* idx, int L, const void* src, void* dst,
                               cudaStream_t st);
moga_status launch_frame_offsets(int32_t* off, int F, int tokens_per_frame, cudaStream_t st);
moga_status launch_mean3(const moga_shape& s, const void* A, const void* Bs, const int32_t* inv_b, const void* C,
                         void* O, cudaStream_t st);
moga_status stga_build_host(int F, int Hh, int Ww, int wh, int ww, const int32_t* shot_starts, int n_shots,
                            int tg, int augment, int32_t* q_idx, int32_t* q_inv, int32_t* q_offsets,
                            int32_t* kv_idx, int32_t* kv_offsets, int32_t* G_out, int32_t* Tkv_out);

// Multiprocessor count of the current device (asked every time: a process may drive several
// kinds of GPU, and the attribute query is a cached host-side lookup).
inline bool current_sm_count(int* n) {
  int dev = 0;
  return cudaGetDevice(&dev) == cudaSuccess &&
         cudaDeviceGetAttribute(n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && *n > 0;
}

#define MOGA_CUDA_OK(expr)                                   \
  do {                                                       \
    cudaError_t e__ = (expr);                                \
    if (e__ != cudaSuccess) return MOGA_ERR_CUDA;            \
  } while (0)

}  // namespace moga
