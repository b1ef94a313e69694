// moga_forward_host: the whole forward from HOST buffers.  The copies over the host link
// are several times longer than the kernels (23 GB in, 5.75 GB out against ~0.19 s of
// compute at the minute-long workload), so the call is organised around them: one stream
// copies X and then Q/K/V head chunk by head chunk, the caller's stream routes, sorts and
// runs gather + group attention per chunk as soon as its inputs have landed, and a third
// stream returns each chunk of O while the next one is computed.  Everything lives in a
// caller-provided device arena; the library creates two streams and a fixed pool of events
// per device on first use and allocates no memory.
#include <mutex>

#include "moga_internal.cuh"

namespace moga {
namespace {

constexpr int kMaxChunks = 64;

struct Pipe {
  bool ready = false;
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start = nullptr, x_in = nullptr;
  cudaEvent_t chunk_in[kMaxChunks], gathered[kMaxChunks], done[kMaxChunks], chunk_out[kMaxChunks];
};

constexpr int kMaxDevices = 64;
Pipe g_pipes[kMaxDevices];
std::mutex g_pipe_mutex;

moga_status get_pipe(Pipe** out) {
  int dev = 0;
  MOGA_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return MOGA_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  Pipe& p = g_pipes[dev];
  if (!p.ready) {
    MOGA_CUDA_OK(cudaStreamCreateWithFlags(&p.in, cudaStreamNonBlocking));
    MOGA_CUDA_OK(cudaStreamCreateWithFlags(&p.out, cudaStreamNonBlocking));
    MOGA_CUDA_OK(cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming));
    MOGA_CUDA_OK(cudaEventCreateWithFlags(&p.x_in, cudaEventDisableTiming));
    for (int i = 0; i < kMaxChunks; ++i) {
      MOGA_CUDA_OK(cudaEventCreateWithFlags(&p.chunk_in[i], cudaEventDisableTiming));
      MOGA_CUDA_OK(cudaEventCreateWithFlags(&p.gathered[i], cudaEventDisableTiming));
      MOGA_CUDA_OK(cudaEventCreateWithFlags(&p.done[i], cudaEventDisableTiming));
      MOGA_CUDA_OK(cudaEventCreateWithFlags(&p.chunk_out[i], cudaEventDisableTiming));
    }
    p.ready = true;
  }
  *out = &p;
  return MOGA_OK;
}

struct Arena {
  size_t scratch, wr, bias, gid, gate, perm, inv, offsets, asg, X;
  size_t in[2][3];      // two staging sets of Q, K, V chunks  [B, hc, N, D]
  size_t Qp, Kp, Vp, Op;  // permuted chunk                    [B, hc, T, D]
  size_t out[2];        // two staging sets of the O chunk     [B, hc, N, D]
  size_t total;
};

Arena arena_layout(const moga_shape& s, int hc) {
  Arena a{};
  const WsLayout L = ws_layout(s);
  const size_t es = elem_size(s.dtype), T = (size_t)s.N * s.k;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t at = off;
    off = align_up(off + bytes, kWsAlign);
    return at;
  };
  a.scratch = take(L.scratch_end);
  a.wr = take(sizeof(float) * (size_t)s.C * s.M);
  a.bias = take(sizeof(float) * s.M);
  a.gid = take(sizeof(int32_t) * s.B * T);
  a.gate = take(sizeof(float) * s.B * T);
  a.perm = take(sizeof(int32_t) * s.B * T);
  a.asg = take(sizeof(int32_t) * s.B * T);
  a.inv = take(sizeof(int32_t) * s.B * T);
  a.offsets = take(sizeof(int32_t) * s.B * (s.M + 1));
  a.X = take(es * s.B * s.N * s.C);
  const size_t tok_chunk = es * s.B * hc * (size_t)s.N * s.D, perm_chunk = es * s.B * hc * T * s.D;
  for (int i = 0; i < 2; ++i)
    for (int j = 0; j < 3; ++j) a.in[i][j] = take(tok_chunk);
  a.Qp = take(perm_chunk);
  a.Kp = take(perm_chunk);
  a.Vp = take(perm_chunk);
  a.Op = take(perm_chunk);
  for (int i = 0; i < 2; ++i) a.out[i] = take(tok_chunk);
  a.total = off;
  return a;
}

bool chunking_ok(const moga_shape& s, int hc) {
  return hc >= 1 && hc <= s.H && (s.H + hc - 1) / hc <= kMaxChunks;
}

// Heads [h0, h0 + nh) of a contiguous host tensor [B, H, N, D] <-> a contiguous device chunk [B, nh, N, D].
moga_status copy_heads(void* dst, const void* src, const moga_shape& s, int h0, int nh, bool to_device,
                       cudaStream_t st) {
  const size_t head = elem_size(s.dtype) * (size_t)s.N * s.D;
  for (int b = 0; b < s.B; ++b) {
    const size_t host_off = ((size_t)b * s.H + h0) * head, dev_off = (size_t)b * nh * head;
    if (to_device)
      MOGA_CUDA_OK(cudaMemcpyAsync(static_cast<char*>(dst) + dev_off, static_cast<const char*>(src) + host_off,
                                   head * nh, cudaMemcpyHostToDevice, st));
    else
      MOGA_CUDA_OK(cudaMemcpyAsync(static_cast<char*>(dst) + host_off, static_cast<const char*>(src) + dev_off,
                                   head * nh, cudaMemcpyDeviceToHost, st));
  }
  return MOGA_OK;
}

}  // namespace
}  // namespace moga

using namespace moga;

extern "C" {

size_t moga_forward_host_bytes(const moga_shape* s, int32_t heads_per_chunk) {
  if (moga_workspace_bytes(s) == 0 || !chunking_ok(*s, heads_per_chunk)) return 0;
  return arena_layout(*s, heads_per_chunk).total;
}

moga_status moga_forward_host(const moga_shape* s, const void* X, const float* Wr, const float* bias,
                              const void* Q, const void* K, const void* V, void* O, int32_t* gid_out,
                              float* gate_out, void* arena, size_t arena_bytes, int32_t heads_per_chunk,
                              void* stream) {
  if (s == nullptr || moga_workspace_bytes(s) == 0) {
    // reuse the shape checks of the device entry points for the precise code
    return s == nullptr ? MOGA_ERR_INVALID_ARG
                        : moga_route(s, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, 0, nullptr);
  }
  if (X == nullptr || Wr == nullptr || Q == nullptr || K == nullptr || V == nullptr || O == nullptr)
    return MOGA_ERR_INVALID_ARG;
  if (s->q_stride_b || s->q_stride_h || s->q_stride_n) return MOGA_ERR_UNSUPPORTED;   // contiguous host tensors
  if (!chunking_ok(*s, heads_per_chunk)) return MOGA_ERR_INVALID_ARG;
  const Arena A = arena_layout(*s, heads_per_chunk);
  if (arena == nullptr || arena_bytes < A.total || (reinterpret_cast<uintptr_t>(arena) & (kWsAlign - 1)))
    return MOGA_ERR_WORKSPACE;
  Pipe* P = nullptr;
  moga_status st = get_pipe(&P);
  if (st != MOGA_OK) return st;

  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  char* a = static_cast<char*>(arena);
  const WsLayout L = ws_layout(*s);
  const size_t es = elem_size(s->dtype), T = (size_t)s->N * s->k;
  const int hc = heads_per_chunk, nchunks = (s->H + hc - 1) / hc;
  char* scratch = a + A.scratch;
  float* wr_d = reinterpret_cast<float*>(a + A.wr);
  float* bias_d = bias != nullptr ? reinterpret_cast<float*>(a + A.bias) : nullptr;
  int32_t* gid = reinterpret_cast<int32_t*>(a + A.gid);
  float* gate = reinterpret_cast<float*>(a + A.gate);
  int32_t* perm = reinterpret_cast<int32_t*>(a + A.perm);
  int32_t* inv = reinterpret_cast<int32_t*>(a + A.inv);
  int32_t* offsets = reinterpret_cast<int32_t*>(a + A.offsets);

  // ---- copy-in stream: X first (routing needs it), then the Q/K/V chunks in order
  MOGA_CUDA_OK(cudaEventRecord(P->start, cs));
  MOGA_CUDA_OK(cudaStreamWaitEvent(P->in, P->start, 0));
  MOGA_CUDA_OK(cudaStreamWaitEvent(P->out, P->start, 0));
  MOGA_CUDA_OK(cudaMemcpyAsync(a + A.X, X, es * s->B * s->N * s->C, cudaMemcpyHostToDevice, P->in));
  MOGA_CUDA_OK(cudaEventRecord(P->x_in, P->in));

  // ---- caller's stream: routing and the sort
  MOGA_CUDA_OK(cudaMemcpyAsync(wr_d, Wr, sizeof(float) * (size_t)s->C * s->M, cudaMemcpyHostToDevice, cs));
  if (bias != nullptr) MOGA_CUDA_OK(cudaMemcpyAsync(bias_d, bias, sizeof(float) * s->M, cudaMemcpyHostToDevice, cs));
  MOGA_CUDA_OK(cudaMemsetAsync(scratch + L.header, 0, 256, cs));
  MOGA_CUDA_OK(cudaStreamWaitEvent(cs, P->x_in, 0));
  st = (s->dtype == MOGA_BF16 && s->route_mode == MOGA_ROUTE_AUTO)
           ? launch_route_mma(*s, L, a + A.X, wr_d, bias_d, gid, gate, nullptr, scratch, cs)
           : launch_route(*s, a + A.X, wr_d, bias_d, gid, gate, nullptr, cs);
  if (st != MOGA_OK) return st;
  // bf16 top-2: the same add epilogue as moga_forward (the results are bit-identical to it)
  const bool add_epilogue = s->dtype == MOGA_BF16 && s->k == 2 && fused_topk();
  int32_t* asg = add_epilogue ? reinterpret_cast<int32_t*>(a + A.asg) : nullptr;
  if ((st = launch_sort(*s, L, gid, perm, inv, offsets, scratch, cs, asg)) != MOGA_OK) return st;
  if (gid_out) MOGA_CUDA_OK(cudaMemcpyAsync(gid_out, gid, sizeof(int32_t) * s->B * T, cudaMemcpyDeviceToHost, cs));
  if (gate_out) MOGA_CUDA_OK(cudaMemcpyAsync(gate_out, gate, sizeof(float) * s->B * T, cudaMemcpyDeviceToHost, cs));

  for (int c = 0; c < nchunks; ++c) {
    const int h0 = c * hc, nh = (s->H - h0) < hc ? (s->H - h0) : hc, set = c & 1;
    moga_shape sub = *s;
    sub.H = nh;
    // copy-in: the staging set is free once the gather of chunk c-2 has read it
    if (c >= 2) MOGA_CUDA_OK(cudaStreamWaitEvent(P->in, P->gathered[c - 2], 0));
    const void* src[3] = {Q, K, V};
    for (int j = 0; j < 3; ++j)
      if ((st = copy_heads(a + A.in[set][j], src[j], *s, h0, nh, true, P->in)) != MOGA_OK) return st;
    MOGA_CUDA_OK(cudaEventRecord(P->chunk_in[c], P->in));
    // compute
    MOGA_CUDA_OK(cudaStreamWaitEvent(cs, P->chunk_in[c], 0));
    if ((st = launch_gather(sub, perm, a + A.in[set][0], a + A.in[set][1], a + A.in[set][2], a + A.Qp, a + A.Kp,
                            a + A.Vp, cs, inv)) != MOGA_OK)
      return st;
    MOGA_CUDA_OK(cudaEventRecord(P->gathered[c], cs));
    if (c >= 2) MOGA_CUDA_OK(cudaStreamWaitEvent(cs, P->chunk_out[c - 2], 0));   // O staging set free again
    void* Oc = a + A.out[set];
    if (s->dtype == MOGA_F32) {
      st = launch_attn_f32(sub, reinterpret_cast<const float*>(a + A.Qp), reinterpret_cast<const float*>(a + A.Kp),
                           reinterpret_cast<const float*>(a + A.Vp), offsets, reinterpret_cast<float*>(a + A.Op),
                           nullptr, cs);
      if (st == MOGA_OK) st = launch_unpermute(sub, a + A.Op, inv, gate, Oc, cs);
    } else if (add_epilogue) {
      MOGA_CUDA_OK(cudaMemsetAsync(Oc, 0, es * (size_t)s->B * nh * s->N * s->D, cs));
      st = launch_attn_bf16_add(sub, L, a + A.Qp, a + A.Kp, a + A.Vp, offsets, asg, gate, Oc, scratch, cs);
    } else if (s->k == 1) {
      st = launch_attn_bf16_scatter(sub, L, a + A.Qp, a + A.Kp, a + A.Vp, offsets, perm, gate, Oc, scratch, cs);
    } else {
      st = launch_attn_bf16(sub, L, a + A.Qp, a + A.Kp, a + A.Vp, offsets, a + A.Op, nullptr, scratch, cs);
      if (st == MOGA_OK) st = launch_unpermute(sub, a + A.Op, inv, gate, Oc, cs);
    }
    if (st != MOGA_OK) return st;
    MOGA_CUDA_OK(cudaEventRecord(P->done[c], cs));
    // copy-out
    MOGA_CUDA_OK(cudaStreamWaitEvent(P->out, P->done[c], 0));
    if ((st = copy_heads(O, Oc, *s, h0, nh, false, P->out)) != MOGA_OK) return st;
    MOGA_CUDA_OK(cudaEventRecord(P->chunk_out[c], P->out));
  }
  // the caller's stream is done when the last chunks of O are back on the host
  MOGA_CUDA_OK(cudaStreamWaitEvent(cs, P->chunk_out[nchunks - 1], 0));
  if (nchunks >= 2) MOGA_CUDA_OK(cudaStreamWaitEvent(cs, P->chunk_out[nchunks - 2], 0));
  return MOGA_OK;
}

}  // extern "C"
