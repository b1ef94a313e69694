// C ABI of libmoga.so: argument validation, workspace carving, stage launches.
#include "moga_internal.cuh"

using namespace moga;

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Shape checks shared by every entry point.  Sets *st and returns false on failure.
bool check_shape(const moga_shape* s, moga_status* st) {
  if (s == nullptr) { *st = MOGA_ERR_INVALID_ARG; return false; }
  if (s->B < 1 || s->N < 0 || s->H < 1 || s->C < 1 || s->D < 1 || s->M < 1 || s->k < 1 ||
      (s->dtype != MOGA_F32 && s->dtype != MOGA_BF16) ||
      (s->gate_mode != MOGA_GATE_SOFTMAX_ALL && s->gate_mode != MOGA_GATE_SOFTMAX_TOPK) ||
      (s->route_mode != MOGA_ROUTE_AUTO && s->route_mode != MOGA_ROUTE_ALU) ||
      !(s->scale >= 0.f) || s->scale > 3.0e38f) {
    *st = MOGA_ERR_INVALID_ARG;
    return false;
  }
  const int epv = 16 / (int)elem_size(s->dtype);
  if (s->M > kMaxM || s->k > s->M || s->k > kMaxK || (s->D != 64 && s->D != 128) ||
      (s->C % epv) != 0 || (long long)s->N * s->k >= (1ll << 31) || s->H > 65535 ||
      s->B > 65535) {
    *st = MOGA_ERR_UNSUPPORTED;
    return false;
  }
  const bool any = s->q_stride_b || s->q_stride_h || s->q_stride_n;
  if (any) {
    if (s->q_stride_b < 0 || s->q_stride_h < 0 || s->q_stride_n < s->D ||
        (s->q_stride_b % epv) || (s->q_stride_h % epv) || (s->q_stride_n % epv)) {
      *st = MOGA_ERR_INVALID_ARG;
      return false;
    }
  }
  *st = MOGA_OK;
  return true;
}

bool check_ws(void* ws, size_t have, size_t need, moga_status* st) {
  if (ws == nullptr || have < need || (reinterpret_cast<uintptr_t>(ws) & (kWsAlign - 1))) {
    *st = MOGA_ERR_WORKSPACE;
    return false;
  }
  return true;
}

moga_status clear_header(char* ws, const WsLayout& L, cudaStream_t st) {
  MOGA_CUDA_OK(cudaMemsetAsync(ws + L.header, 0, 256, st));
  return MOGA_OK;
}

#define PTR_OK(p) ((p) != nullptr && aligned16(p))

// bf16 features go to the tensor-core router when the caller provides scratch for the split
// weights and has not asked for the fp32-ALU kernel; everything else runs on the fp32 ALUs.
bool route_on_tensor_cores(const moga_shape& s, const WsLayout& L, const void* ws, size_t ws_bytes) {
  return s.dtype == MOGA_BF16 && s.route_mode == MOGA_ROUTE_AUTO && ws != nullptr &&
         ws_bytes >= L.scratch_end && (reinterpret_cast<uintptr_t>(ws) & (kWsAlign - 1)) == 0;
}

}  // namespace

extern "C" {

size_t moga_workspace_bytes(const moga_shape* s) {
  moga_status st;
  if (!check_shape(s, &st)) return 0;
  return ws_layout(*s).total;
}

size_t moga_scratch_bytes(const moga_shape* s) {
  moga_status st;
  if (!check_shape(s, &st)) return 0;
  return ws_layout(*s).scratch_end;
}

const char* moga_status_string(moga_status st) {
  switch (st) {
    case MOGA_OK: return "ok";
    case MOGA_ERR_INVALID_ARG: return "invalid argument";
    case MOGA_ERR_UNSUPPORTED: return "unsupported shape or type";
    case MOGA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case MOGA_ERR_CUDA: return "CUDA call failed";
    case MOGA_ERR_TIMEOUT: return "device-side wait timed out";
    case MOGA_ERR_INTERNAL: return "device-side consistency check failed";
  }
  return "unknown status";
}

moga_status moga_route(const moga_shape* s, const void* X, const float* Wr, const float* bias,
                       int32_t* gid, float* gate, float* logits, void* ws, size_t ws_bytes,
                       void* stream) {
  moga_status st;
  if (!check_shape(s, &st)) return st;
  if (s->N == 0) return MOGA_OK;                  // no tokens: nothing to write
  if (!PTR_OK(X) || !PTR_OK(Wr) || !PTR_OK(gid) || !PTR_OK(gate) ||
      (bias != nullptr && !aligned16(bias)) || (logits != nullptr && !aligned16(logits)))
    return MOGA_ERR_INVALID_ARG;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const WsLayout L = ws_layout(*s);
  if (route_on_tensor_cores(*s, L, ws, ws_bytes)) {
    char* w = static_cast<char*>(ws);
    if ((st = clear_header(w, L, cs)) != MOGA_OK) return st;
    return launch_route_mma(*s, L, X, Wr, bias, gid, gate, logits, w, cs);
  }
  return launch_route(*s, X, Wr, bias, gid, gate, logits, cs);
}

moga_status moga_balance_stats(const moga_shape* s, const int32_t* gid, const float* gate, float alpha,
                               float* F, float* P, float* loss, void* ws, size_t ws_bytes, void* stream) {
  moga_status st;
  if (!check_shape(s, &st)) return st;
  if (!PTR_OK(gid) || !PTR_OK(gate) || F == nullptr || P == nullptr || loss == nullptr ||
      (reinterpret_cast<uintptr_t>(F) & 3u) || (reinterpret_cast<uintptr_t>(P) & 3u) ||
      (reinterpret_cast<uintptr_t>(loss) & 3u) || !(alpha == alpha))
    return MOGA_ERR_INVALID_ARG;
  const WsLayout L = ws_layout(*s);
  if (!check_ws(ws, ws_bytes, L.scratch_end, &st)) return st;
  if (s->N == 0) return MOGA_ERR_INVALID_ARG;     // the fractions of Eq. 7-8 divide by N
  return launch_balance_stats(*s, L, gid, gate, alpha, F, P, loss, static_cast<char*>(ws),
                              static_cast<cudaStream_t>(stream));
}

moga_status moga_permute(const moga_shape* s, const int32_t* gid, const void* Q, const void* K,
                         const void* V, int32_t* perm, int32_t* inv, int32_t* offsets, void* Qp,
                         void* Kp, void* Vp, void* ws, size_t ws_bytes, void* stream) {
  moga_status st;
  if (!check_shape(s, &st)) return st;
  if (s->N == 0) {                                // no tokens: every group is empty
    if (!PTR_OK(offsets)) return MOGA_ERR_INVALID_ARG;
    MOGA_CUDA_OK(cudaMemsetAsync(offsets, 0, sizeof(int32_t) * s->B * (s->M + 1), static_cast<cudaStream_t>(stream)));
    return MOGA_OK;
  }
  if (!PTR_OK(gid) || !PTR_OK(perm) || !PTR_OK(inv) || !PTR_OK(offsets)) return MOGA_ERR_INVALID_ARG;
  const int n_out = (Qp != nullptr) + (Kp != nullptr) + (Vp != nullptr);
  if (n_out != 0 && n_out != 3) return MOGA_ERR_INVALID_ARG;
  if (n_out == 3 && (!PTR_OK(Q) || !PTR_OK(K) || !PTR_OK(V) || !aligned16(Qp) || !aligned16(Kp) ||
                     !aligned16(Vp)))
    return MOGA_ERR_INVALID_ARG;
  const WsLayout L = ws_layout(*s);
  if (!check_ws(ws, ws_bytes, L.scratch_end, &st)) return st;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  char* w = static_cast<char*>(ws);
  if ((st = clear_header(w, L, cs)) != MOGA_OK) return st;
  if ((st = launch_sort(*s, L, gid, perm, inv, offsets, w, cs)) != MOGA_OK) return st;
  if (n_out == 3) return launch_gather(*s, perm, Q, K, V, Qp, Kp, Vp, cs, inv);
  return MOGA_OK;
}

moga_status moga_group_attn(const moga_shape* s, const void* Qp, const void* Kp, const void* Vp,
                            const int32_t* offsets, void* Op, float* lse, void* ws,
                            size_t ws_bytes, void* stream) {
  moga_status st;
  if (!check_shape(s, &st)) return st;
  if (s->N == 0) return MOGA_OK;
  if (!PTR_OK(Qp) || !PTR_OK(Kp) || !PTR_OK(Vp) || !PTR_OK(offsets) || !PTR_OK(Op) ||
      (lse != nullptr && !aligned16(lse)))
    return MOGA_ERR_INVALID_ARG;
  const WsLayout L = ws_layout(*s);
  if (!check_ws(ws, ws_bytes, L.scratch_end, &st)) return st;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  char* w = static_cast<char*>(ws);
  if ((st = clear_header(w, L, cs)) != MOGA_OK) return st;
  if (s->dtype == MOGA_F32)
    return launch_attn_f32(*s, static_cast<const float*>(Qp), static_cast<const float*>(Kp),
                           static_cast<const float*>(Vp), offsets, static_cast<float*>(Op), lse, cs);
  return launch_attn_bf16(*s, L, Qp, Kp, Vp, offsets, Op, lse, w, cs);
}

size_t moga_static_scratch_bytes(const moga_shape* s, int32_t G) {
  moga_status st;
  if (!check_shape(s, &st) || G < 0) return 0;
  return align_up(256 + sizeof(int32_t) * (2 * (size_t)s->B * G + 2), kWsAlign);
}

moga_status moga_stga_build(int32_t F, int32_t Hh, int32_t Ww, int32_t wh, int32_t ww,
                            const int32_t* shot_starts, int32_t n_shots, int32_t tg, int32_t augment,
                            int32_t* q_idx, int32_t* q_inv, int32_t* q_offsets, int32_t* kv_idx,
                            int32_t* kv_offsets, int32_t* G_out, int32_t* Tkv_out) {
  return stga_build_host(F, Hh, Ww, wh, ww, shot_starts, n_shots, tg, augment, q_idx, q_inv, q_offsets,
                         kv_idx, kv_offsets, G_out, Tkv_out);
}

moga_status moga_gather_rows(const moga_shape* s, const int32_t* idx, int32_t L, const void* src, void* dst,
                             void* stream) {
  moga_status st;
  if (!check_shape(s, &st)) return st;
  if (L < 0 || !PTR_OK(idx) || !PTR_OK(src) || !PTR_OK(dst)) return MOGA_ERR_INVALID_ARG;
  return launch_gather_list(*s, idx, L, src, dst, static_cast<cudaStream_t>(stream));
}

moga_status moga_static_group_attn(const moga_shape* s, int32_t G, int32_t Tq, int32_t Tkv, const void* Qs,
                                   const void* Ks, const void* Vs, const int32_t* q_offsets,
                                   const int32_t* kv_offsets, void* Os, float* lse, void* ws,
                                   size_t ws_bytes, void* stream) {
  moga_status st;
  if (!check_shape(s, &st)) return st;
  if (G < 0 || Tq < 0 || Tkv < 0 || !PTR_OK(Qs) || !PTR_OK(Ks) || !PTR_OK(Vs) || !PTR_OK(Os) ||
      q_offsets == nullptr || kv_offsets == nullptr || (lse != nullptr && !aligned16(lse)))
    return MOGA_ERR_INVALID_ARG;
  if (!check_ws(ws, ws_bytes, moga_static_scratch_bytes(s, G), &st)) return st;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  char* w = static_cast<char*>(ws);
  MOGA_CUDA_OK(cudaMemsetAsync(w, 0, 256, cs));
  if (s->dtype == MOGA_F32)
    return launch_attn_f32_groups(s->B, s->H, s->D, s->scale, G, Tq, Tkv, static_cast<const float*>(Qs),
                                  static_cast<const float*>(Ks), static_cast<const float*>(Vs), q_offsets,
                                  kv_offsets, 0, static_cast<float*>(Os), lse, cs);
  return launch_attn_bf16_static(*s, G, Tq, Tkv, Qs, Ks, Vs, q_offsets, kv_offsets, Os, lse,
                                 reinterpret_cast<uint32_t*>(w), w + 256, StaticEpilogue{nullptr, nullptr, nullptr}, cs);
}

moga_status moga_mean3(const moga_shape* s, const void* A, const void* Bs, const int32_t* inv_b,
                       const void* C, void* O, void* stream) {
  moga_status st;
  if (!check_shape(s, &st)) return st;
  if (!PTR_OK(A) || !PTR_OK(Bs) || !PTR_OK(C) || !PTR_OK(O)) return MOGA_ERR_INVALID_ARG;
  return launch_mean3(*s, A, Bs, inv_b, C, O, static_cast<cudaStream_t>(stream));
}

moga_status moga_unpermute(const moga_shape* s, const void* Op, const int32_t* inv,
                           const float* gate, void* O, void* stream) {
  moga_status st;
  if (!check_shape(s, &st)) return st;
  if (s->N == 0) return MOGA_OK;
  if (!PTR_OK(Op) || !PTR_OK(inv) || !PTR_OK(gate) || !PTR_OK(O)) return MOGA_ERR_INVALID_ARG;
  return launch_unpermute(*s, Op, inv, gate, O, static_cast<cudaStream_t>(stream));
}

}  // extern "C"

namespace {
// Alg. 1 lines 2-4 and the gate of Eq. 5 from a given routing: sort, gather, group attention,
// gated inverse permutation, with the intermediates in the forward workspace.
moga_status forward_after_route(const moga_shape* s, const WsLayout& L, const int32_t* gid, const float* gate,
                                const void* Q, const void* K, const void* V, void* O, int32_t* perm_out,
                                int32_t* offsets_out, char* w, cudaStream_t cs) {
  moga_status st;
  int32_t* perm = reinterpret_cast<int32_t*>(w + L.perm);
  int32_t* inv = reinterpret_cast<int32_t*>(w + L.inv);
  int32_t* offsets = reinterpret_cast<int32_t*>(w + L.offsets);
  void* Qp = w + L.Qp;
  void* Kp = w + L.Kp;
  void* Vp = w + L.Vp;
  void* Op = w + L.Op;
  // bf16 top-2 with a dense O: the attention epilogue adds gate * row into a zeroed O
  const bool dense_o = !(s->q_stride_b || s->q_stride_h || s->q_stride_n);
  const bool add_epilogue = s->dtype == MOGA_BF16 && s->k == 2 && dense_o && fused_topk();
  int32_t* asg = add_epilogue ? reinterpret_cast<int32_t*>(w + L.asg) : nullptr;
  if ((st = launch_sort(*s, L, gid, perm, inv, offsets, w, cs, asg)) != MOGA_OK) return st;
  if ((st = launch_gather(*s, perm, Q, K, V, Qp, Kp, Vp, cs, inv)) != MOGA_OK) return st;
  if (add_epilogue) {
    MOGA_CUDA_OK(cudaMemsetAsync(O, 0, elem_size(s->dtype) * (size_t)s->B * s->H * s->N * s->D, cs));
    st = launch_attn_bf16_add(*s, L, Qp, Kp, Vp, offsets, asg, gate, O, w, cs);
  } else if (s->dtype == MOGA_F32)
    st = launch_attn_f32(*s, static_cast<const float*>(Qp), static_cast<const float*>(Kp),
                         static_cast<const float*>(Vp), offsets, static_cast<float*>(Op), nullptr, cs);
  else if (s->k == 1)   // one assignment per token: the attention epilogue is the gated scatter
    st = launch_attn_bf16_scatter(*s, L, Qp, Kp, Vp, offsets, perm, gate, O, w, cs);
  else
    st = launch_attn_bf16(*s, L, Qp, Kp, Vp, offsets, Op, nullptr, w, cs);
  if (st != MOGA_OK) return st;
  if (!add_epilogue && (s->dtype == MOGA_F32 || s->k > 1))
    if ((st = launch_unpermute(*s, Op, inv, gate, O, cs)) != MOGA_OK) return st;
  const size_t T = (size_t)s->N * s->k;
  if (perm_out) MOGA_CUDA_OK(cudaMemcpyAsync(perm_out, perm, sizeof(int32_t) * s->B * T, cudaMemcpyDeviceToDevice, cs));
  if (offsets_out) MOGA_CUDA_OK(cudaMemcpyAsync(offsets_out, offsets, sizeof(int32_t) * s->B * (s->M + 1), cudaMemcpyDeviceToDevice, cs));
  return MOGA_OK;
}
}  // namespace

extern "C" {

moga_status moga_forward(const moga_shape* s, const void* X, const float* Wr, const float* bias,
                         const void* Q, const void* K, const void* V, void* O, int32_t* gid_out,
                         float* gate_out, int32_t* perm_out, int32_t* offsets_out, void* ws,
                         size_t ws_bytes, void* stream) {
  moga_status st;
  if (!check_shape(s, &st)) return st;
  if (s->N == 0) {                                // no tokens: only the (all-zero) offsets exist
    if (offsets_out)
      MOGA_CUDA_OK(cudaMemsetAsync(offsets_out, 0, sizeof(int32_t) * s->B * (s->M + 1), static_cast<cudaStream_t>(stream)));
    return MOGA_OK;
  }
  if (!PTR_OK(X) || !PTR_OK(Wr) || !PTR_OK(Q) || !PTR_OK(K) || !PTR_OK(V) || !PTR_OK(O) ||
      (bias != nullptr && !aligned16(bias)))
    return MOGA_ERR_INVALID_ARG;
  const WsLayout L = ws_layout(*s);
  if (!check_ws(ws, ws_bytes, L.total, &st)) return st;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  char* w = static_cast<char*>(ws);
  int32_t* gid = reinterpret_cast<int32_t*>(w + L.gid);
  float* gate = reinterpret_cast<float*>(w + L.gate);
  if ((st = clear_header(w, L, cs)) != MOGA_OK) return st;
  st = route_on_tensor_cores(*s, L, ws, ws_bytes)
           ? launch_route_mma(*s, L, X, Wr, bias, gid, gate, nullptr, w, cs)
           : launch_route(*s, X, Wr, bias, gid, gate, nullptr, cs);
  if (st != MOGA_OK) return st;
  if ((st = forward_after_route(s, L, gid, gate, Q, K, V, O, perm_out, offsets_out, w, cs)) != MOGA_OK) return st;
  const size_t T = (size_t)s->N * s->k;
  if (gid_out) MOGA_CUDA_OK(cudaMemcpyAsync(gid_out, gid, sizeof(int32_t) * s->B * T, cudaMemcpyDeviceToDevice, cs));
  if (gate_out) MOGA_CUDA_OK(cudaMemcpyAsync(gate_out, gate, sizeof(float) * s->B * T, cudaMemcpyDeviceToDevice, cs));
  return MOGA_OK;
}

moga_status moga_forward_routed(const moga_shape* s, const int32_t* gid, const float* gate, const void* Q,
                                const void* K, const void* V, void* O, int32_t* perm_out, int32_t* offsets_out,
                                void* ws, size_t ws_bytes, void* stream) {
  moga_status st;
  if (!check_shape(s, &st)) return st;
  if (s->N == 0) {
    if (offsets_out)
      MOGA_CUDA_OK(cudaMemsetAsync(offsets_out, 0, sizeof(int32_t) * s->B * (s->M + 1), static_cast<cudaStream_t>(stream)));
    return MOGA_OK;
  }
  if (!PTR_OK(gid) || !PTR_OK(gate) || !PTR_OK(Q) || !PTR_OK(K) || !PTR_OK(V) || !PTR_OK(O)) return MOGA_ERR_INVALID_ARG;
  const WsLayout L = ws_layout(*s);
  if (!check_ws(ws, ws_bytes, L.total, &st)) return st;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  char* w = static_cast<char*>(ws);
  if ((st = clear_header(w, L, cs)) != MOGA_OK) return st;
  return forward_after_route(s, L, gid, gate, Q, K, V, O, perm_out, offsets_out, w, cs);
}

}  // extern "C"

extern "C" {

// ---- the whole visual-attention block (Sec. 3.2): routed branch + two static branches + mean
namespace {
struct VisualLayout {
  size_t fwd, st_scratch, fr_scratch, fr_off, A, C, Qs, Ks, Vs, Bs, total;
};
VisualLayout visual_layout(const moga_shape& s, int G, int Tkv, int F) {
  VisualLayout v{};
  const size_t es = elem_size(s.dtype), row = es * (size_t)s.B * s.H * s.D;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t at = off;
    off = align_up(off + bytes, kWsAlign);
    return at;
  };
  v.fwd = take(ws_layout(s).total);
  v.st_scratch = take(moga_static_scratch_bytes(&s, G));
  v.fr_scratch = take(moga_static_scratch_bytes(&s, F));
  v.fr_off = take(sizeof(int32_t) * ((size_t)F + 1));
  v.A = take(row * s.N);
  v.C = take(s.dtype == MOGA_BF16 && s.D == 128 ? 0 : row * s.N);   // the fused path never stores the third branch
  v.Qs = take(row * s.N);
  v.Ks = take(row * Tkv);
  v.Vs = take(row * Tkv);
  v.Bs = take(row * s.N);
  v.total = off;
  return v;
}
bool lists_ok(const moga_shape& s, const moga_static_lists* l) {
  return l != nullptr && l->G >= 1 && l->Tkv >= 1 && l->F >= 1 && l->tokens_per_frame >= 1 &&
         (long long)l->F * l->tokens_per_frame == s.N && l->q_idx && l->q_inv && l->q_offsets && l->kv_idx &&
         l->kv_offsets;
}
}  // namespace

size_t moga_visual_workspace_bytes(const moga_shape* s, const moga_static_lists* lists) {
  moga_status st;
  if (!check_shape(s, &st) || !lists_ok(*s, lists)) return 0;
  return visual_layout(*s, lists->G, lists->Tkv, lists->F).total;
}

moga_status moga_visual_forward(const moga_shape* s, const void* X, const float* Wr, const float* bias,
                                const void* Q, const void* K, const void* V, void* O,
                                const moga_static_lists* lists, void* ws, size_t ws_bytes, void* stream) {
  moga_status st;
  if (!check_shape(s, &st)) return st;
  if (!lists_ok(*s, lists)) return MOGA_ERR_INVALID_ARG;
  if (s->q_stride_b || s->q_stride_h || s->q_stride_n) return MOGA_ERR_UNSUPPORTED;   // per-frame branch reads Q, K, V in place
  const VisualLayout v = visual_layout(*s, lists->G, lists->Tkv, lists->F);
  if (!check_ws(ws, ws_bytes, v.total, &st)) return st;
  char* w = static_cast<char*>(ws);
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  uint32_t* header = reinterpret_cast<uint32_t*>(w);   // == the routed branch's header: all launches report here
  // routed branch -> A (clears the status header)
  st = moga_forward(s, X, Wr, bias, Q, K, V, w + v.A, nullptr, nullptr, nullptr, nullptr, w + v.fwd,
                    ws_layout(*s).total, stream);
  if (st != MOGA_OK) return st;
  // spatial-temporal branch: gather by the lists, attention
  if ((st = launch_gather_list(*s, lists->q_idx, s->N, Q, w + v.Qs, cs)) != MOGA_OK) return st;
  if ((st = launch_gather_list(*s, lists->kv_idx, lists->Tkv, K, w + v.Ks, cs)) != MOGA_OK) return st;
  if ((st = launch_gather_list(*s, lists->kv_idx, lists->Tkv, V, w + v.Vs, cs)) != MOGA_OK) return st;
  int32_t* fr_off = reinterpret_cast<int32_t*>(w + v.fr_off);
  if ((st = launch_frame_offsets(fr_off, lists->F, lists->tokens_per_frame, cs)) != MOGA_OK) return st;
  if (s->dtype == MOGA_BF16 && s->D == 128) {
    // tensor-core path: the spatial-temporal launch writes its rows straight to token order (Bs is
    // then [B, H, N, D] in token order), and the per-frame launch, whose groups are contiguous
    // frames, forms the mean of the three branches in its epilogue: no third tensor, no mean pass
    st = launch_attn_bf16_static(*s, lists->G, s->N, lists->Tkv, w + v.Qs, w + v.Ks, w + v.Vs, lists->q_offsets,
                                 lists->kv_offsets, w + v.Bs, nullptr, header, w + v.st_scratch + 256,
                                 StaticEpilogue{lists->q_idx, nullptr, nullptr}, cs);
    if (st != MOGA_OK) return st;
    return launch_attn_bf16_static(*s, lists->F, s->N, s->N, Q, K, V, fr_off, fr_off, O, nullptr, header,
                                   w + v.fr_scratch + 256, StaticEpilogue{nullptr, w + v.A, w + v.Bs}, cs);
  }
  // other types: the three branches are materialised and averaged by a separate pass
  if (s->dtype == MOGA_BF16) {
    st = launch_attn_bf16_static(*s, lists->G, s->N, lists->Tkv, w + v.Qs, w + v.Ks, w + v.Vs, lists->q_offsets,
                                 lists->kv_offsets, w + v.Bs, nullptr, header, w + v.st_scratch + 256,
                                 StaticEpilogue{nullptr, nullptr, nullptr}, cs);
    if (st != MOGA_OK) return st;
    st = launch_attn_bf16_static(*s, lists->F, s->N, s->N, Q, K, V, fr_off, fr_off, w + v.C, nullptr, header,
                                 w + v.fr_scratch + 256, StaticEpilogue{nullptr, nullptr, nullptr}, cs);
  } else {
    st = launch_attn_f32_groups(s->B, s->H, s->D, s->scale, lists->G, s->N, lists->Tkv,
                                reinterpret_cast<const float*>(w + v.Qs), reinterpret_cast<const float*>(w + v.Ks),
                                reinterpret_cast<const float*>(w + v.Vs), lists->q_offsets, lists->kv_offsets, 0,
                                reinterpret_cast<float*>(w + v.Bs), nullptr, cs);
    if (st != MOGA_OK) return st;
    st = launch_attn_f32_groups(s->B, s->H, s->D, s->scale, lists->F, s->N, s->N, static_cast<const float*>(Q),
                                static_cast<const float*>(K), static_cast<const float*>(V), fr_off, fr_off, 0,
                                reinterpret_cast<float*>(w + v.C), nullptr, cs);
  }
  if (st != MOGA_OK) return st;
  return launch_mean3(*s, w + v.A, w + v.Bs, lists->q_inv, w + v.C, O, cs);
}

namespace {
struct BwdLayout {
  size_t scratch, dOp, delta, dQp, dKp, dVp, total;
};
BwdLayout bwd_layout(const moga_shape& s) {
  BwdLayout b{};
  const size_t T = (size_t)s.N * s.k, row = elem_size(s.dtype) * (size_t)s.B * s.H * T * s.D;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t at = off;
    off = align_up(off + bytes, kWsAlign);
    return at;
  };
  b.scratch = take(ws_layout(s).scratch_end);
  b.dOp = take(row);
  b.delta = take(sizeof(float) * (size_t)s.B * s.H * T);
  b.dQp = take(row);
  b.dKp = take(row);
  b.dVp = take(row);
  b.total = off;
  return b;
}
}  // namespace

size_t moga_backward_workspace_bytes(const moga_shape* s) {
  moga_status st;
  if (!check_shape(s, &st)) return 0;
  return bwd_layout(*s).total;
}

moga_status moga_backward(const moga_shape* s, const void* Qp, const void* Kp, const void* Vp, const void* Op,
                          const float* lse, const float* gate, const int32_t* perm, const int32_t* inv,
                          const int32_t* offsets, const void* dO, void* dQ, void* dK, void* dV, float* dgate,
                          void* ws, size_t ws_bytes, void* stream) {
  moga_status st;
  if (!check_shape(s, &st)) return st;
  if (s->dtype == MOGA_BF16 && s->D != 128) return MOGA_ERR_UNSUPPORTED;
  if (s->N == 0) return MOGA_OK;
  if (!PTR_OK(Qp) || !PTR_OK(Kp) || !PTR_OK(Vp) || !PTR_OK(Op) || !PTR_OK(lse) || !PTR_OK(gate) || !PTR_OK(perm) ||
      !PTR_OK(inv) || !PTR_OK(offsets) || !PTR_OK(dO) || !PTR_OK(dQ) || !PTR_OK(dK) || !PTR_OK(dV) || !PTR_OK(dgate))
    return MOGA_ERR_INVALID_ARG;
  const BwdLayout b = bwd_layout(*s);
  if (!check_ws(ws, ws_bytes, b.total, &st)) return st;
  const WsLayout L = ws_layout(*s);
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  char* w = static_cast<char*>(ws);
  if ((st = clear_header(w, L, cs)) != MOGA_OK) return st;
  if (s->dtype == MOGA_BF16) {
    st = launch_attn_backward(*s, L, Qp, Kp, Vp, Op, lse, gate, perm, inv, offsets, dO, w + b.dOp,
                              reinterpret_cast<float*>(w + b.delta), w + b.dQp, w + b.dKp, w + b.dVp, dgate, w, cs);
  } else {
    auto f = [](const void* x) { return static_cast<const float*>(x); };
    auto g = [&](size_t at) { return reinterpret_cast<float*>(w + at); };
    st = launch_attn_backward_f32(*s, f(Qp), f(Kp), f(Vp), f(Op), lse, gate, perm, inv, offsets, f(dO), g(b.dOp),
                                  g(b.delta), g(b.dQp), g(b.dKp), g(b.dVp), dgate, cs);
  }
  if (st != MOGA_OK) return st;
  // back to token order: a token's gradient is the plain sum over its k assignments
  if ((st = launch_unpermute(*s, w + b.dQp, inv, nullptr, dQ, cs)) != MOGA_OK) return st;
  if ((st = launch_unpermute(*s, w + b.dKp, inv, nullptr, dK, cs)) != MOGA_OK) return st;
  return launch_unpermute(*s, w + b.dVp, inv, nullptr, dV, cs);
}

size_t moga_route_backward_workspace_bytes(const moga_shape* s) {
  moga_status st;
  if (!check_shape(s, &st)) return 0;
  return route_backward_bytes(*s);
}

moga_status moga_route_backward(const moga_shape* s, const void* X, const float* Wr, const float* logits,
                                const int32_t* gid, const float* dgate, void* dX, float* dWr, float* dbias, void* ws,
                                size_t ws_bytes, void* stream) {
  moga_status st;
  if (!check_shape(s, &st)) return st;
  if (!PTR_OK(Wr) || !PTR_OK(dWr) || (dbias != nullptr && (reinterpret_cast<uintptr_t>(dbias) & 3u)) ||
      (dX != nullptr && !aligned16(dX)))
    return MOGA_ERR_INVALID_ARG;
  if (s->N > 0 && (!PTR_OK(X) || !PTR_OK(logits) || !PTR_OK(gid) || !PTR_OK(dgate))) return MOGA_ERR_INVALID_ARG;
  if (!check_ws(ws, ws_bytes, route_backward_bytes(*s), &st)) return st;
  return launch_route_backward(*s, X, Wr, logits, gid, dgate, dX, dWr, dbias, static_cast<char*>(ws),
                               static_cast<cudaStream_t>(stream));
}

moga_status moga_set_fused_topk(int32_t on) {
  set_fused_topk(on != 0);
  return MOGA_OK;
}

moga_status moga_set_attn_kernel(int32_t mode) {
  if (mode != MOGA_ATTN_AUTO && mode != MOGA_ATTN_SINGLE && mode != MOGA_ATTN_PAIR) return MOGA_ERR_INVALID_ARG;
  set_attn_kernel(mode);
  return MOGA_OK;
}

moga_status moga_last_device_status(void* ws, void* stream, uint32_t* detail) {
  if (ws == nullptr) return MOGA_ERR_WORKSPACE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  uint32_t words[2] = {0, 0};
  MOGA_CUDA_OK(cudaMemcpyAsync(words, ws, sizeof(words), cudaMemcpyDeviceToHost, cs));
  MOGA_CUDA_OK(cudaStreamSynchronize(cs));
  if (detail) *detail = words[1];
  if (words[0] != 0) MOGA_CUDA_OK(cudaMemsetAsync(ws, 0, 8, cs));
  return words[0] <= MOGA_ERR_INTERNAL ? static_cast<moga_status>(words[0]) : MOGA_ERR_INTERNAL;
}

}  // extern "C"
