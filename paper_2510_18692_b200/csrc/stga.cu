// Static spatial-temporal groups (Sec. 3.2, "Spatial-Temporal Group Attention"): the host-side
// construction of the group lists, a row gather by a caller-given list, and the mean of the
// three branch outputs.  The attention itself is the same kernel as for routed groups, run
// with separate query and key ranges per group.
#include <vector>

#include "moga_internal.cuh"

namespace moga {
namespace {

constexpr int kMoveThreads = 256;
constexpr int kRowsPerThread = 4;

// dst[b,h,p,:] = src[b,h,idx[p],:]; idx is shared by all batch items and heads.
__global__ void __launch_bounds__(kMoveThreads)
gather_list_kernel(const int32_t* __restrict__ idx, const uint4* __restrict__ src, uint4* __restrict__ dst, int L,
                   int H, int vec_per_row, long long sb, long long sh, long long sn) {
  const int rows_per_pass = kMoveThreads / vec_per_row;
  const int lane_row = threadIdx.x / vec_per_row;
  const int v = threadIdx.x % vec_per_row;
  const int b = blockIdx.z, h = blockIdx.y;
  const int p0 = blockIdx.x * rows_per_pass * kRowsPerThread;
  const long long src_base = (long long)b * sb + (long long)h * sh;
  const long long dst_base = ((long long)b * H + h) * (long long)L * vec_per_row;
  uint4 val[kRowsPerThread];
  int p[kRowsPerThread];
#pragma unroll
  for (int i = 0; i < kRowsPerThread; ++i) {
    p[i] = p0 + i * rows_per_pass + lane_row;
    if (p[i] < L) val[i] = __ldg(src + src_base + (long long)idx[p[i]] * sn + v);
  }
#pragma unroll
  for (int i = 0; i < kRowsPerThread; ++i)
    if (p[i] < L) dst[dst_base + (long long)p[i] * vec_per_row + v] = val[i];
}

__device__ __forceinline__ void add_vec(float (&acc)[8], const uint4& raw, __nv_bfloat16) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    acc[2 * i] += __uint_as_float(w[i] << 16);
    acc[2 * i + 1] += __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ void add_vec(float (&acc)[8], const uint4& raw, float) {
  acc[0] += __uint_as_float(raw.x);
  acc[1] += __uint_as_float(raw.y);
  acc[2] += __uint_as_float(raw.z);
  acc[3] += __uint_as_float(raw.w);
}
__device__ __forceinline__ uint4 third_vec(const float (&acc)[8], __nv_bfloat16) {
  uint4 r;
  __nv_bfloat162 t;
  const float c = 1.f / 3.f;
  t = __floats2bfloat162_rn(acc[0] * c, acc[1] * c); r.x = *reinterpret_cast<uint32_t*>(&t);
  t = __floats2bfloat162_rn(acc[2] * c, acc[3] * c); r.y = *reinterpret_cast<uint32_t*>(&t);
  t = __floats2bfloat162_rn(acc[4] * c, acc[5] * c); r.z = *reinterpret_cast<uint32_t*>(&t);
  t = __floats2bfloat162_rn(acc[6] * c, acc[7] * c); r.w = *reinterpret_cast<uint32_t*>(&t);
  return r;
}
__device__ __forceinline__ uint4 third_vec(const float (&acc)[8], float) {
  return make_uint4(__float_as_uint(acc[0] / 3.f), __float_as_uint(acc[1] / 3.f), __float_as_uint(acc[2] / 3.f),
                    __float_as_uint(acc[3] / 3.f));
}

// O[b,h,n,:] = (A[b,h,n,:] + Bs[b,h,inv_b[n],:] + C[b,h,n,:]) / 3 in fp32, one rounding.
template <typename XT>
__global__ void __launch_bounds__(kMoveThreads)
mean3_kernel(const uint4* __restrict__ A, const uint4* __restrict__ Bs, const int32_t* __restrict__ inv_b,
             const uint4* __restrict__ C, uint4* __restrict__ O, int N, int H, int vec_per_row, long long sb,
             long long sh, long long sn) {
  const int rows_per_pass = kMoveThreads / vec_per_row;
  const int lane_row = threadIdx.x / vec_per_row;
  const int v = threadIdx.x % vec_per_row;
  const int b = blockIdx.z, h = blockIdx.y;
  const int n0 = blockIdx.x * rows_per_pass * kRowsPerThread;
  const long long tok_base = (long long)b * sb + (long long)h * sh;
  const long long flat_base = ((long long)b * H + h) * (long long)N * vec_per_row;
#pragma unroll
  for (int i = 0; i < kRowsPerThread; ++i) {
    const int n = n0 + i * rows_per_pass + lane_row;
    if (n >= N) continue;
    const int pb = inv_b != nullptr ? __ldg(inv_b + n) : n;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    add_vec(acc, __ldg(A + tok_base + (long long)n * sn + v), XT());
    add_vec(acc, __ldg(Bs + flat_base + (long long)pb * vec_per_row + v), XT());
    add_vec(acc, __ldg(C + flat_base + (long long)n * vec_per_row + v), XT());
    O[tok_base + (long long)n * sn + v] = third_vec(acc, XT());
  }
}

// off[f] = f * tokens_per_frame, f = 0..F: the per-frame groups (queries = keys)
__global__ void frame_offsets_kernel(int32_t* __restrict__ off, int F, int tokens_per_frame) {
  for (int f = blockIdx.x * blockDim.x + threadIdx.x; f <= F; f += gridDim.x * blockDim.x) off[f] = f * tokens_per_frame;
}

}  // namespace

moga_status launch_frame_offsets(int32_t* off, int F, int tokens_per_frame, cudaStream_t st) {
  frame_offsets_kernel<<<(F + 256) / 256, 256, 0, st>>>(off, F, tokens_per_frame);
  MOGA_CUDA_OK(cudaGetLastError());
  return MOGA_OK;
}

moga_status launch_gather_list(const moga_shape& s, const int32_t* idx, int L, const void* src, void* dst,
                               cudaStream_t st) {
  if (L == 0) return MOGA_OK;
  const int es = (int)elem_size(s.dtype);
  const int vec_per_row = s.D * es / 16;
  const int epv = 16 / es;
  const Strides sd = qkv_strides(s);
  const int rows_per_block = (kMoveThreads / vec_per_row) * kRowsPerThread;
  dim3 grid((L + rows_per_block - 1) / rows_per_block, s.H, s.B);
  gather_list_kernel<<<grid, kMoveThreads, 0, st>>>(idx, static_cast<const uint4*>(src), static_cast<uint4*>(dst),
                                                    L, s.H, vec_per_row, sd.b / epv, sd.h / epv, sd.n / epv);
  MOGA_CUDA_OK(cudaGetLastError());
  return MOGA_OK;
}

moga_status launch_mean3(const moga_shape& s, const void* A, const void* Bs, const int32_t* inv_b, const void* C,
                         void* O, cudaStream_t st) {
  if (s.N == 0) return MOGA_OK;
  const int es = (int)elem_size(s.dtype);
  const int vec_per_row = s.D * es / 16;
  const int epv = 16 / es;
  const Strides sd = qkv_strides(s);
  const int rows_per_block = (kMoveThreads / vec_per_row) * kRowsPerThread;
  dim3 grid((s.N + rows_per_block - 1) / rows_per_block, s.H, s.B);
  if (s.dtype == MOGA_BF16)
    mean3_kernel<__nv_bfloat16><<<grid, kMoveThreads, 0, st>>>(
        static_cast<const uint4*>(A), static_cast<const uint4*>(Bs), inv_b, static_cast<const uint4*>(C),
        static_cast<uint4*>(O), s.N, s.H, vec_per_row, sd.b / epv, sd.h / epv, sd.n / epv);
  else
    mean3_kernel<float><<<grid, kMoveThreads, 0, st>>>(
        static_cast<const uint4*>(A), static_cast<const uint4*>(Bs), inv_b, static_cast<const uint4*>(C),
        static_cast<uint4*>(O), s.N, s.H, vec_per_row, sd.b / epv, sd.h / epv, sd.n / epv);
  MOGA_CUDA_OK(cudaGetLastError());
  return MOGA_OK;
}

// Host-side construction of the group lists.  Groups are visited shot by shot, run by run
// (at most tg frames, never across a shot boundary), window by window; a group's queries
// are its own tokens in ascending order; its keys are, in this order, the same window of
// the previous shot's last frame (first run of a shot only), its own tokens, and the same
// window of the next shot's first frame (last run of a shot only).
moga_status stga_build_host(int F, int Hh, int Ww, int wh, int ww, const int32_t* shot_starts, int n_shots,
                            int tg, int augment, int32_t* q_idx, int32_t* q_inv, int32_t* q_offsets,
                            int32_t* kv_idx, int32_t* kv_offsets, int32_t* G_out, int32_t* Tkv_out) {
  if (F < 1 || Hh < 1 || Ww < 1 || wh < 1 || ww < 1 || wh > Hh || ww > Ww || n_shots < 1 || tg < 1 ||
      shot_starts == nullptr || shot_starts[0] != 0)
    return MOGA_ERR_INVALID_ARG;
  for (int s = 1; s < n_shots; ++s)
    if (shot_starts[s] <= shot_starts[s - 1] || shot_starts[s] >= F) return MOGA_ERR_INVALID_ARG;
  if ((long long)F * Hh * Ww >= (1ll << 31)) return MOGA_ERR_UNSUPPORTED;
  // tokens of one frame, window by window (window of (y, x) = (y*wh/Hh, x*ww/Ww)), ascending inside
  std::vector<std::vector<int32_t>> win((size_t)wh * ww);
  for (int y = 0; y < Hh; ++y)
    for (int x = 0; x < Ww; ++x) win[(size_t)(y * wh / Hh) * ww + (x * ww / Ww)].push_back(y * Ww + x);
  const int HW = Hh * Ww;
  long long G = 0, nq = 0, nkv = 0;
  auto emit_q = [&](int32_t tok) {
    if (q_idx) q_idx[nq] = tok;
    if (q_inv) q_inv[tok] = (int32_t)nq;
    ++nq;
  };
  auto emit_kv = [&](int32_t tok) {
    if (kv_idx) kv_idx[nkv] = tok;
    ++nkv;
  };
  for (int s = 0; s < n_shots; ++s) {
    const int f0 = shot_starts[s], f1 = s + 1 < n_shots ? shot_starts[s + 1] : F;
    for (int a = f0; a < f1; a += tg) {
      const int b = a + tg < f1 ? a + tg : f1;
      const bool first = a == f0, last = b == f1;
      for (size_t w = 0; w < win.size(); ++w) {
        if (win[w].empty()) continue;
        if (q_offsets) q_offsets[G] = (int32_t)nq;
        if (kv_offsets) kv_offsets[G] = (int32_t)nkv;
        if (augment && first && s > 0)
          for (int32_t t : win[w]) emit_kv((f0 - 1) * HW + t);
        for (int f = a; f < b; ++f)
          for (int32_t t : win[w]) {
            emit_q(f * HW + t);
            emit_kv(f * HW + t);
          }
        if (augment && last && s + 1 < n_shots)
          for (int32_t t : win[w]) emit_kv(f1 * HW + t);
        ++G;
        if (nkv >= (1ll << 31)) return MOGA_ERR_UNSUPPORTED;
      }
    }
  }
  if (q_offsets) q_offsets[G] = (int32_t)nq;
  if (kv_offsets) kv_offsets[G] = (int32_t)nkv;
  if (G_out) *G_out = (int32_t)G;
  if (Tkv_out) *Tkv_out = (int32_t)nkv;
  return MOGA_OK;
}

}  // namespace moga
