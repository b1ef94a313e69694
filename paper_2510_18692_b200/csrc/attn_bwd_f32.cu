// fp32 backward of the per-group attention on the fp32 ALUs (d_head 64 or 128).
//
// The paper states no backward pass; as in the bf16 kernels this is the chain rule on its forward
// (Eq. 1 inside each group, Eq. 5's gate) with the forward's saved log-sum-exp:
//   p = exp(scale * q k^T - lse)    ds = p * (do v^T - delta) * scale    delta = <do, o>
//   dV = p^T do    dK = ds^T q    dQ = ds k
// One kernel template, two launches, shaped like the fp32 forward kernel: a warp owns one
// resident row (a query row for dQ; a key row for dK and dV), the 8 warps of a block share
// 32-row tiles of the other side staged in shared memory; a lane forms the two dot products of
// one streamed row, then the lanes split the channels of the accumulating sums.
#include <math.h>

#include "moga_internal.cuh"

namespace moga {
namespace {

constexpr int kWarps = 8;
constexpr int kRows = 32;
constexpr int kModeQ = 0, kModeKV = 1;

// do_p[b,h,p,:] = gate * dO[b,h,token,:], delta[b,h,p] = gate * <dO, o_p>, dgate[b,a] = sum_h <dO, o_p>
// for the assignment a = token * k + slot at sorted position p.  One warp per (b, p), heads in turn.
template <int D>
__global__ void __launch_bounds__(256)
bwd_prep_f32_kernel(const float* __restrict__ dO, const float* __restrict__ Op, const float* __restrict__ gate,
                    const int32_t* __restrict__ perm, const int32_t* __restrict__ inv, float* __restrict__ dOp,
                    float* __restrict__ delta, float* __restrict__ dgate, int N, int k, int H, long long sb,
                    long long sh, long long sn) {
  const int b = blockIdx.y, lane = threadIdx.x & 31;
  const long long T = (long long)N * k;
  const long long p = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (p >= T) return;
  const int tok = perm[(size_t)b * T + p];
  int slot = 0;
  for (int j = 0; j < k; ++j)
    if (inv[(size_t)b * T + (long long)tok * k + j] == p) slot = j;
  const long long a = (long long)b * T + (long long)tok * k + slot;
  const float g = gate[a];
  float dg = 0.f;
  for (int h = 0; h < H; ++h) {
    const float* d = dO + (long long)b * sb + (long long)h * sh + (long long)tok * sn;
    const size_t at = (((size_t)b * H + h) * T + p) * D;
    float dot = 0.f;
#pragma unroll
    for (int i = 0; i < D / 32; ++i) {
      const float dv = __ldg(d + lane + 32 * i);
      dot = fmaf(dv, __ldg(Op + at + lane + 32 * i), dot);
      dOp[at + lane + 32 * i] = g * dv;
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, s);
    if (lane == 0) delta[((size_t)b * H + h) * T + p] = g * dot;
    dg += dot;
  }
  if (lane == 0) dgate[a] = dg;
}

// kModeQ:  resident (R0, R1) = (q, do) rows, streamed (S0, S1) = (K, V):  out0 = dQ = sum ds * K
// kModeKV: resident (R0, R1) = (k, v) rows,  streamed (S0, S1) = (Q, dO): out0 = dV = sum p * dO,
//                                                                          out1 = dK = sum ds * Q
// In both, s = <R0, S0 row> and dp = <R1, S1 row>; lse and delta belong to the query side.
template <int D, int Mode>
__global__ void __launch_bounds__(kWarps * 32)
attn_bwd_f32_kernel(const float* __restrict__ R0, const float* __restrict__ R1, const float* __restrict__ S0,
                    const float* __restrict__ S1, const float* __restrict__ lse, const float* __restrict__ delta,
                    const int32_t* __restrict__ offsets, float* __restrict__ out0, float* __restrict__ out1, int T,
                    int H, int G, float scale) {
  constexpr int SP = D + 4;   // padded streamed row: 16-byte reads of 8 consecutive rows are conflict-free
  __shared__ __align__(16) float S0s[kRows * SP];
  __shared__ __align__(16) float S1s[kRows * SP];
  __shared__ __align__(16) float Rs[kWarps][2][D];
  __shared__ float s_lse[kRows], s_delta[kRows];
  __shared__ int s_g, s_row0;
  const int b = blockIdx.z, h = blockIdx.y;
  const int32_t* off = offsets + (size_t)b * (G + 1);
  if (threadIdx.x == 0) {
    int acc = 0, found = -1, row0 = 0;
    const int rb = blockIdx.x;
    for (int g = 0; g < G; ++g) {
      const int n = off[g + 1] - off[g];
      const int nb = (n + kWarps - 1) / kWarps;
      if (rb < acc + nb) {
        found = g;
        row0 = off[g] + (rb - acc) * kWarps;
        break;
      }
      acc += nb;
    }
    s_g = found;
    s_row0 = row0;
  }
  __syncthreads();
  if (s_g < 0) return;
  const int lo = off[s_g], hi = off[s_g + 1];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = s_row0 + warp;
  const bool active = row < hi;
  const size_t base = ((size_t)b * H + h) * (size_t)T;
  const size_t rrow = base + (active ? row : lo);
#pragma unroll
  for (int i = 0; i < D / 32; ++i) {
    Rs[warp][0][lane + 32 * i] = __ldg(R0 + rrow * D + lane + 32 * i);
    Rs[warp][1][lane + 32 * i] = __ldg(R1 + rrow * D + lane + 32 * i);
  }
  float row_lse = 0.f, row_delta = 0.f;
  if (Mode == kModeQ) {
    row_lse = __ldg(lse + rrow);
    row_delta = __ldg(delta + rrow);
  }
  float a0[D / 32], a1[D / 32];
#pragma unroll
  for (int i = 0; i < D / 32; ++i) a0[i] = a1[i] = 0.f;

  for (int t = lo; t < hi; t += kRows) {
    __syncthreads();
    for (int idx = threadIdx.x; idx < kRows * (D / 4); idx += kWarps * 32) {
      const int r = idx / (D / 4), c = idx % (D / 4);
      float4 x = make_float4(0.f, 0.f, 0.f, 0.f), y = x;
      if (t + r < hi) {
        x = __ldg(reinterpret_cast<const float4*>(S0 + (base + t + r) * D) + c);
        y = __ldg(reinterpret_cast<const float4*>(S1 + (base + t + r) * D) + c);
      }
      *reinterpret_cast<float4*>(S0s + r * SP + 4 * c) = x;
      *reinterpret_cast<float4*>(S1s + r * SP + 4 * c) = y;
    }
    if (Mode == kModeKV && threadIdx.x < kRows) {
      const bool in = t + (int)threadIdx.x < hi;
      s_lse[threadIdx.x] = in ? __ldg(lse + base + t + threadIdx.x) : 0.f;
      s_delta[threadIdx.x] = in ? __ldg(delta + base + t + threadIdx.x) : 0.f;
    }
    __syncthreads();
    const bool valid = t + lane < hi;
    float s = 0.f, dp = 0.f;
    const float4* x0 = reinterpret_cast<const float4*>(S0s + lane * SP);
    const float4* x1 = reinterpret_cast<const float4*>(S1s + lane * SP);
    const float4* r0 = reinterpret_cast<const float4*>(Rs[warp][0]);
    const float4* r1 = reinterpret_cast<const float4*>(Rs[warp][1]);
#pragma unroll 8
    for (int i = 0; i < D / 4; ++i) {
      const float4 u = r0[i], x = x0[i], w = r1[i], y = x1[i];
      s = fmaf(u.x, x.x, s); s = fmaf(u.y, x.y, s); s = fmaf(u.z, x.z, s); s = fmaf(u.w, x.w, s);
      dp = fmaf(w.x, y.x, dp); dp = fmaf(w.y, y.y, dp); dp = fmaf(w.z, y.z, dp); dp = fmaf(w.w, y.w, dp);
    }
    const float L = Mode == kModeQ ? row_lse : s_lse[lane];
    const float Dl = Mode == kModeQ ? row_delta : s_delta[lane];
    const float p = valid ? expf(s * scale - L) : 0.f;
    const float ds = p * (dp - Dl) * scale;
#pragma unroll 8
    for (int j = 0; j < kRows; ++j) {
      const float dsj = __shfl_sync(0xffffffffu, ds, j);
      if (Mode == kModeQ) {
#pragma unroll
        for (int i = 0; i < D / 32; ++i) a0[i] = fmaf(dsj, S0s[j * SP + lane + 32 * i], a0[i]);
      } else {
        const float pj = __shfl_sync(0xffffffffu, p, j);
#pragma unroll
        for (int i = 0; i < D / 32; ++i) {
          a0[i] = fmaf(pj, S1s[j * SP + lane + 32 * i], a0[i]);
          a1[i] = fmaf(dsj, S0s[j * SP + lane + 32 * i], a1[i]);
        }
      }
    }
  }
  if (active) {
#pragma unroll
    for (int i = 0; i < D / 32; ++i) {
      out0[(base + row) * D + lane + 32 * i] = a0[i];
      if (Mode == kModeKV) out1[(base + row) * D + lane + 32 * i] = a1[i];
    }
  }
}

template <int D>
moga_status launch_d(const moga_shape& s, const float* Qp, const float* Kp, const float* Vp, const float* Op,
                     const float* lse, const float* gate, const int32_t* perm, const int32_t* inv,
                     const int32_t* offsets, const float* dO, float* dOp, float* delta, float* dQp, float* dKp,
                     float* dVp, float* dgate, cudaStream_t st) {
  const long long T = (long long)s.N * s.k;
  const Strides q = qkv_strides(s);
  dim3 pgrid((unsigned)((T + 7) / 8), s.B);
  bwd_prep_f32_kernel<D><<<pgrid, 256, 0, st>>>(dO, Op, gate, perm, inv, dOp, delta, dgate, s.N, s.k, s.H, q.b, q.h,
                                                q.n);
  MOGA_CUDA_OK(cudaGetLastError());
  dim3 grid((unsigned)((T + kWarps - 1) / kWarps + s.M), s.H, s.B);
  attn_bwd_f32_kernel<D, kModeQ><<<grid, kWarps * 32, 0, st>>>(Qp, dOp, Kp, Vp, lse, delta, offsets, dQp, nullptr,
                                                                (int)T, s.H, s.M, s.scale);
  MOGA_CUDA_OK(cudaGetLastError());
  attn_bwd_f32_kernel<D, kModeKV><<<grid, kWarps * 32, 0, st>>>(Kp, Vp, Qp, dOp, lse, delta, offsets, dVp, dKp,
                                                                 (int)T, s.H, s.M, s.scale);
  MOGA_CUDA_OK(cudaGetLastError());
  return MOGA_OK;
}

}  // namespace

moga_status launch_attn_backward_f32(const moga_shape& s, const float* Qp, const float* Kp, const float* Vp,
                                     const float* Op, const float* lse, const float* gate, const int32_t* perm,
                                     const int32_t* inv, const int32_t* offsets, const float* dO, float* dOp,
                                     float* delta, float* dQp, float* dKp, float* dVp, float* dgate,
                                     cudaStream_t st) {
  if ((long long)s.N * s.k == 0) return MOGA_OK;
  if (s.D == 64)
    return launch_d<64>(s, Qp, Kp, Vp, Op, lse, gate, perm, inv, offsets, dO, dOp, delta, dQp, dKp, dVp, dgate, st);
  return launch_d<128>(s, Qp, Kp, Vp, Op, lse, gate, perm, inv, offsets, dO, dOp, delta, dQp, dKp, dVp, dgate, st);
}

}  // namespace moga
