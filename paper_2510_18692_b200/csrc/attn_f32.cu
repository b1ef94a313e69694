// fp32 per-group attention (Eq. 1 inside each group, Alg. 1 line 3) on the fp32 ALUs.
//
// Used when dtype is fp32: a tensor-core path would have to round the operands to
// tf32, whose 10-bit mantissa does not meet the 1e-4 absolute bound.  One warp owns
// one query row (q in registers, online softmax in the exp domain of the running
// maximum); the 8 warps of a block share 32-key K/V tiles staged in shared memory.
#include <math.h>

#include "moga_internal.cuh"

namespace moga {
namespace {

constexpr int kF32Warps = 8;
constexpr int kF32Keys = 32;

template <int D>
__global__ void __launch_bounds__(kF32Warps * 32)
attn_f32_kernel(const float* __restrict__ Qp, const float* __restrict__ Kp,
                const float* __restrict__ Vp, const int32_t* __restrict__ q_offsets,
                const int32_t* __restrict__ kv_offsets, int off_stride, float* __restrict__ Op,
                float* __restrict__ lse, int Tq, int Tkv, int H, int G, float scale) {
  constexpr int KP = D + 4;  // padded K row: 16-byte reads of 8 consecutive rows are conflict-free
  __shared__ __align__(16) float Ks[kF32Keys * KP];
  __shared__ __align__(16) float Vs[kF32Keys * D];
  __shared__ int s_g, s_row0;
  const int b = blockIdx.z, h = blockIdx.y;
  // query rows [off[g], off[g+1]) attend to key rows [koff[g], koff[g+1]); routed groups pass the
  // same array for both, static groups (one list for all batch items) pass stride 0
  const int32_t* off = q_offsets + (size_t)b * off_stride;
  const int32_t* koff = kv_offsets + (size_t)b * off_stride;
  if (threadIdx.x == 0) {
    int acc = 0, found = -1, row0 = 0;
    const int rb = blockIdx.x;
    for (int g = 0; g < G; ++g) {
      int n = koff[g + 1] > koff[g] ? off[g + 1] - off[g] : 0;   // no keys: rows left untouched
      int nb = (n + kF32Warps - 1) / kF32Warps;
      if (rb < acc + nb) {
        found = g;
        row0 = off[g] + (rb - acc) * kF32Warps;
        break;
      }
      acc += nb;
    }
    s_g = found;
    s_row0 = row0;
  }
  __syncthreads();
  if (s_g < 0) return;
  const int qlo = off[s_g], qhi = off[s_g + 1];
  const int lo = koff[s_g], hi = koff[s_g + 1];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = s_row0 + warp;
  const bool active = row < qhi;
  const size_t q_base = ((size_t)b * H + h) * (size_t)Tq;
  const size_t head_base = ((size_t)b * H + h) * (size_t)Tkv;

  float q[D];
  {
    const float4* qr = reinterpret_cast<const float4*>(Qp + (q_base + (active ? row : qlo)) * D);
#pragma unroll
    for (int i = 0; i < D / 4; ++i) {
      float4 t = __ldg(qr + i);
      q[4 * i] = t.x; q[4 * i + 1] = t.y; q[4 * i + 2] = t.z; q[4 * i + 3] = t.w;
    }
  }
  float m = -INFINITY, l = 0.f;
  float o[D / 32];
#pragma unroll
  for (int i = 0; i < D / 32; ++i) o[i] = 0.f;

  for (int kt = lo; kt < hi; kt += kF32Keys) {
    __syncthreads();
    for (int idx = threadIdx.x; idx < kF32Keys * (D / 4); idx += kF32Warps * 32) {
      int r = idx / (D / 4), c = idx % (D / 4);
      float4 kv = make_float4(0.f, 0.f, 0.f, 0.f), vv = kv;
      if (kt + r < hi) {
        kv = __ldg(reinterpret_cast<const float4*>(Kp + (head_base + kt + r) * D) + c);
        vv = __ldg(reinterpret_cast<const float4*>(Vp + (head_base + kt + r) * D) + c);
      }
      *reinterpret_cast<float4*>(Ks + r * KP + 4 * c) = kv;
      *reinterpret_cast<float4*>(Vs + r * D + 4 * c) = vv;
    }
    __syncthreads();
    const bool valid = kt + lane < hi;
    float s = 0.f;
    const float4* kr = reinterpret_cast<const float4*>(Ks + lane * KP);
#pragma unroll
    for (int i = 0; i < D / 4; ++i) {
      float4 t = kr[i];
      s = fmaf(q[4 * i], t.x, s);
      s = fmaf(q[4 * i + 1], t.y, s);
      s = fmaf(q[4 * i + 2], t.z, s);
      s = fmaf(q[4 * i + 3], t.w, s);
    }
    s = valid ? s * scale : -INFINITY;
    float tmax = s;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, d));
    const float m_new = fmaxf(m, tmax);           // finite: key kt is always valid
    const float p = valid ? expf(s - m_new) : 0.f;
    const float alpha = expf(m - m_new);          // exp(-inf) = 0 on the first tile
    float psum = p;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, d);
    l = l * alpha + psum;
#pragma unroll
    for (int i = 0; i < D / 32; ++i) o[i] *= alpha;
#pragma unroll 8
    for (int j = 0; j < kF32Keys; ++j) {
      const float pj = __shfl_sync(0xffffffffu, p, j);
#pragma unroll
      for (int i = 0; i < D / 32; ++i) o[i] = fmaf(pj, Vs[j * D + lane + 32 * i], o[i]);
    }
    m = m_new;
  }
  if (active) {
    const float inv_l = 1.f / l;
#pragma unroll
    for (int i = 0; i < D / 32; ++i) Op[(q_base + row) * D + lane + 32 * i] = o[i] * inv_l;
    if (lse != nullptr && lane == 0) lse[q_base + row] = m + logf(l);
  }
}

}  // namespace

moga_status launch_attn_f32_groups(int B, int H, int D, float scale, int G, int Tq, int Tkv, const float* Qp,
                                   const float* Kp, const float* Vp, const int32_t* q_offsets,
                                   const int32_t* kv_offsets, int off_stride, float* Op, float* lse,
                                   cudaStream_t st) {
  if (Tq == 0 || G == 0) return MOGA_OK;
  dim3 grid((Tq + kF32Warps - 1) / kF32Warps + G, H, B);
  if (D == 64)
    attn_f32_kernel<64><<<grid, kF32Warps * 32, 0, st>>>(Qp, Kp, Vp, q_offsets, kv_offsets, off_stride, Op,
                                                         lse, Tq, Tkv, H, G, scale);
  else
    attn_f32_kernel<128><<<grid, kF32Warps * 32, 0, st>>>(Qp, Kp, Vp, q_offsets, kv_offsets, off_stride, Op,
                                                          lse, Tq, Tkv, H, G, scale);
  MOGA_CUDA_OK(cudaGetLastError());
  return MOGA_OK;
}

moga_status launch_attn_f32(const moga_shape& s, const float* Qp, const float* Kp, const float* Vp,
                            const int32_t* offsets, float* Op, float* lse, cudaStream_t st) {
  const int T = s.N * s.k;
  return launch_attn_f32_groups(s.B, s.H, s.D, s.scale, s.M, T, T, Qp, Kp, Vp, offsets, offsets, s.M + 1, Op,
                                lse, st);
}

}  // namespace moga
