// Backward of the router (Eq. 2-3 and the gate of Eq. 5) on the fp32 ALUs.
//
// The paper states no backward pass; this is the chain rule on its router.  With the logits
// r = X W_r (+ bias) saved by the forward (moga_route's optional output), the fixed routing
// decision gid and dgate = dL/dgate (from moga_backward):
//   gates = softmax over all M logits at the picks:  dr_i = sum_j dgate_j p_{g_j} (delta(i, g_j) - p_i)
//   gates = softmax over the k picked logits:        dr_{g_i} = z_i (dgate_i - sum_j dgate_j z_j), 0 elsewhere
//   dX = dr W_r^T      dW_r = X^T dr      dbias = sum_n dr
// Three kernels: dr per token (with per-block column sums for dbias), dX as a skinny product
// per token tile, and dW_r as per-(channel chunk, token slab) partial sums that a last kernel adds
// in slab order, so the result does not depend on scheduling (no floating-point atomics).
#include "moga_internal.cuh"

namespace moga {
namespace {

constexpr int kDrThreads = 128;       // tokens per block of the dr kernel
constexpr int kSlabs = 32;            // token slabs of the dW_r partial sums
constexpr int kWcChunk = 128;         // channels per block of the dW_r kernel

template <typename XT>
__device__ __forceinline__ float to_f32(XT v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename XT>
__device__ __forceinline__ XT from_f32(float v);
template <>
__device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// dr[t, 0..M) for token t = blockIdx.x * 128 + threadIdx.x (tokens of all batch items in one list),
// and colsum[blockIdx.x, i] = sum of dr[., i] over the block's tokens, added in thread order.
__global__ void __launch_bounds__(kDrThreads)
route_dlogits_kernel(const float* __restrict__ logits, const int32_t* __restrict__ gid, const float* __restrict__ dgate,
                     float* __restrict__ dr, float* __restrict__ colsum, long long tokens, int M, int k, int gate_mode) {
  __shared__ float sdr[kDrThreads][kMaxM + 1];
  const long long t = (long long)blockIdx.x * kDrThreads + threadIdx.x;
  float out[kMaxM];
#pragma unroll
  for (int i = 0; i < kMaxM; ++i) out[i] = 0.f;
  if (t < tokens) {
    const float* r = logits + t * M;
    int g[kMaxK];
    float dg[kMaxK];
#pragma unroll
    for (int j = 0; j < kMaxK; ++j)
      if (j < k) {
        g[j] = gid[t * k + j];
        dg[j] = dgate[t * k + j];
      }
    if (gate_mode == MOGA_GATE_SOFTMAX_ALL) {
      float top = r[0];
      for (int i = 1; i < M; ++i) top = fmaxf(top, r[i]);
      float Z = 0.f;
      for (int i = 0; i < M; ++i) Z += expf(r[i] - top);
      // s = sum_j dgate_j p_{g_j};  dr_i = [i picked as slot j] dgate_j p_i - p_i s
      float s = 0.f;
#pragma unroll
      for (int j = 0; j < kMaxK; ++j)
        if (j < k) s += dg[j] * expf(r[g[j]] - top) / Z;
#pragma unroll
      for (int i = 0; i < kMaxM; ++i)
        if (i < M) {
          const float p = expf(r[i] - top) / Z;
          float v = -p * s;
#pragma unroll
          for (int j = 0; j < kMaxK; ++j)
            if (j < k && g[j] == i) v += dg[j] * p;
          out[i] = v;
        }
    } else {
      float top = r[g[0]];
#pragma unroll
      for (int j = 1; j < kMaxK; ++j)
        if (j < k) top = fmaxf(top, r[g[j]]);
      float z[kMaxK], Z = 0.f, s = 0.f;
#pragma unroll
      for (int j = 0; j < kMaxK; ++j)
        if (j < k) {
          z[j] = expf(r[g[j]] - top);
          Z += z[j];
        }
#pragma unroll
      for (int j = 0; j < kMaxK; ++j)
        if (j < k) {
          z[j] /= Z;
          s += dg[j] * z[j];
        }
#pragma unroll
      for (int i = 0; i < kMaxM; ++i)
        if (i < M) {
#pragma unroll
          for (int j = 0; j < kMaxK; ++j)
            if (j < k && g[j] == i) out[i] = z[j] * (dg[j] - s);
        }
    }
#pragma unroll
    for (int i = 0; i < kMaxM; ++i)
      if (i < M) dr[t * M + i] = out[i];
  }
#pragma unroll
  for (int i = 0; i < kMaxM; ++i)
    if (i < M) sdr[threadIdx.x][i] = out[i];
  __syncthreads();
  if (threadIdx.x < M) {
    float acc = 0.f;
    for (int u = 0; u < kDrThreads; ++u) acc += sdr[u][threadIdx.x];
    colsum[(size_t)blockIdx.x * M + threadIdx.x] = acc;
  }
}

// dX[t, c] = sum_i dr[t, i] W[c, i].  Block: 32 tokens x 128 channels per pass; thread (tx, ty) of
// 16 x 16 owns tokens ty*2, ty*2 + 1 and channels tx + 16 u, u < 8.
constexpr int kDxTok = 32, kDxCh = 128;
template <typename XT>
__global__ void __launch_bounds__(256)
route_dx_kernel(const float* __restrict__ dr, const float* __restrict__ Wr, XT* __restrict__ dX, long long tokens, int C,
                int M) {
  __shared__ float sdr[kDxTok][kMaxM + 1];
  __shared__ float sw[kDxCh][kMaxM + 1];
  const long long t0 = (long long)blockIdx.x * kDxTok;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  for (int idx = threadIdx.x; idx < kDxTok * M; idx += 256) {
    const int tt = idx / M, i = idx % M;
    sdr[tt][i] = t0 + tt < tokens ? dr[(t0 + tt) * M + i] : 0.f;
  }
  for (int c0 = 0; c0 < C; c0 += kDxCh) {
    __syncthreads();
    for (int idx = threadIdx.x; idx < kDxCh * M; idx += 256) {
      const int cc = idx / M, i = idx % M;
      sw[cc][i] = c0 + cc < C ? Wr[(size_t)(c0 + cc) * M + i] : 0.f;
    }
    __syncthreads();
    float acc[2][8];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int u = 0; u < 8; ++u) acc[a][u] = 0.f;
    for (int i = 0; i < M; ++i) {
      float d[2];
#pragma unroll
      for (int a = 0; a < 2; ++a) d[a] = sdr[ty * 2 + a][i];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const float wv = sw[tx + 16 * u][i];
#pragma unroll
        for (int a = 0; a < 2; ++a) acc[a][u] = fmaf(d[a], wv, acc[a][u]);
      }
    }
#pragma unroll
    for (int a = 0; a < 2; ++a) {
      const long long t = t0 + ty * 2 + a;
      if (t < tokens) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int c = c0 + tx + 16 * u;
          if (c < C) dX[t * C + c] = from_f32<XT>(acc[a][u]);
        }
      }
    }
  }
}

// part[slab, c, i] = sum over the slab's tokens of X[t, c] dr[t, i], for the block's 128 channels.
// Thread: channel c = c0 + (threadIdx.x & 127), and half of the M columns (threadIdx.x >> 7).
template <typename XT>
__global__ void __launch_bounds__(256)
route_dw_partial_kernel(const XT* __restrict__ X, const float* __restrict__ dr, float* __restrict__ part,
                        long long tokens, int C, int M) {
  constexpr int kTokTile = 32;
  __shared__ float sdr[kTokTile][kMaxM];
  const int slab = blockIdx.y;
  const int c = blockIdx.x * kWcChunk + (threadIdx.x & (kWcChunk - 1));
  const int half = threadIdx.x >> 7;
  const int mh = (M + 1) / 2, i0 = half * mh, i1 = min(M, i0 + mh);
  const long long per = (tokens + kSlabs - 1) / kSlabs;
  const long long ta = (long long)slab * per, tb = min(tokens, ta + per);
  float acc[kMaxM / 2];
#pragma unroll
  for (int i = 0; i < kMaxM / 2; ++i) acc[i] = 0.f;
  for (long long t0 = ta; t0 < tb; t0 += kTokTile) {
    __syncthreads();
    for (int idx = threadIdx.x; idx < kTokTile * M; idx += 256) {
      const int tt = idx / M, i = idx % M;
      sdr[tt][i] = t0 + tt < tb ? dr[(t0 + tt) * M + i] : 0.f;
    }
    __syncthreads();
    if (c < C) {
#pragma unroll 4
      for (int tt = 0; tt < kTokTile; ++tt) {
        if (t0 + tt >= tb) break;
        const float x = to_f32<XT>(X[(t0 + tt) * C + c]);
#pragma unroll
        for (int i = 0; i < kMaxM / 2; ++i)
          if (i0 + i < i1) acc[i] = fmaf(x, sdr[tt][i0 + i], acc[i]);
      }
    }
  }
  if (c < C)
#pragma unroll
    for (int i = 0; i < kMaxM / 2; ++i)
      if (i0 + i < i1) part[((size_t)slab * C + c) * M + i0 + i] = acc[i];
}

// dWr[c, i] = sum over slabs (in order) of part[slab, c, i];  dbias[i] = sum over blocks of colsum
__global__ void __launch_bounds__(256)
route_dw_reduce_kernel(const float* __restrict__ part, float* __restrict__ dWr, const float* __restrict__ colsum,
                       float* __restrict__ dbias, int C, int M, int nblk) {
  const long long n = (long long)C * M;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < n; idx += (long long)gridDim.x * blockDim.x) {
    float acc = 0.f;
    for (int s = 0; s < kSlabs; ++s) acc += part[(size_t)s * n + idx];
    dWr[idx] = acc;
  }
  if (dbias != nullptr && blockIdx.x == 0 && threadIdx.x < M) {
    float acc = 0.f;
    for (int b = 0; b < nblk; ++b) acc += colsum[(size_t)b * M + threadIdx.x];
    dbias[threadIdx.x] = acc;
  }
}

}  // namespace

size_t route_backward_bytes(const moga_shape& s) {
  const size_t tokens = (size_t)s.B * s.N;
  const size_t nblk = (tokens + kDrThreads - 1) / kDrThreads;
  return align_up(sizeof(float) * tokens * s.M, kWsAlign) + align_up(sizeof(float) * nblk * s.M, kWsAlign) +
         align_up(sizeof(float) * (size_t)kSlabs * s.C * s.M, kWsAlign);
}

moga_status launch_route_backward(const moga_shape& s, const void* X, const float* Wr, const float* logits,
                                  const int32_t* gid, const float* dgate, void* dX, float* dWr, float* dbias, char* ws,
                                  cudaStream_t st) {
  const long long tokens = (long long)s.B * s.N;
  if (tokens == 0) {
    MOGA_CUDA_OK(cudaMemsetAsync(dWr, 0, sizeof(float) * (size_t)s.C * s.M, st));
    if (dbias) MOGA_CUDA_OK(cudaMemsetAsync(dbias, 0, sizeof(float) * s.M, st));
    return MOGA_OK;
  }
  const int nblk = (int)((tokens + kDrThreads - 1) / kDrThreads);
  float* dr = reinterpret_cast<float*>(ws);
  float* colsum = reinterpret_cast<float*>(ws + align_up(sizeof(float) * (size_t)tokens * s.M, kWsAlign));
  float* part = reinterpret_cast<float*>(reinterpret_cast<char*>(colsum) + align_up(sizeof(float) * (size_t)nblk * s.M, kWsAlign));
  route_dlogits_kernel<<<nblk, kDrThreads, 0, st>>>(logits, gid, dgate, dr, colsum, tokens, s.M, s.k, s.gate_mode);
  MOGA_CUDA_OK(cudaGetLastError());
  dim3 wgrid((s.C + kWcChunk - 1) / kWcChunk, kSlabs);
  if (s.dtype == MOGA_BF16) {
    if (dX)
      route_dx_kernel<__nv_bfloat16><<<(unsigned)((tokens + kDxTok - 1) / kDxTok), 256, 0, st>>>(
          dr, Wr, static_cast<__nv_bfloat16*>(dX), tokens, s.C, s.M);
    route_dw_partial_kernel<__nv_bfloat16><<<wgrid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(X), dr, part,
                                                                  tokens, s.C, s.M);
  } else {
    if (dX)
      route_dx_kernel<float><<<(unsigned)((tokens + kDxTok - 1) / kDxTok), 256, 0, st>>>(
          dr, Wr, static_cast<float*>(dX), tokens, s.C, s.M);
    route_dw_partial_kernel<float><<<wgrid, 256, 0, st>>>(static_cast<const float*>(X), dr, part, tokens, s.C, s.M);
  }
  MOGA_CUDA_OK(cudaGetLastError());
  route_dw_reduce_kernel<<<64, 256, 0, st>>>(part, dWr, colsum, dbias, s.C, s.M, nblk);
  MOGA_CUDA_OK(cudaGetLastError());
  return MOGA_OK;
}

}  // namespace moga
