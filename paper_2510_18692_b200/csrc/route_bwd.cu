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

// Loads of four consecutive channels of X as fp32.
__device__ __forceinline__ void load4(const float* p, float (&v)[4]) {
  const float4 t = *reinterpret_cast<const float4*>(p);
  v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
__device__ __forceinline__ void load4(const __nv_bfloat16* p, float (&v)[4]) {
  const uint2 t = *reinterpret_cast<const uint2*>(p);
  v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xffff0000u);
  v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xffff0000u);
}
__device__ __forceinline__ void store4(float* p, const float (&v)[4]) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
__device__ __forceinline__ void store4(__nv_bfloat16* p, const float (&v)[4]) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
  *reinterpret_cast<uint2*>(p) = make_uint2(*reinterpret_cast<uint32_t*>(&a), *reinterpret_cast<uint32_t*>(&b));
}

// WT[i, c] = W[c, i]: the dX kernel stages chunks of 128 channels of every logit column, which are
// contiguous in this order (read from W itself they were 4-byte pieces M floats apart, and the staging took
// longer than the products).
__global__ void __launch_bounds__(256)
route_wt_kernel(const float* __restrict__ Wr, float* __restrict__ WT, int C, int M) {
  const long long n = (long long)C * M;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < n; idx += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(idx / C), c = (int)(idx % C);
    WT[idx] = Wr[(size_t)c * M + i];
  }
}

// dX[t, c] = sum_i dr[t, i] W[c, i].  Block: 64 tokens, all channels in chunks of 128.  Thread
// (lane = channel quad, warp = token octet) owns 8 tokens x 4 channels; per logit column it reads
// two 16-byte words of dr (the same for the whole warp) and one of W, for 32 multiply-adds.
// Dynamic shared memory: drT [M][64] and wT [M][128] floats.
constexpr int kDxTok = 64, kDxCh = 128;
template <typename XT>
__global__ void __launch_bounds__(256)
route_dx_kernel(const float* __restrict__ dr, const float* __restrict__ WT, XT* __restrict__ dX, long long tokens, int C,
                int M) {
  extern __shared__ __align__(16) float dx_smem[];
  float* drT = dx_smem;                   // [M][kDxTok]
  float* wT = dx_smem + M * kDxTok;       // [M][kDxCh]
  const long long t0 = (long long)blockIdx.x * kDxTok;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int idx = threadIdx.x; idx < kDxTok * M; idx += 256) {
    const int i = idx / kDxTok, tt = idx % kDxTok;        // consecutive threads: consecutive tokens (no bank conflicts)
    drT[i * kDxTok + tt] = t0 + tt < tokens ? dr[(t0 + tt) * M + i] : 0.f;
  }
  for (int c0 = 0; c0 < C; c0 += kDxCh) {
    __syncthreads();
    for (int idx = threadIdx.x; idx < kDxCh * M; idx += 256) {
      const int i = idx / kDxCh, cc = idx % kDxCh;        // consecutive threads: consecutive channels
      wT[i * kDxCh + cc] = c0 + cc < C ? WT[(size_t)i * C + c0 + cc] : 0.f;
    }
    __syncthreads();
    float acc[8][4];
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
      for (int u = 0; u < 4; ++u) acc[a][u] = 0.f;
    for (int i = 0; i < M; ++i) {
      const float4 d0 = *reinterpret_cast<const float4*>(drT + i * kDxTok + warp * 8);
      const float4 d1 = *reinterpret_cast<const float4*>(drT + i * kDxTok + warp * 8 + 4);
      const float4 w4 = *reinterpret_cast<const float4*>(wT + i * kDxCh + lane * 4);
      const float d[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
      const float w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
      for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int u = 0; u < 4; ++u) acc[a][u] = fmaf(d[a], w[u], acc[a][u]);
    }
    const int c = c0 + lane * 4;
    if (c < C) {
#pragma unroll
      for (int a = 0; a < 8; ++a) {
        const long long t = t0 + warp * 8 + a;
        if (t < tokens) store4(dX + t * C + c, acc[a]);
      }
    }
  }
}

// part[slab, c, i] = sum over the slab's tokens of X[t, c] dr[t, i], for the block's 128 channels.
// A thread owns 4 channels (lane = channel quad) x COLS logit columns: 4 * COLS accumulators, so that a
// token costs it one 8- or 16-byte load of X and 4 * COLS FMAs against dr values broadcast from shared
// memory.  The 8 warps of a block split into ceil(M / COLS) column blocks (1, 2 or 4: X is read once per
// column block); the warps of a column block take the tile's tokens in turn and their sums are added at the
// end of the slab in warp order through shared memory: a fixed order, no atomics.  Measured at the
// minute-long size (M = 32): 9.0 ms with two 16-column blocks, 14.7 ms with one 32-column block (180
// registers, one block per SM), 17.1 ms for the first form (each warp a column group, X read by all eight).
template <typename XT, int COLS>
__global__ void __launch_bounds__(256)
route_dw_partial_kernel(const XT* __restrict__ X, const float* __restrict__ dr, float* __restrict__ part,
                        long long tokens, int C, int M) {
  constexpr int kTokTile = 128;
  // dr of the tile's tokens; after the last tile the same memory holds the 128 x M sums being added
  __shared__ __align__(16) float sdr[kTokTile][kMaxM];
  static_assert(kTokTile * kMaxM >= kWcChunk * kMaxM, "the sums fit where the dr tile was");
  const int slab = blockIdx.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int c = blockIdx.x * kWcChunk + lane * 4;
  const int ncb = (M + COLS - 1) / COLS;           // 1, 2 or 4 (the launcher picks COLS so)
  const int wpc = 8 / ncb;                         // warps per column block
  const int cb = warp / wpc, wl = warp % wpc;
  const int i0 = cb * COLS;
  const long long per = (tokens + kSlabs - 1) / kSlabs;
  const long long ta = (long long)slab * per, tb = min(tokens, ta + per);
  float acc[4][COLS];
#pragma unroll
  for (int u = 0; u < 4; ++u)
#pragma unroll
    for (int i = 0; i < COLS; ++i) acc[u][i] = 0.f;
  for (long long t0 = ta; t0 < tb; t0 += kTokTile) {
    __syncthreads();
    const int mp = ncb * COLS;                     // columns the threads read (zero beyond M)
    for (int idx = threadIdx.x; idx < kTokTile * mp; idx += 256) {
      const int tt = idx / mp, i = idx % mp;
      sdr[tt][i] = (t0 + tt < tb && i < M) ? dr[(t0 + tt) * M + i] : 0.f;
    }
    __syncthreads();
    if (c < C) {
      const int nt = (int)min((long long)kTokTile, tb - t0);
#pragma unroll 4
      for (int tt = wl; tt < nt; tt += wpc) {
        float x[4];
        load4(X + (t0 + tt) * C + c, x);
#pragma unroll
        for (int i = 0; i < COLS; i += 4) {
          const float4 dv = *reinterpret_cast<const float4*>(&sdr[tt][i0 + i]);
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            acc[u][i] = fmaf(x[u], dv.x, acc[u][i]);
            acc[u][i + 1] = fmaf(x[u], dv.y, acc[u][i + 1]);
            acc[u][i + 2] = fmaf(x[u], dv.z, acc[u][i + 2]);
            acc[u][i + 3] = fmaf(x[u], dv.w, acc[u][i + 3]);
          }
        }
      }
    }
  }
  // the column block's warps add their sums in warp order
  __syncthreads();
  float* r = &sdr[0][0] + (cb * kWcChunk + lane * 4) * COLS;
  for (int w = 0; w < wpc; ++w) {
    __syncthreads();
    if (wl == w) {
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int i = 0; i < COLS; ++i) r[u * COLS + i] = w == 0 ? acc[u][i] : r[u * COLS + i] + acc[u][i];
    }
  }
  __syncthreads();
  if (wl == 0 && c < C)
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int i = 0; i < COLS; ++i)
        if (i0 + i < M) part[((size_t)slab * C + c + u) * M + i0 + i] = r[u * COLS + i];
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

// COLS: 8 for M <= 8, else 16 (1, 2 or 4 column blocks for M <= 16, 32, 64)
template <typename XT>
void launch_dw_partial(const XT* X, const float* dr, float* part, long long tokens, int C, int M, dim3 grid,
                       cudaStream_t st) {
  if (M <= 8)
    route_dw_partial_kernel<XT, 8><<<grid, 256, 0, st>>>(X, dr, part, tokens, C, M);
  else
    route_dw_partial_kernel<XT, 16><<<grid, 256, 0, st>>>(X, dr, part, tokens, C, M);
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
  if (dX) {
    // W transposed, in the head of the partial-sum scratch: the dW_r kernel writes that scratch after the dX kernel has run
    route_wt_kernel<<<64, 256, 0, st>>>(Wr, part, s.C, s.M);
    MOGA_CUDA_OK(cudaGetLastError());
  }
  const size_t dx_smem_bytes = sizeof(float) * (size_t)s.M * (kDxTok + kDxCh);
  if (s.dtype == MOGA_BF16) {
    if (dX) {
      MOGA_CUDA_OK(cudaFuncSetAttribute(route_dx_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)(sizeof(float) * kMaxM * (kDxTok + kDxCh))));
      route_dx_kernel<__nv_bfloat16><<<(unsigned)((tokens + kDxTok - 1) / kDxTok), 256, dx_smem_bytes, st>>>(
          dr, part, static_cast<__nv_bfloat16*>(dX), tokens, s.C, s.M);
    }
    launch_dw_partial(static_cast<const __nv_bfloat16*>(X), dr, part, tokens, s.C, s.M, wgrid, st);
  } else {
    if (dX) {
      MOGA_CUDA_OK(cudaFuncSetAttribute(route_dx_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)(sizeof(float) * kMaxM * (kDxTok + kDxCh))));
      route_dx_kernel<float><<<(unsigned)((tokens + kDxTok - 1) / kDxTok), 256, dx_smem_bytes, st>>>(
          dr, part, static_cast<float*>(dX), tokens, s.C, s.M);
    }
    launch_dw_partial(static_cast<const float*>(X), dr, part, tokens, s.C, s.M, wgrid, st);
  }
  MOGA_CUDA_OK(cudaGetLastError());
  route_dw_reduce_kernel<<<64, 256, 0, st>>>(part, dWr, colsum, dbias, s.C, s.M, nblk);
  MOGA_CUDA_OK(cudaGetLastError());
  return MOGA_OK;
}

}  // namespace moga
