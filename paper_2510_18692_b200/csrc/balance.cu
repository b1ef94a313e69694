// Group-balancing statistics (Eq. 6-8) from a routing result: F_i, the fraction of tokens
// assigned to group i, P_i, the mean routing probability of those assignments, and the
// loss alpha * M * sum_i F_i P_i.  A by-product of routing: 8 bytes per assignment are
// read once.  Deterministic (no floating-point atomics): every thread sums its own strided
// elements per group in shared memory, the block adds the 256 rows in order, and one block
// per batch item adds the block partials in order (in fp64).
#include "moga_internal.cuh"

namespace moga {
namespace {

constexpr int kStatThreads = 256;

__global__ void __launch_bounds__(kStatThreads)
balance_partial_kernel(const int32_t* __restrict__ gid, const float* __restrict__ gate,
                       int32_t* __restrict__ blk_cnt, float* __restrict__ blk_sum, int T, int M, int nblk) {
  extern __shared__ float srow[];                 // [kStatThreads][M] gate sums, then [kStatThreads][M] counts
  int* crow = reinterpret_cast<int*>(srow + kStatThreads * M);
  const int b = blockIdx.y, blk = blockIdx.x, t = threadIdx.x;
  for (int i = 0; i < M; ++i) {
    srow[t * M + i] = 0.f;
    crow[t * M + i] = 0;
  }
  const int begin = blk * kSortChunk, end = min(begin + kSortChunk, T);
  for (int a = begin + t; a < end; a += kStatThreads) {
    int g = gid[(size_t)b * T + a];
    g = g < 0 ? 0 : (g >= M ? M - 1 : g);         // out-of-range ids are reported by the sort; clamp here
    srow[t * M + g] += gate[(size_t)b * T + a];
    crow[t * M + g] += 1;
  }
  __syncthreads();
  if (t < M) {
    float s = 0.f;
    int c = 0;
    for (int r = 0; r < kStatThreads; ++r) {
      s += srow[r * M + t];
      c += crow[r * M + t];
    }
    blk_sum[((size_t)b * nblk + blk) * M + t] = s;
    blk_cnt[((size_t)b * nblk + blk) * M + t] = c;
  }
}

__global__ void __launch_bounds__(kMaxM)
balance_final_kernel(const int32_t* __restrict__ blk_cnt, const float* __restrict__ blk_sum,
                     float* __restrict__ F, float* __restrict__ P, float* __restrict__ loss, int N, int M,
                     int nblk, float alpha) {
  __shared__ double fp[kMaxM];
  const int b = blockIdx.x, i = threadIdx.x;
  if (i < M) {
    long long c = 0;
    double s = 0.0;
    for (int blk = 0; blk < nblk; ++blk) {
      c += blk_cnt[((size_t)b * nblk + blk) * M + i];
      s += (double)blk_sum[((size_t)b * nblk + blk) * M + i];
    }
    const double f = (double)c / (double)N, p = s / (double)N;
    F[(size_t)b * M + i] = (float)f;
    P[(size_t)b * M + i] = (float)p;
    fp[i] = f * p;
  }
  __syncthreads();
  if (i == 0) {
    double acc = 0.0;
    for (int g = 0; g < M; ++g) acc += fp[g];
    loss[b] = (float)((double)alpha * M * acc);
  }
}

}  // namespace

moga_status launch_balance_stats(const moga_shape& s, const WsLayout& L, const int32_t* gid, const float* gate,
                                 float alpha, float* F, float* P, float* loss, char* ws, cudaStream_t st) {
  const int T = s.N * s.k;
  int32_t* blk_cnt = reinterpret_cast<int32_t*>(ws + L.stats);
  float* blk_sum = reinterpret_cast<float*>(blk_cnt + (size_t)s.B * L.nblk * s.M);
  const size_t smem = (size_t)kStatThreads * s.M * 8;
  MOGA_CUDA_OK(cudaFuncSetAttribute(balance_partial_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    kStatThreads * kMaxM * 8));
  balance_partial_kernel<<<dim3(L.nblk, s.B), kStatThreads, smem, st>>>(gid, gate, blk_cnt, blk_sum, T, s.M,
                                                                        L.nblk);
  MOGA_CUDA_OK(cudaGetLastError());
  balance_final_kernel<<<s.B, kMaxM, 0, st>>>(blk_cnt, blk_sum, F, P, loss, s.N, s.M, L.nblk, alpha);
  MOGA_CUDA_OK(cudaGetLastError());
  return MOGA_OK;
}

}  // namespace moga
