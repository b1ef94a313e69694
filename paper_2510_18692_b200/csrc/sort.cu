// Stable counting sort of the N*k assignments of each batch item by group
// (the index part of Alg. 1 line 2): offsets (cu_seqlen), perm (permute_index), inv.
//
// Three small launches: (1) per-block histograms with warp-aggregated shared-memory
// atomics, (2) one block per batch item turns them into group offsets and per-block
// bases (warp shuffle scans), (3) every block re-reads its chunk in order and ranks
// each element inside its 32-wide window with match_any, which keeps the order of
// equal keys (ascending token index).  Integer work only; ~7 MB of traffic at the
// largest case, so this stage is launch-latency bound.
#include "moga_internal.cuh"

namespace moga {
namespace {

constexpr int kSortThreads = 256;
constexpr int kSortWarps = kSortThreads / 32;

__global__ void __launch_bounds__(kSortThreads)
sort_hist_kernel(const int32_t* __restrict__ gid, int32_t* __restrict__ blk_hist, int T, int M,
                 int nblk, uint32_t* header) {
  __shared__ int hist[kMaxM];
  const int b = blockIdx.y, blk = blockIdx.x;
  if (threadIdx.x < kMaxM) hist[threadIdx.x] = 0;
  __syncthreads();
  const int32_t* g = gid + (size_t)b * T;
  const int begin = blk * kSortChunk;
  const int end = min(begin + kSortChunk, T);
  for (int a0 = begin; a0 < end; a0 += kSortThreads) {
    int a = a0 + threadIdx.x;
    bool valid = a < end;
    int key = valid ? g[a] : -1;
    if (valid && (key < 0 || key >= M)) {
      report_status(header, MOGA_ERR_INTERNAL, 0x50000000u | (uint32_t)(a & 0x0fffffff));
      key = key < 0 ? 0 : M - 1;
    }
    unsigned peers = __match_any_sync(0xffffffffu, key);
    if (valid && (int)(__ffs(peers) - 1) == (int)(threadIdx.x & 31))
      atomicAdd(&hist[key], __popc(peers));
  }
  __syncthreads();
  if (threadIdx.x < M) blk_hist[((size_t)b * nblk + blk) * M + threadIdx.x] = hist[threadIdx.x];
}

// One block per batch item; warp w handles groups w, w+32.  In place: blk_hist[b][blk][g]
// becomes the first sorted position block `blk` writes for group g.
__global__ void __launch_bounds__(1024)
sort_scan_kernel(int32_t* __restrict__ blk_hist, int32_t* __restrict__ offsets, int M, int nblk) {
  __shared__ int total[kMaxM];
  __shared__ int start[kMaxM + 1];
  const int b = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int32_t* h = blk_hist + (size_t)b * nblk * M;
  for (int g = warp; g < M; g += 32) {
    int run = 0;
    for (int c0 = 0; c0 < nblk; c0 += 32) {
      int blk = c0 + lane;
      int v = blk < nblk ? h[(size_t)blk * M + g] : 0;
      int inc = v;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += t;
      }
      if (blk < nblk) h[(size_t)blk * M + g] = run + inc - v;   // exclusive, group-relative
      run += __shfl_sync(0xffffffffu, inc, 31);
    }
    if (lane == 0) total[g] = run;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int acc = 0;
    for (int g = 0; g < M; ++g) {
      start[g] = acc;
      acc += total[g];
    }
    start[M] = acc;
  }
  __syncthreads();
  if (threadIdx.x <= M) offsets[(size_t)b * (M + 1) + threadIdx.x] = start[threadIdx.x];
  for (int idx = threadIdx.x; idx < nblk * M; idx += blockDim.x) h[idx] += start[idx % M];
}

__global__ void __launch_bounds__(kSortThreads)
sort_scatter_kernel(const int32_t* __restrict__ gid, const int32_t* __restrict__ blk_base,
                    int32_t* __restrict__ perm, int32_t* __restrict__ inv, int32_t* __restrict__ asg, int T,
                    int M, int k, int nblk) {
  __shared__ int base[kMaxM];
  __shared__ int wcnt[kSortWarps][kMaxM];
  const int b = blockIdx.y, blk = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x < M) base[threadIdx.x] = blk_base[((size_t)b * nblk + blk) * M + threadIdx.x];
  const int32_t* g = gid + (size_t)b * T;
  const int begin = blk * kSortChunk;
  const int end = min(begin + kSortChunk, T);
  for (int a0 = begin; a0 < end; a0 += kSortThreads) {
    for (int i = threadIdx.x; i < kSortWarps * kMaxM; i += kSortThreads) (&wcnt[0][0])[i] = 0;
    __syncthreads();
    int a = a0 + threadIdx.x;
    bool valid = a < end;
    int key = valid ? g[a] : -1;
    if (valid) key = key < 0 ? 0 : (key >= M ? M - 1 : key);
    unsigned peers = __match_any_sync(0xffffffffu, key);
    int rank = __popc(peers & ((1u << lane) - 1u));       // same-key lanes before me
    if (valid && rank == 0) wcnt[warp][key] = __popc(peers);
    __syncthreads();
    if (valid) {
      int pos = base[key] + rank;
      for (int w = 0; w < warp; ++w) pos += wcnt[w][key];
      perm[(size_t)b * T + pos] = a / k;
      inv[(size_t)b * T + a] = pos;
      if (asg != nullptr) asg[(size_t)b * T + pos] = a;     // the assignment (token, slot) at this position
    }
    __syncthreads();
    if (threadIdx.x < M) {
      int add = 0;
#pragma unroll
      for (int w = 0; w < kSortWarps; ++w) add += wcnt[w][threadIdx.x];
      base[threadIdx.x] += add;
    }
    __syncthreads();
  }
}

}  // namespace

moga_status launch_sort(const moga_shape& s, const WsLayout& L, const int32_t* gid, int32_t* perm,
                        int32_t* inv, int32_t* offsets, char* ws, cudaStream_t st, int32_t* asg) {
  const int T = s.N * s.k;
  int32_t* hist = reinterpret_cast<int32_t*>(ws + L.sort_hist);
  uint32_t* header = reinterpret_cast<uint32_t*>(ws + L.header);
  dim3 grid(L.nblk, s.B);
  sort_hist_kernel<<<grid, kSortThreads, 0, st>>>(gid, hist, T, s.M, L.nblk, header);
  MOGA_CUDA_OK(cudaGetLastError());
  sort_scan_kernel<<<s.B, 1024, 0, st>>>(hist, offsets, s.M, L.nblk);
  MOGA_CUDA_OK(cudaGetLastError());
  sort_scatter_kernel<<<grid, kSortThreads, 0, st>>>(gid, hist, perm, inv, asg, T, s.M, s.k, L.nblk);
  MOGA_CUDA_OK(cudaGetLastError());
  return MOGA_OK;
}

}  // namespace moga
