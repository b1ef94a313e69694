// Row gather into group-major order (Alg. 1 line 2, data part) and the gated
// inverse (Alg. 1 line 4 with the gate of Eq. 5).  Pure data movement: 16-byte
// vector loads/stores, one row (D*s = 128..512 bytes) per group of threads, several
// independent rows in flight per thread, 64-bit element offsets throughout.
#include "moga_internal.cuh"

namespace moga {
namespace {

constexpr int kMoveThreads = 256;
constexpr int kRowsPerThread = 4;   // independent 16-byte transfers in flight per tensor

// grid: (ceil(T / rows_per_block), H, B).  vec_per_row = D*s/16.
__global__ void __launch_bounds__(kMoveThreads)
gather_rows_kernel(const int32_t* __restrict__ perm, const uint4* __restrict__ Q,
                   const uint4* __restrict__ K, const uint4* __restrict__ V,
                   uint4* __restrict__ Qp, uint4* __restrict__ Kp, uint4* __restrict__ Vp, int T,
                   int H, int vec_per_row, long long sb, long long sh, long long sn) {
  const int rows_per_pass = kMoveThreads / vec_per_row;
  const int lane_row = threadIdx.x / vec_per_row;
  const int v = threadIdx.x % vec_per_row;
  const int b = blockIdx.z, h = blockIdx.y;
  const int p0 = blockIdx.x * rows_per_pass * kRowsPerThread;
  const int32_t* pm = perm + (size_t)b * T;
  const long long src_base = (long long)b * sb + (long long)h * sh;       // in uint4 units
  const long long dst_base = ((long long)b * H + h) * (long long)T * vec_per_row;
  uint4 q[kRowsPerThread], kk[kRowsPerThread], vv[kRowsPerThread];
  int p[kRowsPerThread];
#pragma unroll
  for (int i = 0; i < kRowsPerThread; ++i) {
    p[i] = p0 + i * rows_per_pass + lane_row;
    if (p[i] < T) {
      long long src = src_base + (long long)pm[p[i]] * sn + v;
      q[i] = __ldg(Q + src);
      kk[i] = __ldg(K + src);
      vv[i] = __ldg(V + src);
    }
  }
#pragma unroll
  for (int i = 0; i < kRowsPerThread; ++i) {
    if (p[i] < T) {
      long long dst = dst_base + (long long)p[i] * vec_per_row + v;
      Qp[dst] = q[i];
      Kp[dst] = kk[i];
      Vp[dst] = vv[i];
    }
  }
}

// The same copy in scatter form, for k > 1: a token's row is read once and written to the k sorted
// positions inv[b, n, 0..k) of its assignments, so the sources cross DRAM once instead of k times.
// grid: (ceil(N / rows_per_block), H, B).
template <int K>
__global__ void __launch_bounds__(kMoveThreads)
scatter_rows_kernel(const int32_t* __restrict__ inv, const uint4* __restrict__ Q, const uint4* __restrict__ K_,
                    const uint4* __restrict__ V, uint4* __restrict__ Qp, uint4* __restrict__ Kp,
                    uint4* __restrict__ Vp, int N, int H, int vec_per_row, long long sb, long long sh,
                    long long sn) {
  const int rows_per_pass = kMoveThreads / vec_per_row;
  const int lane_row = threadIdx.x / vec_per_row;
  const int v = threadIdx.x % vec_per_row;
  const int b = blockIdx.z, h = blockIdx.y;
  const int n0 = blockIdx.x * rows_per_pass * kRowsPerThread;
  const long long T = (long long)N * K;
  const int32_t* iv = inv + (size_t)b * T;
  const long long src_base = (long long)b * sb + (long long)h * sh;       // in uint4 units
  const long long dst_base = ((long long)b * H + h) * T * vec_per_row;
  uint4 q[kRowsPerThread], kk[kRowsPerThread], vv[kRowsPerThread];
  int pos[kRowsPerThread][K];
#pragma unroll
  for (int i = 0; i < kRowsPerThread; ++i) {
    const int n = n0 + i * rows_per_pass + lane_row;
    if (n < N) {
      const long long src = src_base + (long long)n * sn + v;
      q[i] = __ldg(Q + src);
      kk[i] = __ldg(K_ + src);
      vv[i] = __ldg(V + src);
#pragma unroll
      for (int j = 0; j < K; ++j) pos[i][j] = __ldg(iv + (long long)n * K + j);
    }
  }
#pragma unroll
  for (int i = 0; i < kRowsPerThread; ++i) {
    const int n = n0 + i * rows_per_pass + lane_row;
    if (n < N) {
#pragma unroll
      for (int j = 0; j < K; ++j) {
        const long long dst = dst_base + (long long)pos[i][j] * vec_per_row + v;
        Qp[dst] = q[i];
        Kp[dst] = kk[i];
        Vp[dst] = vv[i];
      }
    }
  }
}

__device__ __forceinline__ void fma_vec(float (&acc)[8], const uint4& raw, float g, __nv_bfloat16) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    acc[2 * i] = fmaf(g, __uint_as_float(w[i] << 16), acc[2 * i]);
    acc[2 * i + 1] = fmaf(g, __uint_as_float(w[i] & 0xffff0000u), acc[2 * i + 1]);
  }
}
__device__ __forceinline__ void fma_vec(float (&acc)[8], const uint4& raw, float g, float) {
  acc[0] = fmaf(g, __uint_as_float(raw.x), acc[0]);
  acc[1] = fmaf(g, __uint_as_float(raw.y), acc[1]);
  acc[2] = fmaf(g, __uint_as_float(raw.z), acc[2]);
  acc[3] = fmaf(g, __uint_as_float(raw.w), acc[3]);
}
__device__ __forceinline__ uint4 pack_vec(const float (&acc)[8], __nv_bfloat16) {
  uint4 r;
  __nv_bfloat162 t;
  t = __floats2bfloat162_rn(acc[0], acc[1]); r.x = *reinterpret_cast<uint32_t*>(&t);
  t = __floats2bfloat162_rn(acc[2], acc[3]); r.y = *reinterpret_cast<uint32_t*>(&t);
  t = __floats2bfloat162_rn(acc[4], acc[5]); r.z = *reinterpret_cast<uint32_t*>(&t);
  t = __floats2bfloat162_rn(acc[6], acc[7]); r.w = *reinterpret_cast<uint32_t*>(&t);
  return r;
}
__device__ __forceinline__ uint4 pack_vec(const float (&acc)[8], float) {
  return make_uint4(__float_as_uint(acc[0]), __float_as_uint(acc[1]), __float_as_uint(acc[2]),
                    __float_as_uint(acc[3]));
}

// O[b,h,n,:] = sum_j gate[b,n,j] * Op[b,h,inv[b,n,j],:]   (fp32, slot order, one rounding)
// K > 0: top-k known at compile time, so the index loads of all of a thread's rows go out first
// and all their row loads next (the rows are random 256-byte reads: the more in flight, the
// closer to the copy rate); K == 0: any k, slot loop.
constexpr int kUnpRows = 8;
template <typename XT, int K>
__global__ void __launch_bounds__(kMoveThreads)
unpermute_kernel(const uint4* __restrict__ Op, const int32_t* __restrict__ inv,
                 const float* __restrict__ gate, uint4* __restrict__ O, int N, int k, int H,
                 int vec_per_row, long long sb, long long sh, long long sn) {
  const int rows_per_pass = kMoveThreads / vec_per_row;
  const int lane_row = threadIdx.x / vec_per_row;
  const int v = threadIdx.x % vec_per_row;
  const int b = blockIdx.z, h = blockIdx.y;
  const long long T = (long long)N * k;
  const long long src_base = ((long long)b * H + h) * T * vec_per_row;
  const long long dst_base = (long long)b * sb + (long long)h * sh;
  if (K > 0) {
    constexpr int KK = K > 0 ? K : 1;
    constexpr int R = kUnpRows / KK;           // 8 row loads in flight per thread
    const int n0 = blockIdx.x * rows_per_pass * R;
    int pos[R][KK];
    float g[R][KK];
    uint4 raw[R][KK];
#pragma unroll
    for (int i = 0; i < R; ++i) {
      const int n = n0 + i * rows_per_pass + lane_row;
#pragma unroll
      for (int j = 0; j < KK; ++j) {
        const long long a = (long long)b * T + (long long)(n < N ? n : 0) * KK + j;
        pos[i][j] = __ldg(inv + a);
        g[i][j] = gate != nullptr ? __ldg(gate + a) : 1.f;     // no gates: plain sum over the k assignments
      }
    }
#pragma unroll
    for (int i = 0; i < R; ++i)
#pragma unroll
      for (int j = 0; j < KK; ++j) raw[i][j] = __ldg(Op + src_base + (long long)pos[i][j] * vec_per_row + v);
#pragma unroll
    for (int i = 0; i < R; ++i) {
      const int n = n0 + i * rows_per_pass + lane_row;
      if (n >= N) continue;
      float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int j = 0; j < KK; ++j) fma_vec(acc, raw[i][j], g[i][j], XT());
      O[dst_base + (long long)n * sn + v] = pack_vec(acc, XT());
    }
  } else {
    const int n0 = blockIdx.x * rows_per_pass * kRowsPerThread;
#pragma unroll
    for (int i = 0; i < kRowsPerThread; ++i) {
      const int n = n0 + i * rows_per_pass + lane_row;
      if (n >= N) continue;
      float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      for (int j = 0; j < k; ++j) {
        const long long a = (long long)b * T + (long long)n * k + j;
        const int pos = __ldg(inv + a);
        const float g = gate != nullptr ? __ldg(gate + a) : 1.f;
        const uint4 raw = __ldg(Op + src_base + (long long)pos * vec_per_row + v);
        fma_vec(acc, raw, g, XT());
      }
      O[dst_base + (long long)n * sn + v] = pack_vec(acc, XT());
    }
  }
}

}  // namespace

moga_status launch_gather(const moga_shape& s, const int32_t* perm, const void* Q, const void* K,
                          const void* V, void* Qp, void* Kp, void* Vp, cudaStream_t st, const int32_t* inv) {
  const int T = s.N * s.k;
  if (T == 0) return MOGA_OK;
  const int es = (int)elem_size(s.dtype);
  const int vec_per_row = s.D * es / 16;
  const int epv = 16 / es;
  const Strides sd = qkv_strides(s);
  const int rows_per_block = (kMoveThreads / vec_per_row) * kRowsPerThread;
  const uint4 *q = static_cast<const uint4*>(Q), *k = static_cast<const uint4*>(K), *v = static_cast<const uint4*>(V);
  uint4 *qp = static_cast<uint4*>(Qp), *kp = static_cast<uint4*>(Kp), *vp = static_cast<uint4*>(Vp);
  if (inv != nullptr && s.k >= 2 && s.k <= 4) {
    // top-k > 1: read every token row once, write it to its k positions
    dim3 grid((s.N + rows_per_block - 1) / rows_per_block, s.H, s.B);
    if (s.k == 2)
      scatter_rows_kernel<2><<<grid, kMoveThreads, 0, st>>>(inv, q, k, v, qp, kp, vp, s.N, s.H, vec_per_row,
                                                            sd.b / epv, sd.h / epv, sd.n / epv);
    else if (s.k == 3)
      scatter_rows_kernel<3><<<grid, kMoveThreads, 0, st>>>(inv, q, k, v, qp, kp, vp, s.N, s.H, vec_per_row,
                                                            sd.b / epv, sd.h / epv, sd.n / epv);
    else
      scatter_rows_kernel<4><<<grid, kMoveThreads, 0, st>>>(inv, q, k, v, qp, kp, vp, s.N, s.H, vec_per_row,
                                                            sd.b / epv, sd.h / epv, sd.n / epv);
  } else {
    dim3 grid((T + rows_per_block - 1) / rows_per_block, s.H, s.B);
    gather_rows_kernel<<<grid, kMoveThreads, 0, st>>>(perm, q, k, v, qp, kp, vp, T, s.H, vec_per_row, sd.b / epv,
                                                      sd.h / epv, sd.n / epv);
  }
  MOGA_CUDA_OK(cudaGetLastError());
  return MOGA_OK;
}

template <typename XT>
static moga_status launch_unpermute_t(const moga_shape& s, const void* Op, const int32_t* inv, const float* gate,
                                      void* O, cudaStream_t st) {
  const int es = (int)elem_size(s.dtype);
  const int vec_per_row = s.D * es / 16;
  const int epv = 16 / es;
  const Strides sd = qkv_strides(s);
  const int rows = s.k == 1 ? kUnpRows : (s.k == 2 ? kUnpRows / 2 : kRowsPerThread);
  const int rows_per_block = (kMoveThreads / vec_per_row) * rows;
  dim3 grid((s.N + rows_per_block - 1) / rows_per_block, s.H, s.B);
  const uint4* src = static_cast<const uint4*>(Op);
  uint4* dst = static_cast<uint4*>(O);
  if (s.k == 1)
    unpermute_kernel<XT, 1><<<grid, kMoveThreads, 0, st>>>(src, inv, gate, dst, s.N, s.k, s.H, vec_per_row,
                                                           sd.b / epv, sd.h / epv, sd.n / epv);
  else if (s.k == 2)
    unpermute_kernel<XT, 2><<<grid, kMoveThreads, 0, st>>>(src, inv, gate, dst, s.N, s.k, s.H, vec_per_row,
                                                           sd.b / epv, sd.h / epv, sd.n / epv);
  else
    unpermute_kernel<XT, 0><<<grid, kMoveThreads, 0, st>>>(src, inv, gate, dst, s.N, s.k, s.H, vec_per_row,
                                                           sd.b / epv, sd.h / epv, sd.n / epv);
  MOGA_CUDA_OK(cudaGetLastError());
  return MOGA_OK;
}

moga_status launch_unpermute(const moga_shape& s, const void* Op, const int32_t* inv,
                             const float* gate, void* O, cudaStream_t st) {
  if (s.N == 0) return MOGA_OK;
  return s.dtype == MOGA_BF16 ? launch_unpermute_t<__nv_bfloat16>(s, Op, inv, gate, O, st)
                              : launch_unpermute_t<float>(s, Op, inv, gate, O, st);
}

}  // namespace moga
