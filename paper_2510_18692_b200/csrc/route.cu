// Router (Eq. 2-4): r = X W_r (+ bias) in fp32, top-k groups per token, softmax gate.
//
// A skinny GEMM [tokens x C] . [C x M] on the fp32 FMA pipe.  A block owns TT tokens
// and all M groups; X is streamed once from HBM in 128-byte row pieces with cp.async
// (double buffered), W_r chunks come from L2.  Each thread keeps an RT x 8
// (tokens x groups) register tile.  The logits then go through shared memory to a
// token-per-thread top-k / gate epilogue, so nothing but gid, gate (and optionally
// the logits) is written.
#include "moga_internal.cuh"
#include "route_select.cuh"

namespace moga {
namespace {

constexpr int kRouteThreads = 256;
constexpr int kRowBytes = 128;             // bytes of one token row per K-chunk
constexpr int kRowPitch = kRowBytes + 16;  // padded: 8 consecutive rows hit distinct banks

__device__ __forceinline__ void cp_async16(void* dst, const void* src, bool valid) {
  uint32_t d = (uint32_t)__cvta_generic_to_shared(dst);
  int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(d), "l"(src), "r"(sz));
}
__device__ __forceinline__ void cp_async4(void* dst, const void* src, bool valid) {
  uint32_t d = (uint32_t)__cvta_generic_to_shared(dst);
  int sz = valid ? 4 : 0;
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;\n" ::"r"(d), "l"(src), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

template <typename XT>
struct Chunk {
  static constexpr int EPV = 16 / (int)sizeof(XT);         // elements per 16-byte vector
  static constexpr int CK = kRowBytes / (int)sizeof(XT);   // channels per chunk
};

__device__ __forceinline__ void unpack(const uint4& v, float (&x)[8], __nv_bfloat16) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    x[2 * i] = __uint_as_float(w[i] << 16);
    x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ void unpack(const uint4& v, float (&x)[4], float) {
  x[0] = __uint_as_float(v.x);
  x[1] = __uint_as_float(v.y);
  x[2] = __uint_as_float(v.z);
  x[3] = __uint_as_float(v.w);
}

template <typename XT, int MP, int RT>
__global__ void __launch_bounds__(kRouteThreads)
route_kernel(const XT* __restrict__ X, const float* __restrict__ Wr, const float* __restrict__ bias,
             int32_t* __restrict__ gid, float* __restrict__ gate, float* __restrict__ logits,
             long long total_tokens, int C, int M, int k, int gate_mode) {
  constexpr int EPV = Chunk<XT>::EPV;
  constexpr int CK = Chunk<XT>::CK;
  constexpr int GT = MP / 8;                  // threads across the group dimension
  constexpr int TTH = kRouteThreads / GT;     // threads across the token dimension
  constexpr int TT = TTH * RT;                // tokens per block
  constexpr int XBUF = TT * kRowPitch;        // bytes of one X stage

  extern __shared__ __align__(16) unsigned char smem[];
  unsigned char* xs = smem;                   // 2 stages
  float* wsm = reinterpret_cast<float*>(smem + 2 * XBUF);

  const int tid = threadIdx.x;
  const int gt = tid % GT;
  const int tt = tid / GT;
  const long long tok0 = (long long)blockIdx.x * TT;

  float acc[RT][8];
#pragma unroll
  for (int i = 0; i < RT; ++i)
#pragma unroll
    for (int m = 0; m < 8; ++m) acc[i][m] = 0.f;

  const int nch = (C + CK - 1) / CK;

  auto load_chunk = [&](int ch, int stage) {
    const int c0 = ch * CK;
    unsigned char* xb = xs + stage * XBUF;
    for (int idx = tid; idx < TT * 8; idx += kRouteThreads) {
      int r = idx >> 3, v = idx & 7;
      long long tok = tok0 + r;
      int c = c0 + v * EPV;
      bool ok = tok < total_tokens && c < C;
      const XT* src = ok ? X + tok * C + c : X;
      cp_async16(xb + r * kRowPitch + v * 16, src, ok);
    }
    float* wb = wsm + stage * (CK * MP);
    for (int idx = tid; idx < CK * MP; idx += kRouteThreads) {
      int kk = idx / MP, m = idx % MP;
      bool ok = (c0 + kk) < C && m < M;
      const float* src = ok ? Wr + (size_t)(c0 + kk) * M + m : Wr;
      cp_async4(wb + idx, src, ok);
    }
  };

  load_chunk(0, 0);
  cp_async_commit();
  for (int ch = 0; ch < nch; ++ch) {
    const int stage = ch & 1;
    if (ch + 1 < nch) {
      load_chunk(ch + 1, stage ^ 1);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    const unsigned char* xb = xs + stage * XBUF;
    const float* wb = wsm + stage * (CK * MP) + gt * 8;
#pragma unroll 2
    for (int v = 0; v < 8; ++v) {            // 16-byte vectors along the chunk
      float x[RT][EPV];
#pragma unroll
      for (int i = 0; i < RT; ++i) {
        uint4 raw = *reinterpret_cast<const uint4*>(xb + (tt + i * TTH) * kRowPitch + v * 16);
        unpack(raw, x[i], XT());
      }
#pragma unroll
      for (int e = 0; e < EPV; ++e) {
        const float4 w0 = *reinterpret_cast<const float4*>(wb + (v * EPV + e) * MP);
        const float4 w1 = *reinterpret_cast<const float4*>(wb + (v * EPV + e) * MP + 4);
        const float w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
        for (int i = 0; i < RT; ++i)
#pragma unroll
          for (int m = 0; m < 8; ++m) acc[i][m] = fmaf(x[i][e], w[m], acc[i][m]);
      }
    }
    __syncthreads();
  }

  // Logits to shared memory (reusing the X stages), then one thread per token.
  constexpr int LP = MP + 1;
  float* ls = reinterpret_cast<float*>(smem);
  static_assert(TT * LP * 4 <= 2 * XBUF, "logit tile must fit in the X stages");
#pragma unroll
  for (int i = 0; i < RT; ++i)
#pragma unroll
    for (int m = 0; m < 8; ++m) ls[(tt + i * TTH) * LP + gt * 8 + m] = acc[i][m];
  __syncthreads();
  if (bias != nullptr) {
    for (int idx = tid; idx < TT * M; idx += kRouteThreads) {
      int r = idx / M, m = idx % M;
      ls[r * LP + m] += bias[m];
    }
    __syncthreads();
  }
  if (logits != nullptr) {
    for (int idx = tid; idx < TT * M; idx += kRouteThreads) {
      int r = idx / M, m = idx % M;
      if (tok0 + r < total_tokens) logits[(tok0 + r) * M + m] = ls[r * LP + m];
    }
  }
  for (int r = tid; r < TT; r += kRouteThreads) {
    const long long tok = tok0 + r;
    if (tok >= total_tokens) continue;
    select_and_gate(ls + r * LP, M, k, gate_mode, gid + tok * k, gate + tok * k);
  }
}

template <typename XT, int MP, int RT>
moga_status launch_one(const moga_shape& s, const void* X, const float* Wr, const float* bias,
                       int32_t* gid, float* gate, float* logits, cudaStream_t st) {
  constexpr int GT = MP / 8;
  constexpr int TT = (kRouteThreads / GT) * RT;
  constexpr int CK = Chunk<XT>::CK;
  constexpr int smem = 2 * TT * kRowPitch + 2 * CK * MP * 4;
  auto kern = route_kernel<XT, MP, RT>;
  MOGA_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  long long total = (long long)s.B * s.N;
  if (total == 0) return MOGA_OK;
  long long blocks = (total + TT - 1) / TT;
  kern<<<(unsigned)blocks, kRouteThreads, smem, st>>>(static_cast<const XT*>(X), Wr, bias, gid,
                                                       gate, logits, total, s.C, s.M, s.k,
                                                       s.gate_mode);
  MOGA_CUDA_OK(cudaGetLastError());
  return MOGA_OK;
}

template <typename XT>
moga_status launch_typed(const moga_shape& s, const void* X, const float* Wr, const float* bias,
                         int32_t* gid, float* gate, float* logits, cudaStream_t st) {
  if (s.M <= 8) return launch_one<XT, 8, 2>(s, X, Wr, bias, gid, gate, logits, st);
  if (s.M <= 16) return launch_one<XT, 16, 2>(s, X, Wr, bias, gid, gate, logits, st);
  if (s.M <= 32) return launch_one<XT, 32, 4>(s, X, Wr, bias, gid, gate, logits, st);
  return launch_one<XT, 64, 4>(s, X, Wr, bias, gid, gate, logits, st);
}

}  // namespace

moga_status launch_route(const moga_shape& s, const void* X, const float* Wr, const float* bias,
                         int32_t* gid, float* gate, float* logits, cudaStream_t st) {
  if (s.dtype == MOGA_BF16)
    return launch_typed<__nv_bfloat16>(s, X, Wr, bias, gid, gate, logits, st);
  return launch_typed<float>(s, X, Wr, bias, gid, gate, logits, st);
}

}  // namespace moga
