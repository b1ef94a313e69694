// Router (Eq. 2-4) for bf16 token features on the tcgen05 tensor cores, at fp32 accuracy.
//
// r = X W_r is a skinny GEMM that is bound by the one pass over X (N x C, bf16) only if
// the M multiply-adds per loaded element are cheap.  Each fp32 weight is written as the sum
// of three bf16 numbers (w = hi + mid + lo, 24 mantissa bits in all), so every product
// x * w_part is a bf16 x bf16 product, exact in fp32, and the sums are accumulated in fp32
// in TMEM: the result agrees with an fp32 FMA chain to fp32 rounding.  The three parts are
// stacked along the MMA's N dimension (one instruction per 16-channel step covers all of
// them: the cost of a step is set by streaming the 128-token A operand, not by N), so each
// part has its own accumulator columns.  To keep the accumulation error of the tensor core
// (one rounding per step) near that of an fp32 chain, consecutive 64-channel chunks rotate
// over NACC independent accumulators; the epilogue adds parts and accumulators in fp32.
//
//   prep kernel  splits W_r [C, M] fp32 into Wsplit [3, MP, C] bf16 (K-major rows, MP = M
//                rounded up to 16 / 32 / 64, padding rows zero).
//   main kernel  persistent, one CTA per SM, 128 tokens per tile:
//     warp 0     TMA producer: per chunk one X box [128 tokens x 64 ch] and one Wsplit box
//                [3*MP rows x 64 ch] into a ring of stages (128-byte swizzle).
//     warp 1     MMA issuer: per chunk 4 k-steps of tcgen05.mma 128 x (3*MP) x 16 into
//                accumulator (chunk mod NACC).
//     warps 2-5  epilogue, one thread per token: adds the accumulators, bias, then the
//                top-k / gate selection shared with the fp32-ALU router kernel.
// Every mbarrier wait is bounded; on expiry the CTA records MOGA_ERR_TIMEOUT and leaves.
#include "moga_internal.cuh"
#include "route_select.cuh"
#include "sm100_ptx.cuh"

namespace moga {
namespace {

using namespace sm100;

constexpr int kThreads = 192;
constexpr int kTok = 128;                  // tokens per tile (MMA M)
constexpr int kChunk = 64;                 // channels per stage: 128 bytes per row
constexpr int kXBytes = kTok * 128;

template <int MP>
struct RCfg {
  static constexpr int NACC = 512 / (3 * MP);              // 10, 5, 2 for MP = 16, 32, 64
  static constexpr int kAccCols = 3 * MP;                  // hi | mid | lo partial sums
  static constexpr int kTmemCols = 512;
  static constexpr int kWBytes = 3 * MP * 128;
  static constexpr int kStageBytes = kXBytes + kWBytes;    // a multiple of 1024
  static constexpr int kLogitPitch = MP + 1;
  static constexpr int kLogitBytes = kTok * kLogitPitch * 4;
  static constexpr int NS = (200 * 1024 - kLogitBytes) / kStageBytes;
  static constexpr int kSmemBar = NS * kStageBytes;
  static constexpr int kNumBars = 2 * NS + 2;
  static constexpr int kSmemLogits = kSmemBar + 8 * kNumBars + 16;
  static constexpr int kDynSmem = kSmemLogits + kLogitBytes + 1024;   // slack for 1024-byte alignment
  static_assert(NS >= 3, "ring too shallow");
};

// Wsplit[t][m][c] = t-th bf16 part of W_r[c][m]; rows m >= M are zero.
__global__ void route_split_w_kernel(const float* __restrict__ Wr, __nv_bfloat16* __restrict__ out, int C,
                                     int M, int MP) {
  const long long n = (long long)MP * C;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < n;
       idx += (long long)gridDim.x * blockDim.x) {
    const int m = (int)(idx / C), c = (int)(idx % C);
    const float w = m < M ? Wr[(size_t)c * M + m] : 0.f;
    const __nv_bfloat16 hi = __float2bfloat16_rn(w);
    const float r1 = w - __bfloat162float(hi);          // exact
    const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
    const float r2 = r1 - __bfloat162float(mid);        // exact
    out[idx] = hi;
    out[n + idx] = mid;
    out[2 * n + idx] = __float2bfloat16_rn(r2);
  }
}

template <int MP>
__global__ void __launch_bounds__(kThreads, 1)
route_mma_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW,
                 const float* __restrict__ bias, int32_t* __restrict__ gid, float* __restrict__ gate,
                 float* __restrict__ logits, uint32_t* header, long long total_tokens, int C, int M, int k,
                 int gate_mode, uint64_t wait_limit_ns) {
  using R = RCfg<MP>;
  constexpr int NS = R::NS, NACC = R::NACC;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + R::kSmemBar;
  constexpr int FULL = 0, EMPTY = NS, ACC_FULL = 2 * NS, ACC_EMPTY = 2 * NS + 1;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + R::kSmemBar + 8 * R::kNumBars);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  float* ls = reinterpret_cast<float*>(smem + R::kSmemLogits);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ntiles = (int)((total_tokens + kTok - 1) / kTok);
  const int nch = (C + kChunk - 1) / kChunk;

  if (threadIdx.x == 0) {
    for (int i = 0; i < NS; ++i) {
      mbar_init(bar(FULL + i), 1);
      mbar_init(bar(EMPTY + i), 1);
    }
    mbar_init(bar(ACC_FULL), 1);
    mbar_init(bar(ACC_EMPTY), kTok);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32((const void*)tmem_slot), (uint32_t)R::kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  auto wait = [&](int idx, uint32_t parity, uint32_t where) -> bool {
    const WaitResult res = mbar_wait_bounded(bar(idx), parity, abort_flag, wait_limit_ns);
    if (res == kWaitExpired)
      report_status(header, MOGA_ERR_TIMEOUT,
                    (where << 24) | (1u << 23) | ((uint32_t)blockIdx.x << 8) | (uint32_t)idx);
    return res == kWaitDone;
  };

  if (warp == 0) {
    // ===================================================================== TMA producer
    if (lane == 0) {
      uint32_t n = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < ntiles; tile += gridDim.x) {
        for (int q = 0; q < nch; ++q, ++n) {
          const int s = n % NS;
          ok = wait(EMPTY + s, ((n / NS) & 1u) ^ 1u, 1);
          if (!ok) break;
          const uint32_t dst = base + s * R::kStageBytes;
          mbar_expect_tx(bar(FULL + s), R::kStageBytes);
          tma_load_2d(dst, &mapX, bar(FULL + s), q * kChunk, tile * kTok);
          tma_load_2d(dst + kXBytes, &mapW, bar(FULL + s), q * kChunk, 0);
        }
      }
    }
  } else if (warp == 1) {
    // ===================================================================== MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc(kTok, 3 * MP, false);
      constexpr uint32_t hi = desc_hi(1024);
      uint32_t n = 0, nt = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < ntiles; tile += gridDim.x, ++nt) {
        ok = wait(ACC_EMPTY, (nt & 1u) ^ 1u, 2);     // the epilogue has read the previous tile
        if (!ok) break;
        tc_fence_after();
        for (int q = 0; q < nch; ++q, ++n) {
          const int s = n % NS;
          ok = wait(FULL + s, (n / NS) & 1u, 3);
          if (!ok) break;
          tc_fence_after();
          const uint32_t xa = desc_lo(base + s * R::kStageBytes, 16);
          const uint32_t wb = desc_lo(base + s * R::kStageBytes + kXBytes, 16);
          const uint32_t d = tmem + (uint32_t)((q % NACC) * R::kAccCols);
#pragma unroll
          for (int kk = 0; kk < kChunk / 16; ++kk)
            mma_ss(d, xa + kk * 2, wb + kk * 2, hi, idesc, (q >= NACC || kk > 0) ? 1u : 0u);
          tc_commit(bar(EMPTY + s));
        }
        if (ok) tc_commit(bar(ACC_FULL));
      }
    }
  } else {
    // ===================================================================== epilogue
    const int q4 = warp & 3;                        // TMEM lane quarter this warp may read
    const int row = q4 * 32 + lane;
    const uint32_t taddr = tmem + ((uint32_t)(q4 * 32) << 16);
    const int valid_cols = (nch < NACC ? nch : NACC) * R::kAccCols;
    uint32_t nt = 0;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < ntiles; tile += gridDim.x, ++nt) {
      ok = __all_sync(0xffffffffu, wait(ACC_FULL, nt & 1u, 4));   // warp-uniform: TMEM loads are warp-collective
      if (!ok) break;
      tc_fence_after();
      float r[MP];
#pragma unroll
      for (int i = 0; i < MP; ++i) r[i] = 0.f;
#pragma unroll
      for (int p = 0; p < R::kTmemCols / 32; ++p) {
        if (p * 32 < valid_cols) {
          uint32_t v[32];
          tmem_ld32(taddr + p * 32, v);
          tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; ++c)
            r[(p * 32 + c) % MP] += (p * 32 + c < valid_cols) ? __uint_as_float(v[c]) : 0.f;
        }
      }
      tc_fence_before();
      mbar_arrive(bar(ACC_EMPTY));                  // TMEM may take the next tile
      const long long tok = (long long)tile * kTok + row;
#pragma unroll
      for (int i = 0; i < MP; ++i)
        if (i < M) ls[row * R::kLogitPitch + i] = r[i] + (bias != nullptr ? bias[i] : 0.f);
      // optional output: each thread writes the row it owns, so no role ever waits on another
      // outside the bounded mbarrier waits
      if (logits != nullptr && tok < total_tokens)
        for (int m = 0; m < M; ++m) logits[tok * M + m] = ls[row * R::kLogitPitch + m];
      if (tok < total_tokens)
        select_and_gate(ls + row * R::kLogitPitch, M, k, gate_mode, gid + tok * k, gate + tok * k);
    }
  }

  __syncwarp();
  if (*abort_flag) {
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, (uint32_t)R::kTmemCols);
  }
}

// Row-major [rows, C] bf16 matrix, box 64 channels x box_rows, 128-byte swizzle, zero fill.
bool make_map_2d(CUtensorMap* map, const void* ptr, long long rows, int C, int box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {(cuuint64_t)C, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)C * 2};
  cuuint32_t box[2] = {(cuuint32_t)kChunk, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int MP>
moga_status launch(const moga_shape& s, const WsLayout& L, const void* X, const float* Wr, const float* bias,
                   int32_t* gid, float* gate, float* logits, char* ws, cudaStream_t st) {
  using R = RCfg<MP>;
  const long long total = (long long)s.B * s.N;
  __nv_bfloat16* wsplit = reinterpret_cast<__nv_bfloat16*>(ws + L.wsplit);
  const long long nsplit = (long long)MP * s.C;
  route_split_w_kernel<<<(unsigned)((nsplit + 255) / 256 < 1024 ? (nsplit + 255) / 256 : 1024), 256, 0, st>>>(
      Wr, wsplit, s.C, s.M, MP);
  MOGA_CUDA_OK(cudaGetLastError());
  CUtensorMap mx, mw;
  if (!make_map_2d(&mx, X, total, s.C, kTok) || !make_map_2d(&mw, wsplit, 3 * MP, s.C, 3 * MP))
    return MOGA_ERR_CUDA;
  int num_sms = 0;
  if (!current_sm_count(&num_sms)) return MOGA_ERR_CUDA;
  auto kern = route_mma_kernel<MP>;
  MOGA_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, R::kDynSmem));
  const long long ntiles = (total + kTok - 1) / kTok;
  const int grid = (int)(ntiles < num_sms ? ntiles : num_sms);
  kern<<<grid, kThreads, R::kDynSmem, st>>>(mx, mw, bias, gid, gate, logits,
                                            reinterpret_cast<uint32_t*>(ws + L.header), total, s.C, s.M, s.k,
                                            s.gate_mode, kDefaultWaitLimitNs);
  MOGA_CUDA_OK(cudaGetLastError());
  return MOGA_OK;
}

}  // namespace

moga_status launch_route_mma(const moga_shape& s, const WsLayout& L, const void* X, const float* Wr,
                             const float* bias, int32_t* gid, float* gate, float* logits, char* ws,
                             cudaStream_t st) {
  if ((long long)s.B * s.N == 0) return MOGA_OK;
  if (s.M <= 16) return launch<16>(s, L, X, Wr, bias, gid, gate, logits, ws, st);
  if (s.M <= 32) return launch<32>(s, L, X, Wr, bias, gid, gate, logits, ws, st);
  return launch<64>(s, L, X, Wr, bias, gid, gate, logits, ws, st);
}

}  // namespace moga
