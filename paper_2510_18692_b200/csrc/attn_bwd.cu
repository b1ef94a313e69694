// Backward of the bf16 per-group attention on tcgen05 tensor cores (d_head = 128).
//
// The paper states no backward pass; these kernels apply the chain rule to its forward
// (Eq. 1 inside each group, Eq. 5's gate), with the forward's saved log-sum-exp:
//   p  = exp(scale * q k^T - lse)           (the softmax weights, recomputed)
//   ds = p * (do v^T - delta) * scale       delta = <do, o> per query row
//   dV = p^T do      dK = ds^T q      dQ = ds k
// in sorted (group-major) order, do being the upstream gradient already multiplied by the gate.
//
// Two launches of one kernel template, both shaped like the forward kernel (TMA producer warp,
// one MMA-issuing thread, eight compute warps with two threads per TMEM lane (64 of the 128
// columns each), TMEM accumulators, bounded waits), each work item one 128-row tile that stays resident while the other
// operand's tiles stream past it:
//   kModeQ   item = 128 query rows (Q, dO resident); streams the group's K / V tiles:
//            T0 = Q K^T, T1 = dO V^T  ->  dS (bf16, over T1)  ->  dQ += dS K
//   kModeKV  item = 128 key rows (K, V resident); streams the group's Q / dO tiles:
//            T0 = K Q^T, T1 = V dO^T  ->  P^T (bf16, over T0), dS^T (over T1)
//            ->  dV += P^T dO,  dK += dS^T Q
// Computing the transposed products in the second launch keeps every A operand either K-major
// in shared memory or row-per-lane in TMEM and every streamed tile usable as the MN-major B
// operand of the accumulating MMAs: the same operand forms as the forward kernel, at the price of
// seven GEMMs per tile pair instead of five.
// Overlap inside a CTA (one tile pair's T0 / T1 fill the TMEM beside the accumulators, so there is no
// second buffer): the compute warps take T0 first (the exponentials, kept in registers) and release it,
// so the next tile's T0 product runs while they work on T1; the accumulating MMAs of tile j and the T1
// product of tile j+1 run while they take the exponentials of tile j+1.
// TMEM: T0 [0,128) T1 [128,256) acc0 [256,384) acc1 [384,512).  Both bf16 results of the compute warps
// go over T1: a thread that has read 32 of its T1 columns writes P over the first 16 of them and dS over
// the other 16.
#include <type_traits>

#include "attn_common.cuh"

namespace moga {
namespace {

using namespace attn;
using namespace sm100;

constexpr int kThreads = 384;          // warp 0 producer, warp 1 MMA, warps 4-11 compute (two per TMEM lane quarter)
constexpr int kD = 128;
constexpr int kTile = 128;
constexpr int kBoxBytes = kTile * 128;           // 128 rows x 64 columns
constexpr int kTileBytes = 2 * kBoxBytes;        // 32 KB
constexpr int NS = 2;                            // ring depth of the streamed tile pairs
constexpr int kSmemR = 0;                        // resident pair
constexpr int kSmemS = 2 * kTileBytes;           // streamed pairs
constexpr int kSmemVec = kSmemS + NS * 2 * kTileBytes;   // 8 warps x (64 lse + 64 delta) floats
constexpr int kSmemBar = kSmemVec + 8 * 128 * 4;
constexpr int kNumBars = 2 + 2 * NS + 6;
constexpr int kSmemTotal = kSmemBar + 8 * kNumBars + 16;
constexpr int kDynSmem = kSmemTotal + 1024;
static_assert(kDynSmem <= 227 * 1024, "shared memory");

constexpr int kModeQ = 0, kModeKV = 1;

// Sorted-order tensors of one launch; everything [B*H, T, D] bf16 except lse / delta [B*H, T] fp32.
struct BwdArgs {
  const float* lse;      // natural-log sum-exp of the scaled scores, from the forward
  const float* delta;    // <do, o> per sorted row
  __nv_bfloat16* out0;   // kModeQ: dQ;  kModeKV: dV
  __nv_bfloat16* out1;   // kModeKV: dK
};

template <int Mode>
__global__ void __launch_bounds__(kThreads, 1)
attn_bwd_kernel(const __grid_constant__ CUtensorMap mapR0, const __grid_constant__ CUtensorMap mapR1,
                const __grid_constant__ CUtensorMap mapS0, const __grid_constant__ CUtensorMap mapS1,
                const Groups grp, const int32_t* __restrict__ order, const int32_t* __restrict__ prefix,
                const BwdArgs args, uint32_t* header, int T, int H, int BG, float scale_log2, float scale) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sR = base + kSmemR, sS = base + kSmemS;
  const uint32_t bars = base + kSmemBar;
  constexpr int R_FULL = 0, R_EMPTY = 1, S_FULL = 2, S_EMPTY = 2 + NS, T0_FULL = 2 + 2 * NS, T1_FULL = T0_FULL + 1,
                P_DONE = T0_FULL + 2, E_FULL = T0_FULL + 3, ACC_FULL = T0_FULL + 4, ACC_EMPTY = T0_FULL + 5;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + kSmemBar + 8 * kNumBars);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_items = prefix[BG];

  if (threadIdx.x == 0) {
    mbar_init(bar(R_FULL), 1);
    mbar_init(bar(R_EMPTY), 1);
    for (int i = 0; i < NS; ++i) {
      mbar_init(bar(S_FULL + i), 1);
      mbar_init(bar(S_EMPTY + i), 1);
    }
    mbar_init(bar(T0_FULL), 1);
    mbar_init(bar(T1_FULL), 1);
    mbar_init(bar(P_DONE), 2 * kTile);
    mbar_init(bar(E_FULL), 2 * kTile);
    mbar_init(bar(ACC_FULL), 1);
    mbar_init(bar(ACC_EMPTY), 2 * kTile);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32((const void*)tmem_slot), 512u);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  auto wait = [&](int idx, uint32_t parity, uint32_t where) -> bool {
    const WaitResult res = mbar_wait_bounded(bar(idx), parity, abort_flag, kDefaultWaitLimitNs);
    if (res == kWaitExpired)
      report_status(header, MOGA_ERR_TIMEOUT, (where << 24) | (3u << 20) | ((uint32_t)(blockIdx.x & 0xfff) << 8) | (uint32_t)idx);
    return res == kWaitDone;
  };

  // An item: tile rows [it.row0, it.row0 + 128) of its group stay resident; the group's other
  // side is streamed in tiles of 128 rows from it.klo.  (Routed groups: queries and keys are
  // the same rows, so decode_item's query range serves both launches.)
  if (warp == 0) {
    // ===================================================================== TMA producer
    if (lane == 0) {
      uint32_t nit = 0, ns = 0;
      bool ok = true;
      for (int w = blockIdx.x; ok && w < total_items; w += gridDim.x, ++nit) {
        const Item it = decode_item<kTile>(w, grp, order, prefix, BG, H);
        const int ntiles = (it.khi - it.klo + kTile - 1) / kTile;
        ok = wait(R_EMPTY, (nit & 1u) ^ 1u, 1);
        if (!ok) break;
        mbar_expect_tx(bar(R_FULL), 2 * kTileBytes);
#pragma unroll
        for (int bx = 0; bx < 2; ++bx) {
          tma_load_3d(sR + bx * kBoxBytes, &mapR0, bar(R_FULL), bx * 64, it.row0, it.bh);
          tma_load_3d(sR + kTileBytes + bx * kBoxBytes, &mapR1, bar(R_FULL), bx * 64, it.row0, it.bh);
        }
        for (int j = 0; j < ntiles && ok; ++j, ++ns) {
          const int s = ns % NS;
          ok = wait(S_EMPTY + s, ((ns / NS) & 1u) ^ 1u, 2);
          if (!ok) break;
          mbar_expect_tx(bar(S_FULL + s), 2 * kTileBytes);
          const uint32_t dst = sS + s * 2 * kTileBytes;
#pragma unroll
          for (int bx = 0; bx < 2; ++bx) {
            tma_load_3d(dst + bx * kBoxBytes, &mapS0, bar(S_FULL + s), bx * 64, it.klo + j * kTile, it.bh);
            tma_load_3d(dst + kTileBytes + bx * kBoxBytes, &mapS1, bar(S_FULL + s), bx * 64, it.klo + j * kTile, it.bh);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ===================================================================== MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_t = instr_desc(kTile, kTile, false);   // resident x streamed^T, both K-major
      constexpr uint32_t idesc_a = instr_desc(kTile, kD, true);       // TMEM operand x streamed tile (MN-major)
      constexpr uint32_t hi = desc_hi(1024);
      // T[t] = R[t] S[t]^T
      auto issue_t = [&](int t, uint32_t stage) {
        const uint32_t ra = desc_lo(sR + t * kTileBytes, 16), sb = desc_lo(stage + t * kTileBytes, 16);
#pragma unroll
        for (int kk = 0; kk < kD / 16; ++kk) {
          const uint32_t o = ((kk / 4) * kBoxBytes + (kk % 4) * 32) >> 4;
          mma_ss(tmem + t * kTile, ra + o, sb + o, hi, idesc_t, kk > 0);
        }
      };
      // acc[a] (+)= E[e] S[t]   (E[e]: bf16 over T1; the 16 streamed rows of k-step kk sit in 8 columns
      // of the thread half kk / 4, its chunk (kk % 4) / 2; P first, dS 16 columns on)
      auto issue_acc = [&](int a, int e, int t, uint32_t stage, bool accumulate) {
        const uint32_t vb = desc_lo(stage + t * kTileBytes, kBoxBytes);
#pragma unroll
        for (int kk = 0; kk < kTile / 16; ++kk)
          mma_ts(tmem + 256 + a * 128, tmem + kTile + (kk / 4) * 64 + ((kk % 4) / 2) * 32 + (kk % 2) * 8 + e * 16,
                 vb + ((kk * 2048) >> 4), hi, idesc_a, (accumulate || kk > 0) ? 1u : 0u);
      };
      uint32_t nit = 0, ns = 0, nt = 0;
      bool ok = true;
      for (int w = blockIdx.x; ok && w < total_items; w += gridDim.x, ++nit) {
        const Item it = decode_item<kTile>(w, grp, order, prefix, BG, H);
        const int ntiles = (it.khi - it.klo + kTile - 1) / kTile;
        ok = wait(R_FULL, nit & 1u, 3);
        if (!ok) break;
        // first tile: both products.  T0 is free (P_DONE of the previous item's last tile was waited
        // for below); T1 held that tile's P / dS, whose MMAs were issued before these (the pipe keeps issue order).
        ok = wait(S_FULL + ns % NS, (ns / NS) & 1u, 4);
        if (!ok) break;
        tc_fence_after();
        issue_t(0, sS + (ns % NS) * 2 * kTileBytes);
        tc_commit(bar(T0_FULL));
        issue_t(1, sS + (ns % NS) * 2 * kTileBytes);
        tc_commit(bar(T1_FULL));
        if (ntiles == 1) tc_commit(bar(R_EMPTY));
        for (int j = 0; j < ntiles && ok; ++j, ++ns, ++nt) {
          const uint32_t stage = sS + (ns % NS) * 2 * kTileBytes;
          const uint32_t next = sS + ((ns + 1) % NS) * 2 * kTileBytes;
          const bool more = j + 1 < ntiles;
          ok = wait(P_DONE, nt & 1u, 9);                  // T0 of tile j has been read
          if (!ok) break;
          if (more) {
            ok = wait(S_FULL + (ns + 1) % NS, ((ns + 1) / NS) & 1u, 4);
            if (!ok) break;
            tc_fence_after();
            issue_t(0, next);
            tc_commit(bar(T0_FULL));
          }
          ok = wait(E_FULL, nt & 1u, 5);
          if (!ok) break;
          if (j == 0) {
            ok = wait(ACC_EMPTY, (nit & 1u) ^ 1u, 6);     // the previous item's accumulators have been read
            if (!ok) break;
          }
          tc_fence_after();
          if (Mode == kModeQ) {
            issue_acc(0, 1, 0, stage, j > 0);             // dQ += dS K
          } else {
            issue_acc(0, 0, 1, stage, j > 0);             // dV += P^T dO
            issue_acc(1, 1, 0, stage, j > 0);             // dK += dS^T Q
          }
          tc_commit(bar(S_EMPTY + ns % NS));
          if (more) {
            issue_t(1, next);                             // over the P / dS the MMAs above read
            tc_commit(bar(T1_FULL));
            if (j + 2 == ntiles) tc_commit(bar(R_EMPTY));
          } else {
            tc_commit(bar(ACC_FULL));
          }
        }
      }
    }
  } else if (warp >= 4) {
    // ===================================================================== compute + epilogue
    const int q = warp & 3;
    const int half = (warp - 4) >> 2;              // which 64 of the tile's 128 columns this thread handles
    const int r = q * 32 + lane;                   // row of the resident tile = TMEM lane
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    const uint32_t tT0 = tmem + lane_off + half * 64, tT1 = tmem + lane_off + kTile + half * 64;
    float* wvec = reinterpret_cast<float*>(smem + kSmemVec) + (warp - 4) * 128;   // this warp's column vectors
    const float log2e = 1.4426950408889634f;
    uint32_t nit = 0, nt = 0;
    bool ok = true;
    for (int w = blockIdx.x; ok && w < total_items; w += gridDim.x, ++nit) {
      const Item it = decode_item<kTile>(w, grp, order, prefix, BG, H);
      const int ntiles = (it.khi - it.klo + kTile - 1) / kTile;
      const int row = it.row0 + r;
      const bool live = row < it.qhi;
      const size_t vbase = (size_t)it.bh * T;
      float row_lse = 0.f, row_delta = 0.f;       // minus lse * log2e and minus delta * scale of this row
      if (Mode == kModeQ && live) {
        row_lse = -args.lse[vbase + row] * log2e;
        row_delta = -args.delta[vbase + row] * scale;
      }
      for (int j = 0; j < ntiles && ok; ++j, ++nt) {
        const int col0 = it.klo + j * kTile;
        const int ncols = it.khi - col0;             // valid streamed rows (columns of T) in this tile
        if (Mode == kModeKV) {
          // lse and delta of the streamed query rows, per column: each warp keeps its own copy
          __syncwarp();
#pragma unroll
          for (int m = 0; m < 2; ++m) {
            const int c = lane + 32 * m, col = half * 64 + c;
            const bool in = col < ncols;
            wvec[c] = in ? -args.lse[vbase + col0 + col] * log2e : 0.f;
            wvec[64 + c] = in ? -args.delta[vbase + col0 + col] * scale : 0.f;
          }
          __syncwarp();
        }
        ok = __all_sync(0xffffffffu, wait(T0_FULL, nt & 1u, 7));
        if (!ok) break;
        tc_fence_after();
        // p = 2^(t0 * scale_log2 - lse * log2e), kept in registers; T0 is then free for the next tile.
        // A tile that reaches past the group's end takes the variant that zeroes those columns' p.
        const float2 sl2 = make_float2(scale_log2, scale_log2), sc2 = make_float2(scale, scale);
        float2 p[32];
        auto weights = [&](int ch, auto masked) {
          uint32_t t0[32];
          tmem_ld32(tT0 + ch * 32, t0);
          tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            const int lc = ch * 32 + c;
            const float2 nl2 = Mode == kModeQ ? make_float2(row_lse, row_lse) : *reinterpret_cast<const float2*>(wvec + lc);
            const float2 x = __ffma2_rn(make_float2(__uint_as_float(t0[c]), __uint_as_float(t0[c + 1])), sl2, nl2);
            float2 pe = make_float2(ex2(x.x), ex2(x.y));
            if (decltype(masked)::value) {
              const int col = half * 64 + lc;
              pe.x = col < ncols ? pe.x : 0.f;
              pe.y = col + 1 < ncols ? pe.y : 0.f;
            }
            p[lc >> 1] = pe;
          }
        };
        if (ncols < kTile) {
          weights(0, std::true_type{});
          weights(1, std::true_type{});
        } else {
          weights(0, std::false_type{});
          weights(1, std::false_type{});
        }
        tc_fence_before();
        mbar_arrive(bar(P_DONE));
        ok = __all_sync(0xffffffffu, wait(T1_FULL, nt & 1u, 10));
        if (!ok) break;
        tc_fence_after();
        // ds = p * (t1 * scale - delta * scale).  Chunk ch of this thread's T1 columns has been read when
        // its results are written: P over the chunk's first 16 columns, dS over its last 16.
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t t1[32];
          tmem_ld32(tT1 + ch * 32, t1);
          tmem_wait_ld();
          uint32_t ep[16], ed[16];
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            const int lc = ch * 32 + c;
            const float2 nds = Mode == kModeQ ? make_float2(row_delta, row_delta)
                                              : *reinterpret_cast<const float2*>(wvec + 64 + lc);
            const float2 u = __ffma2_rn(make_float2(__uint_as_float(t1[c]), __uint_as_float(t1[c + 1])), sc2, nds);
            const float2 pe = p[lc >> 1];
            const float2 ds = __fmul2_rn(pe, u);
            __nv_bfloat162 a = __floats2bfloat162_rn(pe.x, pe.y);
            __nv_bfloat162 b = __floats2bfloat162_rn(ds.x, ds.y);
            ep[c >> 1] = *reinterpret_cast<uint32_t*>(&a);
            ed[c >> 1] = *reinterpret_cast<uint32_t*>(&b);
          }
          if (Mode == kModeKV) tmem_st16(tT1 + ch * 32, ep);
          tmem_st16(tT1 + ch * 32 + 16, ed);
        }
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar(E_FULL));
      }
      if (!ok) break;
      // ---- epilogue: accumulators -> bf16 rows of the sorted-order outputs
      ok = __all_sync(0xffffffffu, wait(ACC_FULL, nit & 1u, 8));
      if (!ok) break;
      tc_fence_after();
#pragma unroll
      for (int a = 0; a < (Mode == kModeKV ? 2 : 1); ++a) {
        __nv_bfloat16* out = (a == 0 ? args.out0 : args.out1) + (vbase + row) * kD;
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
          const int ch = half * 2 + cc;            // this thread's half of the accumulator columns
          uint32_t acc[32];
          tmem_ld32(tmem + lane_off + 256 + a * 128 + ch * 32, acc);
          tmem_wait_ld();
          if (live) {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              uint4 pk;
              uint32_t* pw = reinterpret_cast<uint32_t*>(&pk);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                __nv_bfloat162 t = __floats2bfloat162_rn(__uint_as_float(acc[v * 8 + 2 * i]),
                                                         __uint_as_float(acc[v * 8 + 2 * i + 1]));
                pw[i] = *reinterpret_cast<uint32_t*>(&t);
              }
              *reinterpret_cast<uint4*>(out + ch * 32 + v * 8) = pk;
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(bar(ACC_EMPTY));
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
    tmem_dealloc(tmem, 512u);
  }
}

// do_p[b,h,p,:] = gate * dO[b,h,token,:] (bf16), delta[b,h,p] = gate * <dO, o_p>, dgate[b,a] = sum_h <dO, o_p>
// for the assignment a = token * k + slot that sits at sorted position p.  One half-warp per
// (b, p): 16 lanes x 8 channels, all heads in turn (the sum over heads is sequential: deterministic).
__global__ void __launch_bounds__(256)
bwd_prep_kernel(const uint4* __restrict__ dO, const uint4* __restrict__ Op, const float* __restrict__ gate,
                const int32_t* __restrict__ perm, const int32_t* __restrict__ inv, uint4* __restrict__ dOp,
                float* __restrict__ delta, float* __restrict__ dgate, int N, int k, int H, long long sb, long long sh,
                long long sn) {
  const int b = blockIdx.y;
  const long long T = (long long)N * k;
  const int p = blockIdx.x * 16 + (threadIdx.x >> 4);
  const int v = threadIdx.x & 15;
  if (p >= T) return;                       // whole half-warps leave together
  const int tok = perm[(size_t)b * T + p];
  int slot = 0;
  for (int j = 0; j < k; ++j)
    if (inv[(size_t)b * T + (long long)tok * k + j] == p) slot = j;
  const long long a = (long long)b * T + (long long)tok * k + slot;
  const float g = gate[a];
  float dg = 0.f;
  const unsigned mask = 0xffffu << (threadIdx.x & 16);
  for (int h = 0; h < H; ++h) {
    const uint4 d = __ldg(dO + (long long)b * sb + (long long)h * sh + (long long)tok * sn + v);
    const size_t at = (((size_t)b * H + h) * T + p) * 16 + v;
    const uint4 o = __ldg(Op + at);
    const uint32_t dw[4] = {d.x, d.y, d.z, d.w}, ow[4] = {o.x, o.y, o.z, o.w};
    float dot = 0.f;
    uint4 outv;
    uint32_t* pw = reinterpret_cast<uint32_t*>(&outv);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float d0 = __uint_as_float(dw[i] << 16), d1 = __uint_as_float(dw[i] & 0xffff0000u);
      dot = fmaf(d0, __uint_as_float(ow[i] << 16), dot);
      dot = fmaf(d1, __uint_as_float(ow[i] & 0xffff0000u), dot);
      __nv_bfloat162 t = __floats2bfloat162_rn(g * d0, g * d1);
      pw[i] = *reinterpret_cast<uint32_t*>(&t);
    }
    dOp[at] = outv;
#pragma unroll
    for (int s = 8; s > 0; s >>= 1) dot += __shfl_xor_sync(mask, dot, s);
    if (v == 0) delta[((size_t)b * H + h) * T + p] = g * dot;
    dg += dot;
  }
  if (v == 0) dgate[a] = dg;
}

template <int Mode>
moga_status launch_bwd(const Problem& p, const void* R0, const void* R1, const void* S0, const void* S1,
                       const BwdArgs& args, cudaStream_t st) {
  CUtensorMap m0, m1, m2, m3;
  const long long BH = (long long)p.B * p.H;
  if (!make_map(&m0, R0, kD, p.Tq, BH, kTile) || !make_map(&m1, R1, kD, p.Tq, BH, kTile) ||
      !make_map(&m2, S0, kD, p.Tq, BH, kTile) || !make_map(&m3, S1, kD, p.Tq, BH, kTile))
    return MOGA_ERR_CUDA;
  int num_sms = 0;
  if (!current_sm_count(&num_sms)) return MOGA_ERR_CUDA;
  auto kern = attn_bwd_kernel<Mode>;
  MOGA_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmem));
  const long long max_items = ((p.Tq + kTile - 1) / kTile + p.grp.G) * BH;
  const int grid = (int)(max_items < num_sms ? max_items : num_sms);
  const float log2e = 1.4426950408889634f;
  kern<<<grid, kThreads, kDynSmem, st>>>(m0, m1, m2, m3, p.grp, p.order, p.prefix, args, p.header, (int)p.Tq, p.H,
                                          p.B * p.grp.G, p.scale * log2e, p.scale);
  MOGA_CUDA_OK(cudaGetLastError());
  return MOGA_OK;
}

}  // namespace

// Sorted-order gradients dQp, dKp, dVp from the sorted-order saved tensors; ws holds the status
// header and the schedule scratch (WsLayout); dOp / delta are filled first by the prep kernel.
moga_status launch_attn_backward(const moga_shape& s, const WsLayout& L, const void* Qp, const void* Kp,
                                 const void* Vp, const void* Op, const float* lse, const float* gate,
                                 const int32_t* perm, const int32_t* inv, const int32_t* offsets, const void* dO,
                                 void* dOp, float* delta, void* dQp, void* dKp, void* dVp, float* dgate, char* ws,
                                 cudaStream_t st) {
  const long long T = (long long)s.N * s.k;
  if (T == 0) return MOGA_OK;
  const Strides q = qkv_strides(s);
  dim3 pgrid((unsigned)((T + 15) / 16), s.B);
  bwd_prep_kernel<<<pgrid, 256, 0, st>>>(static_cast<const uint4*>(dO), static_cast<const uint4*>(Op), gate, perm, inv,
                                         static_cast<uint4*>(dOp), delta, dgate, s.N, s.k, s.H, q.b / 8, q.h / 8,
                                         q.n / 8);
  MOGA_CUDA_OK(cudaGetLastError());
  int32_t* order = reinterpret_cast<int32_t*>(ws + L.sched);
  const Scatter none{nullptr, nullptr, 0, 0, 0, 0, 0, nullptr, nullptr};
  const Problem p{s.B, s.H, T, T, s.scale, nullptr, nullptr, nullptr, nullptr, nullptr,
                  Groups{offsets, offsets, s.M + 1, s.M}, order, order + (size_t)s.B * s.M, nullptr,
                  reinterpret_cast<uint32_t*>(ws + L.header), none, kEpiDefault};
  attn_schedule_kernel<<<1, 1024, 0, st>>>(p.grp, p.order, p.prefix, p.B, p.H, kTile);
  MOGA_CUDA_OK(cudaGetLastError());
  moga_status rc = launch_bwd<kModeQ>(p, Qp, dOp, Kp, Vp,
                                      BwdArgs{lse, delta, static_cast<__nv_bfloat16*>(dQp), nullptr}, st);
  if (rc != MOGA_OK) return rc;
  return launch_bwd<kModeKV>(p, Kp, Vp, Qp, dOp,
                             BwdArgs{lse, delta, static_cast<__nv_bfloat16*>(dVp), static_cast<__nv_bfloat16*>(dKp)}, st);
}

}  // namespace moga
