// bf16 per-group attention (Eq. 1 inside each group, Alg. 1 line 3) on tcgen05 tensor cores.
//
// One persistent CTA per SM walks a cost-ordered list of work items.  An item is
// (batch, head, group, block of 256 query rows): two 128-row Q tiles (A and B) that
// share every K/V tile of the group, so the tensor pipe works on one tile while the
// other tile's softmax runs.
//
//   warp 0      TMA producer: Q tiles and a ring of K / V tiles, 128B-swizzled,
//               each signalled through an mbarrier (no multicast).
//   warp 1      MMA issuer (one lane): S = Q K^T into TMEM, O += P V with P read
//               from TMEM; owns the TMEM allocation.
//   warps 4-7   softmax of tile A, one thread per query row; warps 8-11 tile B.
//               Online softmax in the log2 domain against a reference maximum taken
//               from the row's first tile; it is raised, and O rescaled in TMEM by
//               the same warps, only when a later tile's row sum exceeds 2^40.
//               They also run the epilogue: O / l -> bf16 -> a 2 KB staging buffer
//               private to the warp -> 64-byte row segments, row-predicated stores.
//               (The Q tiles are released by the MMA warp right after their last
//               use, so the next item's Q loads overlap this item's tail.)
//
// TMEM (512 columns): S_A [0,128) S_B [128,256) O_A [256,256+D) O_B [384,384+D);
// P (bf16, two per column) overwrites the first 64 columns of its S tile.
// Every mbarrier wait is bounded: on expiry the CTA records MOGA_ERR_TIMEOUT in the
// workspace status word, all roles leave their loops, and TMEM is released.
#include "attn_common.cuh"

namespace moga {
namespace attn {

// ----------------------------------------------------------------------------- schedule
__global__ void attn_schedule_kernel(const Groups grp, int32_t* __restrict__ order, int32_t* __restrict__ prefix,
                                     int B, int H, int qblock) {
  const int G = grp.G;
  for (int idx = threadIdx.x; idx < B * G; idx += blockDim.x) {
    const int b = idx / G, g = idx % G;
    int r = g;
    if (G <= kRankLimit) {
      const int32_t* qo = grp.q_off + (size_t)b * grp.stride;
      const int32_t* ko = grp.kv_off + (size_t)b * grp.stride;
      const long long n = (long long)(qo[g + 1] - qo[g]) * (ko[g + 1] - ko[g]);
      r = 0;
      for (int o = 0; o < G; ++o) {
        const long long no = (long long)(qo[o + 1] - qo[o]) * (ko[o + 1] - ko[o]);
        r += (no > n) || (no == n && o < g);
      }
    }
    order[b * G + r] = g;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int acc = 0;
    for (int idx = 0; idx < B * G; ++idx) {
      const int b = idx / G;
      const int g = order[idx];
      const int nq = grp.q_off[(size_t)b * grp.stride + g + 1] - grp.q_off[(size_t)b * grp.stride + g];
      const int nk = grp.kv_off[(size_t)b * grp.stride + g + 1] - grp.kv_off[(size_t)b * grp.stride + g];
      prefix[idx] = acc;
      if (nk > 0) acc += ((nq + qblock - 1) / qblock) * H;
    }
    prefix[B * G] = acc;
  }
}

}  // namespace attn

namespace {

using namespace attn;

constexpr int kThreads = 384;
constexpr int kTileM = 128;       // query rows per tile
constexpr int kTileN = 128;       // keys per K/V tile
constexpr int kQBlock = 2 * kTileM;
constexpr float kRowSumLimit = 1.0995116e12f;      // 2^40: a tile's row sum beyond this forces a new maximum

using namespace sm100;

// ----------------------------------------------------------------------------- the kernel
template <int D>
struct Cfg {
  static constexpr int NS = (D == 128) ? 2 : 4;           // K and V ring depth
  static constexpr int kBoxes = D / 64;                   // 64-column TMA boxes per tile
  static constexpr int kBoxBytes = kTileM * 128;          // 128 rows x 128 bytes
  static constexpr int kTileBytes = kBoxes * kBoxBytes;
  static constexpr int kSmemQ = 0;
  static constexpr int kSmemK = 2 * kTileBytes;
  static constexpr int kSmemV = kSmemK + NS * kTileBytes;
  static constexpr int kSmemStage = kSmemV + NS * kTileBytes;   // 8 softmax warps x 2 KB output staging
  static constexpr int kSmemBar = kSmemStage + 8 * 2048;
  static constexpr int kNumBars = 2 + 2 + 4 * NS + 2 + 2 + 2 + 2;
  static constexpr int kSmemTotal = kSmemBar + 8 * kNumBars + 16;
  static constexpr int kDynSmem = kSmemTotal + 1024;      // slack for 1024-byte alignment
};

// Redo: the work items are those listed in redo[4 ...] (redo[0] of them) instead of all items.
template <int D, bool Redo, int Epi>
__global__ void __launch_bounds__(kThreads, 1)
attn_bf16_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                 const __grid_constant__ CUtensorMap mapV, const Groups grp,
                 const int32_t* __restrict__ order, const int32_t* __restrict__ prefix,
                 __nv_bfloat16* __restrict__ Op, float* __restrict__ lse, uint32_t* header, int T, int H,
                 int BG, float scale_log2, float scale, const Scatter sc, const int32_t* __restrict__ redo) {
  using C = Cfg<D>;
  constexpr int NS = C::NS;
  extern __shared__ unsigned char smem_raw[];
  // 128B-swizzled tiles need 1024-byte aligned bases
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sQ = base + C::kSmemQ, sK = base + C::kSmemK, sV = base + C::kSmemV;
  const uint32_t bars = base + C::kSmemBar;
  constexpr int Q_FULL = 0, Q_EMPTY = 2, K_FULL = 4, K_EMPTY = 4 + NS, V_FULL = 4 + 2 * NS,
                V_EMPTY = 4 + 3 * NS, S_FULL = 4 + 4 * NS, P_FULL = S_FULL + 2, O_FULL = S_FULL + 4,
                O_EMPTY = S_FULL + 6;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + C::kSmemBar + 8 * C::kNumBars);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_items = Redo ? redo[0] : prefix[BG];

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(Q_FULL + i), 1);
      mbar_init(bar(Q_EMPTY + i), 1);
      mbar_init(bar(S_FULL + i), 1);
      mbar_init(bar(P_FULL + i), kTileM);
      mbar_init(bar(O_FULL + i), 1);
      mbar_init(bar(O_EMPTY + i), kTileM);
    }
    for (int i = 0; i < NS; ++i) {
      mbar_init(bar(K_FULL + i), 1);
      mbar_init(bar(K_EMPTY + i), 1);
      mbar_init(bar(V_FULL + i), 1);
      mbar_init(bar(V_EMPTY + i), 1);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32((const void*)tmem_slot)),
                 "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  // Bounded wait.  Returns false when the CTA is aborting (this wait or another one expired).
  auto wait = [&](int idx, uint32_t parity, uint32_t where) -> bool {
    const WaitResult res = mbar_wait_bounded(bar(idx), parity, abort_flag, kDefaultWaitLimitNs);
    if (res == kWaitExpired)
      report_status(header, MOGA_ERR_TIMEOUT, (where << 24) | ((uint32_t)blockIdx.x << 8) | (uint32_t)idx);
    return res == kWaitDone;
  };

  // The producer's waits are long (a ring slot frees once per K/V tile): it parks between polls
  // so that it does not take issue slots from the softmax warps of its sub-partition.
  auto wait_parked = [&](int idx, uint32_t parity, uint32_t where) -> bool {
    const WaitResult res = mbar_wait_bounded_parked(bar(idx), parity, abort_flag, kDefaultWaitLimitNs);
    if (res == kWaitExpired)
      report_status(header, MOGA_ERR_TIMEOUT, (where << 24) | ((uint32_t)blockIdx.x << 8) | (uint32_t)idx);
    return res == kWaitDone;
  };

  // Registers move from the producer / MMA warpgroup (warps 0-3) to the softmax warpgroups:
  // 128 * 80 + 256 * 208 <= 384 * 168.
  // (each setmaxnreg sits at the top of the branch it governs, so the compiler can give
  //  the code it dominates that many registers)
  if (warp < 4) {
    static_assert(128 * 80 + 256 * 208 <= kThreads * 168, "the softmax warps' setmaxnreg.inc would wait forever");
    reg_dec<80>();
  if (warp == 0) {
    // ===================================================================== TMA producer
    if (lane == 0) {
      uint32_t nq[2] = {0, 0}, nkv = 0;
      bool ok = true;
      for (int w = blockIdx.x; ok && w < total_items; w += gridDim.x) {
        const Item it = decode_item<kQBlock>(Redo ? redo[4 + w] : w, grp, order, prefix, BG, H);
        const int ntiles = (it.khi - it.klo + kTileN - 1) / kTileN;
        const bool validB = it.row0 + kTileM < it.qhi;
        for (int x = 0; x < (validB ? 2 : 1) && ok; ++x) {
          ok = wait_parked(Q_EMPTY + x, (nq[x] & 1u) ^ 1u, 1);
          if (!ok) break;
          mbar_expect_tx(bar(Q_FULL + x), C::kTileBytes);
#pragma unroll
          for (int bx = 0; bx < C::kBoxes; ++bx)
            tma_load_3d(sQ + x * C::kTileBytes + bx * C::kBoxBytes, &mapQ, bar(Q_FULL + x), bx * 64,
                        it.row0 + x * kTileM, it.bh);
          ++nq[x];
        }
        for (int j = 0; j < ntiles && ok; ++j) {
          const int s = nkv % NS;
          const uint32_t ph = ((nkv / NS) & 1u) ^ 1u;
          ok = wait_parked(K_EMPTY + s, ph, 2);
          if (!ok) break;
          mbar_expect_tx(bar(K_FULL + s), C::kTileBytes);
#pragma unroll
          for (int bx = 0; bx < C::kBoxes; ++bx)
            tma_load_3d(sK + s * C::kTileBytes + bx * C::kBoxBytes, &mapK, bar(K_FULL + s), bx * 64,
                        it.klo + j * kTileN, it.bh);
          ok = wait_parked(V_EMPTY + s, ph, 3);
          if (!ok) break;
          mbar_expect_tx(bar(V_FULL + s), C::kTileBytes);
#pragma unroll
          for (int bx = 0; bx < C::kBoxes; ++bx)
            tma_load_3d(sV + s * C::kTileBytes + bx * C::kBoxBytes, &mapV, bar(V_FULL + s), bx * 64,
                        it.klo + j * kTileN, it.bh);
          ++nkv;
        }
      }
    }
  } else if (warp == 1) {
    // ===================================================================== MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = instr_desc(kTileM, kTileN, false);
      constexpr uint32_t idesc_pv = instr_desc(kTileM, D, true);
      uint32_t nq[2] = {0, 0}, ns[2] = {0, 0}, np[2] = {0, 0}, no[2] = {0, 0}, nk = 0, nv = 0;
      bool ok = true;
      // S_x = Q_x K^T for the K tile in ring slot s
      constexpr uint32_t hi = desc_hi(1024);   // 8-row groups are 1024 bytes apart in every tile
      auto issue_qk = [&](int x, int s) {
        const uint32_t qa = desc_lo(sQ + x * C::kTileBytes, 16), kb = desc_lo(sK + s * C::kTileBytes, 16);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t o = ((kk / 4) * C::kBoxBytes + (kk % 4) * 32) >> 4;
          mma_ss(tmem + x * kTileN, qa + o, kb + o, hi, idesc_qk, kk > 0);
        }
      };
      // O_x (+)= P_x V for the V tile in ring slot s (V is MN-major: 64-column boxes kBoxBytes apart)
      auto issue_pv = [&](int x, int s, bool accumulate) {
        const uint32_t vb = desc_lo(sV + s * C::kTileBytes, C::kBoxBytes);
#pragma unroll
        for (int kk = 0; kk < kTileN / 16; ++kk)
          mma_ts(tmem + 256 + x * 128, tmem + x * kTileN + kk * 8, vb + ((kk * 2048) >> 4), hi, idesc_pv,
                 (accumulate || kk > 0) ? 1u : 0u);
      };
      for (int w = blockIdx.x; ok && w < total_items; w += gridDim.x) {
        const Item it = decode_item<kQBlock>(Redo ? redo[4 + w] : w, grp, order, prefix, BG, H);
        const int ntiles = (it.khi - it.klo + kTileN - 1) / kTileN;
        const int nx = (it.row0 + kTileM < it.qhi) ? 2 : 1;
        // first S tiles
        for (int x = 0; x < nx && ok; ++x) {
          ok = wait(Q_FULL + x, nq[x] & 1u, 4);
          ++nq[x];
        }
        if (!ok) break;
        ok = wait(K_FULL + nk % NS, (nk / NS) & 1u, 5);
        if (!ok) break;
        tc_fence_after();
        for (int x = 0; x < nx; ++x) {
          issue_qk(x, nk % NS);
          tc_commit(bar(S_FULL + x));
          if (ntiles == 1) tc_commit(bar(Q_EMPTY + x));   // the item's only use of this Q tile
        }
        tc_commit(bar(K_EMPTY + nk % NS));
        ++nk;
        for (int j = 0; j < ntiles && ok; ++j) {
          ok = wait(V_FULL + nv % NS, (nv / NS) & 1u, 6);
          if (!ok) break;
          const bool more = j + 1 < ntiles;
          if (more) {
            ok = wait(K_FULL + nk % NS, (nk / NS) & 1u, 7);
            if (!ok) break;
          }
          // ragged last tile, landed: warp 2 clears its foreign V rows while the softmax runs
          for (int x = 0; x < nx && ok; ++x) {
            ok = wait(P_FULL + x, np[x] & 1u, 8);
            if (!ok) break;
            ++np[x];
            if (j == 0) {
              ok = wait(O_EMPTY + x, (no[x] & 1u) ^ 1u, 9);
              if (!ok) break;
              ++no[x];
            }
            tc_fence_after();
            issue_pv(x, nv % NS, j > 0);
            if (more) {
              issue_qk(x, nk % NS);
              tc_commit(bar(S_FULL + x));
              if (j + 2 == ntiles) tc_commit(bar(Q_EMPTY + x));   // last use of this Q tile: free it early
            } else {
              tc_commit(bar(O_FULL + x));
            }
          }
          if (!ok) break;
          tc_commit(bar(V_EMPTY + nv % NS));
          ++nv;
          if (more) {
            tc_commit(bar(K_EMPTY + nk % NS));
            ++nk;
          }
        }
      }
      (void)ns;
    }
  }
  } else {
    // ===================================================================== softmax + epilogue
    reg_inc<208>();
    const int x = (warp - 4) >> 2;                 // 0: tile A, 1: tile B
    const int q = warp & 3;                        // TMEM lane quarter of this warp
    const int r = q * 32 + lane;                   // row inside the tile
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    const uint32_t tS = tmem + lane_off + x * kTileN;
    const uint32_t tO = tmem + lane_off + 256 + x * 128;
    uint32_t n_s = 0, n_o = 0;
    bool ok = true;
    for (int w = blockIdx.x; ok && w < total_items; w += gridDim.x) {
      const Item it = decode_item<kQBlock>(Redo ? redo[4 + w] : w, grp, order, prefix, BG, H);
      if (x == 1 && !(it.row0 + kTileM < it.qhi)) continue;
      const int ntiles = (it.khi - it.klo + kTileN - 1) / kTileN;
      const int tile_row0 = it.row0 + x * kTileM;
      float m = -INFINITY, l = 0.f;
      for (int j = 0; j < ntiles && ok; ++j) {
        ok = __all_sync(0xffffffffu, wait(S_FULL + x, n_s & 1u, 10));   // warp-uniform: TMEM loads are warp-collective
        if (!ok) break;
        ++n_s;
        tc_fence_after();
        // Tile 0 fixes the row's reference maximum m.  Later tiles exponentiate against the
        // same m without looking for their own maximum: any reference gives the same quotient
        // O / l as long as nothing overflows, and bf16 / fp32 keep their relative precision at
        // any magnitude.  Only when a row sum shows scores far above m (2^40, inf or nan) is the
        // tile redone with its exact maximum, m raised, and O and l rescaled.
        uint32_t preg[64];
        float alpha = 1.f, lsum;
        bool exact = (j == 0), rescale = false;
        const int ncols = it.khi - it.klo - j * kTileN;     // valid keys in this tile (may exceed 128)
        while (true) {
          uint32_t sreg[128];
#pragma unroll
          for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&sreg[c * 32]));
          tmem_wait_ld();
          if (ncols < kTileN) {
            // Columns past the group's last key hold scores against the next group's rows (any
            // value, NaN included): they become -inf before anything reads them, so they never
            // win the maximum and their weight is 2^(-inf) = 0 exactly.  (scale_log2 > 0 always:
            // the launcher replaces a zero scale by the smallest normal float, see there.)
#pragma unroll
            for (int c = 0; c < 128; ++c)
              if (c >= ncols) sreg[c] = 0xff800000u;        // -inf
          }
          if (exact) {
            float mx[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) mx[c] = __uint_as_float(sreg[c]);
#pragma unroll
            for (int c = 8; c < 128; ++c) mx[c & 7] = fmaxf(mx[c & 7], __uint_as_float(sreg[c]));
            const float mt = fmaxf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])),
                                   fmaxf(fmaxf(mx[4], mx[5]), fmaxf(mx[6], mx[7])));
            const float m_new = fmaxf(m, mt);
            alpha = j == 0 ? 0.f : ex2((m - m_new) * scale_log2);
            m = m_new;
            rescale = j > 0;
          }
          const float neg_m = -m * scale_log2;
          const float2 sc2 = make_float2(scale_log2, scale_log2), nm2 = make_float2(neg_m, neg_m);
          float2 ls[4] = {{0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}};
#pragma unroll
          for (int c = 0; c < 64; ++c) {
            const float2 x = __ffma2_rn(make_float2(__uint_as_float(sreg[2 * c]), __uint_as_float(sreg[2 * c + 1])),
                                        sc2, nm2);
            const float2 pe = make_float2(ex2(x.x), ex2(x.y));
            ls[c & 3] = __fadd2_rn(ls[c & 3], pe);
            __nv_bfloat162 pk = __floats2bfloat162_rn(pe.x, pe.y);
            preg[c] = *reinterpret_cast<uint32_t*>(&pk);
          }
          const float2 l01 = __fadd2_rn(__fadd2_rn(ls[0], ls[1]), __fadd2_rn(ls[2], ls[3]));
          lsum = l01.x + l01.y;
          if (exact || !__any_sync(0xffffffffu, !(lsum < kRowSumLimit))) break;
          exact = true;       // S is still intact in TMEM: load it again and take the maximum
        }
        l = l * alpha + lsum;
        tmem_st32(tS, *reinterpret_cast<uint32_t(*)[32]>(&preg[0]));
        tmem_st32(tS + 32, *reinterpret_cast<uint32_t(*)[32]>(&preg[32]));
        if (rescale && j > 0) {
          // the S tile arriving implies the previous P V has completed: O is stable
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t oreg[32];
            tmem_ld32(tO + c * 32, oreg);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) oreg[i] = __float_as_uint(__uint_as_float(oreg[i]) * alpha);
            tmem_st32(tO + c * 32, oreg);
          }
        }
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar(P_FULL + x));
      }
      if (!ok) break;
      // ---- epilogue: O / l -> bf16 -> per-warp staging -> global
      // mean of three branches: the rows of the other two branches this lane will need (4 rows x
      // 4 column chunks x 16 bytes of each) are requested now, so they arrive while the item's
      // last P V runs; the softmax registers are free at this point
      uint4 pre_a[D / 32][4], pre_b[D / 32][4];
      if (Epi == kEpiMean3) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int grow = tile_row0 + q * 32 + i * 8 + (lane >> 2);
          const long long at = ((long long)it.bh * T + (grow < it.qhi ? grow : it.qhi - 1)) * D + (lane & 3) * 8;
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            pre_a[c][i] = __ldg(reinterpret_cast<const uint4*>(sc.mean_a + at + c * 32));
            pre_b[c][i] = __ldg(reinterpret_cast<const uint4*>(sc.mean_b + at + c * 32));
          }
        }
      }
      ok = __all_sync(0xffffffffu, wait(O_FULL + x, n_o & 1u, 11));
      if (!ok) break;
      ++n_o;
      tc_fence_after();
      float inv_l = 1.f / l;
      const bool live = tile_row0 + r < it.qhi;
      const int bb = it.bh / H, hh = it.bh % H;
      if (Epi == kEpiDefault && sc.perm != nullptr && live)
        inv_l *= sc.gate[(size_t)bb * sc.N + sc.perm[(size_t)bb * T + tile_row0 + r]];
      if (Epi == kEpiAdd && live) inv_l *= sc.gate[(size_t)bb * T + sc.perm[(size_t)bb * T + tile_row0 + r]];
      // Each warp stages 32 rows x 32 columns (2 KB) at a time in its own buffer and writes them
      // out itself: lane L stores piece L % 4 of rows i * 8 + L / 4, i = 0..3 (64-byte row segments).
      unsigned char* wst = smem + C::kSmemStage + (x * 4 + q) * 2048;
      __nv_bfloat16* obase[4];
      bool orow_live[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int grow = tile_row0 + q * 32 + i * 8 + (lane >> 2);
        orow_live[i] = grow < it.qhi;
        if (Epi == kEpiAdd) {
          const int tok = orow_live[i] ? sc.perm[(size_t)bb * T + grow] / sc.k : 0;
          obase[i] = Op + bb * sc.sb + hh * sc.sh + (long long)tok * sc.sn;
        } else if (Epi == kEpiList) {
          const int tok = orow_live[i] ? sc.perm[grow] : 0;
          obase[i] = Op + bb * sc.sb + hh * sc.sh + (long long)tok * sc.sn;
        } else if (Epi == kEpiDefault && sc.perm != nullptr) {
          const int tok = orow_live[i] ? sc.perm[(size_t)bb * T + grow] : 0;
          obase[i] = Op + bb * sc.sb + hh * sc.sh + (long long)tok * sc.sn;
        } else {
          obase[i] = Op + ((size_t)it.bh * T + grow) * D;
        }
      }
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t oreg[32];
        tmem_ld32(tO + c * 32, oreg);
        tmem_wait_ld();
        if (c == D / 32 - 1) {
          tc_fence_before();
          mbar_arrive(bar(O_EMPTY + x));    // TMEM O (and S) of this tile may be overwritten
        }
#pragma unroll
        for (int v = 0; v < 4; ++v) {      // four 16-byte chunks (8 bf16 each) per 32 columns
          uint4 pk;
          uint32_t* pw = reinterpret_cast<uint32_t*>(&pk);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 t = __floats2bfloat162_rn(__uint_as_float(oreg[v * 8 + 2 * i]) * inv_l,
                                                     __uint_as_float(oreg[v * 8 + 2 * i + 1]) * inv_l);
            pw[i] = *reinterpret_cast<uint32_t*>(&t);
          }
          *reinterpret_cast<uint4*>(wst + lane * 64 + ((v ^ ((lane >> 1) & 3)) * 16)) = pk;
        }
        __syncwarp();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int row = i * 8 + (lane >> 2), piece = lane & 3;
          uint4 val = *reinterpret_cast<const uint4*>(wst + row * 64 + ((piece ^ ((row >> 1) & 3)) * 16));
          if (Epi == kEpiMean3) {
            // the other two branches' rows live at the same offset of their own tensors
            const uint4 a = pre_a[c][i], b = pre_b[c][i];
            const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
            uint32_t* vw = reinterpret_cast<uint32_t*>(&val);
            const float third = 1.f / 3.f;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float lo = (__uint_as_float(aw[e] << 16) + __uint_as_float(bw[e] << 16)) + __uint_as_float(vw[e] << 16);
              const float hi = (__uint_as_float(aw[e] & 0xffff0000u) + __uint_as_float(bw[e] & 0xffff0000u)) +
                               __uint_as_float(vw[e] & 0xffff0000u);
              __nv_bfloat162 t = __floats2bfloat162_rn(lo * third, hi * third);
              vw[e] = *reinterpret_cast<uint32_t*>(&t);
            }
          }
          if (Epi == kEpiAdd) {
            if (orow_live[i])
              asm volatile("red.relaxed.gpu.global.add.noftz.v4.bf16x2 [%0], {%1, %2, %3, %4};" ::"l"(
                               obase[i] + c * 32 + piece * 8),
                           "r"(val.x), "r"(val.y), "r"(val.z), "r"(val.w)
                           : "memory");
          } else if (orow_live[i]) {
            *reinterpret_cast<uint4*>(obase[i] + c * 32 + piece * 8) = val;
          }
        }
        __syncwarp();
      }
      if (lse != nullptr && live) lse[(size_t)it.bh * T + tile_row0 + r] = m * scale + __logf(l);
    }
  }

  __syncwarp();
  // ----------------------------------------------------------------------------- teardown
  if (*abort_flag) {
    // give copies and MMAs already in flight time to land before the TMEM is released
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

// ----------------------------------------------------------------------------- host side
// Tensor maps, grid and launch of the one-CTA kernel.  Redo: only the items the CTA-pair kernel
// listed in p.redo, whose schedule (the same 256-row items) is already in order / prefix.
template <int D, bool Redo, int Epi>
moga_status launch_one(const Problem& p, cudaStream_t st) {
  CUtensorMap mq, mk, mv;
  const long long BH = (long long)p.B * p.H;
  if (!make_map(&mq, p.Q, D, p.Tq, BH, kTileM) || !make_map(&mk, p.K, D, p.Tkv, BH, kTileN) ||
      !make_map(&mv, p.V, D, p.Tkv, BH, kTileN))
    return MOGA_ERR_CUDA;
  if (!Redo) {
    attn_schedule_kernel<<<1, 1024, 0, st>>>(p.grp, p.order, p.prefix, p.B, p.H, kQBlock);
    MOGA_CUDA_OK(cudaGetLastError());
  }
  int num_sms = 0;
  if (!current_sm_count(&num_sms)) return MOGA_ERR_CUDA;
  auto kern = attn_bf16_kernel<D, Redo, Epi>;
  MOGA_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<D>::kDynSmem));
  const long long max_items = max_items_256(p);
  int grid = (int)(max_items < num_sms ? max_items : num_sms);
  if (Redo && grid > 16) grid = 16;      // the list is normally empty: a few CTAs walk it
  // The kernel works in the log2 domain with scale_log2 = scale * log2(e) and masks columns by
  // setting their score to -inf, which needs scale_log2 > 0 (-inf * 0 is NaN).  A zero scale
  // (uniform weights) is served by the smallest normal float instead: every weight
  // 2^(1.2e-38 * (s - m)) is then exactly 1.0f for all scores below 1e30 in magnitude.
  const float log2e = 1.4426950408889634f;
  const float scale_log2 = p.scale * log2e > 1.17549435e-38f ? p.scale * log2e : 1.17549435e-38f;
  kern<<<grid, kThreads, Cfg<D>::kDynSmem, st>>>(mq, mk, mv, p.grp, p.order, p.prefix,
                                                  static_cast<__nv_bfloat16*>(p.O), p.lse, p.header, (int)p.Tq,
                                                  p.H, p.B * p.grp.G, scale_log2, p.scale, p.sc, p.redo);
  MOGA_CUDA_OK(cudaGetLastError());
  return MOGA_OK;
}

// Which kernel serves a launch.  Default for d_head = 128 launches that have the redo scratch and
// store their rows (sorted order or the top-1 scatter): the kernel with two softmax threads per row
// (attn_bf16_duo.cu), followed by this file's kernel over the items it listed; measured on groups of
// ~17,500 rows, same box, alternating runs: 1,202 TFLOP/s against 1,157 for this file's kernel alone.
// Everything else (d_head = 64, static groups, the adding epilogue) runs this file's kernel.
// The CTA-pair kernel (935 TFLOP/s on the same case) halves the K/V bytes each SM stages and reads
// per flop, but issuing an M = 256, N = 128 instruction for two SMs keeps the issuing thread about as
// long as the instruction runs, so its waits are no longer hidden behind queued MMAs and the tensor
// pipe idles 55 % of the cycles.  It stays selectable (moga_set_attn_kernel).
int g_attn_kernel = MOGA_ATTN_AUTO;

moga_status launch_any(int D, const Problem& p, cudaStream_t st) {
  const bool listable = D == 128 && p.redo != nullptr && p.epi == kEpiDefault;
  if (listable && g_attn_kernel == MOGA_ATTN_PAIR) return launch_pair(p, st);
  if (listable && g_attn_kernel == MOGA_ATTN_AUTO) return launch_duo(p, st);
  return launch_single(D, p, st);
}

// Routed groups: offsets [B, M+1] serve queries and keys alike; scratch from the workspace layout.
Problem routed_problem(const moga_shape& s, const WsLayout& L, const void* Qp, const void* Kp, const void* Vp,
                       const int32_t* offsets, void* O, float* lse, char* ws, const Scatter& sc) {
  const long long T = (long long)s.N * s.k;
  int32_t* order = reinterpret_cast<int32_t*>(ws + L.sched);
  return Problem{s.B, s.H, T, T, s.scale, Qp, Kp, Vp, O, lse, Groups{offsets, offsets, s.M + 1, s.M},
                 order, order + (size_t)s.B * s.M, reinterpret_cast<int32_t*>(ws + L.redo),
                 reinterpret_cast<uint32_t*>(ws + L.header), sc, kEpiDefault};
}

}  // namespace

moga_status attn::launch_single(int D, const attn::Problem& p, cudaStream_t st) {
  if (p.epi == kEpiList) return D == 128 ? launch_one<128, false, kEpiList>(p, st) : MOGA_ERR_UNSUPPORTED;
  if (p.epi == kEpiMean3) return D == 128 ? launch_one<128, false, kEpiMean3>(p, st) : MOGA_ERR_UNSUPPORTED;
  if (p.epi == kEpiAdd) return D == 128 ? launch_one<128, false, kEpiAdd>(p, st) : launch_one<64, false, kEpiAdd>(p, st);
  return D == 128 ? launch_one<128, false, kEpiDefault>(p, st) : launch_one<64, false, kEpiDefault>(p, st);
}

moga_status attn::launch_single_redo(const attn::Problem& p, cudaStream_t st) { return launch_one<128, true, kEpiDefault>(p, st); }

void set_attn_kernel(int mode) { g_attn_kernel = mode; }

moga_status launch_attn_bf16(const moga_shape& s, const WsLayout& L, const void* Qp, const void* Kp,
                             const void* Vp, const int32_t* offsets, void* Op, float* lse, char* ws,
                             cudaStream_t st) {
  if ((long long)s.N * s.k == 0) return MOGA_OK;
  const Scatter none{nullptr, nullptr, 0, 0, 0, 0, 0, nullptr, nullptr};
  return launch_any(s.D, routed_problem(s, L, Qp, Kp, Vp, offsets, Op, lse, ws, none), st);
}

moga_status launch_attn_bf16_scatter(const moga_shape& s, const WsLayout& L, const void* Qp, const void* Kp,
                                     const void* Vp, const int32_t* offsets, const int32_t* perm,
                                     const float* gate, void* O, char* ws, cudaStream_t st) {
  if ((long long)s.N * s.k == 0) return MOGA_OK;
  const Strides q = qkv_strides(s);
  const Scatter sc{perm, gate, q.b, q.h, q.n, s.N, s.k, nullptr, nullptr};
  return launch_any(s.D, routed_problem(s, L, Qp, Kp, Vp, offsets, O, nullptr, ws, sc), st);
}

moga_status launch_attn_bf16_add(const moga_shape& s, const WsLayout& L, const void* Qp, const void* Kp,
                                 const void* Vp, const int32_t* offsets, const int32_t* asg, const float* gate,
                                 void* O, char* ws, cudaStream_t st) {
  if ((long long)s.N * s.k == 0) return MOGA_OK;
  const Strides q = qkv_strides(s);
  const Scatter sc{asg, gate, q.b, q.h, q.n, s.N, s.k, nullptr, nullptr};
  Problem p = routed_problem(s, L, Qp, Kp, Vp, offsets, O, nullptr, ws, sc);
  p.epi = kEpiAdd;
  return launch_any(s.D, p, st);
}

namespace {
// Off by default: measured on the two top-2 workloads it is no faster than the staged path
// (74.6 vs 74.3 ms and 548.8 vs 548.6 ms per forward), which sums in fp32 with one rounding.
int g_fused_topk = 0;
}
void set_fused_topk(int on) { g_fused_topk = on; }
bool fused_topk() { return g_fused_topk != 0; }

moga_status launch_attn_bf16_static(const moga_shape& s, int G, long long Tq, long long Tkv, const void* Qs,
                                    const void* Ks, const void* Vs, const int32_t* q_offsets,
                                    const int32_t* kv_offsets, void* Os, float* lse, uint32_t* header, char* sched,
                                    const StaticEpilogue& epi, cudaStream_t st) {
  if (Tq == 0 || G == 0) return MOGA_OK;
  Scatter sc{nullptr, nullptr, 0, 0, 0, 0, 0, nullptr, nullptr};
  int mode = attn::kEpiDefault;
  if (epi.token_list != nullptr) {          // rows go to token order: Os is [B, H, N, D]
    mode = attn::kEpiList;
    sc.perm = epi.token_list;
    sc.sb = (long long)s.H * s.N * s.D;
    sc.sh = (long long)s.N * s.D;
    sc.sn = s.D;
    sc.N = s.N;
  } else if (epi.mean_a != nullptr) {       // mean with two token-order tensors: rows stay in place
    mode = attn::kEpiMean3;
    sc.mean_a = static_cast<const __nv_bfloat16*>(epi.mean_a);
    sc.mean_b = static_cast<const __nv_bfloat16*>(epi.mean_b);
  }
  int32_t* order = reinterpret_cast<int32_t*>(sched);
  const Problem p{s.B, s.H, Tq, Tkv, s.scale, Qs, Ks, Vs, Os, lse, Groups{q_offsets, kv_offsets, 0, G},
                  order, order + (size_t)s.B * G, nullptr, header, sc, mode};
  return launch_any(s.D, p, st);
}

}  // namespace moga
