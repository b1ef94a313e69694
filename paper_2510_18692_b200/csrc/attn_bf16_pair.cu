// bf16 per-group attention (Eq. 1 inside each group, Alg. 1 line 3) on tcgen05 tensor cores,
// one work item per PAIR of CTAs (a cluster of two, on the two SMs of one TPC), d_head = 128.
//
// A work item is (batch, head, group, block of 512 query rows): two tiles A and B of 256 rows,
// each split over the pair (the CTA of cluster rank r owns rows [r*128, r*128 + 128) of a
// tile).  Every tcgen05.mma covers both CTAs (cta_group::2, M = 256) and is issued by the CTA
// of rank 0; each CTA stages only half of the B operand of every instruction:
//   S = Q K^T : the CTA of rank r holds keys [r*64, r*64 + 64) of the 128-key tile;
//   O += P V  : the CTA of rank r holds value columns [r*64, r*64 + 64) of all 128 keys.
// So a K/V tile costs each SM 32 KB of L2 -> shared-memory traffic and of operand reads per
// 512 query rows, against 64 KB per 256 rows in the one-CTA kernel.  Each CTA loads its halves
// with its own plain TMA copies (no multicast); the copies of both CTAs count into the mbarrier
// of rank 0, which is the one the MMA thread waits on.
//
// Roles per CTA (same warps as the one-CTA kernel):
//   warp 0      TMA producer for this CTA's halves (one lane).
//   warp 1      rank 0: MMA issuer (one lane); both ranks: tensor-memory allocation.
//   warps 4-7   softmax + epilogue of this CTA's 128 rows of tile A; warps 8-11 of tile B.
// Hand-offs: tcgen05.commit arrives on the barrier at the same offset in both CTAs (S ready,
// O ready, ring slot free); the softmax warps of both CTAs arrive, one lane per warp, on the
// P-ready / O-free barriers of rank 0.  TMEM per CTA: S_A [0,128) S_B [128,256) O_A [256,384)
// O_B [384,512); P (bf16) overwrites the first 64 columns of its S tile.
// Every mbarrier wait is bounded; a CTA whose wait runs out raises the abort flag of both CTAs,
// records MOGA_ERR_TIMEOUT, and both leave through the common exit.
#include "attn_common.cuh"

namespace moga {
namespace {

using namespace attn;
using namespace sm100;

constexpr int kThreads = 384;
constexpr int kD = 128;
constexpr int kRows = 128;            // query rows of a tile held by one CTA
constexpr int kTileN = 128;           // keys per K/V tile
constexpr int kPairTile = 2 * kRows;  // query rows of a tile over the pair
constexpr int kQBlock = 2 * kPairTile;
constexpr float kRowSumLimit = 1.0995116e12f;   // 2^40

constexpr int NS = 4;                            // K and V ring depth
constexpr int kQBoxBytes = kRows * 128;          // 128 rows x 64 columns
constexpr int kQTileBytes = 2 * kQBoxBytes;      // 32 KB
constexpr int kKBoxBytes = 64 * 128;             // 64 keys x 64 columns
constexpr int kKHalfBytes = 2 * kKBoxBytes;      // 16 KB: this CTA's 64 keys x 128 columns
constexpr int kVHalfBytes = kTileN * 128;        // 16 KB: 128 keys x this CTA's 64 columns
constexpr int kSmemQ = 0;
constexpr int kSmemK = 2 * kQTileBytes;
constexpr int kSmemV = kSmemK + NS * kKHalfBytes;
constexpr int kSmemStage = kSmemV + NS * kVHalfBytes;   // 8 softmax warps x 2 KB output staging
constexpr int kSmemBar = kSmemStage + 8 * 2048;
constexpr int kNumBars = 2 + 2 + 4 * NS + 2 + 2 + 2 + 2;
constexpr int kSmemTotal = kSmemBar + 8 * kNumBars + 16;
constexpr int kDynSmem = kSmemTotal + 1024;      // slack for 1024-byte alignment
static_assert(kDynSmem <= 227 * 1024, "shared memory");

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
attn_bf16_pair_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                      const __grid_constant__ CUtensorMap mapV, const Groups grp,
                      const int32_t* __restrict__ order, const int32_t* __restrict__ prefix,
                      __nv_bfloat16* __restrict__ Op, float* __restrict__ lse, uint32_t* header, int T, int H,
                      int BG, float scale_log2, float scale, const Scatter sc) {
  extern __shared__ unsigned char smem_raw[];
  // 128B-swizzled tiles need 1024-byte aligned bases (the offset is the same in both CTAs)
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sQ = base + kSmemQ, sK = base + kSmemK, sV = base + kSmemV;
  const uint32_t bars = base + kSmemBar;
  constexpr int Q_FULL = 0, Q_EMPTY = 2, K_FULL = 4, K_EMPTY = 4 + NS, V_FULL = 4 + 2 * NS,
                V_EMPTY = 4 + 3 * NS, S_FULL = 4 + 4 * NS, P_FULL = S_FULL + 2, O_FULL = S_FULL + 4,
                O_EMPTY = S_FULL + 6;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + kSmemBar + 8 * kNumBars);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();       // 0: issues the MMAs and owns the FULL / P / O-free barriers
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const int total_items = prefix[BG];

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(Q_FULL + i), 1);      // rank 0's arrive.expect_tx; bytes of both CTAs
      mbar_init(bar(Q_EMPTY + i), 1);
      mbar_init(bar(S_FULL + i), 1);
      mbar_init(bar(P_FULL + i), 8);      // four softmax warps of each CTA
      mbar_init(bar(O_FULL + i), 1);
      mbar_init(bar(O_EMPTY + i), 8);
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
  if (warp == 1) tmem_alloc_pair(smem_u32((const void*)tmem_slot), 512u);   // the same warp in both CTAs
  tc_fence_before();
  __syncthreads();
  // the partner's barriers and abort flag must exist before anything of this CTA reaches them
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t peer_abort = map_to_rank(smem_u32((const void*)abort_flag), rank ^ 1u);

  // Bounded wait.  Returns false when the pair is aborting (a wait of either CTA ran out).
  auto expired = [&](uint32_t where, int idx) {
    st_cluster_u32(peer_abort, 1u);
    report_status(header, MOGA_ERR_TIMEOUT, (where << 24) | (2u << 20) | ((uint32_t)(blockIdx.x & 0xfff) << 8) | (uint32_t)idx);
  };
  auto wait = [&](int idx, uint32_t parity, uint32_t where) -> bool {
    const WaitResult res = mbar_wait_bounded(bar(idx), parity, abort_flag, kDefaultWaitLimitNs);
    if (res == kWaitExpired) expired(where, idx);
    return res == kWaitDone;
  };
  auto wait_parked = [&](int idx, uint32_t parity, uint32_t where) -> bool {
    const WaitResult res = mbar_wait_bounded_parked(bar(idx), parity, abort_flag, kDefaultWaitLimitNs);
    if (res == kWaitExpired) expired(where, idx);
    return res == kWaitDone;
  };

  if (warp < 4) {
    static_assert(128 * 80 + 256 * 208 <= kThreads * 168, "the softmax warps' setmaxnreg.inc would wait forever");
    reg_dec<80>();
    if (warp == 0) {
      // ===================================================================== TMA producer
      if (lane == 0) {
        // completion bytes of both CTAs are counted by rank 0's barriers
        auto full = [&](int i) { return map_to_rank(bar(i), 0u); };
        uint32_t nq[2] = {0, 0}, nkv = 0;
        bool ok = true;
        for (int w = pair; ok && w < total_items; w += npairs) {
          const Item it = decode_item<kQBlock>(w, grp, order, prefix, BG, H);
          const int ntiles = (it.khi - it.klo + kTileN - 1) / kTileN;
          const bool validB = it.row0 + kPairTile < it.qhi;
          for (int x = 0; x < (validB ? 2 : 1) && ok; ++x) {
            ok = wait_parked(Q_EMPTY + x, (nq[x] & 1u) ^ 1u, 1);
            if (!ok) break;
            if (rank == 0) mbar_expect_tx(bar(Q_FULL + x), 2 * kQTileBytes);
#pragma unroll
            for (int bx = 0; bx < 2; ++bx)
              tma_load_3d_pair(sQ + x * kQTileBytes + bx * kQBoxBytes, &mapQ, full(Q_FULL + x), bx * 64,
                               it.row0 + x * kPairTile + (int)rank * kRows, it.bh);
            ++nq[x];
          }
          for (int j = 0; j < ntiles && ok; ++j) {
            const int s = nkv % NS;
            const uint32_t ph = ((nkv / NS) & 1u) ^ 1u;
            ok = wait_parked(K_EMPTY + s, ph, 2);
            if (!ok) break;
            if (rank == 0) mbar_expect_tx(bar(K_FULL + s), 2 * kKHalfBytes);
#pragma unroll
            for (int bx = 0; bx < 2; ++bx)      // this CTA's 64 keys, both 64-column halves
              tma_load_3d_pair(sK + s * kKHalfBytes + bx * kKBoxBytes, &mapK, full(K_FULL + s), bx * 64,
                               it.klo + j * kTileN + (int)rank * 64, it.bh);
            ok = wait_parked(V_EMPTY + s, ph, 3);
            if (!ok) break;
            if (rank == 0) mbar_expect_tx(bar(V_FULL + s), 2 * kVHalfBytes);
            // all 128 keys, this CTA's 64 value columns
            tma_load_3d_pair(sV + s * kVHalfBytes, &mapV, full(V_FULL + s), (int)rank * 64, it.klo + j * kTileN,
                             it.bh);
            ++nkv;
          }
        }
      }
    } else if (warp == 1 && rank == 0) {
      // ===================================================================== MMA issuer (rank 0 only)
      if (lane == 0) {
        constexpr uint32_t idesc_qk = instr_desc(kPairTile, kTileN, false);
        constexpr uint32_t idesc_pv = instr_desc(kPairTile, kD, true);
        uint32_t nq[2] = {0, 0}, np[2] = {0, 0}, no[2] = {0, 0}, nk = 0, nv = 0;
        bool ok = true;
        constexpr uint32_t hi = desc_hi(1024);   // 8-row groups are 1024 bytes apart in every tile
        // S_x = Q_x K^T for the K tile in ring slot s (the same offsets address both CTAs' halves)
        auto issue_qk = [&](int x, int s) {
          const uint32_t qa = desc_lo(sQ + x * kQTileBytes, 16), kb = desc_lo(sK + s * kKHalfBytes, 16);
#pragma unroll
          for (int kk = 0; kk < kD / 16; ++kk) {
            const uint32_t oq = ((kk / 4) * kQBoxBytes + (kk % 4) * 32) >> 4;
            const uint32_t ok_ = ((kk / 4) * kKBoxBytes + (kk % 4) * 32) >> 4;
            mma_ss_pair(tmem + x * kTileN, qa + oq, kb + ok_, hi, idesc_qk, kk > 0);
          }
        };
        // O_x (+)= P_x V for the V tile in ring slot s (V is MN-major: 16 keys are 2048 bytes apart)
        auto issue_pv = [&](int x, int s, bool accumulate) {
          const uint32_t vb = desc_lo(sV + s * kVHalfBytes, kVHalfBytes);
#pragma unroll
          for (int kk = 0; kk < kTileN / 16; ++kk)
            mma_ts_pair(tmem + 256 + x * 128, tmem + x * kTileN + kk * 8, vb + ((kk * 2048) >> 4), hi, idesc_pv,
                        (accumulate || kk > 0) ? 1u : 0u);
        };
        for (int w = pair; ok && w < total_items; w += npairs) {
          const Item it = decode_item<kQBlock>(w, grp, order, prefix, BG, H);
          const int ntiles = (it.khi - it.klo + kTileN - 1) / kTileN;
          const int nx = (it.row0 + kPairTile < it.qhi) ? 2 : 1;
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
            tc_commit_pair(bar(S_FULL + x));
            if (ntiles == 1) tc_commit_pair(bar(Q_EMPTY + x));   // the item's only use of this Q tile
          }
          tc_commit_pair(bar(K_EMPTY + nk % NS));
          ++nk;
          for (int j = 0; j < ntiles && ok; ++j) {
            ok = wait(V_FULL + nv % NS, (nv / NS) & 1u, 6);
            if (!ok) break;
            const bool more = j + 1 < ntiles;
            if (more) {
              ok = wait(K_FULL + nk % NS, (nk / NS) & 1u, 7);
              if (!ok) break;
            }
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
                tc_commit_pair(bar(S_FULL + x));
                if (j + 2 == ntiles) tc_commit_pair(bar(Q_EMPTY + x));   // last use of this Q tile: free it early
              } else {
                tc_commit_pair(bar(O_FULL + x));
              }
            }
            if (!ok) break;
            tc_commit_pair(bar(V_EMPTY + nv % NS));
            ++nv;
            if (more) {
              tc_commit_pair(bar(K_EMPTY + nk % NS));
              ++nk;
            }
          }
        }
      }
    }
  } else {
    // ===================================================================== softmax + epilogue
    reg_inc<208>();
    const int x = (warp - 4) >> 2;                 // 0: tile A, 1: tile B
    const int q = warp & 3;                        // TMEM lane quarter of this warp
    const int r = q * 32 + lane;                   // row inside this CTA's half of the tile
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    const uint32_t tS = tmem + lane_off + x * kTileN;
    const uint32_t tO = tmem + lane_off + 256 + x * 128;
    // the P-ready and O-free barriers the MMA thread waits on live in rank 0
    const uint32_t p_full = map_to_rank(bar(P_FULL + x), 0u), o_empty = map_to_rank(bar(O_EMPTY + x), 0u);
    uint32_t n_s = 0, n_o = 0;
    bool ok = true;
    for (int w = pair; ok && w < total_items; w += npairs) {
      const Item it = decode_item<kQBlock>(w, grp, order, prefix, BG, H);
      if (x == 1 && !(it.row0 + kPairTile < it.qhi)) continue;
      const int ntiles = (it.khi - it.klo + kTileN - 1) / kTileN;
      const int tile_row0 = it.row0 + x * kPairTile + (int)rank * kRows;
      float m = -INFINITY, l = 0.f;
      for (int j = 0; j < ntiles && ok; ++j) {
        ok = __all_sync(0xffffffffu, wait(S_FULL + x, n_s & 1u, 10));   // warp-uniform: TMEM loads are warp-collective
        if (!ok) break;
        ++n_s;
        tc_fence_after();
        // Tile 0 fixes the row's reference maximum m; later tiles exponentiate against the same m
        // (any reference gives the same quotient O / l while nothing overflows).  Only when a row
        // sum shows scores far above m (2^40, inf or nan) is the tile redone with its exact
        // maximum, m raised, and O and l rescaled.
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
            // columns past the group's last key: -inf before anything reads them (weight exactly 0;
            // scale_log2 > 0 always, see the launcher)
#pragma unroll
            for (int c = 0; c < 128; ++c)
              if (c >= ncols) sreg[c] = 0xff800000u;
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
            const float2 xs = __ffma2_rn(make_float2(__uint_as_float(sreg[2 * c]), __uint_as_float(sreg[2 * c + 1])),
                                         sc2, nm2);
            const float2 pe = make_float2(ex2(xs.x), ex2(xs.y));
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
          for (int c = 0; c < kD / 32; ++c) {
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
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(p_full);
      }
      if (!ok) break;
      // ---- epilogue: O / l -> bf16 -> per-warp staging -> global
      ok = __all_sync(0xffffffffu, wait(O_FULL + x, n_o & 1u, 11));
      if (!ok) break;
      ++n_o;
      tc_fence_after();
      float inv_l = 1.f / l;
      const bool live = tile_row0 + r < it.qhi;
      const int bb = it.bh / H, hh = it.bh % H;
      if (sc.perm != nullptr && live) inv_l *= sc.gate[(size_t)bb * sc.N + sc.perm[(size_t)bb * T + tile_row0 + r]];
      // Each warp stages 32 rows x 32 columns (2 KB) at a time in its own buffer and writes them
      // out itself: lane L stores piece L % 4 of rows i * 8 + L / 4, i = 0..3 (64-byte row segments).
      unsigned char* wst = smem + kSmemStage + (x * 4 + q) * 2048;
      __nv_bfloat16* obase[4];
      bool orow_live[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int grow = tile_row0 + q * 32 + i * 8 + (lane >> 2);
        orow_live[i] = grow < it.qhi;
        if (sc.perm != nullptr) {
          const int tok = orow_live[i] ? sc.perm[(size_t)bb * T + grow] : 0;
          obase[i] = Op + bb * sc.sb + hh * sc.sh + (long long)tok * sc.sn;
        } else {
          obase[i] = Op + ((size_t)it.bh * T + grow) * kD;
        }
      }
#pragma unroll
      for (int c = 0; c < kD / 32; ++c) {
        uint32_t oreg[32];
        tmem_ld32(tO + c * 32, oreg);
        tmem_wait_ld();
        if (c == kD / 32 - 1) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(o_empty);    // TMEM O (and S) of this tile may be overwritten
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
          const uint4 val = *reinterpret_cast<const uint4*>(wst + row * 64 + ((piece ^ ((row >> 1) & 3)) * 16));
          if (orow_live[i]) *reinterpret_cast<uint4*>(obase[i] + c * 32 + piece * 8) = val;
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
  // Neither CTA may leave (or free tensor memory) while its partner can still reach its shared
  // memory, barriers or tensor memory.  Every wait above is bounded, so both arrive here.
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem, 512u);
  }
}

}  // namespace

moga_status attn::launch_pair(const attn::Problem& p, cudaStream_t st) {
  CUtensorMap mq, mk, mv;
  const long long BH = (long long)p.B * p.H;
  if (!make_map(&mq, p.Q, kD, p.Tq, BH, kRows) || !make_map(&mk, p.K, kD, p.Tkv, BH, 64) ||
      !make_map(&mv, p.V, kD, p.Tkv, BH, kTileN))
    return MOGA_ERR_CUDA;
  attn_schedule_kernel<<<1, 1024, 0, st>>>(p.grp, p.order, p.prefix, p.B, p.H, kQBlock);
  MOGA_CUDA_OK(cudaGetLastError());
  int num_sms = 0;
  if (!current_sm_count(&num_sms)) return MOGA_ERR_CUDA;
  MOGA_CUDA_OK(cudaFuncSetAttribute(attn_bf16_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmem));
  const long long max_items = ((p.Tq + kQBlock - 1) / kQBlock + p.grp.G) * BH;
  long long pairs = num_sms / 2;
  if (max_items < pairs) pairs = max_items;
  if (pairs < 1) pairs = 1;
  // log2 domain; a zero scale is served by the smallest normal float (see the one-CTA launcher)
  const float log2e = 1.4426950408889634f;
  const float scale_log2 = p.scale * log2e > 1.17549435e-38f ? p.scale * log2e : 1.17549435e-38f;
  attn_bf16_pair_kernel<<<(unsigned)(2 * pairs), kThreads, kDynSmem, st>>>(
      mq, mk, mv, p.grp, p.order, p.prefix, static_cast<__nv_bfloat16*>(p.O), p.lse, p.header, (int)p.Tq, p.H,
      p.B * p.grp.G, scale_log2, p.scale, p.sc);
  MOGA_CUDA_OK(cudaGetLastError());
  return MOGA_OK;
}

}  // namespace moga
