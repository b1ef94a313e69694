// bf16 per-group attention (Eq. 1 inside each group, Alg. 1 line 3) on tcgen05 tensor cores,
// one work item per PAIR of CTAs (a cluster of two, on the two SMs of one TPC), d_head = 128.
//
// A work item is (batch, head, group, block of 256 query rows); the CTA of cluster rank r owns
// rows [r*128, r*128 + 128).  Every tcgen05.mma covers both CTAs (cta_group::2, M = 256) and is
// issued by the CTA of rank 0; each CTA stages only half of the B operand of every instruction:
//   S = Q K^T : the CTA of rank r holds keys [r*64, r*64 + 64) of the 128-key tile;
//   O += P V  : the CTA of rank r holds value columns [r*64, r*64 + 64) of all 128 keys.
// Each CTA loads its halves with its own plain TMA copies (no multicast); the copies of both
// CTAs count into the mbarrier of rank 0, which is the one the MMA thread waits on.
//
// The score tiles live in a ring of three TMEM buffers, so S = Q K^T runs up to three key tiles
// ahead of the softmax, and the two softmax warpgroups take the key tiles of an item in turn
// (tile t goes to warpgroup t mod 2, both work on the same 128 query rows, thread per row).  A
// warpgroup therefore never waits for the tensor pipe between its tiles, and the tensor pipe
// has a P tile waiting whenever the softmax keeps up: the hand-offs, which cross the pair, are
// off the critical path.  All tiles of an item are exponentiated against one reference maximum
// per row, taken from the item's first key tile and passed to the other warpgroup through
// shared memory, so O is never rescaled.  A row whose later scores exceed that reference by
// more than 2^40 (or hold inf / nan) cannot be finished this way: its item is appended to a
// list in global memory and redone afterwards by the one-CTA kernel, which carries the exact
// running-maximum path.
//
// Roles per CTA:
//   warp 0      TMA producer for this CTA's halves (one lane).
//   warp 1      rank 0: MMA issuer (one lane); both ranks: tensor-memory allocation.
//   warps 4-7   softmax warpgroup 0, warps 8-11 warpgroup 1; at the end of an item both
//               add their row sums and each writes half of the output columns.
// TMEM per CTA: S ring [0,128) [128,256) [256,384), O [384,512); P (bf16) overwrites the first
// 64 columns of its S buffer.  Every mbarrier wait is bounded; a CTA whose wait runs out raises
// the abort flag of both CTAs, records MOGA_ERR_TIMEOUT, and both leave through the common exit.
#include "attn_common.cuh"

namespace moga {
namespace {

using namespace attn;
using namespace sm100;

constexpr int kThreads = 384;
constexpr int kD = 128;
constexpr int kRows = 128;            // query rows of an item held by one CTA
constexpr int kTileN = 128;           // keys per K/V tile
constexpr int kQBlock = 2 * kRows;    // query rows of an item
constexpr int kSRing = 3;             // S buffers in TMEM
constexpr float kRowSumLimit = 1.0995116e12f;   // 2^40

constexpr int NS = 4;                            // K and V ring depth
constexpr int kQBoxBytes = kRows * 128;          // 128 rows x 64 columns
constexpr int kQTileBytes = 2 * kQBoxBytes;      // 32 KB
constexpr int kKBoxBytes = 64 * 128;             // 64 keys x 64 columns
constexpr int kKHalfBytes = 2 * kKBoxBytes;      // 16 KB: this CTA's 64 keys x 128 columns
constexpr int kVHalfBytes = kTileN * 128;        // 16 KB: 128 keys x this CTA's 64 columns
constexpr int kSmemQ = 0;                        // two Q buffers (items alternate)
constexpr int kSmemK = 2 * kQTileBytes;
constexpr int kSmemV = kSmemK + NS * kKHalfBytes;
constexpr int kSmemStage = kSmemV + NS * kVHalfBytes;   // 8 softmax warps x 2 KB output staging
constexpr int kSmemXchg = kSmemStage + 8 * 2048;        // m [2][128], l [2][2][128] floats, flags [2]
constexpr int kXchgBytes = (2 * 128 + 4 * 128) * 4 + 16;
constexpr int kSmemBar = kSmemXchg + kXchgBytes;
// barriers: Q_FULL[2] Q_EMPTY[2] K_FULL[NS] K_EMPTY[NS] V_FULL[NS] V_EMPTY[NS] S_FULL[3] P_FULL[3]
//           O_FULL O_EMPTY M_READY[4] L_READY[2][4]
constexpr int kNumBars = 4 + 4 * NS + 2 * kSRing + 2 + 4 + 8;
constexpr int kSmemTotal = kSmemBar + 8 * kNumBars + 16;
constexpr int kDynSmem = kSmemTotal + 1024;      // slack for 1024-byte alignment
static_assert(kSmemBar % 8 == 0, "barrier alignment");
static_assert(kDynSmem <= 227 * 1024, "shared memory");

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
attn_bf16_pair_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                      const __grid_constant__ CUtensorMap mapV, const Groups grp,
                      const int32_t* __restrict__ order, const int32_t* __restrict__ prefix,
                      __nv_bfloat16* __restrict__ Op, float* __restrict__ lse, uint32_t* header,
                      int32_t* __restrict__ redo, int T, int H, int BG, float scale_log2, float scale,
                      const Scatter sc) {
  extern __shared__ unsigned char smem_raw[];
  // 128B-swizzled tiles need 1024-byte aligned bases (the offset is the same in both CTAs)
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sQ = base + kSmemQ, sK = base + kSmemK, sV = base + kSmemV;
  const uint32_t bars = base + kSmemBar;
  constexpr int Q_FULL = 0, Q_EMPTY = 2, K_FULL = 4, K_EMPTY = 4 + NS, V_FULL = 4 + 2 * NS,
                V_EMPTY = 4 + 3 * NS, S_FULL = 4 + 4 * NS, P_FULL = S_FULL + kSRing, O_FULL = P_FULL + kSRing,
                O_EMPTY = O_FULL + 1, M_READY = O_EMPTY + 1, L_READY = M_READY + 4;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  float* xm = reinterpret_cast<float*>(smem + kSmemXchg);              // [2][128] reference maxima
  float* xl = xm + 2 * 128;                                            // [2][2][128] row sums per warpgroup
  volatile uint32_t* xflag = reinterpret_cast<volatile uint32_t*>(xl + 4 * 128);   // [2] last item sent to the exact path, + 1
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
    }
    for (int i = 0; i < NS; ++i) {
      mbar_init(bar(K_FULL + i), 1);
      mbar_init(bar(K_EMPTY + i), 1);
      mbar_init(bar(V_FULL + i), 1);
      mbar_init(bar(V_EMPTY + i), 1);
    }
    for (int i = 0; i < kSRing; ++i) {
      mbar_init(bar(S_FULL + i), 1);
      mbar_init(bar(P_FULL + i), 8);      // the four warps of one warpgroup in each CTA
    }
    mbar_init(bar(O_FULL), 1);
    mbar_init(bar(O_EMPTY), 16);          // all eight softmax warps of each CTA
    for (int i = 0; i < 4; ++i) mbar_init(bar(M_READY + i), 1);
    for (int i = 0; i < 8; ++i) mbar_init(bar(L_READY + i), 1);
    xflag[0] = 0;
    xflag[1] = 0;
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
    report_status(header, MOGA_ERR_TIMEOUT,
                  (where << 24) | (2u << 20) | ((uint32_t)(blockIdx.x & 0xfff) << 8) | (uint32_t)idx);
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
        uint32_t nit = 0, nkv = 0;
        bool ok = true;
        for (int w = pair; ok && w < total_items; w += npairs, ++nit) {
          const Item it = decode_item<kQBlock>(w, grp, order, prefix, BG, H);
          const int ntiles = (it.khi - it.klo + kTileN - 1) / kTileN;
          const int qb = nit & 1u;
          ok = wait_parked(Q_EMPTY + qb, ((nit >> 1) & 1u) ^ 1u, 1);
          if (!ok) break;
          if (rank == 0) mbar_expect_tx(bar(Q_FULL + qb), 2 * kQTileBytes);
#pragma unroll
          for (int bx = 0; bx < 2; ++bx)
            tma_load_3d_pair(sQ + qb * kQTileBytes + bx * kQBoxBytes, &mapQ, full(Q_FULL + qb), bx * 64,
                             it.row0 + (int)rank * kRows, it.bh);
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
        constexpr uint32_t idesc_qk = instr_desc(kQBlock, kTileN, false);
        constexpr uint32_t idesc_pv = instr_desc(kQBlock, kD, true);
        constexpr uint32_t hi = desc_hi(1024);   // 8-row groups are 1024 bytes apart in every tile
        // S[buf] = Q[qb] K^T for the K tile in ring slot s (the same offsets address both CTAs' halves)
        auto issue_qk = [&](int qb, int s, int buf) {
          const uint32_t qa = desc_lo(sQ + qb * kQTileBytes, 16), kb = desc_lo(sK + s * kKHalfBytes, 16);
#pragma unroll
          for (int kk = 0; kk < kD / 16; ++kk) {
            const uint32_t oq = ((kk / 4) * kQBoxBytes + (kk % 4) * 32) >> 4;
            const uint32_t okk = ((kk / 4) * kKBoxBytes + (kk % 4) * 32) >> 4;
            mma_ss_pair(tmem + buf * kTileN, qa + oq, kb + okk, hi, idesc_qk, kk > 0);
          }
        };
        // O (+)= P[buf] V for the V tile in ring slot s (V is MN-major: 16 keys are 2048 bytes apart)
        auto issue_pv = [&](int s, int buf, bool accumulate) {
          const uint32_t vb = desc_lo(sV + s * kVHalfBytes, kVHalfBytes);
#pragma unroll
          for (int kk = 0; kk < kTileN / 16; ++kk)
            mma_ts_pair(tmem + kSRing * kTileN, tmem + buf * kTileN + kk * 8, vb + ((kk * 2048) >> 4), hi, idesc_pv,
                        (accumulate || kk > 0) ? 1u : 0u);
        };
        // Two cursors over the pair's tiles (item by item, tile by tile): S = Q K^T is issued up to
        // kSRing tiles ahead of O += P V.  tq / tp count the tiles each cursor has passed (ring
        // positions), iq / ip the items.
        int wq = pair, jq = 0, nq_tiles = 0;       // QK cursor: item index, tile in item, tiles of the item
        uint32_t tq = 0, iq = 0;
        if (wq < total_items) {
          const Item it = decode_item<kQBlock>(wq, grp, order, prefix, BG, H);
          nq_tiles = (it.khi - it.klo + kTileN - 1) / kTileN;
        }
        uint32_t tp = 0, ip = 0;
        bool ok = true;
        for (int wp = pair; ok && wp < total_items; wp += npairs, ++ip) {
          const Item itp = decode_item<kQBlock>(wp, grp, order, prefix, BG, H);
          const int np_tiles = (itp.khi - itp.klo + kTileN - 1) / kTileN;
          for (int jp = 0; jp < np_tiles && ok; ++jp, ++tp) {
            // run the QK cursor ahead
            while (ok && wq < total_items && tq < tp + kSRing) {
              if (jq == 0) {
                ok = wait(Q_FULL + (iq & 1u), (iq >> 1) & 1u, 4);
                if (!ok) break;
              }
              ok = wait(K_FULL + tq % NS, (tq / NS) & 1u, 5);
              if (!ok) break;
              tc_fence_after();
              issue_qk(iq & 1u, tq % NS, tq % kSRing);
              tc_commit_pair(bar(S_FULL + tq % kSRing));
              tc_commit_pair(bar(K_EMPTY + tq % NS));
              ++tq;
              if (++jq == nq_tiles) {                 // last use of this item's Q
                tc_commit_pair(bar(Q_EMPTY + (iq & 1u)));
                ++iq;
                jq = 0;
                wq += npairs;
                if (wq < total_items) {
                  const Item it = decode_item<kQBlock>(wq, grp, order, prefix, BG, H);
                  nq_tiles = (it.khi - it.klo + kTileN - 1) / kTileN;
                }
              }
            }
            if (!ok) break;
            ok = wait(V_FULL + tp % NS, (tp / NS) & 1u, 6);
            if (!ok) break;
            ok = wait(P_FULL + tp % kSRing, (tp / kSRing) & 1u, 8);
            if (!ok) break;
            if (jp == 0) {
              ok = wait(O_EMPTY, (ip & 1u) ^ 1u, 9);       // the previous item's epilogue has read O
              if (!ok) break;
            }
            tc_fence_after();
            issue_pv(tp % NS, tp % kSRing, jp > 0);
            tc_commit_pair(bar(V_EMPTY + tp % NS));
            if (jp + 1 == np_tiles) tc_commit_pair(bar(O_FULL));
          }
        }
      }
    }
  } else {
    // ===================================================================== softmax + epilogue
    reg_inc<208>();
    const int wg = (warp - 4) >> 2;                // warpgroup: takes the tiles t with t mod 2 == wg
    const int q = warp & 3;                        // TMEM lane quarter of this warp
    const int r = q * 32 + lane;                   // row inside this CTA's half of the item
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    const uint32_t tO = tmem + lane_off + kSRing * kTileN;
    // the P-ready and O-free barriers the MMA thread waits on live in rank 0
    const uint32_t p_full0 = map_to_rank(bar(P_FULL), 0u), o_empty = map_to_rank(bar(O_EMPTY), 0u);
    uint32_t t0 = 0, nit = 0;                      // tiles of earlier items, items done
    bool ok = true;
    for (int w = pair; ok && w < total_items; w += npairs, ++nit) {
      const Item it = decode_item<kQBlock>(w, grp, order, prefix, BG, H);
      const int ntiles = (it.khi - it.klo + kTileN - 1) / kTileN;
      const int tile_row0 = it.row0 + (int)rank * kRows;
      const uint32_t ipar = nit & 1u;              // exchange buffers alternate between items
      const int j0 = (int)((t0 ^ (uint32_t)wg) & 1u);   // first tile of this item that is mine
      float m = 0.f, l = 0.f;
      bool overflow = false;
      if (j0 != 0) {
        // the other warpgroup owns tile 0 and with it the row's reference maximum
        ok = __all_sync(0xffffffffu, wait(M_READY + q, ipar, 14));
        if (!ok) break;
        m = xm[ipar * 128 + r];
      }
      for (int j = j0; j < ntiles && ok; j += 2) {
        const uint32_t t = t0 + (uint32_t)j, buf = t % kSRing;
        const uint32_t tS = tmem + lane_off + buf * kTileN;
        ok = __all_sync(0xffffffffu, wait(S_FULL + buf, (t / kSRing) & 1u, 10));   // warp-uniform: TMEM loads are warp-collective
        if (!ok) break;
        tc_fence_after();
        uint32_t preg[64];
        {
          uint32_t sreg[128];
#pragma unroll
          for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&sreg[c * 32]));
          tmem_wait_ld();
          const int ncols = it.khi - it.klo - j * kTileN;     // valid keys in this tile (may exceed 128)
          if (ncols < kTileN) {
            // columns past the group's last key: -inf before anything reads them (weight exactly 0;
            // scale_log2 > 0 always, see the launcher)
#pragma unroll
            for (int c = 0; c < 128; ++c)
              if (c >= ncols) sreg[c] = 0xff800000u;
          }
          if (j == 0) {
            // the item's first tile fixes the row's reference maximum for both warpgroups
            float mx[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) mx[c] = __uint_as_float(sreg[c]);
#pragma unroll
            for (int c = 8; c < 128; ++c) mx[c & 7] = fmaxf(mx[c & 7], __uint_as_float(sreg[c]));
            m = fmaxf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])), fmaxf(fmaxf(mx[4], mx[5]), fmaxf(mx[6], mx[7])));
            xm[ipar * 128 + r] = m;
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(M_READY + q));
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
          const float lsum = l01.x + l01.y;
          overflow |= !(lsum < kRowSumLimit);      // scores far above the reference, inf or nan
          l += lsum;
        }
        tmem_st32(tS, *reinterpret_cast<uint32_t(*)[32]>(&preg[0]));
        tmem_st32(tS + 32, *reinterpret_cast<uint32_t(*)[32]>(&preg[32]));
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(p_full0 + 8u * buf);
      }
      if (!ok) break;
      t0 += (uint32_t)ntiles;
      // ---- the two warpgroups add their row sums (thread r of each holds the same row)
      // rows that could not be finished against the fixed reference: the item goes to the exact
      // path, listed once per CTA (the flag holds the last item listed through it)
      if (__any_sync(0xffffffffu, overflow) && lane == 0 &&
          atomicExch(const_cast<uint32_t*>(&xflag[ipar]), (uint32_t)w + 1u) != (uint32_t)w + 1u) {
        const int at = atomicAdd(redo, 1);
        redo[4 + at] = w;
      }
      xl[(ipar * 2 + wg) * 128 + r] = l;
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(L_READY + wg * 4 + q));
      ok = __all_sync(0xffffffffu, wait(L_READY + (wg ^ 1) * 4 + q, ipar, 15));
      if (!ok) break;
      l += xl[(ipar * 2 + (wg ^ 1)) * 128 + r];
      // ---- epilogue: O / l -> bf16 -> per-warp staging -> global; this warpgroup writes columns
      //      [wg * 64, wg * 64 + 64)
      ok = __all_sync(0xffffffffu, wait(O_FULL, ipar, 11));
      if (!ok) break;
      tc_fence_after();
      float inv_l = 1.f / l;
      const bool live = tile_row0 + r < it.qhi;
      const int bb = it.bh / H, hh = it.bh % H;
      if (sc.perm != nullptr && live) inv_l *= sc.gate[(size_t)bb * sc.N + sc.perm[(size_t)bb * T + tile_row0 + r]];
      // Each warp stages 32 rows x 32 columns (2 KB) at a time in its own buffer and writes them
      // out itself: lane L stores piece L % 4 of rows i * 8 + L / 4, i = 0..3 (64-byte row segments).
      unsigned char* wst = smem + kSmemStage + (wg * 4 + q) * 2048;
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
      for (int cc = 0; cc < 2; ++cc) {
        const int c = wg * 2 + cc;           // 32-column chunk of O
        uint32_t oreg[32];
        tmem_ld32(tO + c * 32, oreg);
        tmem_wait_ld();
        if (cc == 1) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(o_empty);    // this warp has read its part of O
        }
#pragma unroll
        for (int v = 0; v < 4; ++v) {      // four 16-byte chunks (8 bf16 each) per 32 columns
          uint4 pk;
          uint32_t* pw = reinterpret_cast<uint32_t*>(&pk);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 tt = __floats2bfloat162_rn(__uint_as_float(oreg[v * 8 + 2 * i]) * inv_l,
                                                      __uint_as_float(oreg[v * 8 + 2 * i + 1]) * inv_l);
            pw[i] = *reinterpret_cast<uint32_t*>(&tt);
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
      if (wg == 0 && lse != nullptr && live) lse[(size_t)it.bh * T + tile_row0 + r] = m * scale + __logf(l);
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

// redo: int32 [4 + 2 * items]: word 0 counts the items the exact path has to redo, the list
// starts at word 4 (both CTAs of a pair may list the same item).
moga_status attn::launch_pair(const attn::Problem& p, cudaStream_t st) {
  CUtensorMap mq, mk, mv;
  const long long BH = (long long)p.B * p.H;
  if (!make_map(&mq, p.Q, kD, p.Tq, BH, kRows) || !make_map(&mk, p.K, kD, p.Tkv, BH, 64) ||
      !make_map(&mv, p.V, kD, p.Tkv, BH, kTileN))
    return MOGA_ERR_CUDA;
  MOGA_CUDA_OK(cudaMemsetAsync(p.redo, 0, 16, st));
  attn_schedule_kernel<<<1, 1024, 0, st>>>(p.grp, p.order, p.prefix, p.B, p.H, kQBlock);
  MOGA_CUDA_OK(cudaGetLastError());
  int num_sms = 0;
  if (!current_sm_count(&num_sms)) return MOGA_ERR_CUDA;
  MOGA_CUDA_OK(cudaFuncSetAttribute(attn_bf16_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmem));
  const long long max_items = max_items_256(p);
  long long pairs = num_sms / 2;
  if (max_items < pairs) pairs = max_items;
  if (pairs < 1) pairs = 1;
  // log2 domain; a zero scale is served by the smallest normal float (see the one-CTA launcher)
  const float log2e = 1.4426950408889634f;
  const float scale_log2 = p.scale * log2e > 1.17549435e-38f ? p.scale * log2e : 1.17549435e-38f;
  attn_bf16_pair_kernel<<<(unsigned)(2 * pairs), kThreads, kDynSmem, st>>>(
      mq, mk, mv, p.grp, p.order, p.prefix, static_cast<__nv_bfloat16*>(p.O), p.lse, p.header, p.redo, (int)p.Tq,
      p.H, p.B * p.grp.G, scale_log2, p.scale, p.sc);
  MOGA_CUDA_OK(cudaGetLastError());
  // the items it listed (normally none) are redone by the one-CTA kernel's exact path
  return launch_single_redo(p, st);
}

}  // namespace moga
