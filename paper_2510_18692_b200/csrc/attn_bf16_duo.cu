// bf16 per-group attention (Eq. 1 inside each group, Alg. 1 line 3) on tcgen05 tensor cores,
// d_head = 128: the kernel with two softmax threads per query row.
//
// Same work items, MMA order and TMEM map as the kernel in attn_bf16.cu (two 128-row Q tiles A and B
// per item, S_A S_B O_A O_B in the 512 TMEM columns, P over S).  Per Q tile the chain
// Q K^T -> softmax -> P V -> next Q K^T is serial (P lives where S was), and the two tiles' chains
// interleave on the one tensor pipe; the softmax link of that chain is what this kernel shortens:
//
//   warps 2-17  softmax, two threads per query row (64 of the tile's 128 columns each; 16 warps, four
//               per scheduler), so a tile's exponentials keep the XU pipe busy instead of one warp
//               per scheduler issuing them in order.  A thread reads its columns in two chunks of 32
//               and writes each chunk's P over columns it has already read (P of keys 64 h .. 64 h + 63
//               sits in columns [64 h, 64 h + 32) of the S tile).
//
// The reference maximum of a row is the exact maximum of its first key tile (the two halves exchange
// theirs through shared memory) and is never raised: any reference gives the same quotient O / l while
// nothing overflows.  A row whose tile sum reaches 2^40 (or is not finite) marks its item: the item
// is appended to the redo list and computed again by the exact kernel of attn_bf16.cu, which runs
// after this one over that list (normally empty) and overwrites the item's rows.  Output placement:
// kEpiDefault (sorted order, or the gated scatter of top-1 routing), both plain stores, so a redone
// item is simply stored twice.
// The K / V ring pairs the tiles the way the MMA issuer uses them: a stage holds the V tile of one key
// tile and the K tile of the next (the next item's first one after an item's last), which are read in the
// same step (P V, then the next Q K^T), so the issuer polls one barrier and commits one per key tile
// for its inputs instead of two (its polls and commits are serial with its MMAs: +1.7 % on groups of
// ~17,500 rows, +2.1 % on the clip's groups, same box, alternating runs).
// Every wait is a bounded mbarrier wait (the exchanges between the two halves too).
#include "attn_common.cuh"

namespace moga {
namespace {

using namespace attn;
using namespace sm100;

constexpr int kThreads = 576;     // warp 0 producer, warp 1 MMA issuer, warps 2-17 softmax: 18 warps, at most 5 per
                                  // scheduler, whose 16,384 registers then allow 96 per thread
constexpr int kD = 128;
constexpr int kTileM = 128;       // query rows per tile
constexpr int kTileN = 128;       // keys per K/V tile
constexpr int kQBlock = 2 * kTileM;
constexpr float kRowSumLimit = 1.0995116e12f;      // 2^40

constexpr int NS = 2;                              // ring depth: stages of one V and one K tile
constexpr int kBoxes = kD / 64;                    // 64-column TMA boxes per tile
constexpr int kBoxBytes = kTileM * 128;            // 128 rows x 128 bytes
constexpr int kTileBytes = kBoxes * kBoxBytes;
constexpr int kSmemQ = 0;
constexpr int kSmemK = 2 * kTileBytes;
constexpr int kSmemV = kSmemK + NS * kTileBytes;
constexpr int kSmemStage = kSmemV + NS * kTileBytes;   // 16 softmax warps x 2 KB output staging
constexpr int kSmemX = kSmemStage + 16 * 2048;         // exchange between the two halves: 2 tiles x 2 halves x 128 floats
constexpr int kSmemBar = kSmemX + 2 * 2 * kTileM * 4;
constexpr int kNumBars = 2 + 2 + 2 * NS + 2 + 2 + 2 + 2 + 2 + 2;
constexpr int kSmemTotal = kSmemBar + 8 * kNumBars + 32;
constexpr int kDynSmem = 227 * 1024;                   // everything a CTA may have; the tiles need a 1024-byte aligned base
static_assert(kSmemTotal <= kDynSmem, "shared memory");

__global__ void __launch_bounds__(kThreads, 1)
attn_bf16_duo_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                     const __grid_constant__ CUtensorMap mapV, const Groups grp,
                     const int32_t* __restrict__ order, const int32_t* __restrict__ prefix,
                     __nv_bfloat16* __restrict__ Op, float* __restrict__ lse, uint32_t* header, int T, int H,
                     int BG, float scale_log2, float scale, const Scatter sc, int32_t* __restrict__ redo) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  // 128B-swizzled tiles need 1024-byte aligned bases; the layout leaves less than 1 KB of slack, so a base
  // that would push it past the allocation is reported instead of used
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  if (base - smem_u32(smem_raw) + kSmemTotal > (uint32_t)kDynSmem) {
    if (threadIdx.x == 0) report_status(header, MOGA_ERR_INTERNAL, 0x5a000000u | blockIdx.x);
    return;
  }
  unsigned char* smem = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sQ = base + kSmemQ, sK = base + kSmemK, sV = base + kSmemV;
  const uint32_t bars = base + kSmemBar;
  constexpr int Q_FULL = 0, Q_EMPTY = 2, IN_FULL = 4, IN_EMPTY = 4 + NS, S_FULL = 4 + 2 * NS, P_FULL = S_FULL + 2, O_FULL = S_FULL + 4,
                O_EMPTY = S_FULL + 6, X_WRITTEN = S_FULL + 8, X_READ = S_FULL + 10;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + kSmemBar + 8 * kNumBars);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  int* listed = reinterpret_cast<int*>(smem + kSmemBar + 8 * kNumBars + 8);   // per tile: the item it last put on the redo list

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_items = prefix[BG];

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(Q_FULL + i), 1);
      mbar_init(bar(Q_EMPTY + i), 1);
      mbar_init(bar(S_FULL + i), 1);
      mbar_init(bar(P_FULL + i), 2 * kTileM);
      mbar_init(bar(O_FULL + i), 1);
      mbar_init(bar(O_EMPTY + i), 2 * kTileM);
      mbar_init(bar(X_WRITTEN + i), 2 * kTileM);
      mbar_init(bar(X_READ + i), 2 * kTileM);
      listed[i] = -1;
    }
    for (int i = 0; i < NS; ++i) {
      mbar_init(bar(IN_FULL + i), 1);
      mbar_init(bar(IN_EMPTY + i), 1);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32((const void*)tmem_slot), 512u);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  // Bounded wait.  Returns false when the CTA is aborting (this wait or another one expired).
  auto wait = [&](int idx, uint32_t parity, uint32_t where) -> bool {
    const WaitResult res = mbar_wait_bounded(bar(idx), parity, abort_flag, kDefaultWaitLimitNs);
    if (res == kWaitExpired)
      report_status(header, MOGA_ERR_TIMEOUT, (where << 24) | (4u << 20) | ((uint32_t)(blockIdx.x & 0xfff) << 8) | (uint32_t)idx);
    return res == kWaitDone;
  };
  // The producer's waits are long (a ring slot frees once per K/V tile): it parks between polls
  // so that it does not take issue slots from the softmax warps of its scheduler.
  auto wait_parked = [&](int idx, uint32_t parity, uint32_t where) -> bool {
    const WaitResult res = mbar_wait_bounded_parked(bar(idx), parity, abort_flag, kDefaultWaitLimitNs);
    if (res == kWaitExpired)
      report_status(header, MOGA_ERR_TIMEOUT, (where << 24) | (4u << 20) | ((uint32_t)(blockIdx.x & 0xfff) << 8) | (uint32_t)idx);
    return res == kWaitDone;
  };

  if (warp == 0) {
    // ===================================================================== TMA producer
    if (lane == 0) {
      // Ring stage c holds the K tile of the c-th key tile this CTA meets (over all its items) and the V
      // tile of the one before it: both are used in the same step of the MMA issuer (P V of a tile, then
      // Q K^T of the next), so one barrier fills and one frees a stage.  The first stage has no V, the
      // last one (after the loop) no K.
      uint32_t nq[2] = {0, 0}, c = 0;
      bool ok = true, have_prev = false;
      int prev_row = 0, prev_bh = 0;
      for (int w = blockIdx.x; ok && w < total_items; w += gridDim.x) {
        const Item it = decode_item<kQBlock>(w, grp, order, prefix, BG, H);
        const int ntiles = (it.khi - it.klo + kTileN - 1) / kTileN;
        const bool validB = it.row0 + kTileM < it.qhi;
        for (int j = 0; j < ntiles && ok; ++j) {
          const int s = c % NS;
          ok = wait_parked(IN_EMPTY + s, ((c / NS) & 1u) ^ 1u, 2);
          if (!ok) break;
          mbar_expect_tx(bar(IN_FULL + s), kTileBytes * (have_prev ? 2 : 1));
#pragma unroll
          for (int bx = 0; bx < kBoxes; ++bx)
            tma_load_3d(sK + s * kTileBytes + bx * kBoxBytes, &mapK, bar(IN_FULL + s), bx * 64, it.klo + j * kTileN, it.bh);
          if (have_prev) {
#pragma unroll
            for (int bx = 0; bx < kBoxes; ++bx)
              tma_load_3d(sV + s * kTileBytes + bx * kBoxBytes, &mapV, bar(IN_FULL + s), bx * 64, prev_row, prev_bh);
          }
          ++c;
          have_prev = true;
          prev_row = it.klo + j * kTileN;
          prev_bh = it.bh;
          if (j == 0) {
            // the item's Q tiles, after the stage that carries its first K tile
            for (int x = 0; x < (validB ? 2 : 1) && ok; ++x) {
              ok = wait_parked(Q_EMPTY + x, (nq[x] & 1u) ^ 1u, 1);
              if (!ok) break;
              mbar_expect_tx(bar(Q_FULL + x), kTileBytes);
#pragma unroll
              for (int bx = 0; bx < kBoxes; ++bx)
                tma_load_3d(sQ + x * kTileBytes + bx * kBoxBytes, &mapQ, bar(Q_FULL + x), bx * 64,
                            it.row0 + x * kTileM, it.bh);
              ++nq[x];
            }
          }
        }
      }
      if (ok && have_prev) {
        const int s = c % NS;
        if (wait_parked(IN_EMPTY + s, ((c / NS) & 1u) ^ 1u, 2)) {
          mbar_expect_tx(bar(IN_FULL + s), kTileBytes);
#pragma unroll
          for (int bx = 0; bx < kBoxes; ++bx)
            tma_load_3d(sV + s * kTileBytes + bx * kBoxBytes, &mapV, bar(IN_FULL + s), bx * 64, prev_row, prev_bh);
        }
      }
    }
  } else if (warp == 1) {
    // ===================================================================== MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = instr_desc(kTileM, kTileN, false);
      constexpr uint32_t idesc_pv = instr_desc(kTileM, kD, true);
      uint32_t nq[2] = {0, 0}, np[2] = {0, 0}, no[2] = {0, 0};
      bool ok = true;
      // S_x = Q_x K^T for the K tile in ring slot s
      constexpr uint32_t hi = desc_hi(1024);   // 8-row groups are 1024 bytes apart in every tile
      auto issue_qk = [&](int x, int s) {
        const uint32_t qa = desc_lo(sQ + x * kTileBytes, 16), kb = desc_lo(sK + s * kTileBytes, 16);
#pragma unroll
        for (int kk = 0; kk < kD / 16; ++kk) {
          const uint32_t o = ((kk / 4) * kBoxBytes + (kk % 4) * 32) >> 4;
          mma_ss(tmem + x * kTileN, qa + o, kb + o, hi, idesc_qk, kk > 0);
        }
      };
      // O_x (+)= P_x V for the V tile in ring slot s (V is MN-major: 64-column boxes kBoxBytes apart)
      auto issue_pv = [&](int x, int s, bool accumulate) {
        const uint32_t vb = desc_lo(sV + s * kTileBytes, kBoxBytes);
#pragma unroll
        for (int kk = 0; kk < kTileN / 16; ++kk)
          mma_ts(tmem + 256 + x * 128, tmem + x * kTileN + (kk / 4) * 64 + (kk % 4) * 8, vb + ((kk * 2048) >> 4), hi, idesc_pv,
                 (accumulate || kk > 0) ? 1u : 0u);
      };
      uint32_t c = 0;                       // ring stage counter (see the producer)
      int w = blockIdx.x;
      if (w < total_items) {
        Item it = decode_item<kQBlock>(w, grp, order, prefix, BG, H);
        int ntiles = (it.khi - it.klo + kTileN - 1) / kTileN;
        int nx = (it.row0 + kTileM < it.qhi) ? 2 : 1;
        // the first item's first S tiles
        for (int x = 0; x < nx && ok; ++x) {
          ok = wait(Q_FULL + x, nq[x] & 1u, 4);
          ++nq[x];
        }
        if (ok) ok = wait(IN_FULL + c % NS, (c / NS) & 1u, 5);
        if (ok) {
          tc_fence_after();
          for (int x = 0; x < nx; ++x) {
            issue_qk(x, c % NS);
            tc_commit(bar(S_FULL + x));
            if (ntiles == 1) tc_commit(bar(Q_EMPTY + x));   // the item's only use of this Q tile
          }
          tc_commit(bar(IN_EMPTY + c % NS));
          ++c;
        }
        while (ok) {
          const int wn = w + (int)gridDim.x;
          const bool has_next = wn < total_items;
          Item nxt = it;
          int ntiles_n = 0, nx_n = 0;
          if (has_next) {
            nxt = decode_item<kQBlock>(wn, grp, order, prefix, BG, H);
            ntiles_n = (nxt.khi - nxt.klo + kTileN - 1) / kTileN;
            nx_n = (nxt.row0 + kTileM < nxt.qhi) ? 2 : 1;
          }
          for (int j = 0; j < ntiles && ok; ++j) {
            // stage c: V of tile j and K of the tile after it (the next item's first tile after this item's last)
            ok = wait(IN_FULL + c % NS, (c / NS) & 1u, 6);
            if (!ok) break;
            const bool more = j + 1 < ntiles;
            const bool cross = !more && has_next;
            if (cross) {
              for (int x = 0; x < nx_n && ok; ++x) {
                ok = wait(Q_FULL + x, nq[x] & 1u, 4);
                ++nq[x];
              }
              if (!ok) break;
            }
            for (int x = 0; x < 2 && ok; ++x) {
              const bool pv = x < nx;
              const bool qk = more ? pv : (cross && x < nx_n);
              if (pv) {
                ok = wait(P_FULL + x, np[x] & 1u, 8);
                if (!ok) break;
                ++np[x];
                if (j == 0) {
                  ok = wait(O_EMPTY + x, (no[x] & 1u) ^ 1u, 9);
                  if (!ok) break;
                  ++no[x];
                }
              }
              tc_fence_after();
              if (pv) issue_pv(x, c % NS, j > 0);
              if (qk) {
                issue_qk(x, c % NS);
                tc_commit(bar(S_FULL + x));
                // last use of this Q tile: free it early
                if (more ? (j + 2 == ntiles) : (ntiles_n == 1)) tc_commit(bar(Q_EMPTY + x));
              }
              if (pv && !more) tc_commit(bar(O_FULL + x));
            }
            if (!ok) break;
            tc_commit(bar(IN_EMPTY + c % NS));
            ++c;
          }
          if (!has_next) break;
          w = wn;
          it = nxt;
          ntiles = ntiles_n;
          nx = nx_n;
        }
      }
    }
  } else {
    // ===================================================================== softmax + epilogue
    const int x = (warp - 2) >> 3;                 // 0: tile A, 1: tile B
    const int h = ((warp - 2) >> 2) & 1;           // which 64 of the tile's 128 columns
    const int q = warp & 3;                        // TMEM lane quarter of this warp
    const int r = q * 32 + lane;                   // row inside the tile
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    const uint32_t tS = tmem + lane_off + x * kTileN + h * 64;
    const uint32_t tO = tmem + lane_off + 256 + x * 128;
    float* xmine = reinterpret_cast<float*>(smem + kSmemX) + (x * 2 + h) * kTileM;
    const float* xother = reinterpret_cast<const float*>(smem + kSmemX) + (x * 2 + (h ^ 1)) * kTileM;
    uint32_t n_s = 0, n_o = 0, n_x = 0;
    bool ok = true;
    // Exchange of one float per row between the two threads of a row: write, wait until all 256 threads of
    // the tile have written, read the other half's value, and say so (the next write waits for that).
    auto exchange = [&](float mine, float& other) -> bool {
      if (!__all_sync(0xffffffffu, wait(X_READ + x, (n_x & 1u) ^ 1u, 12))) return false;
      xmine[r] = mine;
      mbar_arrive(bar(X_WRITTEN + x));
      if (!__all_sync(0xffffffffu, wait(X_WRITTEN + x, n_x & 1u, 13))) return false;
      other = xother[r];
      mbar_arrive(bar(X_READ + x));
      ++n_x;
      return true;
    };
    for (int w = blockIdx.x; ok && w < total_items; w += gridDim.x) {
      const Item it = decode_item<kQBlock>(w, grp, order, prefix, BG, H);
      if (x == 1 && !(it.row0 + kTileM < it.qhi)) continue;
      const int ntiles = (it.khi - it.klo + kTileN - 1) / kTileN;
      const int tile_row0 = it.row0 + x * kTileM;
      float m = 0.f, l = 0.f;
      bool bad = false;
      for (int j = 0; j < ntiles && ok; ++j) {
        ok = __all_sync(0xffffffffu, wait(S_FULL + x, n_s & 1u, 10));   // warp-uniform: TMEM loads are warp-collective
        if (!ok) break;
        ++n_s;
        tc_fence_after();
        const int ncols = it.khi - it.klo - j * kTileN - h * 64;     // valid keys among this thread's 64 columns
        if (j == 0) {
          // the row's reference maximum: the largest score of the first key tile, both halves
          float mt = -INFINITY;
#pragma unroll
          for (int ch = 0; ch < 2; ++ch) {
            uint32_t sreg[32];
            tmem_ld32(tS + ch * 32, sreg);
            tmem_wait_ld();
            float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int c = 0; c < 32; ++c)
              if (ncols >= 64 || ch * 32 + c < ncols) mx[c & 3] = fmaxf(mx[c & 3], __uint_as_float(sreg[c]));
            mt = fmaxf(mt, fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])));
          }
          float mo;
          ok = exchange(mt, mo);
          if (!ok) break;
          m = fmaxf(mt, mo);            // key 0 of the tile is always inside the group: finite unless a score is not
        }
        const float neg_m = -m * scale_log2;
        const float2 sc2 = make_float2(scale_log2, scale_log2), nm2 = make_float2(neg_m, neg_m);
        float2 ls[4] = {{0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}};
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t sreg[32], preg[16];
          tmem_ld32(tS + ch * 32, sreg);
          tmem_wait_ld();
          if (ncols < 64) {
            // Columns past the group's last key hold scores against the next group's rows (any value, NaN
            // included): they become -inf before anything reads them, so their weight is 2^(-inf) = 0
            // exactly.  (scale_log2 > 0 always: the launcher replaces a zero scale by the smallest normal float.)
#pragma unroll
            for (int c = 0; c < 32; ++c)
              if (ch * 32 + c >= ncols) sreg[c] = 0xff800000u;
          }
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            const float2 xx = __ffma2_rn(make_float2(__uint_as_float(sreg[2 * c]), __uint_as_float(sreg[2 * c + 1])),
                                         sc2, nm2);
            const float2 pe = make_float2(ex2(xx.x), ex2(xx.y));
            ls[c & 3] = __fadd2_rn(ls[c & 3], pe);
            __nv_bfloat162 pk = __floats2bfloat162_rn(pe.x, pe.y);
            preg[c] = *reinterpret_cast<uint32_t*>(&pk);
          }
          // this chunk's 32 columns have been read: its P goes over 16 columns of the part already read
          tmem_st16(tS + ch * 16, preg);
        }
        const float2 l01 = __fadd2_rn(__fadd2_rn(ls[0], ls[1]), __fadd2_rn(ls[2], ls[3]));
        const float lsum = l01.x + l01.y;
        bad |= !(lsum < kRowSumLimit);        // scores far above the reference (or not finite): the item is redone
        l += lsum;
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar(P_FULL + x));
      }
      if (!ok) break;
      // the row's sum; NaN from either half marks the row
      float lo;
      ok = exchange(bad ? __int_as_float(0x7fc00000) : l, lo);
      if (!ok) break;
      l += lo;
      if (__any_sync(0xffffffffu, !(l == l)) && lane == 0 && atomicExch(&listed[x], w) != w) {
        const int at = atomicAdd(&redo[0], 1);
        redo[4 + at] = w;
      }
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
      unsigned char* wst = smem + kSmemStage + (warp - 2) * 2048;
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
      for (int c2 = 0; c2 < 2; ++c2) {
        const int c = h * 2 + c2;             // this thread's half of the output columns, 32 at a time
        uint32_t oreg[32];
        tmem_ld32(tO + c * 32, oreg);
        tmem_wait_ld();
        if (c2 == 1) {
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
          const uint4 val = *reinterpret_cast<const uint4*>(wst + row * 64 + ((piece ^ ((row >> 1) & 3)) * 16));
          if (orow_live[i]) *reinterpret_cast<uint4*>(obase[i] + c * 32 + piece * 8) = val;
        }
        __syncwarp();
      }
      if (lse != nullptr && live && h == 0) lse[(size_t)it.bh * T + tile_row0 + r] = m * scale + __logf(l);
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
    tmem_dealloc(tmem, 512u);
  }
}

}  // namespace

// The two-threads-per-row kernel over all items, then the exact kernel over the items it listed.
moga_status attn::launch_duo(const attn::Problem& p, cudaStream_t st) {
  CUtensorMap mq, mk, mv;
  const long long BH = (long long)p.B * p.H;
  if (!make_map(&mq, p.Q, kD, p.Tq, BH, kTileM) || !make_map(&mk, p.K, kD, p.Tkv, BH, kTileN) ||
      !make_map(&mv, p.V, kD, p.Tkv, BH, kTileN))
    return MOGA_ERR_CUDA;
  attn_schedule_kernel<<<1, 1024, 0, st>>>(p.grp, p.order, p.prefix, p.B, p.H, kQBlock);
  MOGA_CUDA_OK(cudaGetLastError());
  MOGA_CUDA_OK(cudaMemsetAsync(p.redo, 0, 4 * sizeof(int32_t), st));
  int num_sms = 0;
  if (!current_sm_count(&num_sms)) return MOGA_ERR_CUDA;
  MOGA_CUDA_OK(cudaFuncSetAttribute(attn_bf16_duo_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmem));
  const long long max_items = max_items_256(p);
  const int grid = (int)(max_items < num_sms ? max_items : num_sms);
  // zero scale: see the one-CTA kernel's launcher (the masking needs scale_log2 > 0)
  const float log2e = 1.4426950408889634f;
  const float scale_log2 = p.scale * log2e > 1.17549435e-38f ? p.scale * log2e : 1.17549435e-38f;
  attn_bf16_duo_kernel<<<grid, kThreads, kDynSmem, st>>>(mq, mk, mv, p.grp, p.order, p.prefix,
                                                         static_cast<__nv_bfloat16*>(p.O), p.lse, p.header, (int)p.Tq,
                                                         p.H, p.B * p.grp.G, scale_log2, p.scale, p.sc, p.redo);
  MOGA_CUDA_OK(cudaGetLastError());
  return launch_single_redo(p, st);
}

}  // namespace moga
