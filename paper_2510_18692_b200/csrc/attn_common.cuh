// Pieces shared by the two bf16 group-attention kernels (one CTA per work item, and a pair of
// CTAs per work item): the group list, the cost-ordered schedule, the output placement and the
// host-side description of one launch.
#pragma once

#include "moga_internal.cuh"
#include "sm100_ptx.cuh"

namespace moga {
namespace attn {

// ----------------------------------------------------------------------------- schedule
// The groups of one launch.  Group g of batch item b owns query rows
// [q_off[b*stride + g], q_off[b*stride + g + 1]) of Q / O and key rows
// [kv_off[b*stride + g], kv_off[b*stride + g + 1]) of K / V.  Routed groups (Alg. 1): q_off and
// kv_off are the same array, stride = G + 1.  Static groups (Sec. 3.2): one list shared by
// all batch items (stride 0), keys may be a superset of the queries.
struct Groups {
  const int32_t* q_off;
  const int32_t* kv_off;
  int stride;
  int G;
};

constexpr int kRankLimit = 256;   // above this many groups per item the list keeps its order

// order[b*G + r]  : group with the r-th largest cost (queries x keys) in batch item b
// prefix[b*G + r] : number of work items before (b, r); prefix[B*G] = total
// A group with queries but no keys gets no work item: its rows are left untouched.
// qblock: query rows per work item (256 for the one-CTA kernel, 512 for the CTA-pair kernel).
__global__ void attn_schedule_kernel(const Groups grp, int32_t* __restrict__ order, int32_t* __restrict__ prefix,
                                     int B, int H, int qblock);

struct Item {
  int bh;          // b * H + h
  int row0;        // first row of the query block
  int qhi;         // end of the group's query rows
  int klo, khi;    // the group's key rows
};

template <int QB>
__device__ __forceinline__ Item decode_item(int w, const Groups& grp, const int32_t* __restrict__ order,
                                            const int32_t* __restrict__ prefix, int BG, int H) {
  int lo = 0, hi = BG;           // largest idx with prefix[idx] <= w (entries without items are skipped)
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (prefix[mid] <= w) lo = mid; else hi = mid;
  }
  const int b = lo / grp.G;
  const int g = order[lo];
  const int32_t* qo = grp.q_off + (size_t)b * grp.stride;
  const int32_t* ko = grp.kv_off + (size_t)b * grp.stride;
  Item it;
  const int qlo = qo[g];
  it.qhi = qo[g + 1];
  it.klo = ko[g];
  it.khi = ko[g + 1];
  const int nqb = (it.qhi - qlo + QB - 1) / QB;
  const int local = w - prefix[lo];
  const int h = local / nqb, qb = local % nqb;
  it.bh = b * H + h;
  it.row0 = qlo + qb * QB;
  return it;
}

// Output placement (the kernels' epilogue).
//   kEpiDefault   perm == nullptr: rows stay in sorted order, Op is [B*H, T, D].  Otherwise
//                 (top-1 routing) the gated inverse permutation of Eq. 5: sorted row p of batch
//                 item b goes to token perm[b, p] of O (element strides sb, sh, sn), multiplied
//                 by gate[b, token] in fp32 before the one rounding to bf16.
//   kEpiList      static groups: row p goes to token perm[p] (one list for all batch items), no
//                 gate.
//   kEpiMean3     last branch of the visual attention block (Sec. 3.2): rows stay in place
//                 (contiguous [B, H, N, D]); the stored value is the mean of this branch's row,
//                 rounded to bf16 as if it had been stored, and the rows of mean_a and mean_b at
//                 the same place: (a + b + c) / 3 in fp32, one rounding.
//   kEpiAdd       top-k routing with k = 2: perm holds the assignment index a = token * k + slot at
//                 each sorted position; gate[b, a] * row is rounded to bf16 and added into token
//                 a / k of a zeroed O with a bf16x2 reduction (two commutative additions per
//                 element, so the result does not depend on their order).
constexpr int kEpiDefault = 0, kEpiList = 1, kEpiMean3 = 2, kEpiAdd = 3;
struct Scatter {
  const int32_t* perm;
  const float* gate;
  long long sb, sh, sn;
  int N;                     // tokens per batch item
  int k;
  const __nv_bfloat16* mean_a;
  const __nv_bfloat16* mean_b;
};

// [B*H, T, D] bf16, box 64 columns x box_rows rows x 1, 128-byte swizzle, out-of-range rows read as zero.
inline bool make_map(CUtensorMap* map, const void* ptr, int D, long long T, long long BH, int box_rows) {
  sm100::EncodeTiledFn fn = sm100::get_encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)T, (cuuint64_t)BH};
  cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)T * D * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// One launch: B*H heads, groups grp, Q / O with Tq rows and K / V with Tkv rows per head.
struct Problem {
  int B, H;
  long long Tq, Tkv;
  float scale;
  const void *Q, *K, *V;
  void* O;
  float* lse;
  Groups grp;
  int32_t *order, *prefix;   // scratch: B*G and B*G + 1 int32
  int32_t* redo;             // scratch of the kernels that hand items to the exact path: int32
                             // [4 + 2 * max_items_256]; nullptr: the launch cannot use those kernels
  uint32_t* header;          // device status word
  Scatter sc;
  int epi;                   // kEpiDefault / kEpiList / kEpiMean3 (the latter two: one-CTA kernel, D = 128)
};


// Upper bound on the work items of 256 query rows in a launch.
inline long long max_items_256(const Problem& p) {
  return ((p.Tq + 255) / 256 + p.grp.G) * (long long)p.B * p.H;
}

// kernels (each in its own file); both read the schedule attn_schedule_kernel wrote for their
// query block
moga_status launch_single(int D, const Problem& p, cudaStream_t st);   // 256 query rows per CTA
moga_status launch_pair(const Problem& p, cudaStream_t st);            // D = 128, 256 query rows per CTA pair
moga_status launch_duo(const Problem& p, cudaStream_t st);             // D = 128, two softmax threads per row
// D = 128: the one-CTA kernel over the items listed in p.redo (their schedule is already in place)
moga_status launch_single_redo(const Problem& p, cudaStream_t st);

}  // namespace attn
}  // namespace moga
