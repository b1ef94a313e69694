/*
 * moga.h -- C ABI of the B200 (sm_100a) MoGA routed group-attention forward.
 *
 * The library implements the forward of Mixture-of-Groups Attention
 * (Sec. 3.2, Eq. 2-5 and Alg. 1 of the paper): a linear router scores each
 * token against M groups, the token joins its top-k groups with a softmax gate,
 * tokens are listed group by group (stable counting sort), Q/K/V rows are
 * gathered into that order, dense softmax attention runs inside every group, and
 * the rows go back to token order multiplied by their gates.
 *
 * Conventions shared by every entry point
 *  - Every data pointer is a DEVICE pointer owned by the caller, 16-byte aligned.
 *    The library allocates and frees nothing; all scratch lives in the caller's
 *    workspace `ws` (device memory, 256-byte aligned).
 *  - `stream` is a cudaStream_t passed as void*.  Calls are asynchronous on that
 *    stream and never synchronise the host, except moga_last_device_status.
 *  - Errors are return codes only.  A non-OK code from argument checking means
 *    nothing was launched.
 *  - Layouts (row-major, last index fastest):
 *      X       [B, N, C]        dtype          token features
 *      Wr      [C, M]           float          router weight
 *      bias    [M]              float          router bias, may be NULL
 *      Q,K,V,O [B, H, N, D]     dtype          element strides q_stride_{b,h,n}; D contiguous.
 *                                              All-zero strides mean contiguous [B,H,N,D];
 *                                              [B,N,H,D] is expressed through the strides.
 *      gid     [B, N, k]        int32          selected groups, descending logit
 *      gate    [B, N, k]        float          gate of each selected group
 *      logits  [B, N, M]        float          optional router scores
 *      perm    [B, T]           int32          token index at each sorted position, T = N*k
 *      inv     [B, N, k]        int32          sorted position of assignment (n, j)
 *      offsets [B, M+1]         int32          group g owns positions [offsets[g], offsets[g+1])
 *      Qp,Kp,Vp,Op [B, H, T, D] dtype          rows in sorted (group-major) order, contiguous
 *      lse     [B, H, T]        float          optional log-sum-exp of the scaled scores
 *  - N = 0 (no tokens) is valid: the stage and forward calls return MOGA_OK without reading the
 *    data pointers; moga_permute / moga_forward still zero the offsets they are given.
 *  - Limits: 1 <= M <= 64, 1 <= k <= min(M, 8), D in {64, 128}, C a multiple of
 *    16 bytes worth of elements, N*k < 2^31.  Outside them: MOGA_ERR_UNSUPPORTED.
 */
#ifndef MOGA_H_
#define MOGA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MOGA_OK = 0,
  MOGA_ERR_INVALID_ARG = 1, /* null / misaligned pointer, non-positive size, bad enum   */
  MOGA_ERR_UNSUPPORTED = 2, /* valid request outside the limits above                   */
  MOGA_ERR_WORKSPACE = 3,   /* ws is NULL or smaller than the entry point requires      */
  MOGA_ERR_CUDA = 4,        /* a CUDA runtime/driver call or a launch failed            */
  MOGA_ERR_TIMEOUT = 5,     /* a bounded device-side wait gave up (see status word)     */
  MOGA_ERR_INTERNAL = 6     /* device-side consistency check failed (e.g. gid range)    */
} moga_status;

typedef enum { MOGA_F32 = 0, MOGA_BF16 = 1 } moga_dtype;

typedef enum {
  MOGA_GATE_SOFTMAX_ALL = 0, /* Eq. 3-5: gate = softmax over all M logits, at the pick  */
  MOGA_GATE_SOFTMAX_TOPK = 1 /* gate = softmax over the k selected logits               */
} moga_gate_mode;

typedef enum {
  MOGA_ROUTE_AUTO = 0, /* bf16 X and a workspace: tensor-core router (fp32 weights as three
                          bf16 parts, exact products, fp32 accumulation); otherwise fp32 ALUs */
  MOGA_ROUTE_ALU = 1   /* always the fp32-ALU router kernel                                 */
} moga_route_mode;

typedef struct {
  int32_t B, N, H, C, D, M, k;
  int32_t dtype;     /* moga_dtype of X, Q, K, V, O and the permuted buffers            */
  int32_t gate_mode; /* moga_gate_mode                                                  */
  float scale;       /* softmax scale of Eq. 1, e.g. 1/sqrt(D); finite, >= 0; never inferred */
  int64_t q_stride_b, q_stride_h, q_stride_n; /* element strides of Q, K, V and O       */
  int32_t route_mode; /* moga_route_mode                                                 */
  int32_t reserved;   /* set to 0                                                        */
} moga_shape;

/* Host-only helpers: no CUDA call is made. */

/* Bytes of `ws` moga_forward needs for this shape (0 if the shape is invalid). */
size_t moga_workspace_bytes(const moga_shape* s);
/* Bytes of `ws` the stage entry points (route, permute, group_attn) need. */
size_t moga_scratch_bytes(const moga_shape* s);
const char* moga_status_string(moga_status st);

/*
 * Router, Eq. 2-4: r = X W_r (+ bias) accumulated in fp32, the k largest logits
 * per token (ties to the lower group index), and their gates (gate_mode).
 * Writes gid, gate and, if non-NULL, logits.
 * Two kernels compute the same thing to fp32 rounding.  The fp32-ALU kernel needs no
 * workspace (ws may be NULL) and serves fp32 X.  For bf16 X, when ws holds at least
 * moga_scratch_bytes and route_mode is MOGA_ROUTE_AUTO, the tensor-core kernel runs: it
 * writes each fp32 weight as the sum of three bf16 numbers (all 24 mantissa bits), so
 * every product with a bf16 feature is exact, and accumulates in fp32.  That call resets
 * and may set the device status word of ws (see moga_last_device_status).
 */
moga_status moga_route(const moga_shape* s, const void* X, const float* Wr, const float* bias,
                       int32_t* gid, float* gate, float* logits, void* ws, size_t ws_bytes,
                       void* stream);

/*
 * Group-balancing statistics of Eq. 6-8 from a routing result (gid, gate as written by
 * moga_route), per batch item b: F[b,i] = (assignments to group i) / N (Eq. 7),
 * P[b,i] = (1/N) * sum of the gates of those assignments (Eq. 8: the routing probability
 * of the chosen group, summed over the tokens routed to i only) and
 * loss[b] = alpha * M * sum_i F[b,i] P[b,i] (Eq. 6).  The paper states them for top-1;
 * with k > 1 every (token, slot) assignment counts once.  F, P: float [B, M]; loss: float
 * [B]; device pointers.  Sums are taken in a fixed order (fp32 inside a block of 4,096
 * assignments, fp64 across blocks), so results are reproducible bit for bit.
 * ws: at least moga_scratch_bytes.  N = 0 is MOGA_ERR_INVALID_ARG.
 */
moga_status moga_balance_stats(const moga_shape* s, const int32_t* gid, const float* gate, float alpha,
                               float* F, float* P, float* loss, void* ws, size_t ws_bytes, void* stream);

/*
 * "permute" of Alg. 1 line 2.  Stable counting sort of the N*k assignments of each
 * batch item by group (ascending token index inside a group): writes perm, inv,
 * offsets.  If Qp, Kp and Vp are all non-NULL the rows of Q, K, V are gathered
 * into sorted order as well; all three NULL computes the indices only (Q, K, V may
 * then be NULL).  ws: at least moga_scratch_bytes.  A gid outside [0, M) raises
 * MOGA_ERR_INTERNAL in the device status word and is clamped.
 */
moga_status moga_permute(const moga_shape* s, const int32_t* gid, const void* Q, const void* K,
                         const void* V, int32_t* perm, int32_t* inv, int32_t* offsets, void* Qp,
                         void* Kp, void* Vp, void* ws, size_t ws_bytes, void* stream);

/*
 * Group sort without a caller workspace (the paper has no counterpart: this entry
 * point exists for the way the library is hosted, not for the method).
 *
 * It computes exactly what moga_permute computes when Qp, Kp and Vp are NULL --
 * perm, inv and offsets from gid -- but keeps its scratch (a 256-byte status header
 * and B * ceil(N*k / 4096) * M int32 block counters) in a 1 MiB device array that is
 * part of the library image, so the call performs no device allocation of any kind.
 * It is meant for hosts that cannot allocate when they need the sort: code running
 * inside another framework's execution step whose pool already owns the GPU's
 * memory, or a service whose device-memory budget was fixed at start-up.
 *
 *  - Shapes whose counters do not fit the array return MOGA_ERR_WORKSPACE and launch
 *    nothing (all of this library's documented workloads fit with room to spare).
 *  - Every GPU that loads the library holds the 1 MiB until the process exits.
 *  - The first call on each device looks the array's address up for that device;
 *    make that first call outside any stream capture.
 *  - All calls on a device share the array.  Each call clears the status header it
 *    needs and overwrites the counters, so consecutive calls on one stream are
 *    independent, but two calls that overlap on the GPU (different streams) race:
 *    serialise them.
 *  - status_out, if non-NULL, is a device pointer to two uint32 (8-byte aligned) that
 *    receives {status, detail} as moga_last_device_status would report them, e.g.
 *    MOGA_ERR_INTERNAL for a gid outside [0, M) (which is clamped).
 *  - N = 0 is valid as everywhere else: offsets are set to zero, gid / perm / inv may be
 *    NULL, the array is not touched.
 */
moga_status moga_sort_static(const moga_shape* s, const int32_t* gid, int32_t* perm, int32_t* inv,
                             int32_t* offsets, uint32_t* status_out, void* stream);

/*
 * Alg. 1 line 3 / Eq. 1 inside each group: for every (b, h, g),
 * Op_g = softmax(Qp_g Kp_g^T * scale) Vp_g, non-causal, no mask but the group
 * boundary.  bf16 runs on tcgen05 tensor cores (fp32 accumulate and softmax);
 * fp32 runs on the fp32 ALUs.  lse may be NULL.  ws: at least moga_scratch_bytes.
 * An empty group does no work; a 1-token group returns its own V row.
 * scale = 0 gives uniform weights (the group mean of V).  Groups are independent for any K:
 * scores against rows of a neighbouring group that share a 128-key tile are masked before they
 * are used.  The bf16 kernel does load such neighbouring V rows and multiplies them by an
 * exact-zero weight, so V must be finite (0 x inf is NaN): a non-finite V row can reach the
 * rows of the group stored just before it.  The fp32 kernel never loads a foreign row.
 */
moga_status moga_group_attn(const moga_shape* s, const void* Qp, const void* Kp, const void* Vp,
                            const int32_t* offsets, void* Op, float* lse, void* ws,
                            size_t ws_bytes, void* stream);

/*
 * ---- Static groups: Sec. 3.2, "Spatial-Temporal Group Attention" -----------------------
 * A token's visual-attention output is the mean of three group attentions: the routed one
 * above and two with fixed groups (spatial window x run of frames inside a shot, and one
 * group per latent frame).  The fixed groups are the same for every batch item and head,
 * and a group's key/value set may be larger than its query set (boundary groups also see
 * one latent frame of the adjacent shot).
 */

/*
 * Host only, no CUDA call: the group lists of the spatial-temporal branch for a latent
 * video of F frames of Hh x Ww tokens (token index (f*Hh + y)*Ww + x), wh x ww spatial
 * windows (window of (y, x) = (y*wh/Hh, x*ww/Ww)), shots starting at the n_shots frames
 * shot_starts[] (ascending, shot_starts[0] = 0), runs of at most tg frames inside a shot.
 * Group order: shot, run, window.  Queries of a group: its own tokens, ascending.  Keys:
 * with augment != 0 the same window of the previous shot's last frame (first run of a shot)
 * and of the next shot's first frame (last run of a shot) are added before / after them.
 * All pointers are HOST pointers and may be NULL (sizes only): q_idx [N] token at each
 * query position, q_inv [N] query position of each token, q_offsets / kv_offsets [G+1],
 * kv_idx [Tkv]; *G_out and *Tkv_out receive the counts (N = F*Hh*Ww, Tkv <= 3*N: size
 * kv_idx from a first call with NULL lists).
 */
moga_status moga_stga_build(int32_t F, int32_t Hh, int32_t Ww, int32_t wh, int32_t ww,
                            const int32_t* shot_starts, int32_t n_shots, int32_t tg, int32_t augment,
                            int32_t* q_idx, int32_t* q_inv, int32_t* q_offsets, int32_t* kv_idx,
                            int32_t* kv_offsets, int32_t* G_out, int32_t* Tkv_out);

/*
 * dst[b,h,p,:] = src[b,h,idx[p],:] for p < L: rows of src (strides from the shape, N rows)
 * listed by the device array idx [L], shared by all batch items and heads, into the
 * contiguous dst [B, H, L, D].  16-byte vector copies; no workspace.
 */
moga_status moga_gather_rows(const moga_shape* s, const int32_t* idx, int32_t L, const void* src, void* dst,
                             void* stream);

/* Bytes of ws moga_static_group_attn needs for G groups (host only; 0 if the shape is invalid). */
size_t moga_static_scratch_bytes(const moga_shape* s, int32_t G);

/*
 * Eq. 1 inside caller-given groups: query rows [q_offsets[g], q_offsets[g+1]) of
 * Qs [B, H, Tq, D] attend to key/value rows [kv_offsets[g], kv_offsets[g+1]) of
 * Ks, Vs [B, H, Tkv, D]; the result goes to the same rows of Os [B, H, Tq, D]
 * (lse [B, H, Tq] optional).  q_offsets, kv_offsets: device int32 [G+1], one list for all
 * batch items and heads.  Same kernels as moga_group_attn (which is the case Tq = Tkv,
 * q_offsets = kv_offsets per batch item).  Rows of a group without keys, and rows outside
 * every group, are left untouched.  M and k of the shape are not used.
 */
moga_status moga_static_group_attn(const moga_shape* s, int32_t G, int32_t Tq, int32_t Tkv, const void* Qs,
                                   const void* Ks, const void* Vs, const int32_t* q_offsets,
                                   const int32_t* kv_offsets, void* Os, float* lse, void* ws,
                                   size_t ws_bytes, void* stream);

/*
 * The mean of the three branch outputs (Sec. 3.2): O[b,h,n,:] = (A[b,h,n,:] +
 * Bs[b,h,inv_b[n],:] + C[b,h,n,:]) / 3, summed in fp32 and rounded once.  A and O use the
 * shape's strides (token order); Bs [B, H, N, D] is contiguous in the spatial-temporal
 * branch's query order, inv_b [N] (device, NULL = identity) gives each token's position in
 * it; C [B, H, N, D] is contiguous in token order (per-frame groups keep token order).
 */
moga_status moga_mean3(const moga_shape* s, const void* A, const void* Bs, const int32_t* inv_b,
                       const void* C, void* O, void* stream);

/*
 * The whole visual-attention block of Sec. 3.2 in one call: the routed forward (moga_forward),
 * the spatial-temporal static branch (gathers by the lists + moga_static_group_attn), the
 * per-frame branch (one group per latent frame of tokens_per_frame consecutive tokens) and
 * their mean into O.  `lists` carries DEVICE copies of what moga_stga_build produced, plus
 * the frame count (F * tokens_per_frame must equal N).  Q, K, V, O contiguous [B, H, N, D]
 * (non-zero strides: MOGA_ERR_UNSUPPORTED).  ws: at least moga_visual_workspace_bytes; it
 * holds the forward's workspace, the three branch outputs and the gathered Q / K / V of the
 * spatial-temporal branch.  The device status word of the routed branch is at the start of
 * ws (moga_last_device_status(ws, ...)).
 */
typedef struct {
  int32_t G, Tkv;                 /* groups and key rows of the spatial-temporal branch        */
  int32_t F, tokens_per_frame;    /* latent frames and tokens per frame (per-frame branch)     */
  const int32_t *q_idx, *q_inv, *q_offsets, *kv_idx, *kv_offsets;   /* device arrays           */
} moga_static_lists;
size_t moga_visual_workspace_bytes(const moga_shape* s, const moga_static_lists* lists);
moga_status moga_visual_forward(const moga_shape* s, const void* X, const float* Wr, const float* bias,
                                const void* Q, const void* K, const void* V, void* O,
                                const moga_static_lists* lists, void* ws, size_t ws_bytes, void* stream);

/*
 * "repermute" of Alg. 1 line 4 with the gate of Eq. 5:
 * O[b,h,n,:] = sum_j gate[b,n,j] * Op[b,h,inv[b,n,j],:], summed in fp32 in slot
 * order and rounded once.  No workspace.
 */
moga_status moga_unpermute(const moga_shape* s, const void* Op, const int32_t* inv,
                           const float* gate, void* O, void* stream);

/*
 * The whole forward: route -> permute -> group_attn -> unpermute with the
 * intermediates in ws (at least moga_workspace_bytes).  gid_out, gate_out,
 * perm_out, offsets_out may each be NULL; when given they receive copies of the
 * routing results.
 */
moga_status moga_forward(const moga_shape* s, const void* X, const float* Wr, const float* bias,
                         const void* Q, const void* K, const void* V, void* O, int32_t* gid_out,
                         float* gate_out, int32_t* perm_out, int32_t* offsets_out, void* ws,
                         size_t ws_bytes, void* stream);

/*
 * The same forward from a routing that is already known (Alg. 1 lines 2-4 and the gate of
 * Eq. 5, without the router of Eq. 2-4): gid and gate [B, N, k] as moga_route writes them.
 * This is the call of a rank that holds only some heads of Q, K, V (shape.H = its heads) and
 * received the routing of the whole sequence from the ranks that hold the token features
 * (Sec. 3.2, last paragraph: routing is computed per token before the model's sequence-to-head
 * exchange and its results are gathered).  Same kernels, workspace (moga_workspace_bytes) and
 * results as moga_forward given the same routing.  perm_out / offsets_out may be NULL.
 */
moga_status moga_forward_routed(const moga_shape* s, const int32_t* gid, const float* gate, const void* Q,
                                const void* K, const void* V, void* O, int32_t* perm_out, int32_t* offsets_out,
                                void* ws, size_t ws_bytes, void* stream);

/*
 * The whole forward from HOST buffers (the call for a caller whose activations live in host
 * memory).  X, Wr, bias, Q, K, V, O, gid_out, gate_out are HOST pointers (page-locked memory
 * is needed for the copies to overlap; pageable memory works but serialises); Q, K, V, O are
 * contiguous [B, H, N, D] (strides in the shape must be zero).  `arena` is device memory of
 * at least moga_forward_host_bytes(s, heads_per_chunk), 256-byte aligned: it holds X, the
 * routing results, two staging sets of heads_per_chunk heads of Q/K/V and of O, and one
 * permuted chunk.  One internal stream copies X and then Q/K/V chunk by chunk, `stream`
 * routes, sorts and runs gather + group attention (+ gated inverse permutation) on each
 * chunk as its inputs land, a second internal stream returns each chunk of O; `stream`
 * finally waits for the last copy, so synchronising it means O is on the host.  Results are
 * bit-identical to moga_forward.  The two streams and a fixed pool of events are created on
 * the first call on each device (no memory is allocated); calls on one device must not
 * overlap (they share those events).  At most 64 chunks.  The device status word is at the
 * start of `arena` (moga_last_device_status(arena, ...)).
 */
size_t moga_forward_host_bytes(const moga_shape* s, int32_t heads_per_chunk);
moga_status moga_forward_host(const moga_shape* s, const void* X, const float* Wr, const float* bias,
                              const void* Q, const void* K, const void* V, void* O, int32_t* gid_out,
                              float* gate_out, void* arena, size_t arena_bytes, int32_t heads_per_chunk,
                              void* stream);

/*
 * Synchronises `stream`, reads the device status word kept at the start of ws and
 * clears it.  Every permute / group_attn / forward call resets the word when it
 * starts, so the result describes the most recent such call on this ws: MOGA_OK,
 * or the first problem a kernel recorded (MOGA_ERR_TIMEOUT, MOGA_ERR_INTERNAL).
 * `detail`, if non-NULL, receives a kernel-specific word saying where.
 */
moga_status moga_last_device_status(void* ws, void* stream, uint32_t* detail);

/*
 * Backward of the routed group attention (the paper states no backward pass: this is the chain
 * rule applied to Eq. 1 inside each group and the gate of Eq. 5; the routing decision carries no
 * gradient).  bf16 with d_head = 128 and fp32 with d_head 64 or 128; bf16 with d_head = 64 returns
 * MOGA_ERR_UNSUPPORTED.
 * Saved from a forward made of the stage calls, all in sorted order: Qp, Kp, Vp (moga_permute),
 * Op and lse (moga_group_attn), [B, H, T, D] / [B, H, T]; the routing: gate [B, N, k] (moga_route),
 * perm [B, T], inv [B, N, k], offsets [B, M+1] (moga_permute).  dO: the gradient with respect to the
 * forward's output O, [B, H, N, D] with the shape's strides.
 * Outputs: dQ, dK, dV [B, H, N, D] (same strides; a token routed to k groups receives the sum of
 * its k contributions) and dgate [B, N, k] fp32 (the derivative with respect to each gate, summed
 * over heads and channels: what the router's gate needs for its own backward).
 * Kernels: one pass that scales and gathers dO and forms delta = <dO, o>, then two tensor-core
 * launches (dQ; dK and dV) that recompute the softmax weights from lse, then the inverse
 * permutation.  P, dS and the sorted-order gradients are rounded to bf16, accumulation is fp32.
 * fp32 tensors take the same three steps on the fp32 ALUs, nothing rounded below fp32.
 * ws: moga_backward_workspace_bytes(s), 256-byte aligned; the device status word is at its start.
 */
size_t moga_backward_workspace_bytes(const moga_shape* s);
moga_status moga_backward(const moga_shape* s, const void* Qp, const void* Kp, const void* Vp, const void* Op,
                          const float* lse, const float* gate, const int32_t* perm, const int32_t* inv,
                          const int32_t* offsets, const void* dO, void* dQ, void* dK, void* dV, float* dgate,
                          void* ws, size_t ws_bytes, void* stream);

/*
 * Backward of the router (the paper states no backward pass: the chain rule on Eq. 2-3 and the
 * gate of Eq. 5; the routing decision gid is a fixed integer choice).  Inputs: X [B, N, C] and W_r
 * [C, M] as in moga_route, the logits [B, N, M] that moga_route wrote (its optional output), gid
 * [B, N, k], and dgate [B, N, k] (from moga_backward); gate_mode as in the forward.
 * Outputs: dWr [C, M] fp32, dbias [M] fp32 (nullable), dX [B, N, C] in the type of X (nullable: the
 * gradient that reaches the token features through the router alone).  Deterministic: the sums over
 * tokens are formed in a fixed order (per-slab partial sums, then a reduction), no atomics.
 * fp32 ALUs throughout.  ws: moga_route_backward_workspace_bytes(s), 256-byte aligned.
 */
size_t moga_route_backward_workspace_bytes(const moga_shape* s);
moga_status moga_route_backward(const moga_shape* s, const void* X, const float* Wr, const float* logits,
                                const int32_t* gid, const float* dgate, void* dX, float* dWr, float* dbias, void* ws,
                                size_t ws_bytes, void* stream);

/*
 * Choice of the bf16 group-attention kernel (the paper has no counterpart: a tuning and test
 * switch).  Three kernels compute Eq. 1 inside the groups on the tensor cores; all give a block
 * of 256 query rows (two 128-row tiles) to one work item.
 * MOGA_ATTN_AUTO (default): for d_head = 128, routed groups and a storing epilogue, the kernel
 * with two softmax threads per query row, which keeps the first key tile's row maximum as the
 * reference and hands any item whose scores outgrow it by 2^40 to the exact kernel; every other
 * launch runs MOGA_ATTN_SINGLE.
 * MOGA_ATTN_SINGLE: one SM per item, one softmax thread per row, the reference raised inside
 * the row when needed (the exact kernel).
 * MOGA_ATTN_PAIR: a pair of SMs per item that issue every tensor-core instruction together and
 * each stage half of every K/V tile (d_head = 128, routed launches only); correct on every shape
 * but measured slower (see the kernel selection comment in csrc/attn_bf16.cu); kept as an option.
 * Process-wide, not thread-safe against concurrent launches; returns MOGA_ERR_INVALID_ARG for
 * another value.
 */
typedef enum { MOGA_ATTN_AUTO = 0, MOGA_ATTN_SINGLE = 1, MOGA_ATTN_PAIR = 2 } moga_attn_kernel;
moga_status moga_set_attn_kernel(int32_t mode);

/*
 * Top-2 output path of moga_forward / moga_forward_routed for bf16 (the paper has no
 * counterpart: a tuning and test switch).  on != 0: the attention epilogue rounds
 * gate * row to bf16 and adds it into a zeroed O in token order (Eq. 5's sum over the two
 * assignments as two commutative bf16 additions: the result does not depend on their order, so
 * runs stay bit-reproducible); no permuted output is written and moga_unpermute is not run.
 * on == 0 (default): the staged path (attention writes the permuted output, moga_unpermute sums
 * in fp32 with one rounding).  The two differ in the last bit and take the same time on the
 * top-2 workloads measured.  O with custom strides, k > 2 and fp32
 * always take the staged path.  Process-wide.
 */
moga_status moga_set_fused_topk(int32_t on);

/*
 * Self-test of the time-out path (the paper has no counterpart: it is a diagnostic).
 * Every wait inside the tensor-core kernels is bounded; when one runs out the kernel writes
 * MOGA_ERR_TIMEOUT and a detail word to the status header and returns normally.  This call
 * runs that same wait routine to its limit in a one-block kernel of its own, on a barrier
 * nothing signals, so a deployment can check that a stuck wait is reported rather than hung.
 * ws: device memory, >= 256 bytes, 256-byte aligned (any workspace of this library will do;
 * its status header is reset).  limit_ns: the bound of the wait, 1 .. 100,000,000 (100 ms),
 * else MOGA_ERR_INVALID_ARG.  Asynchronous on `stream`.  Afterwards moga_last_device_status(ws)
 * returns MOGA_ERR_TIMEOUT with detail = 0x7e000000 | (block << 8) | barrier index (both 0
 * here); words 2-3 of the header hold the nanoseconds the wait lasted and word 4 how the
 * second warp left (1: released by the abort flag).
 */
moga_status moga_selftest_wait_timeout(void* ws, size_t ws_bytes, uint64_t limit_ns, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MOGA_H_ */
