/*
 * usv.h -- C ABI of the USV sparsified-attention hot path for NVIDIA B200 (sm_100a).
 *
 * The library implements, as hand-written CUDA kernels, one sparsified self-attention block of
 * a video diffusion transformer as the USV paper describes it (Fig. 2 right; Sec. 3.2-3.3):
 *
 *     token merge -> block pooling + scores -> top-k key-block selection
 *                 -> block-sparse attention -> token unmerge
 *
 * Conventions that hold for every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller, 16-byte aligned.  Arguments
 *     documented as HOST are ordinary host pointers read before the call returns.
 *   - Nothing is allocated, nothing is freed, the stream is never synchronised: kernels are
 *     enqueued on `stream` (a cudaStream_t passed as void*; NULL = the default stream).
 *     Scratch memory comes from the caller (`ws`, `ws_bytes`); the matching *_workspace()
 *     function gives the size needed.  The workspace may be reused by a later call on the same
 *     stream; concurrent calls on different streams need different workspaces.  The first
 *     USV_WS_HEADER bytes of every workspace are a header whose first word is the device status
 *     word: zero it once after allocating the buffer (usv_workspace_init); the entry points only
 *     ever OR into it, so one usv_workspace_status after many calls sees a wait that gave up in
 *     any of them.
 *   - Every function returns a usv_status.  Arguments are validated on the host before anything
 *     is launched; on a non-zero status nothing has been enqueued (USV_ERR_CUDA excepted, which
 *     reports a failed launch).  usv_last_error() gives a human-readable reason for the calling
 *     thread's last failure.
 *   - bf16 = the upper 16 bits of an IEEE binary32 value, round-to-nearest-even on output.
 *   - Attention blocks are runs of USV_BLOCK = 64 consecutive tokens in the caller's token
 *     order.  A sequence of N tokens has NB = ceil(N/64) blocks; the last one may be partial.
 *     Rows at or beyond N are never read and never written.
 *   - 4-d views [B,H,N,d] are described by element strides (sb, sh, sn) with the d axis
 *     contiguous; strides must be multiples of 8 elements (16 bytes).
 */
#ifndef USV_H_
#define USV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define USV_BLOCK 64
#define USV_MAX_HEADS 128
#define USV_WS_HEADER 256

typedef enum {
    USV_OK = 0,
    USV_ERR_INVALID_ARG = 1, /* null pointer, bad size, k or r out of range ... */
    USV_ERR_UNSUPPORTED = 2, /* valid request outside what the kernels cover (d, alignment) */
    USV_ERR_WORKSPACE = 3,   /* ws_bytes smaller than *_workspace() */
    USV_ERR_CUDA = 4,        /* a CUDA runtime/driver call or a launch failed */
    USV_ERR_TIMEOUT = 5      /* a bounded device-side wait gave up (see usv_workspace_status) */
} usv_status;

/* Element strides of a [B,H,N,d] view whose d axis is contiguous. */
typedef struct {
    int64_t sb, sh, sn;
} usv_strides;

const char* usv_status_string(int status);
const char* usv_last_error(void);
/* Compiled-in build tag, e.g. "usv-b200 sm_100a". */
const char* usv_build_info(void);
/* Kernels this library has launched in the calling process so far (all threads, all devices;
 * memsets and copies are not counted). */
unsigned long long usv_kernel_launches(void);

/* ------------------------------------------------------------------------------------------
 * Coarse stage of "top-k cube selection" (Fig. 2 caption; the paper names the step and leaves
 * the score open).  Reading implemented: per 64-token block the mean of the valid query rows
 * and of the valid key rows (fp32), then
 *     scores[b,h,I,J] = < mean_q[b,h,I,:], mean_k[b,h,J,:] > / sqrt(d)          (fp32).
 *
 * q: bf16 view [B,H,Nq,d], k: bf16 view [B,H,Nk,d]; d in {64,128}.
 * scores: fp32 [B,H,NBq,NBk] contiguous (written).  ws: pooled means (and, at d = 128, the bf16
 * operand planes of the tensor-core product, which is accumulated in fp32 from a three-way split
 * of every fp32 mean and is fp32-accurate), see *_workspace().
 */
size_t usv_block_scores_workspace(int B, int H, int Nq, int Nk, int d);
int usv_block_scores(int B, int H, int Nq, int Nk, int d, const void* q, const usv_strides* sq,
                     const void* k, const usv_strides* sk, float* scores, void* ws,
                     size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------------------------
 * usv_block_scores for callers that cannot hand over scratch memory.  (The paper has no
 * counterpart: this is a packaging variant of the entry point above.  Same definition and fp32-grade
 * results, but not bit-identical at d = 128: this variant takes the scores from the fp32 CUDA-core
 * kernel, usv_block_scores from the three-plane tensor-core product; the two agree to about 2e-6
 * relative, so a top-k taken on a near-tie may resolve differently.)
 *
 * Who needs it: code that runs where device allocation is off limits -- inside a region that
 * must not call cudaMalloc (an allocator-frozen section of a host framework, a plugin
 * that is only given tensors, a real-time loop with a fixed memory budget) and that has no
 * spare buffer to lend as `ws`.  Here the pooled block means live in a fixed array that is part
 * of the library image: USV_NOALLOC_SCRATCH_BYTES of device memory are reserved on every GPU
 * that loads the library, for as long as it stays loaded.
 *
 *   - Same arguments and results as usv_block_scores minus ws/ws_bytes.  Nothing is allocated
 *     or freed, by the CUDA runtime or any other library.
 *   - The request is rejected (USV_ERR_WORKSPACE, nothing launched) when
 *     the pooled means of q and k (B*H*(NBq + NBk)*d fp32 values, each tensor rounded up to
 *     256 bytes) exceed USV_NOALLOC_SCRATCH_BYTES.
 *   - The first call on each device looks up the array's device address (a one-off, synchronous
 *     runtime query with that device current; where the runtime loads device code lazily, this
 *     query or the first launch is also what brings the library's device image, the array
 *     included, onto the GPU).  Make that first call before entering the region in which nothing
 *     may be allocated, and before starting any stream capture on the device.
 *   - All calls on a device share the one array.  It keeps whatever the previous call left; every
 *     element a call reads is first written by that same call, so nothing needs clearing.  Two
 *     calls whose kernels overlap on the GPU (different streams, no ordering) race on it:
 *     serialise them.
 */
#define USV_NOALLOC_SCRATCH_BYTES (8u << 20)
int usv_block_scores_noalloc(int B, int H, int Nq, int Nk, int d, const void* q,
                             const usv_strides* sq, const void* k, const usv_strides* sk,
                             float* scores, void* stream);

/* ------------------------------------------------------------------------------------------
 * Top-k key-block selection (Fig. 2 caption, "top-k cube selection").  For each (b,h,I) the
 * k_per_head[h] key blocks with the largest score are kept; equal scores are resolved in favour
 * of the lower block index.  The kept indices are written in ascending order; the remainder of
 * the kmax-wide row is filled with -1.
 *
 * scores: fp32 [B,H,NBq,NBk].  k_per_head: HOST int32[H], each in [1,NBk].  kmax >= max k.
 * sel: int32 [B,H,NBq,kmax] (written).  NBk <= 8192.
 */
int usv_select_blocks(int B, int H, int NBq, int NBk, const float* scores,
                      const int32_t* k_per_head, int kmax, int32_t* sel, void* stream);

/* ------------------------------------------------------------------------------------------
 * Block-sparse attention forward (Sec. 3.2, Eq. 5 with a block-structured mask):
 *     O_i = sum_j softmax_j( scale * <q_i,k_j> ) v_j ,  j over the valid keys of the key blocks
 *     listed in sel[b,h,block(i),0..k_per_head[h]).
 * bf16 operands on the tensor cores, fp32 online softmax and accumulation, bf16 output.
 *
 * q,k,v: bf16 views [B,H,N,d] (self-attention: one N); d in {64,128}.
 * sel: int32 [B,H,NB,kmax], entries in [0,NB), -1 entries are skipped.
 * k_per_head: HOST int32[H].  o: bf16 view [B,H,N,d] (written, rows < N only).
 * o_f32: optional fp32 [B,H,N,d] contiguous copy of the un-rounded output (NULL to skip).
 * lse: optional fp32 [B,H,N], natural-log of the softmax denominator (NULL to skip).
 * scale: logit scale; 0 selects 1/sqrt(d).
 * impl: 0 = default kernel, 1 = legacy mma.sync kernel (kept as an on-device cross-check).
 *
 * The default kernel (d = 128) computes two neighbouring query blocks together over the union of
 * their key-block lists and gives a key block that only one of them selected zero weight for
 * the other.  Results equal the per-block definition for finite inputs.  A NaN or infinity in K
 * or V inside a block that one query block of a pair selected can also reach the output rows of
 * its partner (0 * inf); blocks that neither selected are never read.  impl 1 keeps query blocks
 * fully separate.  Sequences of more than 4096 key blocks (262 144 tokens), and d = 64, run the
 * impl 1 kernel whatever impl says.
 */
size_t usv_sparse_attn_workspace(int B, int H, int N, int d, int kmax);
int usv_sparse_attn_fwd(int B, int H, int N, int d, const void* q, const usv_strides* sq,
                        const void* k, const usv_strides* sk, const void* v,
                        const usv_strides* sv, const int32_t* sel, const int32_t* k_per_head,
                        int kmax, void* o, const usv_strides* so, float* o_f32, float* lse,
                        float scale, int impl, void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------------------------
 * Attention with the unmerge of Eq. 15 folded into its epilogue (Sec. 3.3: after attention every
 * merged row is sent back to all the original positions it stands for).  Same computation as
 * usv_sparse_attn_fwd on the merged sequence of N tokens, but every output row is stored straight
 * to the original tokens that read it back, y[b, n, h*d ... h*d+d) for every n with pos[b,n] = row,
 * so that no separate usv_token_unmerge pass (a read of the merged output and a launch) is needed.
 *
 * usv_unmerge_map builds the inverse of pos once per merge plan (any pos works, e.g. a cube
 * permutation): unmerge_off int32 [B, Nm+1] (offsets), unmerge_idx int32 [B, N] (original tokens
 * grouped by merged row).  ws: usv_unmerge_map_workspace(B, Nm) bytes.
 *
 * usv_sparse_attn_fwd_unmerge: arguments as usv_sparse_attn_fwd (tcgen05 kernel only: d = 128);
 * N = merged length, N_full = original length, y: bf16 [B, N_full, H*d] contiguous (written: every
 * token whose pos lies in [0, N)).  o is still required: it receives the (normally zero) query
 * blocks that are recomputed exactly before they are copied to y, and is otherwise left
 * undefined.  o_f32 / lse, if given, are written in the merged order as usual.
 */
size_t usv_unmerge_map_workspace(int B, int Nm);
int usv_unmerge_map(int B, int N, int Nm, const int32_t* pos, int32_t* unmerge_off, int32_t* unmerge_idx,
                    void* ws, size_t ws_bytes, void* stream);
int usv_sparse_attn_fwd_unmerge(int B, int H, int N, int d, const void* q, const usv_strides* sq,
                                const void* k, const usv_strides* sk, const void* v,
                                const usv_strides* sv, const int32_t* sel, const int32_t* k_per_head,
                                int kmax, void* o, const usv_strides* so, float* o_f32, float* lse,
                                float scale, void* ws, size_t ws_bytes, int N_full,
                                const int32_t* unmerge_off, const int32_t* unmerge_idx, void* y,
                                void* stream);

/* After usv_sparse_attn_fwd with impl 0: how many query blocks the tcgen05 kernel handed to the
 * exact kernel because their softmax sums left the safe exponent range (normally 0).
 * Synchronises `stream`.  ws is the workspace that call used. */
int usv_sparse_attn_fallbacks(const void* ws, void* stream, int* count);

/* Zeroes the header of a freshly allocated workspace (asynchronous, on `stream`). */
int usv_workspace_init(void* ws, void* stream);

/* Reads the device status word (word 0 of the workspace header) that kernels with bounded waits
 * OR their codes into: the tcgen05 kernels behind usv_block_scores, usv_sparse_attn_fwd,
 * usv_token_merge and usv_attn_entropy.  Synchronises `stream`.  Returns USV_OK, USV_ERR_CUDA, or
 * USV_ERR_TIMEOUT if any call since the last query gave up a wait (its results are then
 * undefined); a reported word is cleared, so the next query starts afresh. */
int usv_workspace_status(void* ws, void* stream);

/* Self-test of the bounded wait (the paper has no counterpart).  Launches one warp that waits,
 * with the same routine the kernels use but a limit of `limit_us` microseconds (1..100000), on a
 * barrier nothing arrives at.  The wait runs out, the warp ORs 0x80000000 into the status word of
 * `ws` and returns: usv_workspace_status(ws) then reports USV_ERR_TIMEOUT and the device context
 * stays usable.  Nothing traps and nothing waits without a limit. */
int usv_selftest_wait_timeout(void* ws, unsigned int limit_us, void* stream);

/* ------------------------------------------------------------------------------------------
 * Token merge (Sec. 3.3, Eq. 6-14).
 *   Partition: token (t,y,x) of the T x Hh x W raster grid is a destination iff
 *   t % st == 0, y % sh == 0 and x % sw == 0 (the first token of its (st,sh,sw) block); every
 *   other token is a source.
 *   Plan (only when metric != NULL): head-averaged unit descriptors of `metric` (Eq. 7-8), best
 *   destination j*(i) and cosine u_i per source over all destinations of the same batch element
 *   (Eq. 9, ties to the lowest j), the r sources with the largest u are merged (Eq. 10-11, ties
 *   to the lowest i).  The plan is written to dst_of / pos.
 *   Apply: destinations become the mean of themselves and their merged sources (Eq. 12-13,
 *   fp32 accumulation, bf16 RNE); output order is [unmerged sources ascending || destinations
 *   ascending] (Eq. 14).
 *
 * x: bf16 [B,N,C] contiguous, N = T*Hh*W, C a multiple of 8.  x_merged: bf16 [B,N-r,C].
 * metric: bf16 [B,N,Hm,dm] contiguous, dm in {64,128}; NULL = reuse the plan already stored in
 *         dst_of/pos (lets one plan merge several tensors).
 * r: number of sources merged per batch element, 0 <= r <= number of sources.
 * dst_of: int32 [B,N], j*(i) for merged sources, -1 for every other token.
 * pos: int32 [B,N], row of the merged sequence each original token reads back from.
 * u_out, jstar_out: optional [B,N] (fp32 / int32): u_i and j*(i) for every source, (NaN,-1) at
 *         destinations.  Only written when metric != NULL.
 */
size_t usv_token_merge_workspace(int B, int N, int C, int Hm, int dm);
int usv_token_merge(int B, int N, int C, const void* x, int Hm, int dm, const void* metric, int T,
                    int Hh, int W, int st, int sh, int sw, int r, void* x_merged, int32_t* dst_of,
                    int32_t* pos, float* u_out, int32_t* jstar_out, void* ws, size_t ws_bytes,
                    void* stream);

/* Token merge with the matching kept local (the closing paragraphs of Sec. 3.3 describe sources
 * and destinations as confined to local 3D blocks, which Eq. 9 as printed does not): j*(i) is
 * the best destination among the partition blocks within (wt, wh, ww) blocks of the source's
 * own block along (t, y, x); window (0,0,0) merges every source into the destination of its own
 * block, a window that covers the grid gives usv_token_merge.  Everything else, the workspace
 * size included, is as for usv_token_merge.  wt, wh, ww >= 0 (else USV_ERR_INVALID_ARG).
 */
int usv_token_merge_local(int B, int N, int C, const void* x, int Hm, int dm, const void* metric,
                          int T, int Hh, int W, int st, int sh, int sw, int wt, int wh, int ww,
                          int r, void* x_merged, int32_t* dst_of, int32_t* pos, float* u_out,
                          int32_t* jstar_out, void* ws, size_t ws_bytes, void* stream);

/* A plan applied to several tensors (Q, K and V of one layer, Fig. 2; hidden states): the lists of
 * merged sources per destination that the merge needs can be built once and kept by the caller,
 * so that every further merge with that plan is the streaming kernel alone (Eq. 12-14).
 *   usv_merge_plan_cache: from dst_of / pos of a plan (as written by usv_token_merge) into `cache`
 *     (device, 16-byte aligned, usv_merge_plan_cache_bytes(B, N) bytes, owned by the caller).
 *   usv_token_merge_apply: x_merged = merge(x) with the cached plan; same result as
 *     usv_token_merge(metric = NULL).  `cache` is not const: a destination with more than 32 merged
 *     sources has its list sorted in place on first use.
 * Grid, partition and r must be those the plan was made with.
 */
size_t usv_merge_plan_cache_bytes(int B, int N);
int usv_merge_plan_cache(int B, int N, int T, int Hh, int W, int st, int sh, int sw, int r,
                         const int32_t* dst_of, const int32_t* pos, void* cache, size_t cache_bytes,
                         void* stream);
int usv_token_merge_apply(int B, int N, int C, const void* x, int T, int Hh, int W, int st, int sh,
                          int sw, int r, void* cache, void* x_merged, void* stream);

/* ------------------------------------------------------------------------------------------
 * Token unmerge (Sec. 3.3, Eq. 15): y[b,n,:] = y_merged[b,pos[b,n],:].
 * y_merged: bf16 [B,Nm,C]; pos: int32 [B,N] with entries in [0,Nm); y: bf16 [B,N,C] (written).
 */
int usv_token_unmerge(int B, int N, int Nm, int C, const void* y_merged, const int32_t* pos,
                      void* y, void* stream);

/* ------------------------------------------------------------------------------------------
 * Entropy-aware scheduler inputs (Sec. 3.4).
 *
 * usv_attn_entropy: key marginal of the block-masked attention weights averaged over heads and
 * queries (Eq. 16), abar[b,j] = 1/(H N) sum_h sum_i A(h,i,j), and its entropy normalised by log N
 * (Eq. 17), h[b] in [0,1].  A is recomputed as exp(scale <q_i,k_j> - lse_i) from the
 * log-sum-exp that usv_sparse_attn_fwd wrote for the same q, k, sel.
 *
 * q,k: bf16 views [B,H,N,d], d in {64,128}.  sel / k_per_head (HOST) / kmax / scale: as passed to
 * usv_sparse_attn_fwd.  lse: fp32 [B,H,N] from that call.  key_marginal: fp32 [B,N] (written;
 * sums to 1 per batch element up to rounding).  entropy: fp32 [B] (written).  The sums use fp32
 * atomic adds: results are reproducible to rounding, not bit for bit.
 * ws: optional device pointer to a workspace header (USV_WS_HEADER bytes are enough) whose status
 * word receives the code of a bounded wait that gave up; NULL = not reported.
 */
int usv_attn_entropy(int B, int H, int N, int d, const void* q, const usv_strides* sq,
                     const void* k, const usv_strides* sk, const int32_t* sel,
                     const int32_t* k_per_head, int kmax, const float* lse, float scale,
                     float* key_marginal, float* entropy, void* ws, void* stream);

/* Entropy-aware allocation over the L layers of one step (Eq. 18-19), plain host arithmetic:
 *     w_l = (1 - h_l)^gamma ,   rho_l = clip(rho_min, rho_max, rho_bar * w_l / mean_l'(w_l')).
 * entropy, rho: HOST arrays of L floats; gamma >= 1; every h_l in [0,1].  If every w_l is zero
 * each layer keeps rho_bar (clipped).  Serves the attention and the token ratio alike.
 */
int usv_allocate_sparsity(int L, const float* entropy, float gamma, float rho_bar, float rho_min,
                          float rho_max, float* rho);

/* ------------------------------------------------------------------------------------------
 * Local 3D cubes (overview figure, Fig. 2: the tokens are grouped into small 3D cubes, and
 * attention inside the own cube runs beside the long-range top-k selection of cubes).
 *
 * usv_cube_order: the token order in which the tokens of one cube are consecutive.  The grid is
 * (T, Hh, W) in raster order, a cube is ct x ch x cw tokens (4 x 4 x 4 makes a cube one 64-token
 * block).  Cubes come in raster order of their cube coordinates, the tokens of a cube in raster
 * order of their offsets inside it; a cube cut by the edge of the grid holds fewer tokens and
 * nothing is padded, so near the edges a 64-token block may straddle cubes.
 *   perm: device int32 [T*Hh*W] (written), perm[p] = raster index of the token at position p.
 *   inv : device int32 [T*Hh*W] or NULL (written), the inverse: inv[perm[p]] = p.
 * To bring a [B,N,C] tensor into cube order call usv_token_unmerge(B, N, N, C, x, perm_b, y) with
 * perm repeated per batch element (y[b,p] = x[b,perm[p]]); the same call with inv takes it back.
 *
 * usv_force_own_block: the local branch as part of the selection.  Sets scores[b,h,I,I] = +inf
 * for I < min(NBq, NBk), in place, so that usv_select_blocks on these scores keeps, for every
 * query block, its own block plus the k_h - 1 best of the others.
 *   scores: device fp32 [B,H,NBq,NBk] (from usv_block_scores; modified).
 * Both return USV_ERR_INVALID_ARG for non-positive sizes or a null pointer; nothing is launched.
 */
int usv_cube_order(int T, int Hh, int W, int ct, int ch, int cw, int32_t* perm, int32_t* inv,
                   void* stream);
int usv_force_own_block(int B, int H, int NBq, int NBk, float* scores, void* stream);

/* ------------------------------------------------------------------------------------------
 * The two-branch form of the same figure (Fig. 2 caption: local cube attention and the long-range
 * top-k attention run apart and their outputs are fused).  The caption does not say how the
 * outputs are fused; the reading implemented weights each branch by its softmax mass, which makes
 * the fused output EQUAL to one attention over the union of the two branches' key sets as long as
 * those sets are disjoint:
 *     o = (e^lse1 o1 + e^lse2 o2) / (e^lse1 + e^lse2),    lse = log(e^lse1 + e^lse2).
 * Recipe: local branch = usv_sparse_attn_fwd with sel[b,h,I,0] = I (k = 1); long-range branch =
 * usv_exclude_own_block on a copy of the scores, usv_select_blocks with k - 1, usv_sparse_attn_fwd;
 * both with lse; then usv_attn_combine.  (After token merging the branches run on the merged
 * sequence and the fused output goes through usv_token_unmerge: "broadcast back to the full grid".)
 *
 * usv_exclude_own_block: scores[b,h,I,I] = -inf for I < min(NBq, NBk), in place, so that
 * usv_select_blocks never keeps a query block's own block (as long as k < NBk).
 *
 * usv_attn_combine: o1, o2: branch outputs, views [B,H,N,d] (element strides, d contiguous) of
 * bf16 (inputs_f32 = 0) or fp32 (inputs_f32 = 1, e.g. the o_f32 outputs of the branches: strides
 * (H*N*d, N*d, d)); lse1, lse2: fp32 [B,H,N] from the branches (-inf or any value with weight 0
 * for a branch without keys: its output is then ignored, NaN included).  o: bf16 view (written);
 * o_f32: optional fp32 [B,H,N,d] contiguous; lse: optional fp32 [B,H,N].  A row both of whose
 * branches are empty gets zeros and lse = -inf.
 */
int usv_exclude_own_block(int B, int H, int NBq, int NBk, float* scores, void* stream);
int usv_attn_combine(int B, int H, int N, int d, const void* o1, const usv_strides* s1,
                     const float* lse1, const void* o2, const usv_strides* s2, const float* lse2,
                     int inputs_f32, void* o, const usv_strides* so, float* o_f32, float* lse,
                     void* stream);

#ifdef __cplusplus
}
#endif
#endif /* USV_H_ */
