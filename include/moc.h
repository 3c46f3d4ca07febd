/*
 * moc.h - C ABI of the Mixture-of-Contexts (MoC) routing + sparse attention library
 * for NVIDIA B200 (sm_100a).
 *
 * One call per step of the per-layer, per-head hot path of "Mixture of Contexts for
 * Long Video Generation" (Sec. 3.1-3.3): pool keys into chunk descriptors, route every
 * query to its top-k chunks under the causal mask and the mandatory anchors, attend
 * exactly over the selected key tokens, and (for training) the backward of that
 * attention with the selection held constant.
 *
 * Conventions
 *   H heads, L tokens, d head_dim, C chunks, k = top_k.
 *   Chunk c holds tokens [chunk_off[c], chunk_off[c+1]); chunk_shot[c] is the id of the
 *   shot it belongs to, chunk_mod[c] its modality (0 video, 1 text).
 *   Q, K, V, O, dO, dQ, dK, dV : DEVICE, bf16, [H][L][d] contiguous, 16-byte aligned.
 *   desc                       : DEVICE, fp32, [H][C][d].
 *   sel_idx                    : DEVICE, int32, [H][L][k]; routed picks only (anchors are
 *                                implied by the plan), descending score, equal scores in
 *                                ascending chunk index, -1 padding when a query has fewer
 *                                than k candidates.
 *   lse                        : DEVICE, fp32, [H][L]; natural log of the sum over the
 *                                selected keys of exp(softmax_scale * q.k).
 *   ws                         : DEVICE scratch of moc_workspace_bytes() bytes, 256-byte
 *                                aligned, owned by the caller.  moc_route (or moc_lists_from_sel)
 *                                writes the chunk -> query lists of the selection into it; the
 *                                same pointer, unchanged, must be given to moc_attend /
 *                                moc_attend_bwd afterwards.
 *   stream                     : a cudaStream_t passed as void* (NULL = default stream).
 *
 * Ownership: the caller owns every buffer.  The library allocates device memory only in
 * moc_plan_create (the chunk tables, a few KB) and frees it in moc_plan_destroy.  No call
 * synchronises the stream or the device; work is enqueued on `stream` in call order.
 *
 * Errors: every function returns MOC_OK (0) or a negative moc_status.  Argument errors
 * are detected before anything is launched.  Nothing throws, aborts or traps.  What only
 * the device can see is reported through a status word in the workspace that
 * moc_get_status() reads back: a bounded wait that ran out (MOC_ERR_TIMEOUT; the kernel
 * drains its copies, frees its tensor memory and returns), or a workspace that does not
 * hold the lists of this plan (MOC_ERR_WORKSPACE; the attention kernels then return
 * without reading or writing anything else).
 */
#ifndef MOC_H_
#define MOC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum moc_status {
    MOC_OK = 0,
    MOC_ERR_NULL = -1,        /* a required pointer is NULL                                  */
    MOC_ERR_SHAPE = -2,       /* H, L, d, C or k out of the supported range                  */
    MOC_ERR_CHUNK_TABLE = -3, /* offsets not strictly increasing from 0 to L, shots decreasing,
                                 or a modality other than 0/1                                */
    MOC_ERR_ALIGN = -4,       /* a device pointer is not aligned as required                 */
    MOC_ERR_WORKSPACE = -5,   /* workspace missing; as a device status: routing (or moc_lists_from_sel)
                                 of this plan has not been run on it                           */
    MOC_ERR_ARCH = -6,        /* the current device is not compute capability 10.x           */
    MOC_ERR_CUDA = -7,        /* a CUDA runtime call failed; see moc_last_cuda_error()       */
    MOC_ERR_TIMEOUT = -8,     /* device status: a bounded wait inside a kernel ran out       */
    MOC_ERR_TOO_LARGE = -9,   /* problem exceeds the fixed scratch of a no-allocation entry point, or the
                                 workspace budget given to moc_plan_set_workspace_budget           */
    MOC_ERR_INDEX = -10       /* device status, debug build (-DMOC_DEBUG) only: an index a kernel took
                                 from the workspace was out of range; the access was skipped       */
} moc_status;

#define MOC_WHOLE_SHOT (-1)   /* window value: every chunk of the query's shot is an anchor  */
#define MOC_FLAG_CAUSAL 0x1u  /* routed candidates are strictly earlier chunks (Sec. 3.2)    */

/* Problem statement (Sec. 3.1 "Dynamic Routing via Top-k Selection", Sec. 3.3).  The three
 * table pointers are HOST pointers, read during moc_plan_create only. */
typedef struct moc_problem {
    int32_t n_heads, n_tokens, head_dim;  /* 1 <= H <= 65535, L >= 1, H * L < 2^31, d in {64, 128} */
    int32_t n_chunks, top_k;              /* C >= 1, 0 <= k <= 512                           */
    int32_t win_back, win_fwd;            /* intra-shot anchor window in chunks before/after
                                             the query's own chunk; MOC_WHOLE_SHOT = the
                                             paper's "each shot always performs self-attention" */
    uint32_t flags;                       /* MOC_FLAG_*                                      */
    float softmax_scale;                  /* 0 => 1/sqrt(d) (Eq. 1)                          */
    const int32_t *chunk_off;             /* [C+1], off[0] = 0, strictly increasing, off[C] = L */
    const int32_t *chunk_shot;            /* [C], non-decreasing                             */
    const uint8_t *chunk_mod;             /* [C], 0 = video, 1 = text                        */
} moc_problem;

typedef struct moc_plan moc_plan;

/* Validate the problem, derive the per-chunk anchor tables and upload them to the current
 * device (Sec. 3.3: boundary tables, forced links as a pre-routing mask). */
int moc_plan_create(const moc_problem *problem, moc_plan **out);
int moc_plan_destroy(moc_plan *plan);

/* Bytes of caller-owned scratch that moc_route / moc_attend (with_bwd = 0) or also
 * moc_attend_bwd (with_bwd = 1) need.  The largest part is the routed partial outputs (Sec. 3.3:
 * every routed (query, chunk) pair is one attention problem; its normalised result and log-sum-exp
 * wait in the workspace until the query's anchor pass merges them): k times the size of O for the
 * heads in flight.  Attention runs over groups of heads so that this part stays within a budget
 * (6 GiB by default; one head at a time is the floor). */
int moc_workspace_bytes(const moc_plan *plan, int with_bwd, size_t *bytes);

/* Chooses the heads per group so that moc_workspace_bytes(plan, 0) <= max_bytes (the with_bwd size
 * adds 4 H L bytes).  MOC_ERR_TOO_LARGE, and the plan unchanged, if one head at a time still needs
 * more.  Call it before asking for the size and allocating; a workspace laid out under another
 * budget must be routed again. */
int moc_plan_set_workspace_budget(moc_plan *plan, size_t max_bytes);

/* Step 1 - chunk descriptors (Eq. 3 text: phi = mean pooling of the chunk's keys).
 * desc[h][c][:] = mean over t in chunk c of K[h][t][:], accumulated in fp32. */
int moc_chunk_pool(const moc_plan *plan, const void *K, float *desc, void *ws, void *stream);

/* (The paper has no counterpart to this entry point; it exists for deployment reasons.)
 * Same result as moc_chunk_pool, for callers that cannot hand over a workspace because they
 * cannot allocate device memory at this point: code running after a serving engine or a
 * training framework has already claimed the whole GPU for its own pool, hosts with a fixed
 * memory budget settled at start-up, and latency-critical loops where cudaMalloc / cudaFree
 * (which may block on the whole device) are forbidden.  The kernel's scratch (per-slice partial
 * sums and per-chunk arrival counters) lives in a fixed array inside the library image: every
 * GPU that loads the library holds those 4 MiB + 64 KiB until the process exits.
 *   Limits: H * units * d * 4 bytes <= 4 MiB and H * C * 4 bytes <= 64 KiB, where the units are the
 *   256-token slices of the chunks (each chunk's last one shorter); beyond that MOC_ERR_TOO_LARGE and nothing is
 *   launched (24 heads of the 33k-token single-shot clip need 1.8 MiB; longer streams, or more than
 *   16384 (head, chunk) pairs, must use moc_chunk_pool with a workspace).
 *   K, desc: as for moc_chunk_pool; the caller still owns inputs and outputs.
 *   The call itself allocates nothing (no cudaMalloc / cudaFree, no allocating library call).
 *   The array's device address is looked up once per device, in the first moc_plan_create on that
 *   device (which also makes the driver load the array there, so this call never has to); a plan
 *   must exist before this call anyway.  Create the first plan before starting any stream capture.
 *   All calls share the one array, which keeps whatever the previous call left (the counters are
 *   cleared on the stream at the start of every call): two calls that may overlap on the GPU
 *   (different streams, no ordering between them) race on it - serialise them. */
int moc_chunk_pool_noalloc(const moc_plan *plan, const void *K, float *desc, void *stream);

/* Steps 2-5 - routing (Eq. 3; Sec. 3.2 causal mask and fixed selections; Sec. 3.3 forced
 * links before top-k).  For every query i in chunk c(i): candidates are the chunks that
 * are not anchors of c(i) and (causal) lie strictly before c(i); score = q_i . desc_j (raw
 * dot product: each fp32 descriptor enters as the exact sum of three bf16 terms, products are
 * exact and the accumulation is fp32); sel_idx gets the min(k, #candidates) best, ties to the
 * lower index.  Also rebuilds, in ws, the per-(head, chunk) lists of the queries that picked
 * it and the routed work items of moc_attend / moc_attend_bwd, and marks ws as holding this
 * plan's lists.  MOC_ERR_SHAPE if the chunk count is beyond what the kernel's shared-memory
 * tables hold (about 8000 chunks). */
int moc_route(const moc_plan *plan, const void *Q, const float *desc, int32_t *sel_idx, void *ws, void *stream);

/* Sec. 3.3 ("head/tail indices of the selected chunks are gathered ... for the attention call"):
 * rebuilds the chunk -> query lists and the routed work items in ws from a sel_idx that the caller
 * has edited after moc_route (the context drop-off / drop-in of Sec. 3.1 is such an edit), so that
 * moc_attend / moc_attend_bwd attend over exactly that selection.  An entry is kept if it names a
 * chunk that may be routed to from its row (0 <= j < C, not an anchor of the row's chunk, strictly
 * earlier when the plan is causal) and does not repeat an earlier slot of the row; every other entry
 * is an empty slot and is overwritten with -1, so that afterwards sel_idx states the selection in force.
 * Slots need not be sorted or packed to the front. */
int moc_lists_from_sel(const moc_plan *plan, int32_t *sel_idx, void *ws, void *stream);

/* Sec. 3.1, "Context drop-off" and "Context drop-in": the training-time regularisers of the routed
 * selection, applied in place to a sel_idx that moc_route wrote (or moc_lists_from_sel checked), after
 * which the lists in ws are rebuilt for the edited selection (as by moc_lists_from_sel).  Per query:
 *   drop-off: p_drop = U p_max, U ~ Uniform[0, 1); floor(p_drop k) of the query's picks are removed (at
 *             most all it has), each chosen uniformly among the picks still there;
 *   drop-in:  m ~ Poisson(lambda) chunks are added, each chosen uniformly among the chunks the query may
 *             route to (not an anchor, strictly earlier if causal) that are neither picks of the query
 *             (kept or just removed) nor added already; they go into the free slots, lowest first, and
 *             stop when the k slots are full or no chunk is left.
 * The paper gives neither p_max nor lambda; here 0 <= p_max <= 1 and 0 <= lambda <= 8 (MOC_ERR_SHAPE
 * otherwise); p_max = 0 and lambda = 0 leave the selection as it is.  The draws are a pure function of
 * (seed, head, token): Philox4x32-10 with the seed as key and (token, head, draw / 4, 0) as counter, so a
 * run is reproducible and independent of launch shape. */
int moc_context_drop(const moc_plan *plan, int32_t *sel_idx, float p_max, float lambda, uint64_t seed, void *ws,
                     void *stream);

/* Step 6 - sparse attention (Eq. 2): O_i = softmax(scale q_i K_Omega^T) V_Omega over the
 * tokens of the chunks in Omega(i) = anchors(c(i)) U sel_idx[i]; lse as defined above.
 * bf16 products, fp32 accumulation and softmax.
 * The kernels walk the selection through the lists that moc_route or moc_lists_from_sel left in
 * ws, not through sel_idx: sel_idx must be the array the last of those calls on ws wrote or
 * checked, unchanged since (after editing it, call moc_lists_from_sel).  A ws that does not hold
 * this plan's lists makes every block return at once with device status MOC_ERR_WORKSPACE. */
int moc_attend(const moc_plan *plan, const void *Q, const void *K, const void *V, const int32_t *sel_idx,
               void *O, float *lse, void *ws, void *stream);

/* Backward of step 6 with the selection held constant (Sec. 3.1: top-k is not
 * differentiated, gradients reach Q, K, V only through the attention over selected
 * chunks; none flows through the descriptors or scores).  bf16 products (P and dS are rounded
 * to bf16 before their contractions), fp32 accumulation.  Needs with_bwd workspace, written by
 * moc_route (or moc_lists_from_sel) and moc_attend for the same inputs; overwrites the forward's
 * routed partials.  sel_idx: as for moc_attend. */
int moc_attend_bwd(const moc_plan *plan, const void *Q, const void *K, const void *V, const void *O,
                   const float *lse, const void *dO, const int32_t *sel_idx, void *dQ, void *dK, void *dV,
                   void *ws, void *stream);

/* Number of selected (query, key-token) pairs summed over all heads and queries (the unit of
 * the FLOP count of Sec. 3.3: 4 d per pair forward): the anchor pairs follow from the plan's
 * tables, the routed pairs from the per-(head, chunk) pick counts that moc_route or
 * moc_lists_from_sel left in ws.  Copies those counts to the host: synchronises `stream`. */
int moc_selected_pairs(const moc_plan *plan, const void *ws, void *stream, int64_t *pairs);

/* Reads the device status word of ws (synchronous copy on `stream`): MOC_OK, MOC_ERR_TIMEOUT
 * or MOC_ERR_WORKSPACE, with `detail` (optional) receiving a kernel-specific code (for a
 * timeout, which wait gave up). */
int moc_get_status(const moc_plan *plan, const void *ws, void *stream, int *device_status, int *detail);

/* Outer-loop context routing (the paper's appendix of that name): before any attention, whole shots of the
 * context are pre-selected for one query block; the selected shots, the mandatory text and the block's own
 * shots form a reduced stream on which the calls above then run with a plan of its own.
 *   High-level chunk Psi_s = every token of shot s (all chunks with that chunk_shot value); S shots.
 *   phi(Psi_s) = mean of the context features over the shot: computed here as the token-weighted mean of
 *                `desc`, the chunk descriptors that moc_chunk_pool made of the context features;
 *   x_g        = mean of the query features Xq ([H][L][d] bf16, each of the H streams on its own) over the
 *                block of tokens [q_tok0, q_tok1);
 *   scores     = <x_g, phi(Psi_s)> for every shot ([H][S], fp32); shot_desc [H][S][d] fp32;
 *   sel_shot   = [H][top_m] int32: the top_m best shots among those that END before the block begins (a
 *                shot holding a token >= q_tok0 is not history), best first, equal scores to the earlier
 *                shot, -1 padded.  ws: scratch of moc_workspace_bytes (its pooling area is used). */
int moc_outer_num_shots(const moc_plan *plan, int32_t *n_shots);
int moc_outer_route(const moc_plan *plan, const void *Xq, const float *desc, int32_t q_tok0, int32_t q_tok1, int32_t top_m,
                    float *shot_desc, float *scores, int32_t *sel_shot, void *ws, void *stream);

/* HOST only (no device work): the chunk table of the reduced stream for one selection.  Kept, in stream
 * order: every text chunk (the mandatory elements), the chunks of the n_sel shots in sel_shot (HOST, -1
 * entries skipped) and the chunks of the shots that overlap the block [q_tok0, q_tok1).  Outputs (HOST,
 * sized by the caller for the original stream: C + 1, C, C and L entries): the reduced chunk_off /
 * chunk_shot / chunk_mod, ready for moc_plan_create, and tok_map[r] = original token of reduced token r. */
int moc_outer_reduced_layout(const moc_plan *plan, const int32_t *sel_shot, int32_t n_sel, int32_t q_tok0, int32_t q_tok1,
                             int32_t *n_chunks, int32_t *n_tokens, int32_t *chunk_off, int32_t *chunk_shot,
                             uint8_t *chunk_mod, int32_t *tok_map);

/* out[h][r][:] = X[h][tok_map[r]][:] for r < n_out: the rows of a [H][L][d] bf16 tensor that the reduced
 * stream keeps (tok_map: DEVICE int32; out: DEVICE [H][n_out][d] bf16). */
int moc_gather_tokens(const moc_plan *plan, const void *X, const int32_t *tok_map, int32_t n_out, void *out, void *stream);

/* How many kernel launches the library has enqueued since it was loaded. */
int64_t moc_launch_count(void);

const char *moc_strerror(int status);
const char *moc_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* MOC_H_ */
