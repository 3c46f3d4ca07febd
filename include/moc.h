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
 *                                aligned, owned by the caller.  moc_route writes the
 *                                chunk -> query lists into it; the same pointer, unchanged,
 *                                must be given to moc_attend / moc_attend_bwd afterwards.
 *   stream                     : a cudaStream_t passed as void* (NULL = default stream).
 *
 * Ownership: the caller owns every buffer.  The library allocates device memory only in
 * moc_plan_create (the chunk tables, a few KB) and frees it in moc_plan_destroy.  No call
 * synchronises the stream or the device; work is enqueued on `stream` in call order.
 *
 * Errors: every function returns MOC_OK (0) or a negative moc_status.  Argument errors
 * are detected before anything is launched.  Nothing throws, aborts or traps.  Kernels
 * bound every wait; a wait that runs out sets a status word in the workspace that
 * moc_get_status() reads back (after the caller has synchronised the stream).
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
    MOC_ERR_WORKSPACE = -5,   /* workspace missing, or routing has not been run on it        */
    MOC_ERR_ARCH = -6,        /* the current device is not compute capability 10.x           */
    MOC_ERR_CUDA = -7,        /* a CUDA runtime call failed; see moc_last_cuda_error()       */
    MOC_ERR_TIMEOUT = -8,     /* device status: a bounded wait inside a kernel ran out       */
    MOC_ERR_TOO_LARGE = -9    /* problem exceeds the fixed scratch of a no-allocation entry point */
} moc_status;

#define MOC_WHOLE_SHOT (-1)   /* window value: every chunk of the query's shot is an anchor  */
#define MOC_FLAG_CAUSAL 0x1u  /* routed candidates are strictly earlier chunks (Sec. 3.2)    */
#define MOC_FLAG_SCALAR_ATTEND 0x2u /* run attention on the plain fp32 CUDA-core kernels     */

/* Problem statement (Sec. 3.1 "Dynamic Routing via Top-k Selection", Sec. 3.3).  The three
 * table pointers are HOST pointers, read during moc_plan_create only. */
typedef struct moc_problem {
    int32_t n_heads, n_tokens, head_dim;  /* H >= 1, L >= 1, d in {64, 128}                  */
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
 * moc_attend_bwd (with_bwd = 1) need. */
int moc_workspace_bytes(const moc_plan *plan, int with_bwd, size_t *bytes);

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
 *   The first call on each device looks up the array's device address; make that first call
 *   before starting any stream capture on that device.
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
 * it and the routed work items of moc_attend / moc_attend_bwd.  MOC_ERR_SHAPE if the chunk
 * count is beyond what the kernel's shared-memory tables hold (about 8000 chunks). */
int moc_route(const moc_plan *plan, const void *Q, const float *desc, int32_t *sel_idx, void *ws, void *stream);

/* Step 6 - sparse attention (Eq. 2): O_i = softmax(scale q_i K_Omega^T) V_Omega over the
 * tokens of the chunks in Omega(i) = anchors(c(i)) U sel_idx[i]; lse as defined above.
 * bf16 products, fp32 accumulation and softmax. */
int moc_attend(const moc_plan *plan, const void *Q, const void *K, const void *V, const int32_t *sel_idx,
               void *O, float *lse, void *ws, void *stream);

/* Backward of step 6 with the selection held constant (Sec. 3.1: top-k is not
 * differentiated, gradients reach Q, K, V only through the attention over selected
 * chunks; none flows through the descriptors or scores).  bf16 products (P and dS are rounded
 * to bf16 before their contractions), fp32 accumulation.  Needs with_bwd workspace, written by
 * moc_route and moc_attend for the same inputs; overwrites the forward's routed partials. */
int moc_attend_bwd(const moc_plan *plan, const void *Q, const void *K, const void *V, const void *O,
                   const float *lse, const void *dO, const int32_t *sel_idx, void *dQ, void *dK, void *dV,
                   void *ws, void *stream);

/* Number of selected (query, key-token) pairs summed over all heads and queries, from the
 * plan's anchor tables and a HOST copy of the per-(head, chunk) pick counts is not needed:
 * this reads the counts that moc_route left in ws (synchronises `stream`). */
int moc_selected_pairs(const moc_plan *plan, const void *ws, void *stream, int64_t *pairs);

/* Reads the device status word of ws (synchronous copy on `stream`): MOC_OK or
 * MOC_ERR_TIMEOUT, with `detail` (optional) receiving a kernel-specific code. */
int moc_get_status(const moc_plan *plan, const void *ws, void *stream, int *device_status, int *detail);

/* How many kernel launches the library has enqueued since it was loaded. */
int64_t moc_launch_count(void);

const char *moc_strerror(int status);
const char *moc_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* MOC_H_ */
