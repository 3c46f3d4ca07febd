// Shared declarations of the MoC library: plan object, workspace layout, launch helpers.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <atomic>
#include <vector>

#include "../../include/moc.h"
#include <nvtx3/nvToolsExt.h>

namespace moc {

constexpr int kQTileRows = 256;     // query rows per attention work item (two 128-row MMA tiles)
constexpr int kPoolSlice = 256;     // tokens per chunk-pool work unit
constexpr int kStatusWords = 16;    // status area at the head of the workspace (int32 each):
// [0] device status (a moc_status), [1] detail code, [2] cookie of the plan whose lists the workspace holds,
// [3] limit of every bounded wait in microseconds (0 = the default of one second), [4] routing blocks that have finished
enum StatusWord { ST_STATUS = 0, ST_DETAIL = 1, ST_COOKIE = 2, ST_WAIT_US = 3, ST_ARRIVE = 4 };
constexpr int kQueueHeader = 4;     // queue area: [0] next item to claim, [1] items, [2] phases, [3] spare; then 3 ints per phase
constexpr unsigned kPrivFlagCudaCoreAttend = 0x80000000u;   // plan flag outside the public header: test hook

// One contiguous range of key tokens [t0, t1).
struct KeyRange { int32_t t0, t1; };

// One attention work item: up to kQTileRows query rows of head h against the key ranges
// rng[rng_off .. rng_off + nrng) (ntiles key tiles of 128; [t0, t1) repeats the first range).  Anchor pass: `first` is the first of `rows`
// consecutive query rows of one chunk (h is implied by the item index).  Routed pass: `first` is the
// offset, inside the head's list area, of the `rows` entries of one chunk's query list.
struct WorkItem { int32_t h, first, rows, ntiles, rng_off, nrng, t0, t1; };

// One tile of up to 128 consecutive key tokens of chunk c (backward, key-stationary pass).
struct KTile { int32_t chunk, t0, valid, pad; };

struct WsLayout {
    size_t status;      // int32[kStatusWords], see StatusWord
    size_t cnt;         // int32[H][C]     routed picks per (head, chunk); doubles as the list cursor while routing
    size_t tile_off;    // int32[H*C+1]    running count of routed attention tiles over (head, chunk) pairs
    size_t rtiles;      // WorkItem[H * (ceil(L k / 256) + C)]  routed work items, written after routing
    size_t qlist;       // int32[H][cap_total]  per (head, chunk) list at cap_off[c]: entries i*k+s of the picks of c
    size_t desc3;       // bf16 [H][3][Cpad][d]  descriptors split into three bf16 terms (hi + mid + lo)
    size_t pool_part;   // float[H][n_pool_units][d] partial key sums
    size_t pool_done;   // int32[H][C] arrival counters (cleared at the start of every pooling call)
    size_t queue;       // int32[kQueueHeader + 6 groups] work queue of the forward attention kernel
    size_t part_o;      // bf16 [1 or 2][Hg][L][k][d] routed partial outputs (normalised) of one group of Hg heads; with
                        // several groups, two buffers that consecutive groups alternate between
    size_t part_lse;    // float[H][L][k]    routed partial log-sum-exp (-inf = unused slot)
    size_t fwd_end;
    size_t delta;       // float[H][L]       rowsum(dO * O)
    size_t bwd_end;
};

}  // namespace moc

struct moc_plan {
    int H, L, d, C, k, win_back, win_fwd;
    unsigned flags;
    float scale;
    int device;
    int n_sm;
    bool pool_direct = false;    // descriptors by one block per (head, chunk): every block resident at once, no long chunk
    std::vector<int32_t> off, shot;
    std::vector<uint8_t> mod;
    // host-side derived tables
    std::vector<int32_t> anc_off;            // [C+1] into anc_rng
    std::vector<moc::KeyRange> anc_rng;      // merged anchor token ranges per query chunk
    std::vector<int64_t> anc_tokens;         // [C] anchor key tokens per query chunk
    std::vector<int32_t> ranc_off, ranc;     // reverse anchors: key chunk -> query chunks
    std::vector<moc::WorkItem> qitems;       // anchor-pass work items of one head
    std::vector<moc::KTile> ktiles;          // key tiles of one head: the long ones (see moc_plan_create) first, then chunk by chunk
    int n_long_ktiles = 0;
    std::vector<int32_t> pool_unit_off;      // [C+1] prefix of pool units per chunk
    std::vector<moc::KeyRange> shot_chunks;  // [S] chunk range [t0, t1) of every shot (outer-loop routing)
    int words;                               // uint32 words per anchor bitmap row
    std::vector<int32_t> cap_off;            // [C+1] start of chunk c's query list inside a head's list area
    // Routing scores only the chunks that can ever be picked: text chunks are anchors of every query, so the score
    // matrix has one column per non-text chunk ("column" = index among those, in chunk order).
    int ncol;                                // number of columns
    int cwords;                              // uint32 words per candidate bitmap row (over columns)
    int prefix_mode;                         // 1: every query chunk's candidates are exactly the columns [0, lim[c])
    int c_pad;                               // columns rounded up to a multiple of 16 (MMA N granularity)
    int n_pool_units;
    int heads_per_group;                     // Hg: heads whose routed partials are held at once (attention runs group by group)
    size_t partials_budget;                  // bytes the routed partials may take; sets Hg
    uint32_t cookie;                         // hash of the problem, written into a workspace this plan has routed on
    uint32_t wait_us;                        // limit of the kernels' bounded waits (0 = default); tests shorten it
    // device tables (one allocation)
    void *d_blob;
    int32_t *d_off, *d_shot, *d_tok_chunk, *d_anc_off, *d_ranc_off, *d_ranc, *d_pool_unit_off, *d_pool_unit_chunk, *d_cap_off;
    uint8_t *d_mod;
    uint32_t *d_anc_bits;
    uint32_t *d_cand_c;                      // [C][cwords] candidate columns of a query in chunk c (causality included)
    int32_t *d_lim, *d_reach, *d_col_chunk;  // [C] prefix length (-1: not a prefix); [C] columns any query up to chunk c can reach; [ncol] chunk of a column
    moc::KeyRange *d_anc_rng;
    moc::WorkItem *d_qitems;
    moc::KeyRange *d_chunk_rng;              // [C] token range of every chunk
    moc::KTile *d_ktiles;
    moc::KeyRange *d_shot_chunks;            // [S]
    moc::WsLayout ws;
};

namespace moc {

extern std::atomic<long long> g_launches;
void set_cuda_error(cudaError_t e, const char *where);

#define MOC_CUDA_TRY(expr)                                         \
    do {                                                           \
        cudaError_t e_ = (expr);                                   \
        if (e_ != cudaSuccess) {                                   \
            moc::set_cuda_error(e_, #expr);                        \
            return MOC_ERR_CUDA;                                   \
        }                                                          \
    } while (0)

#define MOC_LAUNCH_CHECK()                                         \
    do {                                                           \
        moc::g_launches.fetch_add(1);                              \
        cudaError_t e_ = cudaGetLastError();                       \
        if (e_ != cudaSuccess) {                                   \
            moc::set_cuda_error(e_, "kernel launch");              \
            return MOC_ERR_CUDA;                                   \
        }                                                          \
    } while (0)

template <typename T>
static inline T *ws_ptr(void *ws, size_t off) { return reinterpret_cast<T *>(static_cast<char *>(ws) + off); }
template <typename T>
static inline const T *ws_ptr(const void *ws, size_t off) { return reinterpret_cast<const T *>(static_cast<const char *>(ws) + off); }

#ifdef __CUDACC__
// Debug build (-DMOC_DEBUG): every index a kernel takes from the workspace (list entries, list positions,
// work-item fields) is checked before it is used as an address; a bad one records MOC_ERR_INDEX with `code`
// in the status area and the access is skipped.  In the release build the checks cost nothing.
enum IndexCheck { IX_ITEM_FIELDS = 200, IX_LIST_POSITION, IX_LIST_ENTRY, IX_APPEND_POSITION, IX_BWD_ITEM_FIELDS,
                  IX_BWD_LIST_POSITION, IX_BWD_LIST_ENTRY };
#ifdef MOC_DEBUG
__device__ __forceinline__ bool index_ok(bool cond, int *status, int code) {
    if (!cond && atomicCAS(status, 0, MOC_ERR_INDEX) == 0) status[ST_DETAIL] = code;
    return cond;
}
#else
__device__ __forceinline__ bool index_ok(bool, int *, int) { return true; }
#endif

// Layout of the routed partial outputs.  The row of one (query, slot) is written by one thread of a routed item
// and read by one thread of the query's anchor item, 16 bytes (a "piece": eight columns) at a time.  Anchor items
// hold consecutive queries in consecutive lanes, so the pieces are laid out query-innermost: within a block of 128
// queries, the pieces 2 c2 and 2 c2 + 1 (a pair: one 32-byte sector) of slot s of the block's queries are 128 x 32
// contiguous bytes.  A warp's load of one pair for its 32 queries is then 1024 contiguous bytes instead of 32
// scattered requests, and a routed item, whose rows are scattered queries, still writes whole sectors (a store of
// half a sector makes the memory system read the other half first).
//   index (in 16-byte units) of piece c of (head-in-group hl, query qi, slot s); NP = d / 8 pieces per row,
//   LB = ceil(L / 128) blocks per head
__device__ __forceinline__ size_t part_piece(int hl, int LB, int k, int NP, int qi, int s, int c) {
    return ((((((size_t)hl * LB + (qi >> 7)) * k + s) * (NP >> 1) + (c >> 1)) * 128 + (qi & 127)) << 1) + (c & 1);
}

// A named range around a call of the boundary, for timeline tools (NVTX; a no-op when no tool is attached).
struct NvtxRange {
    explicit NvtxRange(const char *name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
    NvtxRange(const NvtxRange &) = delete;
    NvtxRange &operator=(const NvtxRange &) = delete;
};

// Walks the 128-key tiles of a list of key ranges (a tile never straddles two ranges).
struct TileIter {
    const KeyRange *rng;
    int n, ri, t, end;      // the current range's end is kept: one load per range, not per tile
    __device__ TileIter(const KeyRange *r, int n_) : rng(r), n(n_), ri(0), t(n_ > 0 ? r[0].t0 : 0), end(n_ > 0 ? r[0].t1 : 0) {}
    __device__ bool next(int &t0, int &valid) {
        if (ri >= n) return false;
        t0 = t;
        valid = min(128, end - t);
        t += 128;
        if (t >= end) {
            ++ri;
            if (ri < n) { t = rng[ri].t0; end = rng[ri].t1; }
        }
        return true;
    }
};
#endif

void layout_workspace(moc_plan *p);

static inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// kernels' host launchers (each returns a moc_status)
int launch_chunk_pool(const moc_plan *p, const __nv_bfloat16 *K, float *desc, void *ws, cudaStream_t s);
int launch_route(const moc_plan *p, const __nv_bfloat16 *Q, const float *desc, int32_t *sel, void *ws, cudaStream_t s);
int launch_lists_from_sel(const moc_plan *p, int32_t *sel, void *ws, cudaStream_t s);
int launch_context_drop(const moc_plan *p, int32_t *sel, float p_max, float lambda, uint64_t seed, cudaStream_t s);
int pool_scratch_prepare(int device);     // looks up (once per device) the fixed scratch array of moc_chunk_pool_noalloc
int launch_attend_scalar(const moc_plan *p, const __nv_bfloat16 *Q, const __nv_bfloat16 *K, const __nv_bfloat16 *V,
                         const int32_t *sel, __nv_bfloat16 *O, float *lse, void *ws, cudaStream_t s);
int launch_attend_bwd_scalar(const moc_plan *p, const __nv_bfloat16 *Q, const __nv_bfloat16 *K, const __nv_bfloat16 *V,
                             const __nv_bfloat16 *O, const float *lse, const __nv_bfloat16 *dO, const int32_t *sel,
                             __nv_bfloat16 *dQ, __nv_bfloat16 *dK, __nv_bfloat16 *dV, void *ws, cudaStream_t s);
int launch_attend_bwd_tc(const moc_plan *p, const __nv_bfloat16 *Q, const __nv_bfloat16 *K, const __nv_bfloat16 *V,
                         const __nv_bfloat16 *O, const float *lse, const __nv_bfloat16 *dO, const int32_t *sel,
                         __nv_bfloat16 *dQ, __nv_bfloat16 *dK, __nv_bfloat16 *dV, void *ws, cudaStream_t s);
int launch_delta(const moc_plan *p, const __nv_bfloat16 *O, const __nv_bfloat16 *dO, float *delta, cudaStream_t s);
int launch_attend_tc(const moc_plan *p, const __nv_bfloat16 *Q, const __nv_bfloat16 *K, const __nv_bfloat16 *V,
                     const int32_t *sel, __nv_bfloat16 *O, float *lse, void *ws, cudaStream_t s);

}  // namespace moc

// Test hooks: exported, but not part of the public header (tests declare them themselves).
extern "C" {
// attention and its backward on the plain fp32 CUDA-core kernels (an in-library cross-check that reads
// the selection straight from sel_idx)
int moc_debug_use_cuda_core_attention(moc_plan *plan, int on);
// limit of every bounded device-side wait, in microseconds, for workspaces routed from now on (0 = default)
int moc_debug_set_wait_limit_us(moc_plan *plan, unsigned us);
// one block whose only wait is on a barrier that nothing ever arrives on: it must give up after the limit,
// record MOC_ERR_TIMEOUT with detail `code` in ws, and return
int moc_debug_wait_probe(const moc_plan *plan, void *ws, int code, void *stream);
}
