// Tensor-core sparse attention forward (tcgen05 MMA, TMEM accumulators, TMA-fed Q/K/V), one persistent
// kernel over a single queue of work items.
//
// Two kinds of items:
//   routed (key-chunk stationary): (head, chunk c, up to 256 entries of the list of (query, slot) pairs that
//     picked c).  The Q rows are gathered by TMA (four rows per copy), the keys are exactly the tokens of chunk
//     c, and each (query, slot) gets a partial result (normalised output + log-sum-exp) in the workspace;
//   anchor (query-tile stationary): (head, up to 256 consecutive rows of one chunk); keys are the chunk's
//     mandatory anchors (merged token ranges).  Its epilogue merges the row's <= k routed partials by
//     log-sum-exp and writes O and LSE.
// The queue holds, group of heads by group of heads, the group's routed items and then its anchor items.  One
// CTA per SM claims items in queue order (a global counter), so the two kinds need no separate launches and no
// CTA is set up or torn down per item: the tensor memory, the barriers and the K/V ring live for the whole
// kernel, and the next item's Q tiles and first K/V tiles are on their way while the current item finishes.
// What an anchor item needs from the routed items of its group (their partials) is awaited late, just before
// its merge, on a count of completed rows; by then every routed item of the group has long been claimed, by a
// CTA that is running, so the wait ends.  Partials of consecutive groups alternate between two buffers; a
// routed item waits, before it stores, for the anchor items that read its buffer two groups ago.
//
// 12 warps in three warpgroups (the third gives most of its registers to the other two); an item is two 128-row
// query tiles that share every K/V tile:
//   warps 0-3 / 4-7  softmax group of query tile 0 / 1, one row per thread (TMEM lane = row): read S from TMEM,
//              online softmax, write P back to TMEM as packed bf16 (aliasing S; the first 64 keys are released
//              to the issuer before the exponentials of the other 64), lazily rescale O, epilogue.  The
//              exponentials of the two tiles take turns;
//   warp 8     lane 0, TMA producer: the K and V tiles of 128 keys, two stages each, 128-byte swizzle; the ring
//              runs across items.  Lane 16, bookkeeping: waits for what an item depends on, and when the item's
//              rows are stored adds them to the queue's count of completed rows (the one thread that pays for
//              a device-wide fence per item);
//   warps 9, 10  one MMA-issuing thread per query tile g:  S_g(0), then  O_g += P_g V(j),  S_g(j + 1)  per key
//              tile.  S = Q K^T takes both operands from shared memory, O += P V takes P from TMEM and V as an
//              MN-major shared-memory operand; all accumulators live in TMEM (S0, S1, O0, O1 = 512 columns);
//   warp 11    scheduler and Q loader: lane 0 claims the next item and hands its description to the others
//              through a two-slot ring; then the warp loads the item's Q tiles (plain tiles for anchor items,
//              row gathers, four rows per lane, for routed ones) into a ring of three tile buffers, so the next
//              item's first query tile is in place before the current item ends.
// Every wait (mbarrier or global counter) is bounded; one that runs out flags the workspace status word and
// the CTA drains its copies and leaves.
#include <algorithm>

#include "moc_common.cuh"
#include "moc_tc.cuh"

namespace moc {

using namespace tc;

struct AttendParams {
    const __nv_bfloat16 *Q;
    __nv_bfloat16 *O;
    float *lse;
    __nv_bfloat16 *part_o;      // [2 or 1] buffers of the group in flight's partials (even / odd groups alternate), laid
                                // out query-innermost in blocks of 128 queries (part_piece)
    float *part_lse;            // [H][L][k]
    size_t part_stride;         // elements between the two partial buffers (0 with a single group)
    const KeyRange *chunk_rng;  // [C] key range of a routed item (its chunk)
    const KeyRange *anc_rng;    // merged anchor ranges, indexed by the anchor items
    const WorkItem *ritems;     // routed items of every head, (head, chunk) order
    const WorkItem *aitems;     // anchor items of one head
    const int *tile_off;        // [H C + 1] running count of routed items over (head, chunk)
    const int32_t *qlist;       // [H][cap_total]
    int *queue;
    size_t cap_total;
    int *status;
    int H, L, C, k, hg, n_groups, n_aitems;
    float scale_log2;           // softmax scale * log2(e)
    uint32_t cookie;
};

constexpr int kBN = 128;               // keys per tile
constexpr int kThreads = 384;          // three warpgroups: softmax 0, softmax 1, {producer, two MMA issuers, scheduler}
constexpr int kTmemCols = 512;         // S0/P0 [0,128) S1/P1 [128,256) O0 [256,384) O1 [384,512)
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.0f;    // log2 units: O is rescaled only when the row max grows by more

enum WaitCode { W_QFULL = 1, W_KFULL, W_VFULL, W_SFULL, W_PFULL, W_OFULL, W_KEMPTY, W_VEMPTY, W_TURN, W_PHALF,
                W_QEMPTY, W_OFREE, W_ITEMFULL, W_ITEMEMPTY, W_ROWSDONE, W_DEPEND };

// One claimed item, as the scheduler hands it over.
struct ItemSlot {
    int valid;          // 0: the queue is empty, everyone leaves
    int routed, h, first, rows, nrng, ntiles, phase;
    const KeyRange *rng;
};

// Queue bookkeeping in the workspace (kQueueHeader ints, then three per phase: first item, rows that must
// complete, rows completed), written before the persistent kernel starts.  Phase 2 g is the routed items of head
// group g (rows = the group's list entries), phase 2 g + 1 its anchor items (rows = its query rows).  One block.
__global__ void attend_queue_kernel(int *__restrict__ queue, const int *__restrict__ tile_off, const int *__restrict__ cnt,
                                    const int *__restrict__ status, uint32_t cookie, int H, int L, int C, int k, int hg, int n_groups,
                                    int n_aitems) {
    __shared__ int red[256];
    const bool routed_ok = status[ST_STATUS] == 0 && (uint32_t)status[ST_COOKIE] == cookie;     // else nothing may be read
    int first = 0;
    for (int g = 0; g < n_groups; ++g) {
        const int h0 = g * hg, h1 = min(H, h0 + hg);
        int entries = 0;
        if (routed_ok && k > 0)
            for (int x = h0 * C + threadIdx.x; x < h1 * C; x += blockDim.x) entries += cnt[x];
        red[threadIdx.x] = entries;
        __syncthreads();
        for (int o = 128; o > 0; o >>= 1) {
            if ((int)threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
            __syncthreads();
        }
        if (threadIdx.x == 0) {
            const int n_r = (routed_ok && k > 0) ? tile_off[h1 * C] - tile_off[h0 * C] : 0;
            int *ph = queue + kQueueHeader + 3 * (2 * g);
            ph[0] = first; ph[1] = red[0]; ph[2] = 0;
            first += n_r;
            ph[3] = first; ph[4] = (h1 - h0) * L; ph[5] = 0;
            first += (h1 - h0) * n_aitems;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) { queue[0] = 0; queue[1] = routed_ok ? first : 0; queue[2] = 2 * n_groups; queue[3] = 0; }
}

// a bounded wait on a counter in global memory (another CTA adds to it)
__device__ __forceinline__ bool wait_count(const int *ctr, int need, volatile int *abort_flag, int *status, int code) {
    if (*(volatile const int *)ctr >= need) return true;
    const uint64_t t0 = global_timer_ns();
    for (uint32_t it = 1;; ++it) {
        if (*(volatile const int *)ctr >= need) return true;
        __nanosleep(200);
        if ((it & 0x3f) == 0) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > wait_limit_ns(status)) {
                *abort_flag = 1;
                if (atomicCAS(status, 0, MOC_ERR_TIMEOUT) == 0) status[ST_DETAIL] = code;
                return false;
            }
        }
    }
}

// four rows of a 2-D tensor, 64 columns from column x on, into four consecutive 128-byte rows of shared memory
__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap *map, int x, int r0, int r1, int r2, int r3, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cta.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(r0), "r"(r1), "r"(r2), "r"(r3), "r"(bar)
                 : "memory");
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1) attend_tc_kernel(const __grid_constant__ CUtensorMap tmQ,
                                                                const __grid_constant__ CUtensorMap tmQrow,
                                                                const __grid_constant__ CUtensorMap tmK,
                                                                const __grid_constant__ CUtensorMap tmV,
                                                                const AttendParams p) {
    constexpr int TILE_BYTES = 128 * D * 2;
    constexpr int SUB = D / 64;            // 64-column (128-byte) sub-tiles per row
    constexpr int SUB_BYTES = 128 * 128;   // one sub-tile: 128 rows of 128 bytes
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[36];
    __shared__ uint32_t tmem_slot;
    __shared__ int s_abort;
    __shared__ ItemSlot s_item[2];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    // shared tiles: Q ring of three | K stage 0,1 | V stage 0,1
    const uint32_t sQ = sbase, sK = sbase + 3 * TILE_BYTES, sV = sbase + 5 * TILE_BYTES;
    auto bar = [&](int i) { return smem_u32(&bars[i]); };
    // barrier indices (pairs: per query tile g, per K/V stage, or per item slot)
    constexpr int Q_FULL = 0, Q_EMPTY = 3, K_FULL = 6, K_EMPTY = 8, V_FULL = 10, V_EMPTY = 12, S_FULL = 14, P_HALF = 16, P_FULL = 18,
                  O_FULL = 20, O_FREE = 22, TURN = 24, ITEM_FULL = 26, ITEM_EMPTY = 28, ROWS_DONE = 30, DEPEND = 32;
    constexpr int kItemReaders = 2 + 2 + 256;          // producer and bookkeeping lanes, two issuers, every softmax thread

    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int t = 0; t < 3; ++t) {
            mbar_init(bar(Q_FULL + t), 1);
            mbar_init(bar(Q_EMPTY + t), 1);
        }
        mbar_init(bar(DEPEND), 1);
        for (int t = 0; t < 2; ++t) {
            mbar_init(bar(K_FULL + t), 1);
            mbar_init(bar(K_EMPTY + t), 2);            // one arrival per MMA issuer
            mbar_init(bar(V_FULL + t), 1);
            mbar_init(bar(V_EMPTY + t), 2);
            mbar_init(bar(S_FULL + t), 1);
            mbar_init(bar(P_HALF + t), 128);
            mbar_init(bar(P_FULL + t), 128);
            mbar_init(bar(O_FULL + t), 1);
            mbar_init(bar(O_FREE + t), 128);
            mbar_init(bar(TURN + t), 128);
            mbar_init(bar(ITEM_FULL + t), 1);
            mbar_init(bar(ITEM_EMPTY + t), kItemReaders);
            mbar_init(bar(ROWS_DONE + t), 128);
        }
        fence_barrier_init();
    }
    __syncthreads();
    if (warp == 8) {
        tmem_alloc(smem_u32(&tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    volatile int *abort_flag = &s_abort;
    int *phase_tab = p.queue + kQueueHeader;

    if (warp < 8) {
        // ------------------------------------------------------------ softmax / epilogue groups
        // the row-per-thread softmax holds a whole 128-key row of S in registers: take the
        // registers the third warpgroup gives up
        asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
        const int g = warp >> 2;                       // query tile of this group
        const int r = threadIdx.x & 127;               // row within the tile = TMEM lane
        const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + g * 128 + lane_off, tP = tS, tO = tmem + 256 + g * 128 + lane_off;
        const float c = p.scale_log2;
        // running counts that give every barrier's phase: items seen, items this group worked on, key tiles it
        // processed, key tiles processed in two-tile items (the turn-taking of the exponentials)
        int n_item = 0, n_mine = 0, n_s = 0, n_turn = 0, n_dep = 0;
        bool ok = true;
        while (ok) {
            const int sl = n_item & 1;
            ok = mbar_wait(bar(ITEM_FULL + sl), (n_item >> 1) & 1, abort_flag, p.status, W_ITEMFULL);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const ItemSlot it_ = s_item[sl];
            mbar_arrive(bar(ITEM_EMPTY + sl));
            ++n_item;
            if (!it_.valid) break;
            const int h = it_.h, rows = it_.rows, first = it_.first, group = it_.phase >> 1;
            const bool routed = it_.routed != 0, two = rows > 128;
            // an item that depends on other items' rows (see the bookkeeping lane) is released through DEPEND, whose
            // phase counts those items only
            const bool dep = routed ? group >= 2 : p.k > 0;
            const int dep_phase = n_dep & 1;
            if (dep) ++n_dep;
            if (g == 1 && !two) continue;               // this item has one query tile
            const int rt = g * 128 + r;                 // row within the work item
            int qi = -1, slot = 0;
            if (rt < rows) {
                if (routed) {
                    const bool at_ok = index_ok((size_t)first + rt < p.cap_total, p.status, IX_LIST_POSITION);
                    const int e = at_ok ? p.qlist[(size_t)h * p.cap_total + first + rt] : -1;
                    qi = e / p.k;
                    slot = e - qi * p.k;
                    (void)index_ok(e >= 0 && qi < p.L, p.status, IX_LIST_ENTRY);
                    if (e < 0 || qi >= p.L) qi = -1;         // never follow an entry that is not a row of this head
                } else {
                    qi = first + rt;
                }
            }
            // partials of the group in flight: even and odd groups alternate between two buffers
            __nv_bfloat16 *part_o = p.part_o + (size_t)(group & 1) * p.part_stride;
            const int h_loc = h - group * p.hg;
            constexpr int NP = D / 8;                   // 16-byte pieces per row
            const int LB = (p.L + 127) >> 7;
            uint4 *part16 = reinterpret_cast<uint4 *>(part_o);
            if (!routed && qi >= 0 && p.k > 0) {
                // the epilogue will merge this row's routed partials: start them on their way into L2 now.  A 128-byte
                // line holds one pair of pieces of four consecutive queries: every fourth query (and the tile's first) asks
                asm volatile("prefetch.global.L2 [%0];" ::"l"(p.part_lse + ((size_t)h * p.L + qi) * p.k));
                if ((qi & 3) == 0 || r == 0)
                    for (int s = 0; s < p.k; ++s)
                        for (int cc = 0; cc < NP; cc += 2)
                            asm volatile("prefetch.global.L2 [%0];" ::"l"(part16 + part_piece(h_loc, LB, p.k, NP, qi, s, cc)));
            }

            float m_run = -INFINITY, l_run = 0.f;
            TileIter it(it_.rng, it_.nrng);
            int t0, valid, jt = 0;
            while (it.next(t0, valid)) {
                ok = mbar_wait(bar(S_FULL + g), n_s & 1, abort_flag, p.status, W_SFULL);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                uint32_t v[4][32];
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) tmem_ld32(tS + ch * 32, v[ch]);
                tmem_wait_ld();
                if (valid < kBN) {
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch)
#pragma unroll
                        for (int x = 0; x < 32; ++x)
                            if (ch * 32 + x >= valid) v[ch][x] = 0xff800000u;   // -inf
                }
                float m4[4];
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    m4[ch] = -INFINITY;
#pragma unroll
                    for (int x = 0; x < 32; x += 2) m4[ch] = max3(m4[ch], __uint_as_float(v[ch][x]), __uint_as_float(v[ch][x + 1]));
                }
                const float m_new = fmaxf(m_run, fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])) * c);
                float alpha = 1.f;
                if (jt == 0) {
                    m_run = m_new;
                } else if (m_new - m_run > kRescaleThreshold) {
                    alpha = exp2f(m_run - m_new);
                    m_run = m_new;
                }
                // The exponentials of the two query tiles take turns (tile 0 of key tile j, tile 1
                // of j, tile 0 of j + 1, ...): each then has the arithmetic pipes to itself while
                // the other tile's MMAs run, instead of both drifting into lock step.
                // TURN + g is arrived on by group g when its exponentials of a key tile are done.  (Tile 0 waits for
                // tile 1's previous turn even at the start of an item: the barrier must never get two phases ahead of
                // a group that has yet to wait on it.)
                if (two && (g == 1 || n_turn > 0)) {
                    ok = mbar_wait(bar(TURN + (g ^ 1)), (g == 1 ? n_turn : n_turn - 1) & 1, abort_flag, p.status, W_TURN);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                }
                if (__any_sync(0xffffffffu, alpha != 1.f)) {
                    // this group's PV of the previous tile has completed (its commit precedes this tile's S)
#pragma unroll 1
                    for (int ch = 0; ch < D / 32; ++ch) {
                        uint32_t o[32];
                        tmem_ld32(tO + ch * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int x = 0; x < 32; ++x) o[x] = __float_as_uint(__uint_as_float(o[x]) * alpha);
                        tmem_st32(tO + ch * 32, o);
                    }
                }
                // P = exp2(s * c - m), packed bf16 into the P columns (aliasing S).  The first 64 keys
                // are handed to the MMA issuer as soon as they are stored: their P V product overlaps
                // the exponentials of the other 64.
                const uint64_t c2 = pack2(c, c), nm2 = pack2(-m_run, -m_run);
                uint64_t sum_a = 0ull, sum_b = 0ull;   // two packed partial row sums
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t u[16];
#pragma unroll
                    for (int x = 0; x < 16; ++x) {
                        float a0, a1;
                        unpack2(fma2(pack2(__uint_as_float(v[ch][2 * x]), __uint_as_float(v[ch][2 * x + 1])), c2, nm2), a0, a1);
                        a0 = ex2(a0);
                        a1 = ex2(a1);
                        if (x & 1) sum_b = add2(sum_b, pack2(a0, a1));
                        else sum_a = add2(sum_a, pack2(a0, a1));
                        u[x] = bf16x2(a0, a1);
                    }
                    tmem_st16(tP + ch * 16, u);
                    if (ch == 1) {
                        tmem_wait_st();
                        tc_fence_before();
                        mbar_arrive(bar(P_HALF + g));
                    }
                }
                if (two) mbar_arrive(bar(TURN + g));
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(bar(P_FULL + g));
                float s0, s1;
                unpack2(add2(sum_a, sum_b), s0, s1);
                l_run = l_run * alpha + (s0 + s1);
                ++jt;
                ++n_s;
                if (two) ++n_turn;
            }
            if (!ok) break;
            // ---- epilogue
            // The merge weights of the routed partials depend only on log-sum-exps: have them ready before
            // the last P V lands.  wslot[s] = exp(lse_s - lse_total), w_own likewise for this pass's own part.
            const float inv_l = 1.f / l_run;
            const float lse_own = (m_run + log2f(l_run)) * kLn2;
            float w_own = inv_l, big = lse_own, wsum = 1.f;
            constexpr int KW = 8;                     // slots whose weights live in registers
            float wslot[KW];
#pragma unroll
            for (int s = 0; s < KW; ++s) wslot[s] = 0.f;
            const float *pl = nullptr;
            // what this item depends on (an anchor item: the routed items of its group have stored all their partials;
            // a routed item: the anchor items two groups back have read the buffer it is about to store into) has been
            // awaited by the bookkeeping lane, which then arrives on DEPEND, once per item
            if (dep) {
                ok = mbar_wait(bar(DEPEND), dep_phase, abort_flag, p.status, W_DEPEND);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
            }
            if (!routed && qi >= 0 && p.k > 0) {
                pl = p.part_lse + ((size_t)h * p.L + qi) * p.k;
                if (p.k <= KW) {
                    float plv[KW];
#pragma unroll
                    for (int s = 0; s < KW; ++s) plv[s] = s < p.k ? __ldcg(pl + s) : -INFINITY;
#pragma unroll
                    for (int s = 0; s < KW; ++s) big = fmaxf(big, plv[s]);
                    wsum = __expf(lse_own - big);
#pragma unroll
                    for (int s = 0; s < KW; ++s) { wslot[s] = __expf(plv[s] - big); wsum += wslot[s]; }     // exp(-inf) = 0: empty slot
#pragma unroll
                    for (int s = 0; s < KW; ++s) wslot[s] /= wsum;
                } else {
                    for (int s = 0; s < p.k; ++s) big = fmaxf(big, __ldcg(pl + s));
                    wsum = __expf(lse_own - big);
                    for (int s = 0; s < p.k; ++s) wsum += __expf(__ldcg(pl + s) - big);
                }
                w_own = __expf(lse_own - big) / wsum * inv_l;
            }
            ok = mbar_wait(bar(O_FULL + g), n_mine & 1, abort_flag, p.status, W_OFULL);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
#pragma unroll 1
            for (int ch = 0; ch < D / 32; ++ch) {
                uint32_t v[32];
                __syncwarp();
                tmem_ld32(tO + ch * 32, v);
                tmem_wait_ld();
                if (ch == D / 32 - 1) {
                    // O has been read: the issuer may start the next item's P V (which overwrites it)
                    tc_fence_before();
                    mbar_arrive(bar(O_FREE + g));
                }
                float acc[32];
#pragma unroll
                for (int x = 0; x < 32; ++x) acc[x] = __uint_as_float(v[x]) * w_own;
                if (pl && p.k <= KW) {
                    // four slots' pieces of this column block are requested together: one round trip, not four
#pragma unroll
                    for (int s0 = 0; s0 < KW; s0 += 4) {
                        if (s0 >= p.k) break;
                        uint4 raw[4][4];
#pragma unroll
                        for (int s = 0; s < 4; ++s)
#pragma unroll
                            for (int q4 = 0; q4 < 4; q4 += 2) {
                                raw[s][q4] = raw[s][q4 + 1] = make_uint4(0, 0, 0, 0);
                                if (s0 + s < p.k && wslot[s0 + s] != 0.f)
                                    ld_cg_256(part16 + part_piece(h_loc, LB, p.k, NP, qi, s0 + s, ch * 4 + q4), raw[s][q4], raw[s][q4 + 1]);
                            }
#pragma unroll
                        for (int s = 0; s < 4; ++s) {
                            const float w = wslot[s0 + s];
#pragma unroll
                            for (int q4 = 0; q4 < 4; ++q4) {
                                const __nv_bfloat162 *b = reinterpret_cast<const __nv_bfloat162 *>(&raw[s][q4]);
#pragma unroll
                                for (int y = 0; y < 4; ++y) {
                                    const float2 f = __bfloat1622float2(b[y]);
                                    acc[q4 * 8 + 2 * y] = fmaf(w, f.x, acc[q4 * 8 + 2 * y]);
                                    acc[q4 * 8 + 2 * y + 1] = fmaf(w, f.y, acc[q4 * 8 + 2 * y + 1]);
                                }
                            }
                        }
                    }
                } else if (pl) {
                    for (int s = 0; s < p.k; ++s) {
                        const float ls = __ldcg(pl + s);
                        if (ls == -INFINITY) continue;
                        const float w = __expf(ls - big) / wsum;
                        uint4 raw[4];
                        ld_cg_256(part16 + part_piece(h_loc, LB, p.k, NP, qi, s, ch * 4), raw[0], raw[1]);
                        ld_cg_256(part16 + part_piece(h_loc, LB, p.k, NP, qi, s, ch * 4 + 2), raw[2], raw[3]);
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            const __nv_bfloat162 *b = reinterpret_cast<const __nv_bfloat162 *>(&raw[q4]);
#pragma unroll
                            for (int y = 0; y < 4; ++y) {
                                const float2 f = __bfloat1622float2(b[y]);
                                acc[q4 * 8 + 2 * y] = fmaf(w, f.x, acc[q4 * 8 + 2 * y]);
                                acc[q4 * 8 + 2 * y + 1] = fmaf(w, f.y, acc[q4 * 8 + 2 * y + 1]);
                            }
                        }
                    }
                }
                if (qi < 0) continue;
                uint4 *dst_row = reinterpret_cast<uint4 *>(p.O + ((size_t)h * p.L + qi) * D + ch * 32);
                uint4 out[4];
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    uint32_t *o32 = reinterpret_cast<uint32_t *>(&out[q4]);
#pragma unroll
                    for (int y = 0; y < 4; ++y) {
                        __nv_bfloat162 b = __floats2bfloat162_rn(acc[q4 * 8 + 2 * y], acc[q4 * 8 + 2 * y + 1]);
                        o32[y] = *reinterpret_cast<uint32_t *>(&b);
                    }
                }
                if (routed) {            // whole 32-byte sectors
                    st_256(part16 + part_piece(h_loc, LB, p.k, NP, qi, slot, ch * 4), out[0], out[1]);
                    st_256(part16 + part_piece(h_loc, LB, p.k, NP, qi, slot, ch * 4 + 2), out[2], out[3]);
                } else {
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) dst_row[q4] = out[q4];
                }
            }
            if (qi >= 0) {
                if (routed) p.part_lse[((size_t)h * p.L + qi) * p.k + slot] = lse_own;
                else p.lse[(size_t)h * p.L + qi] = (pl ? big + __logf(wsum) : lse_own);
            }
            // this tile's rows are stored; the bookkeeping lane counts them once all 128 threads are here
            mbar_arrive(bar(ROWS_DONE + g));
            ++n_mine;
        }
    } else if (warp == 8) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
        if (lane == 0) {
            // ------------------------------------------------------------ TMA producer of the K and V tiles
            prefetch_tensormap(&tmK);
            prefetch_tensormap(&tmV);
            int n_item = 0, n_kv = 0;                         // items seen, K/V tiles issued
            int k_last = -1, v_last = -1;                     // last tile whose K / V copy was issued
            bool ok = true;
            while (ok) {
                const int sl = n_item & 1;
                if (!mbar_wait(bar(ITEM_FULL + sl), (n_item >> 1) & 1, abort_flag, p.status, W_ITEMFULL)) break;
                const ItemSlot it_ = s_item[sl];
                mbar_arrive(bar(ITEM_EMPTY + sl));
                ++n_item;
                if (!it_.valid) break;
                const int h = it_.h;
                // the ring of stages runs on from the previous item
                TileIter it(it_.rng, it_.nrng);
                int t0, valid;
                while (it.next(t0, valid)) {
                    const int st = n_kv & 1;
                    const uint32_t ph = (n_kv >> 1) & 1;
                    if (!mbar_wait(bar(K_EMPTY + st), ph ^ 1, abort_flag, p.status, W_KEMPTY)) { ok = false; break; }
                    mbar_expect_tx(bar(K_FULL + st), TILE_BYTES);
#pragma unroll
                    for (int sub = 0; sub < SUB; ++sub)
                        tma_load_2d(sK + st * TILE_BYTES + sub * SUB_BYTES, &tmK, sub * 64, h * p.L + t0, bar(K_FULL + st));
                    k_last = n_kv;
                    if (!mbar_wait(bar(V_EMPTY + st), ph ^ 1, abort_flag, p.status, W_VEMPTY)) { ok = false; break; }
                    mbar_expect_tx(bar(V_FULL + st), TILE_BYTES);
#pragma unroll
                    for (int sub = 0; sub < SUB; ++sub)
                        tma_load_2d(sV + st * TILE_BYTES + sub * SUB_BYTES, &tmV, sub * 64, h * p.L + t0, bar(V_FULL + st));
                    v_last = n_kv;
                    ++n_kv;
                }
            }
            if (*abort_flag) {
                // drain: copies already issued must land before the CTA's shared memory is released
                int dummy_flag = 0;
                for (int b = 0; b < 2; ++b) {
                    const int kj = k_last - b, vj = v_last - b;
                    if (kj >= 0) mbar_wait(bar(K_FULL + (kj & 1)), (kj >> 1) & 1, &dummy_flag, p.status, W_KFULL);
                    if (vj >= 0) mbar_wait(bar(V_FULL + (vj & 1)), (vj >> 1) & 1, &dummy_flag, p.status, W_VFULL);
                }
            }
        } else if (lane == 16) {
            // ------------------------------------------------------------ bookkeeping, item by item:
            // first what the item depends on - an anchor item: the routed items of its group have stored all their
            // partials; a routed item: the anchor items two groups back have read the buffer it will store into -
            // then, when the softmax groups have stored the item's rows, the rows join the phase's count.  The
            // groups' arrivals order their stores before this thread (CTA scope); its fence makes them visible
            // device-wide before the count moves.
            // An item that depends on nothing does not go through DEPEND at all; the rows of an item are counted when
            // the next item has been seen, so that the fence before the count (it waits for the item's stores to
            // land) is not in the way of the next item.  DEPEND is arrived on after the previous item's rows were
            // counted, that is after every softmax thread has passed its previous wait on it.
            int n_item = 0, n_tile[2] = {0, 0};
            int pend_phase = -1, pend_rows = 0;                 // the item whose rows are still to be counted
            bool ok = true;
            while (ok) {
                const int sl = n_item & 1;
                if (!mbar_wait(bar(ITEM_FULL + sl), (n_item >> 1) & 1, abort_flag, p.status, W_ITEMFULL)) break;
                const ItemSlot it_ = s_item[sl];
                mbar_arrive(bar(ITEM_EMPTY + sl));
                ++n_item;
                const int group = it_.phase >> 1;
                const bool dep_anchor = it_.valid && !it_.routed && p.k > 0, dep_routed = it_.valid && it_.routed && group >= 2;
                if (pend_phase >= 0) {
                    const int n_qt = pend_rows > 128 ? 2 : 1;
                    for (int g = 0; ok && g < n_qt; ++g) {
                        ok = mbar_wait(bar(ROWS_DONE + g), n_tile[g] & 1, abort_flag, p.status, W_ROWSDONE);
                        ++n_tile[g];
                    }
                    if (!ok) break;
                    __threadfence();
                    atomicAdd(&phase_tab[3 * pend_phase + 2], pend_rows);
                    pend_phase = -1;
                }
                if (!it_.valid) break;
                if (dep_anchor)
                    ok = wait_count(&phase_tab[3 * (2 * group) + 2], phase_tab[3 * (2 * group) + 1], abort_flag, p.status, W_DEPEND);
                if (dep_routed)
                    ok = wait_count(&phase_tab[3 * (2 * (group - 2) + 1) + 2], phase_tab[3 * (2 * (group - 2) + 1) + 1], abort_flag, p.status, W_DEPEND);
                if (!ok) break;
                if (dep_anchor || dep_routed) {
                    __threadfence();
                    mbar_arrive(bar(DEPEND));
                }
                pend_phase = it_.phase;
                pend_rows = it_.rows;
            }
        }
    } else if (warp < 11) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
        // ------------------------------------------------------------ MMA issuers (one per query tile)
        const int g = warp - 9;
        if (lane == 0) {
            constexpr uint32_t IDESC_PV = idesc_bf16_f32(128, D, 0, 1);
            // Descriptors are built once; inside the issue loops only the 14-bit start-address field
            // (low word, 16-byte units) moves, so one tcgen05.mma costs the issuing thread a few
            // integer instructions.
            const uint64_t q_desc0 = smem_desc_sw128(sQ, 16, 1024), k_desc0 = smem_desc_sw128(sK, 16, 1024);
            const uint64_t v_desc0 = smem_desc_sw128(sV, SUB_BYTES, 1024);
            constexpr uint64_t STAGE = TILE_BYTES >> 4;   // next tile / next stage, in address-field units
            int qb = 0;                                   // Q buffer of this tile in the current item
            auto issue_qk = [&](int st, int valid) {
                const int n_qk = max(16, (valid + 15) & ~15);
                const uint32_t idesc_qk = idesc_bf16_f32(128, n_qk, 0, 0);
                const uint64_t qd = q_desc0 + qb * STAGE, kd = k_desc0 + (st ? STAGE : 0);
                const uint32_t q_lo = (uint32_t)qd, q_hi = (uint32_t)(qd >> 32), k_lo = (uint32_t)kd, k_hi = (uint32_t)(kd >> 32);
                const uint32_t d_s = tmem + g * 128;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t o = ((ks >> 2) * SUB_BYTES + (ks & 3) * 32) >> 4;     // never carries out of the address field
                    mma_ss_lo(d_s, q_lo + o, q_hi, k_lo + o, k_hi, idesc_qk, ks > 0);
                }
            };
            // k-steps [ks0, ks1) of  O_g += P_g V(stage st)  (16 keys each)
            auto issue_pv = [&](int st, int ks0, int ks1, bool accumulate) {
                const uint64_t vd = v_desc0 + (st ? STAGE : 0);
                const uint32_t v_lo = (uint32_t)vd, v_hi = (uint32_t)(vd >> 32);
                const uint32_t d_o = tmem + 256 + g * 128, a_p = tmem + g * 128;
                if (ks1 - ks0 == 4) {
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        mma_ts_lo(d_o, a_p + (ks0 + ks) * 8, v_lo + (ks0 + ks) * (2048 >> 4), v_hi, IDESC_PV, accumulate || ks > 0);
                } else {
                    for (int ks = ks0; ks < ks1; ++ks) mma_ts_lo(d_o, a_p + ks * 8, v_lo + ks * (2048 >> 4), v_hi, IDESC_PV, accumulate || ks > ks0);
                }
            };
            // items seen, items with this tile, K/V tiles seen, P tiles consumed, query tiles loaded before this item
            int n_item = 0, n_mine = 0, n_kv = 0, n_p = 0, n_qtile = 0;
            bool ok = true;
            while (ok) {
                const int sl = n_item & 1;
                if (!mbar_wait(bar(ITEM_FULL + sl), (n_item >> 1) & 1, abort_flag, p.status, W_ITEMFULL)) break;
                const ItemSlot it_ = s_item[sl];
                mbar_arrive(bar(ITEM_EMPTY + sl));
                ++n_item;
                if (!it_.valid) break;
                const int n_tiles = it_.ntiles;
                const int q_seq = n_qtile + g;                      // this tile's place in the sequence of Q loads
                n_qtile += it_.rows > 128 ? 2 : 1;
                if (g == 1 && it_.rows <= 128) {
                    // no second query tile: this issuer only keeps the K/V ring's accounting (each stage is
                    // released by two arrivals)
                    for (int jt = 0; ok && jt < n_tiles; ++jt) {
                        const int st = n_kv & 1;
                        const uint32_t ph = (n_kv >> 1) & 1;
                        ok = mbar_wait(bar(K_FULL + st), ph, abort_flag, p.status, W_KFULL) &&
                             mbar_wait(bar(V_FULL + st), ph, abort_flag, p.status, W_VFULL);
                        if (!ok) break;
                        mbar_arrive(bar(K_EMPTY + st));
                        mbar_arrive(bar(V_EMPTY + st));
                        ++n_kv;
                    }
                    continue;
                }
                qb = q_seq % 3;
                // this issuer serves query tile g: S_g(0), then per key tile  O_g += P_g V(j),  S_g(j + 1)
                TileIter it(it_.rng, it_.nrng);
                int t0, valid, valid_next = 0;
                ok = it.next(t0, valid);
                ok = ok && mbar_wait(bar(Q_FULL + qb), (q_seq / 3) & 1, abort_flag, p.status, W_QFULL);
                ok = ok && mbar_wait(bar(K_FULL + (n_kv & 1)), (n_kv >> 1) & 1, abort_flag, p.status, W_KFULL);
                if (!ok) break;
                tc_fence_after();
                issue_qk(n_kv & 1, valid);
                tc_commit(bar(S_FULL + g));
                tc_commit(bar(K_EMPTY + (n_kv & 1)));
                if (n_tiles == 1) tc_commit(bar(Q_EMPTY + qb));       // that was the item's only S: its Q buffer may be refilled
                for (int jt = 0; ok && jt < n_tiles; ++jt) {
                    const int st = n_kv & 1, sn = (n_kv + 1) & 1;
                    const uint32_t ph = (n_kv >> 1) & 1, phn = ((n_kv + 1) >> 1) & 1;
                    const bool more = it.next(t0, valid_next);
                    if (!mbar_wait(bar(V_FULL + st), ph, abort_flag, p.status, W_VFULL)) { ok = false; break; }
                    if (more && !mbar_wait(bar(K_FULL + sn), phn, abort_flag, p.status, W_KFULL)) { ok = false; break; }
                    const int steps = (valid + 15) >> 4, half = min(steps, 4);
                    if (!mbar_wait(bar(P_HALF + g), n_p & 1, abort_flag, p.status, W_PHALF)) { ok = false; break; }
                    // the first P V of an item overwrites O: the previous item's epilogue must have read it
                    if (jt == 0 && n_mine > 0 && !mbar_wait(bar(O_FREE + g), (n_mine - 1) & 1, abort_flag, p.status, W_OFREE)) { ok = false; break; }
                    tc_fence_after();
                    issue_pv(st, 0, half, jt > 0);
                    if (!mbar_wait(bar(P_FULL + g), n_p & 1, abort_flag, p.status, W_PFULL)) { ok = false; break; }
                    tc_fence_after();
                    if (steps > half) issue_pv(st, half, steps, true);
                    // a commit between two groups of MMAs leaves the pipe idle: the next S goes out first, then all commits
                    if (more) {
                        issue_qk(sn, valid_next);
                        tc_commit(bar(S_FULL + g));
                        tc_commit(bar(V_EMPTY + st));
                        tc_commit(bar(K_EMPTY + sn));
                        if (jt + 2 == n_tiles) tc_commit(bar(Q_EMPTY + qb));      // the item's last S: its Q buffer may be refilled
                    } else {
                        tc_commit(bar(V_EMPTY + st));
                        tc_commit(bar(O_FULL + g));
                    }
                    valid = valid_next;
                    ++n_kv;
                    ++n_p;
                }
                ++n_mine;
            }
        }
    } else {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
        // ------------------------------------------------------------ scheduler (lane 0 claims items in queue order) and
        // Q loader (the whole warp): a claimed item is published at once, then its query tiles are loaded as their
        // buffers come free, which for the first tile is before the previous item has finished
        bool usable = false;
        int total = 0, n_phases = 0;
        if (lane == 0) {
            usable = *(volatile int *)p.status == 0 && (uint32_t)((volatile int *)p.status)[ST_COOKIE] == p.cookie;
            if (!usable) atomicCAS(p.status, 0, MOC_ERR_WORKSPACE);      // not this plan's lists: report, touch nothing else
            total = usable ? p.queue[1] : 0;
            n_phases = p.queue[2];
            prefetch_tensormap(&tmQ);
            prefetch_tensormap(&tmQrow);
        }
        int n_item = 0, n_qtile = 0;
        bool ok = true;
        while (ok) {
            const int sl = n_item & 1;
            ItemSlot s;
            s.valid = 0; s.routed = 0; s.h = 0; s.first = 0; s.rows = 0; s.nrng = 0; s.ntiles = 0; s.phase = 0; s.rng = nullptr;
            if (lane == 0) {
                if (n_item >= 2) ok = mbar_wait(bar(ITEM_EMPTY + sl), ((n_item - 2) >> 1) & 1, abort_flag, p.status, W_ITEMEMPTY);
                const int t = (ok && usable && !*abort_flag && *(volatile int *)p.status == 0) ? atomicAdd(&p.queue[0], 1) : total;
                if (t < total) {
                    int ph = 0;
                    while (ph + 1 < n_phases && phase_tab[3 * (ph + 1)] <= t) ++ph;
                    const int local = t - phase_tab[3 * ph], group = ph >> 1, h0 = group * p.hg;
                    WorkItem w;
                    s.routed = (ph & 1) == 0;
                    if (s.routed) {
                        w = p.ritems[p.tile_off[(size_t)h0 * p.C] + local];
                        s.h = w.h;
                        s.rng = p.chunk_rng + w.rng_off;
                    } else {
                        w = p.aitems[local % p.n_aitems];
                        s.h = h0 + local / p.n_aitems;
                        s.rng = p.anc_rng + w.rng_off;
                    }
                    s.first = w.first; s.rows = w.rows; s.nrng = w.nrng; s.ntiles = w.ntiles; s.phase = ph;
                    s.valid = 1;
                    if (s.routed && !index_ok((unsigned)w.h < (unsigned)p.H && w.rows > 0 && w.rows <= kQTileRows && w.first >= 0 &&
                                              (size_t)w.first + w.rows <= p.cap_total && w.nrng == 1, p.status, IX_ITEM_FIELDS))
                        s.valid = 0;
                }
                s_item[sl] = s;
                __threadfence_block();
                mbar_arrive(bar(ITEM_FULL + sl));
            }
            ++n_item;
            // the rest of the warp learns the item from lane 0
            const int valid = __shfl_sync(0xffffffffu, s.valid, 0), routed = __shfl_sync(0xffffffffu, s.routed, 0);
            const int h = __shfl_sync(0xffffffffu, s.h, 0), first = __shfl_sync(0xffffffffu, s.first, 0), rows = __shfl_sync(0xffffffffu, s.rows, 0);
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            if (!valid || !ok) break;
            const int n_qt = rows > 128 ? 2 : 1;
            for (int g = 0; ok && g < n_qt; ++g) {
                const int qb = n_qtile % 3;
                ok = mbar_wait(bar(Q_EMPTY + qb), ((n_qtile / 3) & 1) ^ 1, abort_flag, p.status, W_QEMPTY);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (lane == 0) mbar_expect_tx(bar(Q_FULL + qb), TILE_BYTES);
                __syncwarp();
                if (!routed) {
                    if (lane == 0) {
#pragma unroll
                        for (int sub = 0; sub < SUB; ++sub)
                            tma_load_2d(sQ + qb * TILE_BYTES + sub * SUB_BYTES, &tmQ, sub * 64, h * p.L + first + g * 128, bar(Q_FULL + qb));
                    }
                } else {
                    // lane l gathers rows 4 l .. 4 l + 3 of the tile; a row past the item's end repeats the item's
                    // first query (its result is never stored)
                    int row[4];
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        const int rt = g * 128 + lane * 4 + x;
                        const size_t at = (size_t)first + (rt < rows ? rt : 0);
                        const int e = at < p.cap_total ? p.qlist[(size_t)h * p.cap_total + at] : 0;
                        int qi = e / p.k;
                        if (e < 0 || qi >= p.L) qi = 0;
                        row[x] = h * p.L + qi;
                    }
#pragma unroll
                    for (int sub = 0; sub < SUB; ++sub)
                        tma_gather4(sQ + qb * TILE_BYTES + sub * SUB_BYTES + lane * 512, &tmQrow, sub * 64, row[0], row[1], row[2], row[3],
                                    bar(Q_FULL + qb));
                }
                ++n_qtile;
            }
        }
        if (*abort_flag && lane == 0) {
            // drain: the Q copies already issued must land before the CTA's shared memory is released
            int dummy_flag = 0;
            for (int b = 1; b <= 3; ++b) {
                const int qj = n_qtile - b;
                if (qj >= 0) mbar_wait(bar(Q_FULL + qj % 3), (qj / 3) & 1, &dummy_flag, p.status, W_QFULL);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 8) tmem_dealloc(tmem, kTmemCols);
}

// ---- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int make_tmap_2d_bf16(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        MOC_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q));
        if (!sym || q != cudaDriverEntryPointSuccess) { set_cuda_error(cudaErrorUnknown, "cuTensorMapEncodeTiled not found"); return MOC_ERR_CUDA; }
        fn = (EncodeTiledFn)sym;
    }
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled"); return MOC_ERR_CUDA; }
    return MOC_OK;
}

template <int D>
static int attend_tc_d(const moc_plan *p, const __nv_bfloat16 *Q, const __nv_bfloat16 *K, const __nv_bfloat16 *V,
                       __nv_bfloat16 *O, float *lse, void *ws, cudaStream_t s) {
    CUtensorMap tmQ, tmQrow, tmK, tmV;
    if (int r = make_tmap_2d_bf16(&tmQ, Q, (uint64_t)p->H * p->L, D, 128)) return r;
    if (int r = make_tmap_2d_bf16(&tmQrow, Q, (uint64_t)p->H * p->L, D, 1)) return r;      // row gathers: a box one row high
    if (int r = make_tmap_2d_bf16(&tmK, K, (uint64_t)p->H * p->L, D, kBN)) return r;
    if (int r = make_tmap_2d_bf16(&tmV, V, (uint64_t)p->H * p->L, D, kBN)) return r;
    const int n_groups = (p->H + p->heads_per_group - 1) / p->heads_per_group;
    AttendParams a;
    a.Q = Q; a.O = O; a.lse = lse;
    a.part_o = ws_ptr<__nv_bfloat16>(ws, p->ws.part_o);
    a.part_lse = ws_ptr<float>(ws, p->ws.part_lse);
    a.part_stride = n_groups > 1 ? (size_t)p->heads_per_group * ((p->L + 127) / 128 * 128) * p->k * D : 0;
    a.chunk_rng = p->d_chunk_rng; a.anc_rng = p->d_anc_rng;
    a.ritems = ws_ptr<WorkItem>(ws, p->ws.rtiles);
    a.aitems = p->d_qitems;
    a.tile_off = ws_ptr<int>(ws, p->ws.tile_off);
    a.qlist = ws_ptr<int32_t>(ws, p->ws.qlist);
    a.queue = ws_ptr<int>(ws, p->ws.queue);
    a.cap_total = (size_t)p->cap_off[p->C];
    a.status = ws_ptr<int>(ws, p->ws.status);
    a.H = p->H; a.L = p->L; a.C = p->C; a.k = p->k; a.hg = p->heads_per_group; a.n_groups = n_groups;
    a.n_aitems = (int)p->qitems.size();
    a.scale_log2 = p->scale * 1.4426950408889634f;
    a.cookie = p->cookie;
    attend_queue_kernel<<<1, 256, 0, s>>>(a.queue, a.tile_off, ws_ptr<int>(ws, p->ws.cnt), a.status, p->cookie, p->H, p->L, p->C, p->k,
                                          p->heads_per_group, n_groups, a.n_aitems);
    MOC_LAUNCH_CHECK();
    // always the d = 128 footprint: more than half an SM's shared memory, so CTAs (which each
    // take all 512 TMEM columns) never share an SM
    const size_t smem = 7 * (size_t)128 * 128 * 2 + 1024;      // Q ring of three, K and V two stages each
    MOC_CUDA_TRY(cudaFuncSetAttribute(attend_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    // one CTA per SM, never more than there are anchor items (the least the queue can hold)
    const long long most = (long long)p->H * a.n_aitems;
    const unsigned grid = (unsigned)std::max(1LL, std::min<long long>(p->n_sm, most));
    attend_tc_kernel<D><<<grid, kThreads, smem, s>>>(tmQ, tmQrow, tmK, tmV, a);
    MOC_LAUNCH_CHECK();
    return MOC_OK;
}

int launch_attend_tc(const moc_plan *p, const __nv_bfloat16 *Q, const __nv_bfloat16 *K, const __nv_bfloat16 *V,
                     const int32_t *, __nv_bfloat16 *O, float *lse, void *ws, cudaStream_t s) {
    return p->d == 128 ? attend_tc_d<128>(p, Q, K, V, O, lse, ws, s) : attend_tc_d<64>(p, Q, K, V, O, lse, ws, s);
}

}  // namespace moc
