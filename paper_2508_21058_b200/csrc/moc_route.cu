// Routing: scores of every query against every chunk descriptor, causal chunk mask,
// anchors removed from the candidates, top-k per query (ties to the lower chunk index),
// and the inverse index (per head and chunk, the list of (query, slot) pairs that
// picked it) which the key-stationary attention pass consumes.
//
// The scores are a dense [L, d] x [d, C] contraction per head, so they run on the tensor
// cores.  Q is bf16 already; each fp32 descriptor is split once into three bf16 terms
// (hi + mid + lo carries its 24-bit mantissa), and S = Q hi^T + Q mid^T + Q lo^T is
// accumulated in fp32 in TMEM: every product is exact, only the fp32 accumulation rounds.
//
// route_prep_kernel   splits the descriptors, clears the pick counters and the status words (few chunks: the
//                     routing kernel splits them itself and a memset does the clearing).
// route_tc_kernel     H x (SMs / H) CTAs; the 128-query tiles ("units") of a head are dealt round-robin
//                     to the head's CTAs:
//     warp 0      TMA producer: Q tiles (ring of stages) and the head's descriptor block;
//     warps 1, 10 MMA issuers: 3 x d/16 MMAs per 128 chunks into one of two TMEM accumulators
//                 (warp 1 the even units, warp 10 the odd ones);
//     warps 2-5 / 6-9   selection groups (one, two or four: the units in turn), one query per thread (TMEM
//                 lane = query): read the scores 32 chunks at a time, drop non-candidates,
//                 keep a sorted top-k in registers (at most 64 entries; more picks are taken in
//                 passes of 64 over recomputed scores), then write sel_idx and append the picks
//                 to the per-(head, chunk) query lists (tile-local ranks from a shared-memory
//                 histogram, one global atomic per (tile, chunk) to reserve the range).
//   The head's descriptors stay in shared memory for the CTA's lifetime (C <= 192) and are scored
//   in steps of at most 128 chunks; with more chunks they are streamed in blocks of 128 and warp 1
//   alone issues.
//   With at most 32 padded chunks (and k <= 8) the three terms of the split descriptors form one MMA
//   operand, the selection adds the three column groups and every candidate sinks through the sorted
//   list in one pass (template parameter FEW).
// route_tiles_kernel  running count of attention tiles over (head, chunk) from the pick counts;
// route_items_kernel  the routed attention work items (one per 256 picks of a chunk).
// Every mbarrier wait is bounded; a wait that runs out flags the workspace status word.
#include <float.h>
#include <algorithm>

#include "moc_common.cuh"
#include "moc_tc.cuh"

namespace moc {

using namespace tc;

constexpr int kRtRows = 128;          // queries per tile
__host__ __device__ constexpr int rt_threads(int ng) { return 64 + 128 * ng + 64; }   // producer, issuer | NG selection groups | second issuer, idle
constexpr int kRtResident = 192;      // up to this many (padded) chunks the whole block stays resident
constexpr int kRtBlock = 128;         // otherwise chunks are streamed in blocks of this many
constexpr int kRtDeferredChunks = 512; // up to this many chunks (and 8 picks) a unit's list append is finished behind the next unit's selection

enum RouteWait { RW_QFULL = 32, RW_QEMPTY, RW_DFULL, RW_DEMPTY, RW_ACCFULL, RW_ACCEMPTY, RW_GROUP };

template <int KMAX>
struct TopK {
    float s[KMAX];
    int j[KMAX];
    __device__ __forceinline__ void init() {
#pragma unroll
        for (int x = 0; x < KMAX; ++x) { s[x] = -INFINITY; j[x] = -1; }
    }
};

// desc3[h][t][col][:] for t = 0, 1, 2: bf16 terms of the descriptor of score column col (the col-th non-text
// chunk; rows beyond the last column are zero); also clears the pick counters and the status words (the workspace holds no plan's lists until they
// are complete) and states the limit of the bounded waits.  With desc == nullptr only the clearing is done.
__global__ void route_prep_kernel(const float *__restrict__ desc, __nv_bfloat16 *__restrict__ desc3, int *__restrict__ cnt,
                                  int *__restrict__ status, const int32_t *__restrict__ col_chunk, int H, int C, int ncol,
                                  int c_pad, int d, unsigned wait_us) {
    const size_t n = desc ? (size_t)H * c_pad * d : 0;
    const size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    if (i < (size_t)H * C) cnt[i] = 0;
    if (i < kStatusWords) status[i] = i == ST_WAIT_US ? (int)wait_us : 0;
    if (i >= n) return;
    const int x = (int)(i % d);
    const int c = (int)((i / d) % c_pad);
    const int h = (int)(i / ((size_t)d * c_pad));
    float v = c < ncol ? desc[((size_t)h * C + col_chunk[c]) * d + x] : 0.f;
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    v -= __bfloat162float(hi);
    const __nv_bfloat16 mid = __float2bfloat16_rn(v);
    v -= __bfloat162float(mid);
    const __nv_bfloat16 lo = __float2bfloat16_rn(v);
    const size_t plane = (size_t)c_pad * d, base = (size_t)h * 3 * plane + (size_t)c * d + x;
    desc3[base] = hi;
    desc3[base + plane] = mid;
    desc3[base + 2 * plane] = lo;
}

struct RouteParams {
    const float *desc;      // few-chunk case: the fp32 descriptors, split into their three terms by the kernel itself (else nullptr)
    unsigned wait_us;       // limit of the bounded waits, stated in the status words by the kernel in that case
    int32_t *sel;
    float *part_lse;
    int *cnt;
    int32_t *qlist;
    const int32_t *tok_chunk;
    const uint32_t *cand_c;     // [C][cwords] candidate columns per query chunk
    const int32_t *lim;         // [C] prefix mode: the candidates of a query in chunk c are the columns [0, lim[c])
    const int32_t *reach;       // [C] columns any query up to chunk c can pick from
    const int32_t *col_chunk;   // [ncol] chunk of a score column
    const int32_t *cap_off;
    int *status;
    int H, L, C, ncol, c_pad, k, cwords, prefix;
    int tiles_per_head;     // ceil(L / 128)
    int ctas_per_head;      // the grid is H * ctas_per_head
    int sb_rows;            // chunks per scoring step (one accumulator's worth)
    int d_rows;             // descriptor rows per term held in shared memory: c_pad (resident) or sb_rows (streamed)
    int q_stages;
    int n_pass;             // selection passes over a tile's scores: 64 picks each (the scores are recomputed per pass)
    int surv_cap;           // threshold selection: survivor slots per query row in shared memory (0 = not used)
    int *tile_off;          // [H C + 1] running tile counts, written by the last block to finish
    uint32_t cookie;
    size_t cap_total;
};

// score columns a tile can pick from: what the chunk of its last row can reach
__device__ __forceinline__ int chunks_in_reach(const RouteParams &p, int t) {
    return p.reach[p.tok_chunk[min(p.L, (t + 1) * kRtRows) - 1]];
}

// FEW (at most 32 padded chunks, k <= 8): the three descriptor terms form one B operand of 3 c_pad rows, so a
// tile costs one MMA chain instead of three (an MMA costs the same for any N <= 128); the selection adds the
// three column groups and lets every candidate in reach sink through the sorted list in one pass.
template <int D, int KMAX, int NG, bool FEW>
__global__ void __launch_bounds__(rt_threads(NG), 1) route_tc_kernel(const __grid_constant__ CUtensorMap tmQ,
                                                                 const __grid_constant__ CUtensorMap tmD,
                                                                 const RouteParams p) {
    constexpr int SUB = D / 64;
    constexpr int Q_SUB_BYTES = kRtRows * 128, Q_TILE_BYTES = SUB * Q_SUB_BYTES;
    constexpr int kMaxStages = 4;
    extern __shared__ uint8_t smem_raw[];
    constexpr int kRtThreads = rt_threads(NG);
    __shared__ __align__(8) uint64_t bars[2 * kMaxStages + 2 + 3 * NG];
    __shared__ uint32_t tmem_slot;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gbase = smem_raw + (sbase - smem_u32(smem_raw));
    // shared memory: descriptor block (3 terms x SUB sub-tiles of d_rows x 128 bytes) | Q stages | histograms
    const int d_sub_bytes = p.d_rows * 128;
    const uint32_t sD = sbase;
    const uint32_t sQ = sD + ((3 * SUB * d_sub_bytes + 1023) & ~1023);
    int *hist_base = reinterpret_cast<int *>(gbase + (sQ - sbase) + p.q_stages * Q_TILE_BYTES);
    // per selection group: one histogram of C counters, or (deferred list append) two alternating histograms and
    // two alternating tables of list bases
    const int hist_ints = (KMAX <= 8 && p.C <= kRtDeferredChunks ? 4 : 1) * p.C;
    int *s_cap = hist_base + NG * hist_ints;                             // copy of cap_off[0 .. C)
    int *s_col = s_cap + p.C;                                            // copy of col_chunk[0 .. ncol)
    // per unit of this CTA, packed: columns in reach (bits 0-15), scoring steps (16-23), Q stage (24-27) and the parity
    // of that stage's use (28): worked out once by all threads, so that the single threads that load and issue never divide
    uint32_t *s_unit = reinterpret_cast<uint32_t *>(s_col + p.ncol);
    // threshold selection: per group, surv_cap slots of (score, column) per query row; slot e of row r at [e][r]
    float *surv_base = reinterpret_cast<float *>(reinterpret_cast<uintptr_t>(s_unit + p.tiles_per_head / p.ctas_per_head + 16) + 15 & ~(uintptr_t)15);
    auto bar = [&](int i) { return smem_u32(&bars[i]); };
    constexpr int Q_FULL = 0, Q_EMPTY = kMaxStages, D_FULL = 2 * kMaxStages, D_EMPTY = D_FULL + 1, ACC_FULL = D_FULL + 2,
                  ACC_EMPTY = ACC_FULL + NG, GROUP = ACC_EMPTY + NG;

    if (threadIdx.x == 0) {
        s_abort = 0;
        if (FEW && p.desc) p.status[ST_WAIT_US] = (int)p.wait_us;       // every block writes the same value, before any of its waits
        for (int t = 0; t < kMaxStages; ++t) { mbar_init(bar(Q_FULL + t), 1); mbar_init(bar(Q_EMPTY + t), 1); }
        mbar_init(bar(D_FULL), 1);
        mbar_init(bar(D_EMPTY), 1);
        for (int t = 0; t < NG; ++t) {
            mbar_init(bar(ACC_FULL + t), 1);
            mbar_init(bar(ACC_EMPTY + t), 128);
            mbar_init(bar(GROUP + t), 128);
        }
        fence_barrier_init();
    }
    __syncthreads();
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    volatile int *abort_flag = &s_abort;

    // this CTA's units: 128-query tiles of ONE head (u counts tiles of that head), so its descriptor block
    // never changes while it fits in shared memory
    const int h = blockIdx.x / p.ctas_per_head, part = blockIdx.x % p.ctas_per_head;
    // the head's tiles are dealt round-robin to its CTAs: a tile's work grows with the chunks in its causal
    // reach, i.e. with its position, and contiguous ranges would leave the last CTA of a head the slowest
    const int nu = (p.tiles_per_head - part + p.ctas_per_head - 1) / p.ctas_per_head;      // units of this CTA
    auto unit_of = [&](int n) { return part + n * p.ctas_per_head; };
    for (int x = threadIdx.x; x < p.C; x += kRtThreads) s_cap[x] = p.cap_off[x];
    for (int x = threadIdx.x; x < p.ncol; x += kRtThreads) s_col[x] = p.col_chunk[x];
    for (int x = threadIdx.x; x < nu; x += kRtThreads) {
        const int reach = chunks_in_reach(p, unit_of(x));
        s_unit[x] = (uint32_t)reach | (uint32_t)max(1, (reach + p.sb_rows - 1) / p.sb_rows) << 16 | (uint32_t)(x % p.q_stages) << 24 |
                    (uint32_t)((x / p.q_stages) & 1) << 28;
    }
    if (FEW && p.desc) {
        // Few chunks: the head's descriptor block is small enough for the block to split it into its three bf16 terms
        // itself, straight into the swizzled operand layout (what the copy of the pre-split block would have
        // written), which saves the launch that prepares the split block.  One 16-byte piece (8 columns) per thread.
        constexpr int PIECES = D / 8;
        for (int x = threadIdx.x; x < p.c_pad * PIECES; x += kRtThreads) {
            const int col = x / PIECES, pc = x % PIECES;
            float v[8];
#pragma unroll
            for (int y = 0; y < 8; ++y) v[y] = 0.f;
            if (col < p.ncol) {
                const float4 *src = reinterpret_cast<const float4 *>(p.desc + ((size_t)h * p.C + p.col_chunk[col]) * D + pc * 8);
                const float4 a = __ldg(src), b = __ldg(src + 1);
                v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
            }
            uint32_t t3[3][4];
#pragma unroll
            for (int y = 0; y < 4; ++y) {
                float r0 = v[2 * y], r1 = v[2 * y + 1];
#pragma unroll
                for (int term = 0; term < 3; ++term) {
                    const __nv_bfloat16 b0 = __float2bfloat16_rn(r0), b1 = __float2bfloat16_rn(r1);
                    r0 -= __bfloat162float(b0);
                    r1 -= __bfloat162float(b1);
                    t3[term][y] = (uint32_t)__bfloat16_as_ushort(b0) | ((uint32_t)__bfloat16_as_ushort(b1) << 16);
                }
            }
            const int sub = pc >> 3, c16 = pc & 7;
#pragma unroll
            for (int term = 0; term < 3; ++term)
                *reinterpret_cast<uint4 *>(gbase + (sub * 3 + term) * d_sub_bytes + sw128_offset(col, c16)) =
                    make_uint4(t3[term][0], t3[term][1], t3[term][2], t3[term][3]);
        }
        fence_proxy_async_smem();       // the tensor core reads these through the async proxy
    }
    auto reach_of = [&](int n) { return (int)(s_unit[n] & 0xffffu); };
    auto steps_of = [&](int n) { return (int)((s_unit[n] >> 16) & 0xffu); };
    auto qstage_of = [&](int n) { return (int)((s_unit[n] >> 24) & 0xfu); };
    auto qparity_of = [&](int n) { return (int)((s_unit[n] >> 28) & 1u); };
    __syncthreads();
    constexpr int ACC_COLS = 512 / NG;   // TMEM columns per accumulator (NG = 4 only with sb_rows <= 128)
    const int n_pass = KMAX == 64 ? p.n_pass : 1;     // only the 64-entry list is used for more picks than it holds
    const bool resident = p.d_rows == p.c_pad;       // every chunk's descriptor is held: loaded once, two MMA issuers

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tensormap(&tmQ);
            prefetch_tensormap(&tmD);
            int res_sb = -1, qn = 0, dn = 0;
            bool ok = true;
            // Streamed descriptor blocks are shared by a round of NG consecutive units (one per selection group):
            // the round's Q tiles are loaded first, then every block is loaded once and scored against all of
            // them.  With a resident block a round is one unit.
            const int grp = resident ? 1 : NG;
            for (int n0 = 0; ok && n0 < nu; n0 += grp) {
                const int n1 = min(n0 + grp, nu);
                int n_sb = 1;
                for (int n = n0; n < n1; ++n) n_sb = max(n_sb, steps_of(n));   // blocks that hold a column in reach
                for (int n = n0; ok && n < n1; ++n) {
                    const int st = qstage_of(n);                          // qn == n: one Q tile per unit, in unit order
                    ok = mbar_wait(bar(Q_EMPTY + st), qparity_of(n) ^ 1, abort_flag, p.status, RW_QEMPTY);
                    if (!ok) break;
                    mbar_expect_tx(bar(Q_FULL + st), Q_TILE_BYTES);
#pragma unroll
                    for (int sub = 0; sub < SUB; ++sub)
                        tma_load_2d(sQ + st * Q_TILE_BYTES + sub * Q_SUB_BYTES, &tmQ, sub * 64, h * p.L + unit_of(n) * kRtRows, bar(Q_FULL + st));
                    ++qn;
                }
                for (int rep = 0; ok && rep < n_pass; ++rep)
                for (int sb = 0; ok && sb < n_sb; ++sb) {
                    if (resident ? dn == 0 : sb != res_sb) {
                        ok = mbar_wait(bar(D_EMPTY), (dn & 1) ^ 1, abort_flag, p.status, RW_DEMPTY);
                        if (!ok) break;
                        if (FEW && p.desc) {
                            mbar_arrive(bar(D_FULL));       // the block wrote the terms itself, before the roles parted
                        } else {
                            mbar_expect_tx(bar(D_FULL), 3 * SUB * d_sub_bytes);
                            for (int term = 0; term < 3; ++term)
#pragma unroll
                                for (int sub = 0; sub < SUB; ++sub)
                                    tma_load_2d(sD + (sub * 3 + term) * d_sub_bytes, &tmD, sub * 64,
                                                (h * 3 + term) * p.c_pad + (resident ? 0 : sb * p.sb_rows), bar(D_FULL));
                        }
                        ++dn;
                        res_sb = sb;
                    }
                }
            }
            if (*abort_flag) {
                // drain: copies already issued must land before the CTA's shared memory is released
                int dummy_flag = 0;
                for (int b = 1; b <= p.q_stages; ++b) {
                    const int qj = qn - b;
                    if (qj >= 0) mbar_wait(bar(Q_FULL + qj % p.q_stages), (qj / p.q_stages) & 1, &dummy_flag, p.status, RW_QFULL);
                }
                if (dn > 0) mbar_wait(bar(D_FULL), (dn - 1) & 1, &dummy_flag, p.status, RW_DFULL);
            }
        }
    } else if (warp == 1 || warp == 2 + 4 * NG) {
        // ------------------------------------------------------------ MMA issuers
        // With a resident descriptor block, warp 1 serves the even units and the last warpgroup's first warp
        // the odd ones (each its own accumulators), so one issuer's waits and instruction overhead hide behind the other's
        // MMAs; when blocks are streamed, warp 1 serves every unit and follows the reloads.
        const bool dual = resident && NG > 1;          // one selection group has one accumulator: one issuer
        const int first = warp == 1 ? 0 : 1, stride = dual ? 2 : 1;
        if (lane == 0 && (warp == 1 || dual)) {
            // descriptors are built once: issuing an MMA should cost this thread a few integer instructions
            const uint64_t q_desc0 = smem_desc_sw128(sQ, 16, 1024);
            uint64_t d_term[3 * SUB];
#pragma unroll
            for (int x = 0; x < 3 * SUB; ++x)            // the three terms of a 64-column slice lie one after another
                d_term[x] = smem_desc_sw128(sD + ((x % SUB) * 3 + x / SUB) * d_sub_bytes, 16, 1024);
            int res_sb = -1, dn = 0;
            int nacc_total[NG];
#pragma unroll
            for (int x = 0; x < NG; ++x) nacc_total[x] = 0;
            bool ok = true;
            // a round: one unit (resident block; the two issuers take alternate units), or NG consecutive units that
            // share every streamed block
            const int grp = resident ? 1 : NG;
            for (int n0 = first; ok && n0 < nu; n0 += resident ? stride : grp) {
                const int n1 = min(n0 + grp, nu);
                int n_sb = 1;
                for (int n = n0; n < n1; ++n) n_sb = max(n_sb, steps_of(n));
                for (int n = n0; ok && n < n1; ++n)
                    ok = mbar_wait(bar(Q_FULL + qstage_of(n)), qparity_of(n), abort_flag, p.status, RW_QFULL);
                for (int rep = 0; ok && rep < n_pass; ++rep)
                for (int sb = 0; ok && sb < n_sb; ++sb) {
                    if (resident ? dn == 0 : sb != res_sb) {
                        ok = mbar_wait(bar(D_FULL), dn & 1, abort_flag, p.status, RW_DFULL);
                        if (!ok) break;
                        ++dn;
                        res_sb = sb;
                    }
                    for (int n = n0; ok && n < n1; ++n) {
                        const int reach = reach_of(n);
                        if (sb >= steps_of(n)) continue;       // this unit needs no such block
                        const int buf = n % NG, st = qstage_of(n);
                        int uses = 0;                          // how often this accumulator has been filled (no indexed array:
#pragma unroll                                                 // the counters stay in registers)
                        for (int x = 0; x < NG; ++x) uses = x == buf ? nacc_total[x] : uses;
                        ok = mbar_wait(bar(ACC_EMPTY + buf), (uses & 1) ^ 1, abort_flag, p.status, RW_ACCEMPTY);
                        if (!ok) break;
                        tc_fence_after();
                        const int rows_sb = max(16, min(min(p.sb_rows, p.c_pad - sb * p.sb_rows), (reach - sb * p.sb_rows + 15) & ~15));
                        const uint64_t qd = q_desc0 + (uint64_t)(st * (Q_TILE_BYTES >> 4));
                        if (FEW) {
                            // one chain: B = the 3 c_pad rows (hi, mid, lo terms) of the block, three column groups out
                            const uint32_t idesc = idesc_bf16_f32(128, 3 * p.c_pad, 0, 0);
                            const uint32_t acc = tmem + buf * ACC_COLS;
#pragma unroll
                            for (int ks = 0; ks < D / 16; ++ks)
                                mma_ss_lo(acc, (uint32_t)qd + (((ks >> 2) * Q_SUB_BYTES + (ks & 3) * 32) >> 4), (uint32_t)(qd >> 32),
                                          (uint32_t)d_term[ks >> 2] + (((ks & 3) * 32) >> 4), (uint32_t)(d_term[ks >> 2] >> 32), idesc, ks != 0);
                        } else {
                            // one instruction spans the step's columns (at most 256)
                            const uint32_t idesc = idesc_bf16_f32(128, rows_sb, 0, 0);
                            const uint32_t acc = tmem + buf * ACC_COLS;
                            const uint32_t nofs = (uint32_t)((resident ? sb * p.sb_rows : 0) * 128) >> 4;
#pragma unroll
                            for (int term = 0; term < 3; ++term) {
#pragma unroll
                                for (int ks = 0; ks < D / 16; ++ks)
                                    mma_ss_lo(acc, (uint32_t)qd + (((ks >> 2) * Q_SUB_BYTES + (ks & 3) * 32) >> 4), (uint32_t)(qd >> 32),
                                              (uint32_t)d_term[term * SUB + (ks >> 2)] + nofs + (((ks & 3) * 32) >> 4),
                                              (uint32_t)(d_term[term * SUB + (ks >> 2)] >> 32), idesc, (term | ks) != 0);
                            }
                        }
                        tc_commit(bar(ACC_FULL + buf));
#pragma unroll
                        for (int x = 0; x < NG; ++x) nacc_total[x] += x == buf ? 1 : 0;
                    }
                    // streamed blocks: the next step, if it needs another block, may overwrite this one once
                    // these MMAs are done
                    if (ok && !resident) {
                        int nsb = sb + 1;
                        bool more = true;
                        if (nsb >= n_sb) { nsb = 0; more = rep + 1 < n_pass || n1 < nu; }
                        if (more && nsb != sb) tc_commit(bar(D_EMPTY));
                    }
                }
                for (int n = n0; ok && n < n1; ++n) tc_commit(bar(Q_EMPTY + qstage_of(n)));
            }
        }
    } else if (warp < 2 + 4 * NG) {
        // ------------------------------------------------------------ selection groups
        const int sg = (warp - 2) >> 2;                        // group (warps 2-5, 6-9, ...); its units are those with n % NG == sg
        const int gt = threadIdx.x - 64 - sg * 128;            // thread within the group
        const int r = (warp & 3) * 32 + lane;                  // TMEM lane = query row of the tile
        const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t acc = tmem + sg * ACC_COLS + lane_off;
        int *hist = hist_base + sg * hist_ints;
        int nacc = 0, ngs = 0;
        bool ok = true;
        auto group_sync = [&]() {     // all 128 threads of the group, bounded
            mbar_arrive(bar(GROUP + sg));
            bool o = mbar_wait_spin(bar(GROUP + sg), ngs & 1, abort_flag, p.status, RW_GROUP);   // polled: a parked thread wakes late
            ++ngs;
            return o;
        };
        // the sorted list of this pass's picks lives in registers (a 64-entry list leaves room for one selection group)
        constexpr int KR = KMAX;
        // With at most kRtDeferredChunks chunks the list append of a unit is finished after the next unit's selection,
        // so the round trip of the range-reserving atomics is hidden; `pend` is the unit whose append is open.
        const bool deferred = KMAX <= 8 && p.C <= kRtDeferredChunks;
        constexpr int NB = kRtDeferredChunks / 128;           // chunks a thread owns in the deferred append
        struct Pending { int h, i, j[KR], rank[KR], base[NB]; bool live, open; } pend;
        pend.open = false; pend.live = false; pend.h = 0; pend.i = 0;
#pragma unroll
        for (int y = 0; y < NB; ++y) pend.base[y] = 0;
        // Deferred append, one group barrier per unit.  Unit n uses histogram n & 1 and base table n & 1:
        //   before the barrier: the bases that unit n - 1's range-reserving atomics returned go into the table,
        //     and unit n's picks take their tile-local ranks from the histogram;
        //   after it: unit n - 1's list entries are written (base + rank), and each thread reserves, for the
        //     chunk it owns, unit n's range in that chunk's list and clears the counter it has just read.
        // The same histogram and table are next written two units later, with unit n + 1's barrier in between.
        int ndef = 0;                          // units this group has appended so far
        auto write_bases = [&]() {
            int *baseb = hist + (2 + (ndef & 1)) * p.C;
#pragma unroll
            for (int y = 0; y < NB; ++y)
                if (gt + 128 * y < p.C) baseb[gt + 128 * y] = pend.base[y];
        };
        auto write_entries = [&]() {
            const int *baseb = hist + (2 + (ndef & 1)) * p.C;
            if (pend.live) {
                int32_t *list = p.qlist + (size_t)pend.h * p.cap_total;
#pragma unroll
                for (int x = 0; x < KR; ++x)           // j holds (chunk << 8 | rank) here: a tile has 128 rows
                    if (x < p.k && pend.j[x] >= 0) {
                        const size_t at = (size_t)s_cap[pend.j[x] >> 8] + baseb[pend.j[x] >> 8] + (pend.j[x] & 255);
                        if (index_ok(at < p.cap_total, p.status, IX_APPEND_POSITION)) list[at] = pend.i * p.k + x;
                    }
            }
        };
        if (deferred) {
            for (int x = gt; x < 2 * p.C; x += 128) hist[x] = 0;
            ok = group_sync();
        }
        // Candidates of a row, over score columns.  Prefix mode (the causal rule): the columns [0, lim); else a
        // bitmap row.  Both are fetched a unit ahead, so that these dependent loads are never waited for.
        int nx_ci = 0, nx_lim = 0;
        uint32_t nx_w0 = 0u;
        auto fetch_row = [&](int i0, bool live0) {
            nx_ci = live0 ? p.tok_chunk[i0] : 0;
        };
        auto fetch_cand = [&](bool live0) {
            nx_lim = live0 ? (p.prefix ? p.lim[nx_ci] : 0) : 0;
            nx_w0 = (live0 && !p.prefix) ? p.cand_c[(size_t)nx_ci * p.cwords] : 0u;
        };
        if (sg < nu) {
            const int i0 = unit_of(sg) * kRtRows + r;
            fetch_row(i0, i0 < p.L);
            fetch_cand(i0 < p.L);
        }
        for (int n = sg; ok && n < nu; n += NG) {
            const int u = unit_of(n);
            const int reach = reach_of(n), n_sb = steps_of(n);   // blocks that hold a column in reach
            const int i = u * kRtRows + r;
            const bool live = i < p.L;
            const int ci = nx_ci, lim_i = nx_lim;
            const uint32_t w0 = nx_w0;
            const int i2 = unit_of(n + NG) * kRtRows + r;
            const bool live2 = n + NG < nu && i2 < p.L;
            fetch_row(i2, live2);       // the next unit's chunk, loaded a unit ahead (its candidates follow below)
            // candidate bits of the 32 columns from j0 on
            auto cand_bits = [&](int j0) -> uint32_t {
                if (p.prefix) {
                    const int m = lim_i - j0;
                    return m <= 0 ? 0u : (m >= 32 ? 0xffffffffu : ((1u << m) - 1u));
                }
                return j0 == 0 ? w0 : (live ? p.cand_c[(size_t)ci * p.cwords + (j0 >> 5)] : 0u);
            };
            // More than 64 picks are taken 64 at a time: every pass sees the tile's scores again (the issuer
            // recomputes them) and considers only the columns that come after the previous pass's last pick in
            // the order of the result (score descending, then column ascending).
            [[maybe_unused]] float prev_s = INFINITY;
            [[maybe_unused]] int prev_j = -1;
            for (int pass = 0; ok && pass < n_pass; ++pass) {
            const int kp = min(p.k - pass * 64, KMAX);      // picks of this pass
            TopK<KMAX> top;
            top.init();
            [[maybe_unused]] float kth = -INFINITY;
            // One candidate into the sorted list (descending; equal scores keep their arrival order, which is
            // ascending column): it goes behind every entry that is at least as large, the entries after it move
            // down one slot and the last falls off.  Every slot is decided on its own from the compare of its
            // entry and of the entry before it, so the slots do not wait for one another.
            auto insert = [&](float cv, int cj) {
                bool ge[KR];
#pragma unroll
                for (int x = 0; x < KR; ++x) ge[x] = top.s[x] >= cv;
#pragma unroll
                for (int x = KR - 1; x >= 0; --x) {
                    const bool here = x == 0 ? true : ge[x - 1];             // the new entry's slot is x, or before x
                    const float ps = x == 0 ? cv : top.s[x - 1];
                    const int pj = x == 0 ? cj : top.j[x - 1];
                    top.s[x] = ge[x] ? top.s[x] : (here ? cv : ps);
                    top.j[x] = ge[x] ? top.j[x] : (here ? cj : pj);
                }
            };
            auto update_kth = [&]() {
                kth = top.s[0];
#pragma unroll
                for (int x = 1; x < KR; ++x) kth = (x < kp) ? top.s[x] : kth;
            };
            for (int sb = 0; ok && sb < n_sb; ++sb) {
                ok = mbar_wait_spin(bar(ACC_FULL + sg), nacc & 1, abort_flag, p.status, RW_ACCFULL);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                ++nacc;
                tc_fence_after();
                const int rows_sb = max(16, min(min(p.sb_rows, p.c_pad - sb * p.sb_rows), (reach - sb * p.sb_rows + 15) & ~15));
                if (FEW) {
                    // at most 32 columns, all in this block.  The scores of the columns in the tile's reach come eight
                    // at a time, each the sum of its three terms (hi, mid, lo, in that order), and go into the list.
                    const uint32_t cand = cand_bits(0);
                    uint32_t a[8], b[8], c3[8];
                    tmem_ld8(acc, a);
                    tmem_ld8(acc + p.c_pad, b);
                    tmem_ld8(acc + 2 * p.c_pad, c3);
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        if (g * 8 < rows_sb) {
                            tmem_wait_ld();
                            float f[8];
#pragma unroll
                            for (int c = 0; c < 8; ++c) f[c] = (__uint_as_float(a[c]) + __uint_as_float(b[c])) + __uint_as_float(c3[c]);
                            if (g < 3 && (g + 1) * 8 < rows_sb) {       // the next eight, in flight behind this group's work
                                tmem_ld8(acc + (g + 1) * 8, a);
                                tmem_ld8(acc + p.c_pad + (g + 1) * 8, b);
                                tmem_ld8(acc + 2 * p.c_pad + (g + 1) * 8, c3);
                            }
#pragma unroll
                            for (int c = 0; c < 8; ++c) {
                                insert(((cand >> (g * 8 + c)) & 1u) ? f[c] : -INFINITY, g * 8 + c);     // -inf changes nothing
                            }
                        }
                    }
                } else {
                // Best-first extraction: up to k members of a 32-column block can enter the list; they are taken one
                // per round, the block's best first, while any row of the warp still has one above its k-th score.
                auto extract_blocks = [&](int cc0, int cc1) {
                for (int cc = cc0; cc < cc1; cc += 32) {
                    uint32_t v[32];
                    tmem_ld32(acc + cc, v);
                    const int j0 = sb * p.sb_rows + cc;
                    const uint32_t cand = cand_bits(j0);
                    tmem_wait_ld();
                    {
                        float f[32];
#pragma unroll
                        for (int c = 0; c < 32; ++c) f[c] = ((cand >> c) & 1u) ? __uint_as_float(v[c]) : -INFINITY;
                        if (KMAX == 64 && pass > 0) {
#pragma unroll
                            for (int c = 0; c < 32; ++c) {
                                const bool after = f[c] < prev_s || (f[c] == prev_s && j0 + c > prev_j);
                                f[c] = after ? f[c] : -INFINITY;
                            }
                        }
#pragma unroll 1
                        for (int round = 0; round < kp; ++round) {
                            float m8[4];
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const float a = max3(f[q * 8], f[q * 8 + 1], f[q * 8 + 2]);
                                const float b = max3(f[q * 8 + 3], f[q * 8 + 4], f[q * 8 + 5]);
                                m8[q] = max3(a, b, fmaxf(f[q * 8 + 6], f[q * 8 + 7]));
                            }
                            const float m = fmaxf(fmaxf(m8[0], m8[1]), fmaxf(m8[2], m8[3]));
                            const bool want = m > kth;                                          // above the list's k-th score
                            if (!__any_sync(0xffffffffu, want)) break;
                            uint32_t eq = 0u;                                                   // lowest index among equals
#pragma unroll
                            for (int c = 0; c < 32; ++c) eq |= (f[c] == m) ? (1u << c) : 0u;
                            const int idx = __ffs(eq) - 1;
                            if (want) {
                                insert(m, j0 + idx);
                                update_kth();
                            }
                            const uint32_t clr = want ? (1u << idx) : 0u;
#pragma unroll
                            for (int c = 0; c < 32; ++c) f[c] = ((clr >> c) & 1u) ? -INFINITY : f[c];
                        }
                    }
                }
                };
                // Threshold selection (lists of at most 16 picks).  A lower bound `thr` of the row's final k-th score
                // is known before any candidate is inserted: in the tile's first scoring step it is the k-th largest
                // of G group maxima (group = columns with equal index mod G: k groups whose maximum is at least thr
                // hold k different candidates at least thr), later the list's own k-th score.  Only the candidates at
                // least thr - a few more than k per row - go through the sorted insertion, which is where the work
                // is: each row's survivors are queued in shared memory (score and column, in column order: the lower
                // half of the step's blocks fills the queue from the front, the upper half from the back, two
                // independent streams of instructions) and the warp inserts every row's e-th survivor together, so
                // the insertion runs max-over-rows(survivors) times per warp instead of once per column.  A row with
                // more survivors than slots (many equal scores) sends its warp through the best-first extraction
                // instead, which needs no queue.  A block all of whose columns are candidates for all 32 rows (most
                // blocks: the candidates are a prefix of the columns) skips the candidate masks.
                bool fast = p.surv_cap > 0;
                if (fast) {
                    constexpr int G = KMAX <= 8 ? 16 : 32;
                    const int jb = sb * p.sb_rows;
                    float thr = kth;
                    if (KMAX <= 16 && sb == 0) {
                        float gm[G];
#pragma unroll
                        for (int x = 0; x < G; ++x) gm[x] = -INFINITY;
#pragma unroll 1
                        for (int cc = 0; cc < rows_sb; cc += 64) {          // two blocks of 32 columns in flight
                            const bool two = cc + 32 < rows_sb;
                            uint32_t v[32], w[32];
                            tmem_ld32(acc + cc, v);
                            if (two) tmem_ld32(acc + cc + 32, w);
                            const uint32_t cand = cand_bits(jb + cc), cand2 = two ? cand_bits(jb + cc + 32) : 0u;
                            tmem_wait_ld();
                            if (__all_sync(0xffffffffu, cand == 0xffffffffu && (!two || cand2 == 0xffffffffu))) {
#pragma unroll
                                for (int x = 0; x < G; ++x)
                                    gm[x] = G == 16 ? max3(gm[x], __uint_as_float(v[x]), __uint_as_float(v[x + 16])) : fmaxf(gm[x], __uint_as_float(v[x]));
                                if (two) {
#pragma unroll
                                    for (int x = 0; x < G; ++x)
                                        gm[x] = G == 16 ? max3(gm[x], __uint_as_float(w[x]), __uint_as_float(w[x + 16])) : fmaxf(gm[x], __uint_as_float(w[x]));
                                }
                            } else {
#pragma unroll
                                for (int c = 0; c < 32; ++c) {
                                    const float f = ((cand >> c) & 1u) ? __uint_as_float(v[c]) : -INFINITY;
                                    const float f2 = ((cand2 >> c) & 1u) ? __uint_as_float(w[c]) : -INFINITY;
                                    gm[c % G] = max3(gm[c % G], f, f2);
                                }
                            }
                        }
                        // sort the group maxima, descending (bitonic network: a fixed sequence of compare-exchange
                        // steps, every index a compile-time constant), and take the k-th
#pragma unroll
                        for (int k2 = 2; k2 <= G; k2 <<= 1)
#pragma unroll
                            for (int jj = k2 >> 1; jj > 0; jj >>= 1)
#pragma unroll
                                for (int ii = 0; ii < G; ++ii) {
                                    const int ll = ii ^ jj;
                                    if (ll > ii) {
                                        const float hi = fmaxf(gm[ii], gm[ll]), lo = fminf(gm[ii], gm[ll]);
                                        const bool desc = (ii & k2) == 0;
                                        gm[ii] = desc ? hi : lo;
                                        gm[ll] = desc ? lo : hi;
                                    }
                                }
                        thr = gm[0];
#pragma unroll
                        for (int y = 1; y < KR; ++y) thr = (y < kp) ? gm[y] : thr;
                    }
                    thr = fmaxf(thr, -FLT_MAX);          // a column that is not a candidate (-inf) never survives
                    const int cap = p.surv_cap;
                    float *sv = surv_base + (size_t)sg * cap * 160 + gt;          // 128 floats + 128 bytes per slot
                    uint8_t *sj = reinterpret_cast<uint8_t *>(surv_base + (size_t)sg * cap * 160 + (size_t)cap * 128) + gt;
                    const int nblk = (rows_sb + 31) >> 5, half = (nblk + 1) >> 1;
                    // Queue cursors as shared-memory addresses: the front stream moves up from slot 0, the back stream
                    // down from slot cap - 1.  A survivor is stored while its stream's cursor is inside the queue and the
                    // cursor moves whether it was stored or not, so the count stays exact; the two streams have run into
                    // each other (or out of the queue) exactly when the counts add up to more than cap.  The stores are
                    // predicated instructions, written out so that no branch is made of them.
                    const uint32_t q_v = smem_u32(sv), q_j = smem_u32(sj);
                    uint32_t lo_v = q_v, lo_j = q_j, hi_v = q_v + (cap - 1) * 512, hi_j = q_j + (cap - 1) * 128;
                    const uint32_t lo_end = q_v + cap * 512;
                    // the cursors advance by multiply-add with a factor of one the compiler cannot see through: that
                    // instruction runs on the multiply-add pipe, while the compares around it fill the other one
                    int one;
                    asm volatile("mov.u32 %0, 1;" : "=r"(one));
                    // the 32-column blocks at cl (front stream) and, if `two`, at ch (back stream): survivors into the queue
                    auto scan = [&](int cl, int ch, bool two) {
                        uint32_t vl[32], vh[32];
                        tmem_ld32(acc + cl, vl);
                        if (two) tmem_ld32(acc + ch, vh);
                        const uint32_t cand_l = cand_bits(jb + cl), cand_h = two ? cand_bits(jb + ch) : 0u;
                        tmem_wait_ld();
                        const bool later_pass = KMAX == 64 && pass > 0;
                        const bool plain = !later_pass && __all_sync(0xffffffffu, cand_l == 0xffffffffu && (!two || cand_h == 0xffffffffu));
                        if (!plain) {
#pragma unroll
                            for (int c = 0; c < 32; ++c) {
                                vl[c] = ((cand_l >> c) & 1u) ? vl[c] : 0xff800000u;      // -inf
                                vh[c] = ((cand_h >> c) & 1u) ? vh[c] : 0xff800000u;
                            }
                            if (later_pass) {               // only what comes after the previous pass's last pick
#pragma unroll
                                for (int c = 0; c < 32; ++c) {
                                    const float fl = __uint_as_float(vl[c]), fh = __uint_as_float(vh[c]);
                                    vl[c] = (fl < prev_s || (fl == prev_s && jb + cl + c > prev_j)) ? vl[c] : 0xff800000u;
                                    vh[c] = (fh < prev_s || (fh == prev_s && jb + ch + c > prev_j)) ? vh[c] : 0xff800000u;
                                }
                            }
                        }
                        if (two) {
#pragma unroll
                            for (int c = 0; c < 32; ++c) {
                                asm volatile(
                                    "{\n\t.reg .pred p, q;\n\t"
                                    "setp.ge.f32 p, %3, %4;\n\t"
                                    "setp.lt.and.u32 q, %0, %5, p;\n\t"
                                    "@q st.shared.f32 [%0], %3;\n\t"
                                    "@q st.shared.u8 [%1], %2;\n\t"
                                    "@p mad.lo.s32 %0, %6, 512, %0;\n\t"
                                    "@p mad.lo.s32 %1, %6, 128, %1;\n\t}"
                                    : "+r"(lo_v), "+r"(lo_j)
                                    : "r"(cl + c), "f"(__uint_as_float(vl[c])), "f"(thr), "r"(lo_end), "r"(one)
                                    : "memory");
                                asm volatile(
                                    "{\n\t.reg .pred p, q;\n\t"
                                    "setp.ge.f32 p, %3, %4;\n\t"
                                    "setp.ge.and.s32 q, %0, %5, p;\n\t"
                                    "@q st.shared.f32 [%0], %3;\n\t"
                                    "@q st.shared.u8 [%1], %2;\n\t"
                                    "@p mad.lo.s32 %0, %6, -512, %0;\n\t"
                                    "@p mad.lo.s32 %1, %6, -128, %1;\n\t}"
                                    : "+r"(hi_v), "+r"(hi_j)
                                    : "r"(ch + c), "f"(__uint_as_float(vh[c])), "f"(thr), "r"(q_v), "r"(one)
                                    : "memory");
                            }
                        } else {
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                asm volatile(
                                    "{\n\t.reg .pred p, q;\n\t"
                                    "setp.ge.f32 p, %3, %4;\n\t"
                                    "setp.lt.and.u32 q, %0, %5, p;\n\t"
                                    "@q st.shared.f32 [%0], %3;\n\t"
                                    "@q st.shared.u8 [%1], %2;\n\t"
                                    "@p mad.lo.s32 %0, %6, 512, %0;\n\t"
                                    "@p mad.lo.s32 %1, %6, 128, %1;\n\t}"
                                    : "+r"(lo_v), "+r"(lo_j)
                                    : "r"(cl + c), "f"(__uint_as_float(vl[c])), "f"(thr), "r"(lo_end), "r"(one)
                                    : "memory");
                        }
                    };
                    // the queue's survivors into the list (front stream, then back stream: column order), unless a
                    // row of the warp has more than fit; the cursors start again
                    auto drain = [&]() -> bool {
                        const int cnt_lo = (int)(lo_v - q_v) >> 9, cnt_hi = (int)(q_v + (cap - 1) * 512 - hi_v) >> 9;
                        lo_v = q_v; lo_j = q_j; hi_v = q_v + (cap - 1) * 512; hi_j = q_j + (cap - 1) * 128;
                        if (__any_sync(0xffffffffu, cnt_lo + cnt_hi > cap)) return false;
                        // every row's e-th survivor goes into its list together; a row that has none left inserts
                        // -inf, which changes nothing, so there is no branch; the next survivor is fetched ahead
                        const int nlo = __reduce_max_sync(0xffffffffu, cnt_lo), nhi = __reduce_max_sync(0xffffffffu, cnt_hi);
                        const int ntot = nlo + nhi;
                        auto slot_of = [&](int e) { return e < nlo ? e : cap - 1 - (e - nlo); };
                        auto live_of = [&](int e) { return e < nlo ? e < cnt_lo : e - nlo < cnt_hi; };
                        float nv = 0.f;
                        int nj = 0;
                        if (ntot > 0) { nv = sv[slot_of(0) * 128]; nj = sj[slot_of(0) * 128]; }
#pragma unroll 1
                        for (int e = 0; e < ntot; ++e) {
                            const float cv = live_of(e) ? nv : -INFINITY;
                            const int cj = jb + nj;
                            if (e + 1 < ntot) { nv = sv[slot_of(e + 1) * 128]; nj = sj[slot_of(e + 1) * 128]; }
                            insert(cv, cj);
                        }
                        update_kth();
                        return true;
                    };
                    if (KMAX <= 16) {
                        // one scan of the whole step against the threshold found above, then one drain
#pragma unroll 1
                        for (int b = 0; b < half; ++b) scan(b * 32, (b + half) * 32, b + half < nblk);
                        fast = drain();
                    } else {
                        // Long lists: no group maxima (a list of k needs more groups than registers hold); the columns
                        // go 64 at a time against the list's own k-th score, which rises as they go: after n columns
                        // about k / n of the next ones survive.  A pair of blocks whose survivors do not fit the
                        // queue (the first ones, when everything survives and the queue is short) is extracted
                        // best-first instead.
#pragma unroll 1
                        for (int b0 = 0; b0 < nblk; b0 += 2) {
                            thr = fmaxf(kth, -FLT_MAX);
                            const bool two = b0 + 1 < nblk;
                            scan(b0 * 32, (b0 + 1) * 32, two);
                            if (!drain()) extract_blocks(b0 * 32, min(rows_sb, (b0 + 2) * 32));
                        }
                    }
                }
                if (!fast) extract_blocks(0, rows_sb);
                }
                tc_fence_before();
                mbar_arrive(bar(ACC_EMPTY + sg));
            }
            if (!ok) break;
            fetch_cand(live2);
            if (KMAX == 64) {                           // the next pass starts after this pass's last pick
#pragma unroll
                for (int x = 0; x < KR; ++x)
                    if (x == kp - 1) { prev_s = top.s[x]; prev_j = top.j[x]; }
            }
            // columns -> chunks; sel_idx and the empty slots' partial log-sum-exp
#pragma unroll
            for (int x = 0; x < KR; ++x) top.j[x] = top.j[x] >= 0 ? s_col[top.j[x]] : -1;
            int32_t *out = p.sel + ((size_t)h * p.L + i) * p.k + pass * 64;
            float *pl = p.part_lse + ((size_t)h * p.L + i) * p.k + pass * 64;
            if (live) {
#pragma unroll
                for (int x = 0; x < KR; ++x)
                    if (x < kp) {
                        out[x] = top.j[x];
                        if (top.j[x] < 0) pl[x] = -INFINITY;
                    }
            }
            if (deferred) {
                int *cntb = hist + (ndef & 1) * p.C;
                if (pend.open) write_bases();
                int njr[KR];                           // chunk << 8 | tile-local rank, or -1
#pragma unroll
                for (int x = 0; x < KR; ++x) {
                    const int j = (live && x < kp) ? top.j[x] : -1;
                    njr[x] = j >= 0 ? ((j << 8) | atomicAdd(&cntb[j], 1)) : -1;
                }
                ok = group_sync();
                if (!ok) break;
                if (pend.open) write_entries();
#pragma unroll
                for (int y = 0; y < NB; ++y) {
                    pend.base[y] = 0;
                    if (gt + 128 * y < p.C) {
                        const int n = cntb[gt + 128 * y];
                        if (n) { pend.base[y] = atomicAdd(&p.cnt[h * p.C + gt + 128 * y], n); cntb[gt + 128 * y] = 0; }
                    }
                }
#pragma unroll
                for (int x = 0; x < KR; ++x) pend.j[x] = njr[x];
                pend.h = h; pend.i = i; pend.live = live; pend.open = true;
                ++ndef;
                continue;
            }
            // tile-local rank of every pick (shared-memory histogram), then one global atomic per picked
            // chunk reserves this tile's range in that chunk's list
            for (int x = gt; x < p.C; x += 128) hist[x] = 0;
            ok = group_sync();
            if (!ok) break;
            if (live) {
#pragma unroll
                for (int x = 0; x < KR; ++x) {
                    pend.j[x] = x < kp ? top.j[x] : -1;
                    pend.rank[x] = 0;
                    if (pend.j[x] >= 0) pend.rank[x] = atomicAdd(&hist[pend.j[x]], 1);
                }
            } else {
#pragma unroll
                for (int x = 0; x < KR; ++x) { pend.j[x] = -1; pend.rank[x] = 0; }
            }
            ok = group_sync();
            if (!ok) break;
            {
                for (int x = gt; x < p.C; x += 128) {
                    const int n = hist[x];
                    if (n) hist[x] = atomicAdd(&p.cnt[h * p.C + x], n);
                }
                ok = group_sync();
                if (!ok) break;
                if (live) {
                    int32_t *list = p.qlist + (size_t)h * p.cap_total;
#pragma unroll
                    for (int x = 0; x < KR; ++x)
                        if (pend.j[x] >= 0) {
                            const size_t at = (size_t)s_cap[pend.j[x]] + hist[pend.j[x]] + pend.rank[x];
                            if (index_ok(at < p.cap_total, p.status, IX_APPEND_POSITION)) list[at] = i * p.k + pass * 64 + x;
                        }
                }
                ok = group_sync();
                if (!ok) break;
            }
            }   // pass
        }
        if (ok && pend.open) {                 // the last unit's entries
            write_bases();
            if (group_sync()) write_entries();
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
    // The last block to get here turns the pick counts into the running counts of attention tiles over the (head,
    // chunk) pairs and marks the workspace (what route_tiles_kernel does on the paths that have no such block): one
    // launch less.  Every block's counts are in place before it arrives (the atomics that made them have
    // returned), and the fence orders them before the arrival.
    __shared__ int s_last, s_wsum[32];
    if (threadIdx.x == 0) {
        __threadfence();
        s_last = atomicAdd(&p.status[ST_ARRIVE], 1) == (int)gridDim.x - 1;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const int HC = p.H * p.C, T = kRtThreads, t = threadIdx.x;
    const int per = (HC + T - 1) / T, i0 = min(t * per, HC), i1 = min(i0 + per, HC);
    int mine = 0;
    for (int i = i0; i < i1; ++i) mine += (__ldcg(p.cnt + i) + kQTileRows - 1) / kQTileRows;
    int incl = mine;                                     // inclusive scan over the block: warps by shuffles, then warp totals
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) s_wsum[warp] = incl;
    __syncthreads();
    int at = incl - mine;
    for (int w = 0; w < warp; ++w) at += s_wsum[w];
    for (int i = i0; i < i1; ++i) {
        p.tile_off[i] = at;
        at += (__ldcg(p.cnt + i) + kQTileRows - 1) / kQTileRows;
    }
    if (t == T - 1) {
        p.tile_off[HC] = at;
        p.status[ST_COOKIE] = (int)p.cookie;
    }
}

// gtile[i] = attention tiles (of kQTileRows picks) before (head, chunk) pair i, with a final total;
// marks the workspace as holding the lists of the plan with this cookie.
__global__ void __launch_bounds__(1024) route_tiles_kernel(const int *__restrict__ cnt, int *__restrict__ gtile,
                                                           int *__restrict__ status, int HC, uint32_t cookie) {
    __shared__ int st[1024];
    const int t = threadIdx.x;
    const int per = (HC + 1023) / 1024;
    const int i0 = min(t * per, HC), i1 = min(i0 + per, HC);
    int b = 0;
    for (int i = i0; i < i1; ++i) b += (cnt[i] + kQTileRows - 1) / kQTileRows;
    st[t] = b;
    __syncthreads();
    for (int o = 1; o < 1024; o <<= 1) {   // inclusive scan
        int xb = 0;
        if (t >= o) xb = st[t - o];
        __syncthreads();
        st[t] += xb;
        __syncthreads();
    }
    int eb = st[t] - b;    // exclusive
    for (int i = i0; i < i1; ++i) {
        gtile[i] = eb;
        eb += (cnt[i] + kQTileRows - 1) / kQTileRows;
    }
    if (t == 1023) { gtile[HC] = st[1023]; status[ST_COOKIE] = (int)cookie; }
}

// The routed work items of (head, chunk) pair i: one per kQTileRows entries of its query list.
__global__ void route_items_kernel(const int *__restrict__ cnt, const int *__restrict__ gtile, WorkItem *__restrict__ items,
                                   const int32_t *__restrict__ off, const int32_t *__restrict__ cap_off, int H, int C) {
    const int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;     // one warp per pair
    if (i >= H * C) return;
    const int h = i / C, c = i % C, n = cnt[i];
    const int key_tiles = (off[c + 1] - off[c] + 127) / 128;
    const int at = gtile[i];
    for (int x = lane; x * kQTileRows < n; x += 32)
        items[at + x] = WorkItem{h, cap_off[c] + x * kQTileRows, min(kQTileRows, n - x * kQTileRows), key_tiles, c, 1, off[c], off[c + 1]};
}


// Tile counts, routed work items and the cookie, from the per-(head, chunk) pick counts and lists.
static int finish_lists(const moc_plan *p, void *ws, cudaStream_t s, bool count_tiles) {
    int *cnt = ws_ptr<int>(ws, p->ws.cnt);
    if (count_tiles) {
        route_tiles_kernel<<<1, 1024, 0, s>>>(cnt, ws_ptr<int>(ws, p->ws.tile_off), ws_ptr<int>(ws, p->ws.status), p->H * p->C, p->cookie);
        MOC_LAUNCH_CHECK();
    }
    if (p->k > 0) {
        route_items_kernel<<<(unsigned)((p->H * p->C + 3) / 4), 128, 0, s>>>(cnt, ws_ptr<int>(ws, p->ws.tile_off),
                                                                               ws_ptr<WorkItem>(ws, p->ws.rtiles), p->d_off,
                                                                               p->d_cap_off, p->H, p->C);
        MOC_LAUNCH_CHECK();
    }
    return MOC_OK;
}

// Inverse index of a given sel_idx: 256 consecutive rows of one head per block.  Pass 1 checks every entry
// (a chunk that may be routed to from the row, not a repeat of an earlier slot), blanks the others, marks the
// empty slots' partial log-sum-exp and counts the block's picks per chunk in shared memory; then one global
// atomic per picked chunk reserves the block's range in that chunk's list, and pass 2 writes the entries.
__global__ void __launch_bounds__(256) lists_from_sel_kernel(int32_t *__restrict__ sel, float *__restrict__ part_lse,
                                                             int *__restrict__ cnt, int32_t *__restrict__ qlist,
                                                             const int32_t *__restrict__ tok_chunk, const uint32_t *__restrict__ anc_bits,
                                                             const int32_t *__restrict__ cap_off, int *__restrict__ status,
                                                             int L, int C, int k, int words, int causal, size_t cap_total) {
    extern __shared__ int sh[];
    int *hist = sh, *base = sh + C;
    const int h = blockIdx.y, i = blockIdx.x * 256 + threadIdx.x;
    for (int x = threadIdx.x; x < C; x += 256) hist[x] = 0;
    __syncthreads();
    int32_t *row = sel + ((size_t)h * L + i) * k;
    if (i < L) {
        const int ci = tok_chunk[i];
        float *pl = part_lse + ((size_t)h * L + i) * k;
        for (int s = 0; s < k; ++s) {
            const int j = row[s];
            bool ok = j >= 0 && j < C && (!causal || j < ci);
            if (ok) ok = !((anc_bits[(size_t)ci * words + (j >> 5)] >> (j & 31)) & 1u);
            for (int e = 0; ok && e < s; ++e) ok = row[e] != j;        // earlier slots are already checked
            if (ok) atomicAdd(&hist[j], 1);
            else {
                if (j != -1) row[s] = -1;
                pl[s] = -INFINITY;
            }
        }
    }
    __syncthreads();
    for (int x = threadIdx.x; x < C; x += 256) {
        const int n = hist[x];
        base[x] = n ? atomicAdd(&cnt[h * C + x], n) : 0;
        hist[x] = 0;
    }
    __syncthreads();
    if (i < L) {
        int32_t *list = qlist + (size_t)h * cap_total;
        for (int s = 0; s < k; ++s) {
            const int j = row[s];
            if (j >= 0) {
                const int at = cap_off[j] + base[j] + atomicAdd(&hist[j], 1);
                if (index_ok(at < cap_off[j + 1], status, IX_APPEND_POSITION)) list[at] = i * k + s;
            }
        }
    }
}

int launch_lists_from_sel(const moc_plan *p, int32_t *sel, void *ws, cudaStream_t s) {
    int *cnt = ws_ptr<int>(ws, p->ws.cnt);
    int *status = ws_ptr<int>(ws, p->ws.status);
    const size_t n = std::max((size_t)p->H * p->C, (size_t)kStatusWords);
    route_prep_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(nullptr, nullptr, cnt, status, nullptr, p->H, p->C, p->ncol, p->c_pad, p->d, p->wait_us);
    MOC_LAUNCH_CHECK();
    if (p->k > 0) {
        const size_t smem = 2 * sizeof(int) * (size_t)p->C;
        if (smem > 200 * 1024) return MOC_ERR_SHAPE;
        MOC_CUDA_TRY(cudaFuncSetAttribute(lists_from_sel_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        lists_from_sel_kernel<<<dim3((unsigned)((p->L + 255) / 256), (unsigned)p->H), 256, smem, s>>>(
            sel, ws_ptr<float>(ws, p->ws.part_lse), cnt, ws_ptr<int32_t>(ws, p->ws.qlist), p->d_tok_chunk, p->d_anc_bits,
            p->d_cap_off, status, p->L, p->C, p->k, p->words, (p->flags & MOC_FLAG_CAUSAL) ? 1 : 0, (size_t)p->cap_off[p->C]);
        MOC_LAUNCH_CHECK();
    }
    return finish_lists(p, ws, s, true);
}

template <int D>
static int launch_route_d(const moc_plan *p, const __nv_bfloat16 *Q, const float *desc, int32_t *sel, void *ws,
                          cudaStream_t s) {
    int *cnt = ws_ptr<int>(ws, p->ws.cnt);
    int *status = ws_ptr<int>(ws, p->ws.status);
    __nv_bfloat16 *desc3 = ws_ptr<__nv_bfloat16>(ws, p->ws.desc3);
    // Few chunks: the routing kernel splits the descriptors itself, and the status words and pick counters (next to
    // each other in the workspace) are cleared by one memset instead of a kernel.
    const bool few = p->k > 0 && p->c_pad <= 32 && p->k <= 8;
    const bool fused_prep = few && (reinterpret_cast<uintptr_t>(desc) & 15) == 0 && p->ws.cnt > p->ws.status;
    if (fused_prep) {
        MOC_CUDA_TRY(cudaMemsetAsync(status, 0, (p->ws.cnt - p->ws.status) + sizeof(int) * (size_t)p->H * p->C, s));
    } else {
        const size_t n = std::max((size_t)p->H * p->c_pad * D, (size_t)kStatusWords);   // covers H * C too
        route_prep_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(desc, desc3, cnt, status, p->d_col_chunk, p->H, p->C, p->ncol, p->c_pad, D, p->wait_us);
        MOC_LAUNCH_CHECK();
    }
    if (p->k > 0) {
        RouteParams a;
        a.desc = fused_prep ? desc : nullptr; a.wait_us = p->wait_us;
        a.sel = sel; a.part_lse = ws_ptr<float>(ws, p->ws.part_lse); a.cnt = cnt;
        a.qlist = ws_ptr<int32_t>(ws, p->ws.qlist);
        a.tok_chunk = p->d_tok_chunk; a.cand_c = p->d_cand_c; a.lim = p->d_lim; a.reach = p->d_reach;
        a.col_chunk = p->d_col_chunk; a.cap_off = p->d_cap_off; a.status = status;
        a.H = p->H; a.L = p->L; a.C = p->C; a.ncol = p->ncol; a.c_pad = p->c_pad; a.k = p->k; a.cwords = p->cwords;
        a.prefix = p->prefix_mode;
        a.tiles_per_head = (p->L + kRtRows - 1) / kRtRows;
        a.d_rows = p->c_pad <= kRtResident ? p->c_pad : kRtBlock;
        // a scoring step fills one accumulator: a quarter of TMEM (128 chunks) with four selection groups, half of it
        // (256 chunks) with two, which is every case but the few-chunk one; streamed blocks are 128 chunks
        a.sb_rows = std::min(a.d_rows, p->c_pad <= 32 ? kRtBlock : 2 * kRtBlock);
        a.cap_total = (size_t)p->cap_off[p->C];
        a.tile_off = ws_ptr<int>(ws, p->ws.tile_off);
        a.cookie = p->cookie;
        const size_t q_tile = (size_t)kRtRows * D * 2, d_block = ((size_t)3 * a.d_rows * D * 2 + 1023) & ~(size_t)1023;
        a.ctas_per_head = std::max(1, std::min(p->n_sm / p->H, a.tiles_per_head));
        const unsigned grid = (unsigned)(p->H * a.ctas_per_head);
        // Four selection groups with few chunks (more warps to hide the selection's latencies); one when the
        // 64-entry list takes nearly all of a thread's registers; two otherwise.
        const int ng = few ? 4 : p->k > 32 ? 1 : 2;
        a.n_pass = p->k > 64 ? (p->k + 63) / 64 : 1;
        // one histogram per group, the list offsets, and one byte per unit of a CTA
        const size_t hist = (ng * (p->k <= 8 && p->C <= kRtDeferredChunks ? 4 : 1) + 1) * sizeof(int) * (size_t)p->C + sizeof(int) * (size_t)p->ncol +
                            4 * (size_t)(a.tiles_per_head / a.ctas_per_head + 16),
                     budget = 227 * 1024 - 1024 - 512;      // what an SM has, less the alignment slack and the kernel's static variables
        if (d_block + q_tile + hist > budget) return MOC_ERR_SHAPE;
        // threshold selection (not the few-chunk case): survivor slots per row, as many as fit beside two Q stages
        // (too few: the best-first extraction alone is used)
        a.surv_cap = 0;
        size_t surv = 0;
        if (!few && budget > d_block + hist + 2 * q_tile + 16) {
            const size_t room = budget - d_block - hist - 2 * q_tile - 16, per_slot = (size_t)ng * 160 * sizeof(float);
            // short lists: one scan per scoring step, a few more than k survive; long lists: 64 columns at a time,
            // all of which survive at first
            const int want = p->k <= 16 ? std::max(12, 2 * p->k + 12) : 64, need = p->k <= 16 ? p->k + 4 : 32;
            const int have = (int)std::min<size_t>(room / per_slot, 255);
            if (have >= need) a.surv_cap = std::min(want, have);
            surv = 16 + a.surv_cap * per_slot;
        }
        a.q_stages = (int)std::min<size_t>(4, (budget - d_block - hist - surv) / q_tile);
        if (a.d_rows != p->c_pad && a.q_stages < ng) return MOC_ERR_SHAPE;      // streamed blocks: a round's Q tiles are held together
        const size_t smem = 1024 + d_block + a.q_stages * q_tile + hist + surv;
        CUtensorMap tmQ, tmD;
        if (int r = make_tmap_2d_bf16(&tmQ, Q, (uint64_t)p->H * p->L, D, kRtRows)) return r;
        if (int r = make_tmap_2d_bf16(&tmD, desc3, (uint64_t)p->H * 3 * p->c_pad, D, (uint32_t)a.d_rows)) return r;
#define MOC_ROUTE_CASE(KM, NG, FW)                                                                                          \
    do {                                                                                                                \
        MOC_CUDA_TRY(cudaFuncSetAttribute(route_tc_kernel<D, KM, NG, FW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
        route_tc_kernel<D, KM, NG, FW><<<grid, rt_threads(NG), smem, s>>>(tmQ, tmD, a);                                     \
    } while (0)
        if (p->k <= 4) { if (few) MOC_ROUTE_CASE(4, 4, true); else MOC_ROUTE_CASE(4, 2, false); }
        else if (p->k <= 6 && !few) MOC_ROUTE_CASE(6, 2, false);
        else if (p->k <= 8) { if (few) MOC_ROUTE_CASE(8, 4, true); else MOC_ROUTE_CASE(8, 2, false); }
        else if (p->k <= 16) MOC_ROUTE_CASE(16, 2, false);
        else if (p->k <= 32) MOC_ROUTE_CASE(32, 2, false);
        else MOC_ROUTE_CASE(64, 1, false);                 // beyond 64 picks: several passes of 64
#undef MOC_ROUTE_CASE
        MOC_LAUNCH_CHECK();
        return finish_lists(p, ws, s, false);       // the routing kernel's last block has counted the tiles
    }
    return finish_lists(p, ws, s, true);
}

int launch_route(const moc_plan *p, const __nv_bfloat16 *Q, const float *desc, int32_t *sel, void *ws, cudaStream_t s) {
    return p->d == 128 ? launch_route_d<128>(p, Q, desc, sel, ws, s) : launch_route_d<64>(p, Q, desc, sel, ws, s);
}

}  // namespace moc
