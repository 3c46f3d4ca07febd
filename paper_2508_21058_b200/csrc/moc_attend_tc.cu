// Tensor-core sparse attention forward (tcgen05 MMA, TMEM accumulators, TMA-fed K/V).
//
// Two passes share one kernel:
//   routed pass (key-chunk stationary): work item = (head, chunk c, up to 256 entries of the
//     list of (query, slot) pairs that picked c).  The Q rows are gathered into shared
//     memory, the keys are exactly the tokens of chunk c, and each (query, slot) gets a
//     partial result (normalised output + log-sum-exp) in the workspace.
//   anchor pass (query-tile stationary): work item = (head, up to 256 consecutive rows of
//     one chunk); keys are the chunk's mandatory anchors (merged token ranges).  Its
//     epilogue merges the row's <= k routed partials by log-sum-exp and writes O and LSE.
//
// One CTA per SM, 12 warps in three warpgroups (the third gives most of its registers to the
// other two), two 128-row query tiles that share every K/V tile:
//   warps 0-3 / 4-7  softmax group of query tile 0 / 1, one row per thread (TMEM lane = row):
//              load or gather Q into the swizzled shared tile, read S from TMEM, online
//              softmax, write P back to TMEM as packed bf16 (aliasing S; the first 64 keys are
//              released to the issuer before the exponentials of the other 64), lazily rescale
//              O, epilogue.  The exponentials of the two tiles take turns;
//   warp 8     TMA producer: K and V tiles of 128 keys, two stages each, 128-byte swizzle;
//   warps 9, 10  one MMA-issuing thread per query tile g:  S_g(0), then  O_g += P_g V(j),
//              S_g(j + 1)  per key tile.  The tensor pipe takes the next MMA only as the
//              previous one retires, so an issuer that waits on a barrier idles the pipe; with
//              one issuer per tile the other tile's MMAs fill that time, and one tile's softmax
//              overlaps the other tile's MMAs.  S = Q K^T takes both operands from shared
//              memory, O += P V takes P from TMEM and V as an MN-major shared-memory operand;
//              all accumulators live in TMEM (S0, S1, O0, O1 = 512 columns);
//   warp 11    idle (fills the third warpgroup).
// Every mbarrier wait is bounded; a wait that runs out flags the workspace status word
// and the CTA drains and leaves.
#include <algorithm>

#include "moc_common.cuh"
#include "moc_tc.cuh"

namespace moc {

using namespace tc;

struct AttendParams {
    const __nv_bfloat16 *Q;
    __nv_bfloat16 *O;
    float *lse;
    __nv_bfloat16 *part_o;
    float *part_lse;
    const KeyRange *rng;        // key ranges the items index: merged anchor ranges, or the chunks
    const WorkItem *items;      // anchor pass: one head's items (blockIdx.y = head - h0); routed pass: every item
    const int *item_lo_dev, *item_hi_dev;   // routed pass: the group's item range [*lo, *hi) lives on the device
    int h0;                     // first head of the group in flight (its partials are part_o[h - h0])
    uint32_t cookie;            // what the workspace's status area must hold
    const int32_t *qlist;       // [H][cap_total]
    size_t cap_total;
    int *status;
    int H, L, k;
    float scale_log2;       // softmax scale * log2(e)
};

constexpr int kBN = 128;               // keys per tile
constexpr int kThreads = 384;          // three warpgroups: softmax 0, softmax 1, {producer, two MMA issuers, one idle warp}
constexpr int kTmemCols = 512;         // S0/P0 [0,128) S1/P1 [128,256) O0 [256,384) O1 [384,512)
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.0f;
   // log2 units: O is rescaled only when the row max grows by more

enum WaitCode { W_QFULL = 1, W_KFULL, W_VFULL, W_SFULL, W_PFULL, W_OFULL, W_KEMPTY, W_VEMPTY, W_TURN, W_PHALF };

template <int D, bool ROUTED>
__global__ void __launch_bounds__(kThreads, 1) attend_tc_kernel(const __grid_constant__ CUtensorMap tmK,
                                                                const __grid_constant__ CUtensorMap tmV,
                                                                const AttendParams p) {
    constexpr int TILE_BYTES = 128 * D * 2;
    constexpr int SUB = D / 64;            // 64-column (128-byte) sub-tiles per row
    constexpr int SUB_BYTES = 128 * 128;   // one sub-tile: 128 rows of 128 bytes
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[20];
    __shared__ uint32_t tmem_slot;
    __shared__ int s_abort;
    __shared__ int w_valid, w_h, w_rows, w_first, w_nrng, w_ntiles;
    __shared__ int s_qrow[kQTileRows];              // query row behind each row of the item (-1 = padding)
    __shared__ const KeyRange *w_rng;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gbase = smem_raw + (sbase - smem_u32(smem_raw));
    // shared tiles: Q0 Q1 | K stage 0,1 | V stage 0,1
    const uint32_t sQ = sbase, sK = sbase + 2 * TILE_BYTES, sV = sbase + 4 * TILE_BYTES;
    auto bar = [&](int i) { return smem_u32(&bars[i]); };
    // barrier indices
    constexpr int Q_FULL = 0, K_FULL = 2, K_EMPTY = 4, V_FULL = 6, V_EMPTY = 8, S_FULL = 10, P_FULL = 12, O_FULL = 14, TURN = 16, P_HALF = 18;

    if (threadIdx.x == 0) {
        s_abort = 0;
        int valid = (*(volatile int *)p.status == 0);
        if (valid && (uint32_t)((volatile int *)p.status)[ST_COOKIE] != p.cookie) {
            // the workspace does not hold this plan's lists: report, touch nothing else
            atomicCAS(p.status, 0, MOC_ERR_WORKSPACE);
            valid = 0;
        }
        int item = blockIdx.x;
        if (ROUTED && valid) {
            item += *p.item_lo_dev;
            if (item >= *p.item_hi_dev) valid = 0;
        }
        WorkItem w = {};
        if (valid) {
            w = p.items[item];
            if (ROUTED && !index_ok((unsigned)w.h < (unsigned)p.H && w.rows > 0 && w.rows <= kQTileRows && w.first >= 0 &&
                                    (size_t)w.first + w.rows <= p.cap_total && w.nrng == 1, p.status, IX_ITEM_FIELDS))
                valid = 0;
        }
        if (valid) {
            w_h = ROUTED ? w.h : p.h0 + (int)blockIdx.y;
            w_first = w.first;
            w_rows = w.rows;
            w_rng = p.rng + w.rng_off;
            w_nrng = w.nrng;
            w_ntiles = w.ntiles;
        }
        w_valid = valid;
        for (int t = 0; t < 2; ++t) {
            mbar_init(bar(Q_FULL + t), 128);
            mbar_init(bar(K_FULL + t), 1);
            mbar_init(bar(K_EMPTY + t), valid && w_rows > 128 ? 2 : 1);   // one commit per MMA issuer
            mbar_init(bar(V_FULL + t), 1);
            mbar_init(bar(V_EMPTY + t), valid && w_rows > 128 ? 2 : 1);
            mbar_init(bar(S_FULL + t), 1);
            mbar_init(bar(P_FULL + t), 128);
            mbar_init(bar(O_FULL + t), 1);
            mbar_init(bar(TURN + t), 128);
            mbar_init(bar(P_HALF + t), 128);
        }
        fence_barrier_init();
    }
    __syncthreads();
    if (!w_valid) return;
    if (warp == 8) {
        tmem_alloc(smem_u32(&tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    const uint32_t tmem = tmem_slot;
    const int h = w_h, rows = w_rows, first = w_first, n_tiles = w_ntiles;
    const bool two = rows > 128;            // is query tile 1 populated?
    volatile int *abort_flag = &s_abort;

    if (warp < 8) {
        // ------------------------------------------------------------ softmax / epilogue groups
        // the row-per-thread softmax holds a whole 128-key row of S in registers: take the
        // registers the third warpgroup gives up
        asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
        const int g = warp >> 2;                       // query tile of this group
        const int r = threadIdx.x & 127;               // row within the tile = TMEM lane
        const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + g * 128 + lane_off, tP = tS, tO = tmem + 256 + g * 128 + lane_off;
        if (g == 0 || two) {
            const int rt = g * 128 + r;                // row within the work item
            int qi = -1, slot = 0;
            if (rt < rows) {
                if (ROUTED) {
                    const int e = p.qlist[(size_t)h * p.cap_total + first + rt];
                    qi = e / p.k;
                    slot = e - qi * p.k;
                    (void)index_ok(e >= 0 && qi < p.L, p.status, IX_LIST_ENTRY);
                    if ((unsigned)qi >= (unsigned)p.L) qi = -1;      // never follow an entry that is not a row of this head
                } else {
                    qi = first + rt;
                }
            }
            {
                // The group stages its Q tile together: consecutive threads take consecutive 16-byte pieces
                // of a row, so every request covers whole 128-byte lines even when the rows are gathered.
                s_qrow[g * 128 + r] = qi;
                asm volatile("bar.sync %0, 128;" ::"r"(1 + g) : "memory");     // the group's 128 threads; nothing can have failed yet
                constexpr int CH = D / 8, RP = 128 / CH;       // pieces per row, rows per pass
                const int c16 = r % CH;
                uint8_t *dstq = gbase + g * TILE_BYTES + (c16 >> 3) * SUB_BYTES;
                uint4 v[CH];
#pragma unroll
                for (int ps = 0; ps < CH; ++ps) {
                    const int rr = ps * RP + r / CH, q = s_qrow[g * 128 + rr];
                    v[ps] = make_uint4(0, 0, 0, 0);
                    if (q >= 0) v[ps] = __ldg(reinterpret_cast<const uint4 *>(p.Q + ((size_t)h * p.L + q) * D) + c16);
                }
#pragma unroll
                for (int ps = 0; ps < CH; ++ps)
                    *reinterpret_cast<uint4 *>(dstq + sw128_offset(ps * RP + r / CH, c16 & 7)) = v[ps];
            }
            fence_proxy_async_smem();
            mbar_arrive(bar(Q_FULL + g));
            if (!ROUTED && qi >= 0) {
                // the epilogue will merge this row's routed partials: start them on their way into L2 now
                const char *po = reinterpret_cast<const char *>(p.part_o + ((size_t)(h - p.h0) * p.L + qi) * p.k * D);
                for (int b = 0; b < p.k * D * 2; b += 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(po + b));
                asm volatile("prefetch.global.L2 [%0];" ::"l"(p.part_lse + ((size_t)h * p.L + qi) * p.k));
            }

            float m_run = -INFINITY, l_run = 0.f;
            const float c = p.scale_log2;
            TileIter it(w_rng, w_nrng);
            int t0, valid, jt = 0;
            bool ok = true;
            while (it.next(t0, valid)) {
                ok = mbar_wait(bar(S_FULL + g), jt & 1, abort_flag, p.status, W_SFULL);
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
                // TURN + g is arrived on by group g when its exponentials of a key tile are done.
                if (two && (g == 1 || jt > 0)) {
                    ok = mbar_wait(bar(TURN + (g ^ 1)), (g == 1 ? jt : jt - 1) & 1, abort_flag, p.status, W_TURN);
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
            }
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
            const __nv_bfloat16 *po = nullptr;
            if (!ROUTED && ok && qi >= 0 && p.k > 0) {
                pl = p.part_lse + ((size_t)h * p.L + qi) * p.k;
                po = p.part_o + ((size_t)(h - p.h0) * p.L + qi) * p.k * D;
                if (p.k <= KW) {
                    float plv[KW];
#pragma unroll
                    for (int s = 0; s < KW; ++s) plv[s] = s < p.k ? pl[s] : -INFINITY;
#pragma unroll
                    for (int s = 0; s < KW; ++s) big = fmaxf(big, plv[s]);
                    wsum = __expf(lse_own - big);
#pragma unroll
                    for (int s = 0; s < KW; ++s) { wslot[s] = __expf(plv[s] - big); wsum += wslot[s]; }     // exp(-inf) = 0: empty slot
#pragma unroll
                    for (int s = 0; s < KW; ++s) wslot[s] /= wsum;
                } else {
                    for (int s = 0; s < p.k; ++s) big = fmaxf(big, pl[s]);
                    wsum = __expf(lse_own - big);
                    for (int s = 0; s < p.k; ++s) wsum += __expf(pl[s] - big);
                }
                w_own = __expf(lse_own - big) / wsum * inv_l;
            }
            if (ok) {
                ok = mbar_wait(bar(O_FULL + g), 0, abort_flag, p.status, W_OFULL);
                ok = __all_sync(0xffffffffu, ok);
            }
            if (ok) {
                tc_fence_after();
#pragma unroll 1
                for (int ch = 0; ch < D / 32; ++ch) {
                    uint32_t v[32];
                    __syncwarp();
                    tmem_ld32(tO + ch * 32, v);
                    tmem_wait_ld();
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
                                for (int q4 = 0; q4 < 4; ++q4)
                                    raw[s][q4] = (s0 + s < p.k && wslot[s0 + s] != 0.f)
                                                     ? __ldcg(reinterpret_cast<const uint4 *>(po + (size_t)(s0 + s) * D + ch * 32) + q4)
                                                     : make_uint4(0, 0, 0, 0);
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
                            const float ls = pl[s];
                            if (ls == -INFINITY) continue;
                            const float w = __expf(ls - big) / wsum;
                            const uint4 *src = reinterpret_cast<const uint4 *>(po + (size_t)s * D + ch * 32);
#pragma unroll
                            for (int q4 = 0; q4 < 4; ++q4) {
                                const uint4 raw = __ldcg(src + q4);
                                const __nv_bfloat162 *b = reinterpret_cast<const __nv_bfloat162 *>(&raw);
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
                    __nv_bfloat16 *dst = ROUTED ? p.part_o + (((size_t)(h - p.h0) * p.L + qi) * p.k + slot) * D + ch * 32
                                                : p.O + ((size_t)h * p.L + qi) * D + ch * 32;
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        uint4 out;
                        uint32_t *o32 = reinterpret_cast<uint32_t *>(&out);
#pragma unroll
                        for (int y = 0; y < 4; ++y) {
                            __nv_bfloat162 b = __floats2bfloat162_rn(acc[q4 * 8 + 2 * y], acc[q4 * 8 + 2 * y + 1]);
                            o32[y] = *reinterpret_cast<uint32_t *>(&b);
                        }
                        reinterpret_cast<uint4 *>(dst)[q4] = out;
                    }
                }
                if (qi >= 0) {
                    if (ROUTED) p.part_lse[((size_t)h * p.L + qi) * p.k + slot] = lse_own;
                    else p.lse[(size_t)h * p.L + qi] = (pl ? big + __logf(wsum) : lse_own);
                }
            }
        }
    } else if (warp == 8) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tensormap(&tmK);
            prefetch_tensormap(&tmV);
            TileIter it(w_rng, w_nrng);
            int t0, valid, jt = 0;
            int k_last = -1, v_last = -1;   // last tile whose K / V copy was issued
            while (it.next(t0, valid)) {
                const int st = jt & 1;
                const uint32_t ph = (jt >> 1) & 1;
                if (!mbar_wait(bar(K_EMPTY + st), ph ^ 1, abort_flag, p.status, W_KEMPTY)) break;
                mbar_expect_tx(bar(K_FULL + st), TILE_BYTES);
#pragma unroll
                for (int sub = 0; sub < SUB; ++sub)
                    tma_load_2d(sK + st * TILE_BYTES + sub * SUB_BYTES, &tmK, sub * 64, h * p.L + t0, bar(K_FULL + st));
                k_last = jt;
                if (!mbar_wait(bar(V_EMPTY + st), ph ^ 1, abort_flag, p.status, W_VEMPTY)) break;
                mbar_expect_tx(bar(V_FULL + st), TILE_BYTES);
#pragma unroll
                for (int sub = 0; sub < SUB; ++sub)
                    tma_load_2d(sV + st * TILE_BYTES + sub * SUB_BYTES, &tmV, sub * 64, h * p.L + t0, bar(V_FULL + st));
                v_last = jt;
                ++jt;
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
        }
    } else {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
        // ------------------------------------------------------------ MMA issuers (one per query tile); warp 11 idles
        const int g = warp - 9;
        if (lane == 0 && g < 2 && (g == 0 || two)) {
            constexpr uint32_t IDESC_PV = idesc_bf16_f32(128, D, 0, 1);
            // Descriptors are built once; inside the issue loops only the 14-bit start-address field
            // (low word, 16-byte units) moves, so one tcgen05.mma costs the issuing thread a few
            // integer instructions.
            const uint64_t q_desc0 = smem_desc_sw128(sQ, 16, 1024), k_desc0 = smem_desc_sw128(sK, 16, 1024);
            const uint64_t v_desc0 = smem_desc_sw128(sV, SUB_BYTES, 1024);
            constexpr uint64_t STAGE = TILE_BYTES >> 4;   // next tile / next stage, in address-field units
            auto issue_qk = [&](int g, int st, int valid) {
                const int n_qk = max(16, (valid + 15) & ~15);
                const uint32_t idesc_qk = idesc_bf16_f32(128, n_qk, 0, 0);
                const uint64_t qd = q_desc0 + (g ? STAGE : 0), kd = k_desc0 + (st ? STAGE : 0);
                const uint32_t q_lo = (uint32_t)qd, q_hi = (uint32_t)(qd >> 32), k_lo = (uint32_t)kd, k_hi = (uint32_t)(kd >> 32);
                const uint32_t d_s = tmem + g * 128;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t o = ((ks >> 2) * SUB_BYTES + (ks & 3) * 32) >> 4;     // never carries out of the address field
                    mma_ss_lo(d_s, q_lo + o, q_hi, k_lo + o, k_hi, idesc_qk, ks > 0);
                }
            };
            // k-steps [ks0, ks1) of  O_g += P_g V(stage st)  (16 keys each)
            auto issue_pv = [&](int g, int st, int ks0, int ks1, bool accumulate) {
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
            // this issuer serves query tile g: S_g(0), then per key tile  O_g += P_g V(j),  S_g(j + 1)
            TileIter it(w_rng, w_nrng);
            int t0, valid, valid_next = 0;
            bool ok = it.next(t0, valid);
            ok = ok && mbar_wait(bar(Q_FULL + g), 0, abort_flag, p.status, W_QFULL);
            ok = ok && mbar_wait(bar(K_FULL + 0), 0, abort_flag, p.status, W_KFULL);
            if (ok) {
                tc_fence_after();
                issue_qk(g, 0, valid);
                tc_commit(bar(S_FULL + g));
                tc_commit(bar(K_EMPTY + 0));
            }
            for (int jt = 0; ok && jt < n_tiles; ++jt) {
                const int st = jt & 1, sn = (jt + 1) & 1;
                const uint32_t ph = (jt >> 1) & 1, phn = ((jt + 1) >> 1) & 1;
                const bool more = it.next(t0, valid_next);
                if (!mbar_wait(bar(V_FULL + st), ph, abort_flag, p.status, W_VFULL)) break;
                if (more && !mbar_wait(bar(K_FULL + sn), phn, abort_flag, p.status, W_KFULL)) break;
                const int steps = (valid + 15) >> 4, half = min(steps, 4);
                if (!mbar_wait(bar(P_HALF + g), jt & 1, abort_flag, p.status, W_PHALF)) break;
                tc_fence_after();
                issue_pv(g, st, 0, half, jt > 0);
                if (!mbar_wait(bar(P_FULL + g), jt & 1, abort_flag, p.status, W_PFULL)) break;
                tc_fence_after();
                if (steps > half) issue_pv(g, st, half, steps, true);
                // a commit between two groups of MMAs leaves the pipe idle: the next S goes out first, then all commits
                if (more) {
                    issue_qk(g, sn, valid_next);
                    tc_commit(bar(S_FULL + g));
                    tc_commit(bar(V_EMPTY + st));
                    tc_commit(bar(K_EMPTY + sn));
                } else {
                    tc_commit(bar(V_EMPTY + st));
                    tc_commit(bar(O_FULL + g));
                }
                valid = valid_next;
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
    CUtensorMap tmK, tmV;
    if (int r = make_tmap_2d_bf16(&tmK, K, (uint64_t)p->H * p->L, D, kBN)) return r;
    if (int r = make_tmap_2d_bf16(&tmV, V, (uint64_t)p->H * p->L, D, kBN)) return r;
    AttendParams a;
    a.Q = Q; a.O = O; a.lse = lse;
    a.part_o = ws_ptr<__nv_bfloat16>(ws, p->ws.part_o);
    a.part_lse = ws_ptr<float>(ws, p->ws.part_lse);
    a.qlist = ws_ptr<int32_t>(ws, p->ws.qlist);
    a.cap_total = (size_t)p->cap_off[p->C];
    a.status = ws_ptr<int>(ws, p->ws.status);
    a.H = p->H; a.L = p->L; a.k = p->k;
    a.scale_log2 = p->scale * 1.4426950408889634f;
    a.cookie = p->cookie;
    // always the d = 128 footprint: more than half an SM's shared memory, so CTAs (which each
    // take all 512 TMEM columns) never share an SM
    const size_t smem = 6 * (size_t)128 * 128 * 2 + 1024;
    MOC_CUDA_TRY(cudaFuncSetAttribute(attend_tc_kernel<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    MOC_CUDA_TRY(cudaFuncSetAttribute(attend_tc_kernel<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    // group by group of heads: the routed pass leaves the group's partials in the workspace, the anchor
    // pass merges them
    const int *tile_off = ws_ptr<int>(ws, p->ws.tile_off);
    for (int h0 = 0; h0 < p->H; h0 += p->heads_per_group) {
        const int hg = std::min(p->heads_per_group, p->H - h0);
        a.h0 = h0;
        if (p->k > 0) {
            // routed pass: the items and their count were left in the workspace with the lists; the grid
            // covers the most the group can have
            a.rng = p->d_chunk_rng;
            a.items = ws_ptr<WorkItem>(ws, p->ws.rtiles);
            a.item_lo_dev = tile_off + (size_t)h0 * p->C;
            a.item_hi_dev = tile_off + (size_t)(h0 + hg) * p->C;
            const long long bound = (long long)hg * (((long long)p->L * p->k + kQTileRows - 1) / kQTileRows + p->C);
            attend_tc_kernel<D, true><<<(unsigned)bound, kThreads, smem, s>>>(tmK, tmV, a);
            MOC_LAUNCH_CHECK();
        }
        a.rng = p->d_anc_rng;
        a.items = p->d_qitems;
        a.item_lo_dev = a.item_hi_dev = nullptr;
        dim3 grid((unsigned)p->qitems.size(), (unsigned)hg);
        attend_tc_kernel<D, false><<<grid, kThreads, smem, s>>>(tmK, tmV, a);
        MOC_LAUNCH_CHECK();
    }
    return MOC_OK;
}

int launch_attend_tc(const moc_plan *p, const __nv_bfloat16 *Q, const __nv_bfloat16 *K, const __nv_bfloat16 *V,
                     const int32_t *, __nv_bfloat16 *O, float *lse, void *ws, cudaStream_t s) {
    return p->d == 128 ? attend_tc_d<128>(p, Q, K, V, O, lse, ws, s) : attend_tc_d<64>(p, Q, K, V, O, lse, ws, s);
}

}  // namespace moc
