// Tensor-core backward of the sparse attention (selection held constant): dQ, dK, dV from
// Q, K, V, dO, the forward's log-sum-exp and delta_i = sum_x dO_ix O_ix.
//
// For a selected (query i, key t) pair:  P = exp(scale q.k - lse_i),  dP = dO_i . v_t,
// dS = P (dP - delta_i);  dV_t += P dO_i,  dK_t += scale dS q_i,  dQ_i += scale dS k_t.
//
// One kernel, three modes, one tile engine.  A CTA holds a STATIONARY pair of 128-row tiles
// (X1, X2) in shared memory and streams pairs of 128-row tiles (Y1, Y2) through three and two stages:
//     T1 = X1 Y1^T,  T2 = X2 Y2^T        (both operands from shared memory, into TMEM)
//     threads (two per TMEM lane) turn T1 into P, then (P, T2) into dS, written back to TMEM as bf16
//     ACC1 += dS Y1,  ACC2 += P Y2       (A from TMEM, B the streamed tile as an MN-major operand)
//   dQ modes (query stationary, the forward's work items, 128 rows per CTA):  X = (Q, dO) rows of
//     the item, Y = (K, V) tiles of its key ranges by TMA; lse and delta belong to the lane;
//     ACC1 is the item's dQ.  The routed mode leaves one partial per (query, slot) in the
//     workspace; the anchor mode adds them to its own part and writes dQ.
//   dK/dV mode (key stationary, one CTA per 128 keys of a chunk):  X = (K, V) rows of the key
//     tile by TMA, Y = (Q, dO) rows of every query that attends to the chunk - the query rows of
//     the chunks that have it as an anchor, then the chunk's routed query list - copied by four
//     producer warps with 16-byte asynchronous copies; lse and delta belong to the column; ACC1 is
//     dK, ACC2 is dV.  Each key tile is owned by one CTA: no atomics, no partial sums.
// The tensor pipe and the lanes overlap across tiles.  dK/dV: the issue order is ACC2(j), T1(j+1),
// ACC1(j), T2(j+1), so that while the lanes form P(j+1) the pipe runs ACC1(j) and T2(j+1), and T1 / T2
// are rewritten only after the contraction that reads the P / dS stored over them; ACC2(j) starts on the
// first half of P(j) while the lanes form the second.  dQ: no ACC2, so its columns serve as a second T2:
// T1(j+1) and T2(j+1) are issued once the lanes have read T1(j) and run while they form dS(j).
// 16 warps: 0-7 the lane threads (two per TMEM lane), 8-11 the producers, 12 and 13 the MMA issuers,
// 14-15 idle (they complete the fourth warpgroup; the lanes take the registers the others give up).  Every mbarrier wait is
// bounded; a wait that runs out flags the workspace status word and the CTA drains and leaves.
#include <algorithm>

#include "moc_common.cuh"
#include "moc_tc.cuh"

namespace moc {

using namespace tc;

enum BwdMode { DQ_ROUTED = 0, DQ_ANCHOR = 1, DKV = 2 };
enum BwdWait { BW_XFULL = 64, BW_YFULL, BW_YEMPTY, BW_T1FULL, BW_T2FULL, BW_PDONE, BW_DSDONE, BW_ACCFULL, BW_SMEM, BW_READ };

struct BwdParams {
    const __nv_bfloat16 *Q, *K, *V, *dO;
    const float *lse, *delta;
    __nv_bfloat16 *dQ, *dK, *dV;
    __nv_bfloat16 *part;          // [Hg][L][k][d] routed dQ partials of the group of heads in flight
    const float *part_lse;        // [H][L][k] the forward's routed log-sum-exps: -inf marks an empty slot
    const KeyRange *rng;          // dQ modes: key ranges the items index
    const WorkItem *items;
    const int *item_lo_dev, *item_hi_dev;   // routed mode: the group's item range [*lo, *hi) on the device
    int h0;                       // first head of the group in flight
    uint32_t cookie;              // what the workspace's status area must hold
    const KTile *ktiles;          // dK/dV mode
    int n_ktiles, n_long;         // tiles per head, and how many of them come first for every head
    const int32_t *off, *ranc_off, *ranc, *cap_off;
    const int *cnt;
    const int32_t *qlist;
    size_t cap_total;
    int *status;
    int H, L, C, k;
    float scale, scale_log2;
};

constexpr int kY1Stages = 3, kY2Stages = 2;   // stages of the streamed tiles Y1 (read twice per tile) and Y2
constexpr int kBwdThreads = 512;
constexpr float kLog2e = 1.4426950408889634f;

template <int D, int MODE>
__global__ void __launch_bounds__(kBwdThreads, 1) attend_bwd_tc_kernel(const __grid_constant__ CUtensorMap tmK,
                                                                       const __grid_constant__ CUtensorMap tmV,
                                                                       const BwdParams p) {
    constexpr int TILE_BYTES = 128 * D * 2;
    constexpr int SUB = D / 64;
    constexpr int SUB_BYTES = 128 * 128;
    constexpr int CH = D / 8;               // 16-byte pieces per row
    constexpr int N_TILES_SMEM = 2 + kY1Stages + kY2Stages;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[23];
    __shared__ uint32_t tmem_slot;
    __shared__ int s_abort;
    __shared__ int w_valid, w_h, w_rows, w_first, w_nrng, w_ntiles, w_chunk, w_t0;
    __shared__ const KeyRange *w_rng;
    // dK/dV mode: per streamed query, (lse * log2(e), delta), for tiles j and j + 1;
    // dQ modes: the first 128 words hold the item's query rows while they are staged
    __shared__ __align__(8) float s_ld[2][2][128];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gbase = smem_raw + (sbase - smem_u32(smem_raw));
    // shared tiles: X1 X2 | Y1 stages | Y2 stages
    const uint32_t sX = sbase, sY1 = sbase + 2 * TILE_BYTES, sY2 = sbase + (2 + kY1Stages) * TILE_BYTES;
    auto bar = [&](int i) { return smem_u32(&bars[i]); };
    constexpr int X_FULL = 0, Y1_FULL = 1, Y1_EMPTY = 4, Y2_FULL = 7, Y2_EMPTY = 9, T1_FULL = 11, T2_FULL = 13,
                  P_HALF = 15, P_DONE = 16, DS_DONE = 17, ACC_FULL = 19, T1_ISSUED = 20, RD1 = 21, RD2 = 22;

    if (threadIdx.x == 0) {
        s_abort = 0;
        int valid = (*(volatile int *)p.status == 0);
        if (valid && (uint32_t)((volatile int *)p.status)[ST_COOKIE] != p.cookie) {
            atomicCAS(p.status, 0, MOC_ERR_WORKSPACE);      // not this plan's lists: report, touch nothing else
            valid = 0;
        }
        uint32_t dyn_bytes;
        asm volatile("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn_bytes));
        if (valid && (sbase - smem_u32(smem_raw)) + (uint32_t)N_TILES_SMEM * TILE_BYTES > dyn_bytes) {
            // the launch gave less shared memory than the tiles need: report, touch nothing
            if (atomicCAS(p.status, 0, MOC_ERR_TIMEOUT) == 0) p.status[1] = BW_SMEM;
            valid = 0;
        }
        if (MODE != DKV) {
            int item = blockIdx.x >> 1;
            const int half = blockIdx.x & 1;
            if (MODE == DQ_ROUTED && valid) {
                item += *p.item_lo_dev;
                if (item >= *p.item_hi_dev) valid = 0;
            }
            WorkItem w = {};
            if (valid) {
                w = p.items[item];
                if (MODE == DQ_ROUTED && !index_ok((unsigned)w.h < (unsigned)p.H && w.rows > 0 && w.rows <= kQTileRows && w.first >= 0 &&
                                                   (size_t)w.first + w.rows <= p.cap_total && w.nrng == 1, p.status, IX_BWD_ITEM_FIELDS))
                    valid = 0;
            }
            if (valid) {
                w_h = MODE == DQ_ROUTED ? w.h : p.h0 + (int)blockIdx.y;
                w_first = w.first + half * 128;
                w_rows = min(128, w.rows - half * 128);
                w_rng = p.rng + w.rng_off;
                w_nrng = w.nrng;
                w_ntiles = w.ntiles;
                if (w_rows <= 0) valid = 0;
            }
        } else {
            // block order: the long key tiles of every head, then the others head by head (tiles of one chunk next
            // to each other: they stream the same query rows)
            const int n_long_all = p.n_long * p.H;
            int b = blockIdx.x, hh, ti;
            if (b < n_long_all) { hh = b / p.n_long; ti = b - hh * p.n_long; }
            else { b -= n_long_all; const int n_rest = p.n_ktiles - p.n_long; hh = b / n_rest; ti = p.n_long + b - hh * n_rest; }
            const KTile kt = p.ktiles[ti];
            w_h = hh;
            w_chunk = kt.chunk;
            w_t0 = kt.t0;
            w_rows = kt.valid;
            // query tiles: merged row ranges of the chunks that have this chunk as an anchor, then the routed list
            int nt = 0;
            const int a0 = p.ranc_off[kt.chunk], a1 = p.ranc_off[kt.chunk + 1];
            for (int a = a0; a < a1;) {
                int qc = p.ranc[a], r0 = p.off[qc], r1 = p.off[qc + 1];
                for (++a; a < a1 && p.ranc[a] == qc + 1; ++a) { qc = p.ranc[a]; r1 = p.off[qc + 1]; }
                nt += (r1 - r0 + 127) / 128;
            }
            nt += (p.cnt[w_h * p.C + kt.chunk] + 127) / 128;
            w_ntiles = nt;
        }
        w_valid = valid;
        mbar_init(bar(X_FULL), MODE == DKV ? 1 : 256);
        for (int t = 0; t < kY1Stages; ++t) {
            mbar_init(bar(Y1_FULL + t), MODE == DKV ? 128 : 1);
            mbar_init(bar(Y1_EMPTY + t), 1);
        }
        for (int t = 0; t < kY2Stages; ++t) {
            mbar_init(bar(Y2_FULL + t), MODE == DKV ? 128 : 1);
            mbar_init(bar(Y2_EMPTY + t), MODE == DKV ? 2 : 1);     // dK/dV: T2 and ACC2 both read the stage
            mbar_init(bar(T1_FULL + t), 1);
            mbar_init(bar(T2_FULL + t), 1);
            mbar_init(bar(DS_DONE + t), 256);
        }
        mbar_init(bar(P_HALF), 256);
        mbar_init(bar(P_DONE), 256);
        mbar_init(bar(T1_ISSUED), 1);
        mbar_init(bar(RD1), 256);
        mbar_init(bar(RD2), 256);
        mbar_init(bar(ACC_FULL), 2);                                // both issuers
        fence_barrier_init();
    }
    __syncthreads();
    if (!w_valid) return;
    if (warp == 8) {
        tmem_alloc(smem_u32(&tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    // TMEM columns: T1 [0,128)  T2 [128,256)  ACC1 [256,384)  ACC2 [384,512); the dQ modes have no ACC2
    // and use its columns as a second T2, for the odd tiles
    const uint32_t tmem = tmem_slot;
    const int h = w_h, rows = w_rows, n_tiles = w_ntiles;
    volatile int *abort_flag = &s_abort;

    if (warp < 8) {
        // ------------------------------------------------------------ lane threads: two per TMEM lane (warps w and
        // w + 4 reach the same lanes).  Of the four 32-column chunks of a tile, thread `half` takes chunks half and
        // 2 + half, so that the first two chunks - the first half of P for ACC2 - are finished first.  A thread
        // keeps its 64 P values between the two halves of a tile.
        asm volatile("setmaxnreg.inc.sync.aligned.u32 168;");
        const int r = threadIdx.x & 127;              // row of the stationary tile = TMEM lane
        const int half = warp >> 2;
        const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
        int qi = -1, slot = 0;
        float lse2 = INFINITY, dlt = 0.f;             // dQ modes: this lane's query
        if (MODE != DKV) {
            if (r < rows) {
                if (MODE == DQ_ROUTED) {
                    const int e = p.qlist[(size_t)h * p.cap_total + w_first + r];
                    qi = e / p.k;
                    slot = e - qi * p.k;
                    (void)index_ok(e >= 0 && qi < p.L, p.status, IX_BWD_LIST_ENTRY);
                    if ((unsigned)qi >= (unsigned)p.L) qi = -1;      // never follow an entry that is not a row of this head
                } else {
                    qi = w_first + r;
                }
                if (qi >= 0) {
                    lse2 = p.lse[(size_t)h * p.L + qi] * kLog2e;
                    dlt = p.delta[(size_t)h * p.L + qi];
                }
            }
            // stage the item's rows, one half Q and the other dO: consecutive threads take consecutive 16-byte pieces
            int *s_row = reinterpret_cast<int *>(&s_ld[0][0][0]);
            if (half == 0) s_row[r] = qi;
            asm volatile("bar.sync 1, 256;" ::: "memory");
            constexpr int RP = 128 / CH;
            const int c16 = r % CH;
            {
                const __nv_bfloat16 *src = half ? p.dO : p.Q;
                uint8_t *dst = gbase + half * TILE_BYTES + (c16 >> 3) * SUB_BYTES;
                uint4 v[CH];
#pragma unroll
                for (int ps = 0; ps < CH; ++ps) {
                    const int rr = ps * RP + r / CH, q = s_row[rr];
                    v[ps] = make_uint4(0, 0, 0, 0);
                    if (q >= 0) v[ps] = __ldg(reinterpret_cast<const uint4 *>(src + ((size_t)h * p.L + q) * D) + c16);
                }
#pragma unroll
                for (int ps = 0; ps < CH; ++ps) *reinterpret_cast<uint4 *>(dst + sw128_offset(ps * RP + r / CH, c16 & 7)) = v[ps];
            }
            fence_proxy_async_smem();
            mbar_arrive(bar(X_FULL));
        }
        const float c = p.scale_log2;
        TileIter it(w_rng, MODE == DKV ? 0 : w_nrng);
        bool ok = true;
        int s3 = 0, ph3 = 0;                          // Y1 stage of tile jt and its phase
        for (int jt = 0; jt < n_tiles; ++jt) {
            const int st = jt & 1;
            int valid = 128, t0;
            if (MODE != DKV) it.next(t0, valid);
            ok = mbar_wait_spin(bar(T1_FULL + st), (jt >> 1) & 1, abort_flag, p.status, BW_T1FULL);
            if (MODE == DKV) ok = ok && mbar_wait(bar(Y1_FULL + s3), ph3, abort_flag, p.status, BW_YFULL);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            // ---- P = exp2(scale log2(e) S - lse log2(e)) from T1
            const uint32_t t2c = (MODE != DKV && st) ? 384u : 128u;       // T2 (then dS) of this tile
            float pv[64];
#pragma unroll
            for (int rd = 0; rd < 2; ++rd) {
                const int ch = rd * 2 + half;
                uint32_t s[32];
                tmem_ld32(tmem + lane_off + ch * 32, s);
                tmem_wait_ld();
                // dK/dV: P goes over T1 columns that the other thread of the lane reads in its first round; that
                // read is announced here and waited for (bounded, like every wait) just before the first store
                if (MODE == DKV && rd == 0) mbar_arrive(bar(RD1));
#pragma unroll
                for (int x = 0; x < 32; x += 2) {
                    float l0 = lse2, l1 = lse2;
                    if (MODE == DKV) {
                        const float2 l = *reinterpret_cast<const float2 *>(&s_ld[st][0][ch * 32 + x]);
                        l0 = l.x; l1 = l.y;
                    }
                    float p0 = ex2(fmaf(__uint_as_float(s[x]), c, -l0)), p1 = ex2(fmaf(__uint_as_float(s[x + 1]), c, -l1));
                    if (MODE != DKV) {
                        if (ch * 32 + x >= valid) p0 = 0.f;
                        if (ch * 32 + x + 1 >= valid) p1 = 0.f;
                    }
                    pv[rd * 32 + x] = p0;
                    pv[rd * 32 + x + 1] = p1;
                }
                if (MODE == DKV) {
                    uint32_t ups[16];
#pragma unroll
                    for (int x = 0; x < 16; ++x) ups[x] = bf16x2(pv[rd * 32 + 2 * x], pv[rd * 32 + 2 * x + 1]);
                    if (rd == 0) {
                        ok = mbar_wait_spin(bar(RD1), jt & 1, abort_flag, p.status, BW_READ);
                        ok = __all_sync(0xffffffffu, ok);
                    }
                    if (ok) {
                        tmem_st16(tmem + lane_off + ch * 16, ups);
                        tmem_wait_st();
                        tc_fence_before();
                        mbar_arrive(bar(rd == 0 ? P_HALF : P_DONE));      // the first, then the second 64 columns of P
                    }
                }
            }
            if (!ok) break;
            if (MODE != DKV) {                                            // T1 has been read and may be overwritten
                tc_fence_before();
                mbar_arrive(bar(P_DONE));
            }
            // ---- dS = P (dP - delta) from T2, written over T2 columns that have been read
            ok = mbar_wait_spin(bar(T2_FULL + st), (jt >> 1) & 1, abort_flag, p.status, BW_T2FULL);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int rd = 0; rd < 2; ++rd) {
                const int ch = rd * 2 + half;
                uint32_t dp[32], uds[16];
                tmem_ld32(tmem + lane_off + t2c + ch * 32, dp);
                tmem_wait_ld();
                if (rd == 0) mbar_arrive(bar(RD2));                     // this thread's first-round columns have been read
#pragma unroll
                for (int x = 0; x < 32; x += 2) {
                    float d0 = dlt, d1 = dlt;
                    if (MODE == DKV) {
                        const float2 d = *reinterpret_cast<const float2 *>(&s_ld[st][1][ch * 32 + x]);
                        d0 = d.x; d1 = d.y;
                    }
                    uds[x >> 1] = bf16x2(pv[rd * 32 + x] * (__uint_as_float(dp[x]) - d0),
                                         pv[rd * 32 + x + 1] * (__uint_as_float(dp[x + 1]) - d1));
                }
                if (rd == 0) {
                    ok = mbar_wait_spin(bar(RD2), jt & 1, abort_flag, p.status, BW_READ);
                    ok = __all_sync(0xffffffffu, ok);
                }
                if (ok) tmem_st16(tmem + lane_off + t2c + ch * 16, uds);
            }
            if (!ok) break;
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar(DS_DONE + st));
            if (++s3 == kY1Stages) { s3 = 0; ph3 ^= 1; }
        }
        // ---- epilogue
        if (ok) {
            ok = mbar_wait(bar(ACC_FULL), 0, abort_flag, p.status, BW_ACCFULL);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            tc_fence_after();
#pragma unroll 1
            for (int ch = half; ch < D / 32; ch += 2) {
                uint32_t v[32];
                __syncwarp();
                tmem_ld32(tmem + lane_off + 256 + ch * 32, v);
                tmem_wait_ld();
                float acc[32];
#pragma unroll
                for (int x = 0; x < 32; ++x) acc[x] = __uint_as_float(v[x]) * p.scale;
                auto store_row = [&](__nv_bfloat16 *dst) {
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        uint4 out;
                        out.x = bf16x2(acc[q4 * 8 + 0], acc[q4 * 8 + 1]);
                        out.y = bf16x2(acc[q4 * 8 + 2], acc[q4 * 8 + 3]);
                        out.z = bf16x2(acc[q4 * 8 + 4], acc[q4 * 8 + 5]);
                        out.w = bf16x2(acc[q4 * 8 + 6], acc[q4 * 8 + 7]);
                        reinterpret_cast<uint4 *>(dst)[q4] = out;
                    }
                };
                // the routed dQ partials use the forward's layout of routed partials: query-innermost pieces
                constexpr int NP = D / 8;
                const int LB = (p.L + 127) >> 7;
                uint4 *part16 = reinterpret_cast<uint4 *>(p.part);
                if (MODE == DQ_ROUTED) {
                    if (qi >= 0) {
                        uint4 out[4];
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            out[q4].x = bf16x2(acc[q4 * 8 + 0], acc[q4 * 8 + 1]);
                            out[q4].y = bf16x2(acc[q4 * 8 + 2], acc[q4 * 8 + 3]);
                            out[q4].z = bf16x2(acc[q4 * 8 + 4], acc[q4 * 8 + 5]);
                            out[q4].w = bf16x2(acc[q4 * 8 + 6], acc[q4 * 8 + 7]);
                        }
                        // whole 32-byte sectors (pairs of pieces)
                        st_256(part16 + part_piece(h - p.h0, LB, p.k, NP, qi, slot, ch * 4), out[0], out[1]);
                        st_256(part16 + part_piece(h - p.h0, LB, p.k, NP, qi, slot, ch * 4 + 2), out[2], out[3]);
                    }
                } else if (MODE == DQ_ANCHOR) {
                    if (qi >= 0) {
                        // the routed partials of this query, four slots requested together; a slot is in use
                        // if the forward left a finite log-sum-exp for it
                        const float *pl = p.part_lse + ((size_t)h * p.L + qi) * p.k;
                        for (int s0 = 0; s0 < p.k; s0 += 4) {
                            uint4 raw[4][4];
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                const bool used = s0 + u < p.k && pl[s0 + u] != -INFINITY;
#pragma unroll
                                for (int q4 = 0; q4 < 4; q4 += 2) {
                                    raw[u][q4] = raw[u][q4 + 1] = make_uint4(0, 0, 0, 0);
                                    if (used) ld_cg_256(part16 + part_piece(h - p.h0, LB, p.k, NP, qi, s0 + u, ch * 4 + q4), raw[u][q4], raw[u][q4 + 1]);
                                }
                            }
#pragma unroll
                            for (int u = 0; u < 4; ++u)
#pragma unroll
                                for (int q4 = 0; q4 < 4; ++q4) {
                                    const __nv_bfloat162 *b = reinterpret_cast<const __nv_bfloat162 *>(&raw[u][q4]);
#pragma unroll
                                    for (int y = 0; y < 4; ++y) {
                                        const float2 f = __bfloat1622float2(b[y]);
                                        acc[q4 * 8 + 2 * y] += f.x;
                                        acc[q4 * 8 + 2 * y + 1] += f.y;
                                    }
                                }
                        }
                        store_row(p.dQ + ((size_t)h * p.L + qi) * D + ch * 32);
                    }
                } else {
                    if (r < rows) store_row(p.dK + ((size_t)h * p.L + w_t0 + r) * D + ch * 32);
                    // dV = ACC2, not scaled
                    __syncwarp();
                    tmem_ld32(tmem + lane_off + 384 + ch * 32, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int x = 0; x < 32; ++x) acc[x] = __uint_as_float(v[x]);
                    if (r < rows) store_row(p.dV + ((size_t)h * p.L + w_t0 + r) * D + ch * 32);
                }
            }
        }
    } else if (warp < 12) {
        // ------------------------------------------------------------ producers
        asm volatile("setmaxnreg.dec.sync.aligned.u32 80;");
        if (MODE != DKV) {
            if (warp == 8 && lane == 0) {
                prefetch_tensormap(&tmK);
                prefetch_tensormap(&tmV);
                TileIter it(w_rng, w_nrng);
                int t0, valid, jt = 0, s3 = 0, ph3 = 0, n_k = 0;      // jt counts the V copies issued, n_k the K copies
                while (it.next(t0, valid)) {
                    const int s2 = jt & 1;
                    if (!mbar_wait(bar(Y1_EMPTY + s3), ph3 ^ 1, abort_flag, p.status, BW_YEMPTY)) break;
                    mbar_expect_tx(bar(Y1_FULL + s3), TILE_BYTES);
#pragma unroll
                    for (int sub = 0; sub < SUB; ++sub)
                        tma_load_2d(sY1 + s3 * TILE_BYTES + sub * SUB_BYTES, &tmK, sub * 64, h * p.L + t0, bar(Y1_FULL + s3));
                    ++n_k;
                    if (!mbar_wait(bar(Y2_EMPTY + s2), ((jt >> 1) & 1) ^ 1, abort_flag, p.status, BW_YEMPTY)) break;
                    mbar_expect_tx(bar(Y2_FULL + s2), TILE_BYTES);
#pragma unroll
                    for (int sub = 0; sub < SUB; ++sub)
                        tma_load_2d(sY2 + s2 * TILE_BYTES + sub * SUB_BYTES, &tmV, sub * 64, h * p.L + t0, bar(Y2_FULL + s2));
                    ++jt;
                    if (++s3 == kY1Stages) { s3 = 0; ph3 ^= 1; }
                }
                if (*abort_flag) {      // copies already issued must land before the shared memory is released
                    int dummy_flag = 0;
                    for (int b = 1; b <= kY1Stages; ++b)
                        if (n_k - b >= 0) mbar_wait(bar(Y1_FULL + ((n_k - b) % kY1Stages)), ((n_k - b) / kY1Stages) & 1, &dummy_flag, p.status, BW_YFULL);
                    for (int b = 1; b <= kY2Stages; ++b)
                        if (jt - b >= 0) mbar_wait(bar(Y2_FULL + ((jt - b) & 1)), ((jt - b) >> 1) & 1, &dummy_flag, p.status, BW_YFULL);
                }
            }
        } else {
            // the key tile itself: K -> X1, V -> X2
            if (warp == 8 && lane == 0) {
                mbar_expect_tx(bar(X_FULL), 2 * TILE_BYTES);
#pragma unroll
                for (int sub = 0; sub < SUB; ++sub) {
                    tma_load_2d(sX + sub * SUB_BYTES, &tmK, sub * 64, h * p.L + w_t0, bar(X_FULL));
                    tma_load_2d(sX + TILE_BYTES + sub * SUB_BYTES, &tmV, sub * 64, h * p.L + w_t0, bar(X_FULL));
                }
            }
            // the queries that attend to this chunk, 128 at a time: Q rows -> Y1, dO rows -> Y2; each of the
            // four producer warps copies 32 rows of every tile
            const int pw = warp - 8;
            const int chunk = w_chunk;
            const int a1 = p.ranc_off[chunk + 1];
            int a = p.ranc_off[chunk], r0 = 0, r1 = 0;       // current row range [r0, r1)
            const int n_list = p.cnt[h * p.C + chunk];
            const int32_t *list = p.qlist + (size_t)h * p.cap_total + p.cap_off[chunk];
            int e0 = 0;                                        // next entry of the routed list
            int s3 = 0, ph3 = 0;
            bool ok = true;
            const int i = pw * 32 + lane;                      // this lane's row of every tile
            // the query behind this lane's row of the next tile, with its lse and delta; loaded one tile ahead so
            // that these dependent loads are never waited for
            int q = -1;
            float q_lse = INFINITY, q_del = 0.f;
            auto next_rows = [&]() {
                if (r0 >= r1 && a < a1) {                      // next merged range of anchor query rows
                    int qc = p.ranc[a];
                    r0 = p.off[qc]; r1 = p.off[qc + 1];
                    for (++a; a < a1 && p.ranc[a] == qc + 1; ++a) { qc = p.ranc[a]; r1 = p.off[qc + 1]; }
                }
                q = -1;
                if (r0 < r1) { if (r0 + i < r1) q = r0 + i; }
                else if (e0 + i < n_list && index_ok((size_t)p.cap_off[chunk] + e0 + i < p.cap_total, p.status, IX_BWD_LIST_POSITION)) {
                    q = list[e0 + i] / p.k;
                    if (!index_ok((unsigned)q < (unsigned)p.L, p.status, IX_BWD_LIST_ENTRY)) q = -1;
                }
                if (r0 < r1) r0 += 128; else e0 += 128;
                // a column without a query gets lse = +inf: its P and dS come out as exact zeros
                q_lse = q >= 0 ? p.lse[(size_t)h * p.L + q] * kLog2e : INFINITY;
                q_del = q >= 0 ? p.delta[(size_t)h * p.L + q] : 0.f;
            };
            if (n_tiles > 0) next_rows();
            for (int jt = 0; ok && jt < n_tiles; ++jt) {
                const int s2 = jt & 1;
                ok = mbar_wait(bar(Y1_EMPTY + s3), ph3 ^ 1, abort_flag, p.status, BW_YEMPTY);
                ok = ok && mbar_wait(bar(Y2_EMPTY + s2), ((jt >> 1) & 1) ^ 1, abort_flag, p.status, BW_YEMPTY);
                // the lanes have finished with the lse / delta of tile jt - 2
                if (jt >= 2) ok = ok && mbar_wait(bar(DS_DONE + s2), ((jt - 2) >> 1) & 1, abort_flag, p.status, BW_DSDONE);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                s_ld[s2][0][i] = q_lse;
                s_ld[s2][1][i] = q_del;
                constexpr int RP = 32 / CH;                    // rows per instruction
                const int c16 = lane % CH;
#pragma unroll
                for (int rb = 0; rb < 32; rb += RP) {
                    const int rl = rb + lane / CH, rr = pw * 32 + rl;
                    const int qq = __shfl_sync(0xffffffffu, q, rl);
                    const size_t src = ((size_t)h * p.L + max(qq, 0)) * D + c16 * 8;
                    const uint32_t dst = (c16 >> 3) * SUB_BYTES + sw128_offset(rr, c16 & 7);
                    cp_async16(sY1 + s3 * TILE_BYTES + dst, p.Q + src, qq >= 0 ? 16u : 0u);
                    cp_async16(sY2 + s2 * TILE_BYTES + dst, p.dO + src, qq >= 0 ? 16u : 0u);
                }
                if (jt + 1 < n_tiles) next_rows();
                cp_async_wait_all();
                fence_proxy_async_smem();
                mbar_arrive(bar(Y1_FULL + s3));
                mbar_arrive(bar(Y2_FULL + s2));
                if (++s3 == kY1Stages) { s3 = 0; ph3 ^= 1; }
            }
        }
    } else {
        // ------------------------------------------------------------ MMA issuers: warp 12 owns the T1 / P side
        // (T1, ACC2), warp 13 the T2 / dS side (T2, ACC1); each side's TMEM columns are touched by its issuer only,
        // so the two instruction streams need no ordering between them and one's waits and commits are
        // covered by the other's MMAs.  Warps 14 and 15 idle.
        asm volatile("setmaxnreg.dec.sync.aligned.u32 88;");
        if (warp <= 13 && lane == 0) {
            const bool side1 = warp == 12;
            constexpr uint32_t IDESC_T = idesc_bf16_f32(128, 128, 0, 0);      // T = X Y^T, both K-major
            constexpr uint32_t IDESC_ACC = idesc_bf16_f32(128, D, 0, 1);      // ACC += (TMEM) Y, Y MN-major
            constexpr uint64_t STAGE = TILE_BYTES >> 4;
            const uint64_t x1 = smem_desc_sw128(sX, 16, 1024), x2 = smem_desc_sw128(sX + TILE_BYTES, 16, 1024);
            const uint64_t y1k = smem_desc_sw128(sY1, 16, 1024), y2k = smem_desc_sw128(sY2, 16, 1024);
            const uint64_t y1m = smem_desc_sw128(sY1, SUB_BYTES, 1024), y2m = smem_desc_sw128(sY2, SUB_BYTES, 1024);
            // only the start-address field (low word) of a descriptor moves: 32-bit arithmetic, never a carry out of it
            auto lo = [](uint64_t d) { return (uint32_t)d; };
            auto hi = [](uint64_t d) { return (uint32_t)(d >> 32); };
            bool ok = true;
            auto wait = [&](int b, int parity, int code) { ok = ok && mbar_wait_spin(bar(b), parity, abort_flag, p.status, code); };
            // the MMA groups, without their waits and commits
            // (s3 = j mod the Y1 stage count is carried along by the callers: no division on this thread)
            auto t1 = [&](int j, int s3) {  // T1(j) = X1 Y1(j)^T
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t o = ((ks >> 2) * SUB_BYTES + (ks & 3) * 32) >> 4;
                    mma_ss_lo(tmem, lo(x1) + o, hi(x1), lo(y1k) + s3 * (uint32_t)STAGE + o, hi(y1k), IDESC_T, ks > 0);
                }
            };
            auto t2 = [&](int j) {          // T2(j) = X2 Y2(j)^T
                const int s2 = j & 1;
                const uint32_t d = tmem + ((MODE != DKV && s2) ? 384u : 128u);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t o = ((ks >> 2) * SUB_BYTES + (ks & 3) * 32) >> 4;
                    mma_ss_lo(d, lo(x2) + o, hi(x2), lo(y2k) + s2 * (uint32_t)STAGE + o, hi(y2k), IDESC_T, ks > 0);
                }
            };
            auto acc1 = [&](int j, int s3) {   // ACC1 += dS(j) Y1(j)
                const uint32_t ds = tmem + ((MODE != DKV && (j & 1)) ? 384u : 128u);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    mma_ts_lo(tmem + 256, ds + ks * 8, lo(y1m) + s3 * (uint32_t)STAGE + ks * (2048 >> 4), hi(y1m), IDESC_ACC, j > 0 || ks > 0);
            };
            auto acc2 = [&](int j, int half) {   // ACC2 += P(j) Y2(j), the K steps of one half of P
                const int s2 = j & 1;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    mma_ts_lo(tmem + 384, tmem + (half * 4 + ks) * 8, lo(y2m) + s2 * (uint32_t)STAGE + (half * 4 + ks) * (2048 >> 4), hi(y2m),
                              IDESC_ACC, j > 0 || half > 0 || ks > 0);
            };
            // A wait, a fence or a commit between two groups leaves the pipe idle for longer than it takes, so each
            // side waits early for the tiles it will read, fences once per hand-over from the lanes, and commits
            // after the last group it has to issue at that point.
            wait(X_FULL, 0, BW_XFULL);
            if (side1) {
                // dK/dV: ACC2(j) starts on the first half of P(j); T1(j+1) follows ACC2(j), which reads the P
                // written over T1(j).  dQ: T1(j+1) follows the lanes' read of T1(j).
                if (n_tiles > 0) {
                    wait(Y1_FULL, 0, BW_YFULL);
                    if (ok) {
                        tc_fence_after();
                        t1(0, 0);
                        tc_commit(bar(T1_FULL));
                    }
                }
                int s3n = 1 % kY1Stages, ph3n = 0;                       // stage and phase of tile j + 1
                for (int j = 0; ok && j < n_tiles; ++j) {
                    const bool more = j + 1 < n_tiles;
                    if (MODE == DKV) {
                        wait(P_HALF, j & 1, BW_PDONE);
                        if (!ok) break;
                        tc_fence_after();
                        acc2(j, 0);
                    }
                    if (more) wait(Y1_FULL + s3n, ph3n, BW_YFULL);
                    if (MODE == DKV || more) wait(P_DONE, j & 1, BW_PDONE);
                    if (!ok) break;
                    tc_fence_after();
                    if (MODE == DKV) acc2(j, 1);
                    if (more) {
                        t1(j + 1, s3n);
                        tc_commit(bar(T1_FULL + ((j + 1) & 1)));
                    }
                    if (++s3n == kY1Stages) { s3n = 0; ph3n ^= 1; }
                    if (MODE == DKV) {
                        tc_commit(bar(Y2_EMPTY + (j & 1)));                 // the second of two arrivals
                        if (more) mbar_arrive(bar(T1_ISSUED));              // the other side may use the pipe again
                    }
                }
            } else {
                // The lanes wait for T1(j+1) as soon as dS(j) is done, so this side keeps out of the pipe while the
                // other issues it.  dK/dV: ACC1(j) waits for that issue, and T2(j+1) follows ACC1(j), which reads the
                // dS written over T2(j).  dQ: two T2 buffers; ACC1(j) then T2(j+2), both while the lanes form P(j+1).
                constexpr int AHEAD = MODE == DKV ? 1 : 2;
                for (int j = 0; ok && j < AHEAD && j < n_tiles; ++j) {
                    wait(Y2_FULL + (j & 1), 0, BW_YFULL);
                    if (!ok) break;
                    tc_fence_after();
                    t2(j);
                    tc_commit(bar(T2_FULL + (j & 1)));
                    tc_commit(bar(Y2_EMPTY + (j & 1)));
                }
                int s3 = 0;                                               // Y1 stage of tile j
                for (int j = 0; ok && j < n_tiles; ++j) {
                    const int jn = j + AHEAD;
                    const bool more = jn < n_tiles;
                    if (MODE == DKV && j + 1 < n_tiles) wait(T1_ISSUED, j & 1, BW_T1FULL);
                    wait(DS_DONE + (j & 1), (j >> 1) & 1, BW_DSDONE);
                    if (!ok) break;
                    tc_fence_after();
                    acc1(j, s3);
                    tc_commit(bar(Y1_EMPTY + s3));                  // at once: the next K tile waits for this stage
                    if (++s3 == kY1Stages) s3 = 0;
                    if (more) {
                        wait(Y2_FULL + (jn & 1), (jn >> 1) & 1, BW_YFULL);
                        if (!ok) break;
                        t2(jn);
                        tc_commit(bar(T2_FULL + (jn & 1)));
                        tc_commit(bar(Y2_EMPTY + (jn & 1)));    // dQ modes: V is read here only; dK/dV: the first of two arrivals
                    }
                }
            }
            if (ok) tc_commit(bar(ACC_FULL));
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 8) tmem_dealloc(tmem, 512);
}

template <int D>
static int attend_bwd_tc_d(const moc_plan *p, const __nv_bfloat16 *Q, const __nv_bfloat16 *K, const __nv_bfloat16 *V,
                           const __nv_bfloat16 *O, const float *lse, const __nv_bfloat16 *dO, const int32_t *sel,
                           __nv_bfloat16 *dQ, __nv_bfloat16 *dK, __nv_bfloat16 *dV, void *ws, cudaStream_t s) {
    float *delta = ws_ptr<float>(ws, p->ws.delta);
    if (int r = launch_delta(p, O, dO, delta, s)) return r;
    CUtensorMap tmK, tmV;
    if (int r = make_tmap_2d_bf16(&tmK, K, (uint64_t)p->H * p->L, D, 128)) return r;
    if (int r = make_tmap_2d_bf16(&tmV, V, (uint64_t)p->H * p->L, D, 128)) return r;
    BwdParams a;
    a.Q = Q; a.K = K; a.V = V; a.dO = dO; a.lse = lse; a.delta = delta;
    a.part_lse = ws_ptr<float>(ws, p->ws.part_lse);
    a.cookie = p->cookie; a.h0 = 0; a.item_lo_dev = a.item_hi_dev = nullptr;
    a.dQ = dQ; a.dK = dK; a.dV = dV;
    a.part = ws_ptr<__nv_bfloat16>(ws, p->ws.part_o);      // the forward's partial outputs are no longer needed
    a.ktiles = p->d_ktiles; a.n_ktiles = (int)p->ktiles.size(); a.n_long = p->n_long_ktiles; a.off = p->d_off; a.ranc_off = p->d_ranc_off; a.ranc = p->d_ranc; a.cap_off = p->d_cap_off;
    a.cnt = ws_ptr<int>(ws, p->ws.cnt);
    a.qlist = ws_ptr<int32_t>(ws, p->ws.qlist);
    a.cap_total = (size_t)p->cap_off[p->C];
    a.status = ws_ptr<int>(ws, p->ws.status);
    a.H = p->H; a.L = p->L; a.C = p->C; a.k = p->k;
    a.scale = p->scale; a.scale_log2 = p->scale * kLog2e;
    // seven tiles (X1 X2, three Y1 stages, two Y2 stages) and the slack that aligns them to 1024 bytes; at
    // d = 128 that is all an SM has, so the request is what the kernel's static variables leave of the limit
    const size_t tiles = (size_t)(2 + kY1Stages + kY2Stages) * 128 * D * 2;
    size_t smem[3];
    {
        int optin = 0;
        MOC_CUDA_TRY(cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, p->device));
        const void *fn[3] = {(const void *)attend_bwd_tc_kernel<D, DQ_ROUTED>, (const void *)attend_bwd_tc_kernel<D, DQ_ANCHOR>,
                             (const void *)attend_bwd_tc_kernel<D, DKV>};
        for (int m = 0; m < 3; ++m) {
            cudaFuncAttributes fa;
            MOC_CUDA_TRY(cudaFuncGetAttributes(&fa, fn[m]));
            smem[m] = std::min(tiles + 1024, (size_t)optin - fa.sharedSizeBytes);
            if (smem[m] < tiles) return MOC_ERR_SHAPE;
            MOC_CUDA_TRY(cudaFuncSetAttribute(fn[m], cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem[m]));
        }
    }
    // dQ group by group of heads (the routed mode leaves the group's partials in the workspace, the
    // anchor mode adds them up), then dK / dV of every key tile
    const int *tile_off = ws_ptr<int>(ws, p->ws.tile_off);
    for (int h0 = 0; h0 < p->H; h0 += p->heads_per_group) {
        const int hg = std::min(p->heads_per_group, p->H - h0);
        a.h0 = h0;
        if (p->k > 0) {
            a.rng = p->d_chunk_rng;
            a.items = ws_ptr<WorkItem>(ws, p->ws.rtiles);
            a.item_lo_dev = tile_off + (size_t)h0 * p->C;
            a.item_hi_dev = tile_off + (size_t)(h0 + hg) * p->C;
            const long long bound = (long long)hg * (((long long)p->L * p->k + kQTileRows - 1) / kQTileRows + p->C);
            attend_bwd_tc_kernel<D, DQ_ROUTED><<<(unsigned)(2 * bound), kBwdThreads, smem[DQ_ROUTED], s>>>(tmK, tmV, a);
            MOC_LAUNCH_CHECK();
        }
        a.rng = p->d_anc_rng;
        a.items = p->d_qitems;
        a.item_lo_dev = a.item_hi_dev = nullptr;
        attend_bwd_tc_kernel<D, DQ_ANCHOR><<<dim3((unsigned)(2 * p->qitems.size()), (unsigned)hg), kBwdThreads, smem[DQ_ANCHOR], s>>>(tmK, tmV, a);
        MOC_LAUNCH_CHECK();
    }
    attend_bwd_tc_kernel<D, DKV><<<(unsigned)(p->ktiles.size() * (size_t)p->H), kBwdThreads, smem[DKV], s>>>(tmK, tmV, a);
    MOC_LAUNCH_CHECK();
    return MOC_OK;
}

int launch_attend_bwd_tc(const moc_plan *p, const __nv_bfloat16 *Q, const __nv_bfloat16 *K, const __nv_bfloat16 *V,
                         const __nv_bfloat16 *O, const float *lse, const __nv_bfloat16 *dO, const int32_t *sel,
                         __nv_bfloat16 *dQ, __nv_bfloat16 *dK, __nv_bfloat16 *dV, void *ws, cudaStream_t s) {
    return p->d == 128 ? attend_bwd_tc_d<128>(p, Q, K, V, O, lse, dO, sel, dQ, dK, dV, ws, s)
                       : attend_bwd_tc_d<64>(p, Q, K, V, O, lse, dO, sel, dQ, dK, dV, ws, s);
}

}  // namespace moc
