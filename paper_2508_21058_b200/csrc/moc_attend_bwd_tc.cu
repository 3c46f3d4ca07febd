// Tensor-core backward of the sparse attention (selection held constant): dQ, dK, dV from
// Q, K, V, dO, the forward's log-sum-exp and delta_i = sum_x dO_ix O_ix.
//
// For a selected (query i, key t) pair:  P = exp(scale q.k - lse_i),  dP = dO_i . v_t,
// dS = P (dP - delta_i);  dV_t += P dO_i,  dK_t += scale dS q_i,  dQ_i += scale dS k_t.
//
// One kernel, three modes, one tile engine.  A CTA holds a STATIONARY pair of 128-row tiles
// (X1, X2) in shared memory and streams pairs of 128-row tiles (Y1, Y2) through two stages:
//     T1 = X1 Y1^T,  T2 = X2 Y2^T        (two MMAs, both operands from shared memory, into TMEM)
//     threads (one TMEM lane each) turn (T1, T2) into P and dS, written back to TMEM as bf16
//     ACC1 += dS Y1,  ACC2 += P Y2       (A from TMEM, B the streamed tile as an MN-major operand)
//   dQ modes (query stationary, the forward's work items, 128 rows per CTA):  X = (Q, dO) rows of
//     the item, Y = (K, V) tiles of its key ranges by TMA; lse and delta belong to the lane;
//     ACC1 is the item's dQ.  The routed mode leaves one partial per (query, slot) in the
//     workspace; the anchor mode adds them to its own part and writes dQ.
//   dK/dV mode (key stationary, one CTA per 128 keys of a chunk):  X = (K, V) rows of the key
//     tile by TMA, Y = (Q, dO) rows of every query that attends to the chunk - the query rows of
//     the chunks that have it as an anchor, then the chunk's routed query list - copied by the
//     producer warp with 16-byte asynchronous copies; lse and delta belong to the column; ACC1 is
//     dK, ACC2 is dV.  Each key tile is owned by one CTA: no atomics, no partial sums.
// 6 warps: 0-3 the lane threads, 4 the producer, 5 the MMA issuer.  Every mbarrier wait is
// bounded; a wait that runs out flags the workspace status word and the CTA drains and leaves.
#include <algorithm>

#include "moc_common.cuh"
#include "moc_tc.cuh"

namespace moc {

using namespace tc;

enum BwdMode { DQ_ROUTED = 0, DQ_ANCHOR = 1, DKV = 2 };
enum BwdWait { BW_XFULL = 64, BW_YFULL, BW_YEMPTY, BW_TFULL, BW_DFULL, BW_ACCFULL };

struct BwdParams {
    const __nv_bfloat16 *Q, *K, *V, *dO;
    const float *lse, *delta;
    const int32_t *sel;
    __nv_bfloat16 *dQ, *dK, *dV;
    __nv_bfloat16 *part;          // [H][L][k][d] routed dQ partials
    const KeyRange *rng;          // dQ modes: key ranges the items index
    const WorkItem *items;
    const int *n_items_dev;       // routed mode: item count on the device
    const KTile *ktiles;          // dK/dV mode
    const int32_t *off, *ranc_off, *ranc, *cap_off;
    const int *cnt;
    const int32_t *qlist;
    size_t cap_total;
    int *status;
    int H, L, C, k;
    float scale, scale_log2;
};

constexpr int kBwdThreads = 192;
constexpr float kLog2e = 1.4426950408889634f;

template <int D, int MODE>
__global__ void __launch_bounds__(kBwdThreads, 1) attend_bwd_tc_kernel(const __grid_constant__ CUtensorMap tmK,
                                                                       const __grid_constant__ CUtensorMap tmV,
                                                                       const BwdParams p) {
    constexpr int TILE_BYTES = 128 * D * 2;
    constexpr int SUB = D / 64;
    constexpr int SUB_BYTES = 128 * 128;
    constexpr int CH = D / 8;               // 16-byte pieces per row
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[10];
    __shared__ uint32_t tmem_slot;
    __shared__ int s_abort;
    __shared__ int w_valid, w_h, w_rows, w_first, w_nrng, w_ntiles, w_chunk, w_t0;
    __shared__ const KeyRange *w_rng;
    __shared__ int s_row[2][128];           // query row behind each row of the staged tile (-1 = none)
    __shared__ float s_lse[2][128], s_del[2][128];   // dK/dV mode: per streamed query, lse * log2(e) and delta

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gbase = smem_raw + (sbase - smem_u32(smem_raw));
    // shared tiles: X1 X2 | Y1 stage 0,1 | Y2 stage 0,1
    const uint32_t sX = sbase, sY1 = sbase + 2 * TILE_BYTES, sY2 = sbase + 4 * TILE_BYTES;
    auto bar = [&](int i) { return smem_u32(&bars[i]); };
    constexpr int X_FULL = 0, Y_FULL = 1, Y_EMPTY = 3, T_FULL = 5, D_FULL = 6, ACC_FULL = 7;

    if (threadIdx.x == 0) {
        s_abort = 0;
        int valid = (*(volatile int *)p.status == 0);
        if (MODE != DKV) {
            const int item = blockIdx.x >> 1, half = blockIdx.x & 1;
            if (MODE == DQ_ROUTED && valid && item >= *p.n_items_dev) valid = 0;
            if (valid) {
                const WorkItem w = p.items[item];
                w_h = MODE == DQ_ROUTED ? w.h : (int)blockIdx.y;
                w_first = w.first + half * 128;
                w_rows = min(128, w.rows - half * 128);
                w_rng = p.rng + w.rng_off;
                w_nrng = w.nrng;
                w_ntiles = w.ntiles;
                if (w_rows <= 0) valid = 0;
            }
        } else {
            const KTile kt = p.ktiles[blockIdx.x];
            w_h = blockIdx.y;
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
        mbar_init(bar(X_FULL), MODE == DKV ? 1 : 128);
        for (int t = 0; t < 2; ++t) {
            mbar_init(bar(Y_FULL + t), MODE == DKV ? 32 : 1);
            mbar_init(bar(Y_EMPTY + t), 1);
        }
        mbar_init(bar(T_FULL), 1);
        mbar_init(bar(D_FULL), 128);
        mbar_init(bar(ACC_FULL), 1);
        fence_barrier_init();
    }
    __syncthreads();
    if (!w_valid) return;
    if (warp == 4) {
        tmem_alloc(smem_u32(&tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    const uint32_t tmem = tmem_slot;      // T1 [0,128)  T2 [128,256)  ACC1 [256,384)  ACC2 [384,512)
    const int h = w_h, rows = w_rows, n_tiles = w_ntiles;
    volatile int *abort_flag = &s_abort;

    if (warp < 4) {
        // ------------------------------------------------------------ lane threads
        const int r = threadIdx.x;                    // row of the stationary tile = TMEM lane
        const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
        int qi = -1, slot = 0;
        float lse2 = INFINITY, dlt = 0.f;             // dQ modes: this lane's query
        if (MODE != DKV) {
            if (r < rows) {
                if (MODE == DQ_ROUTED) {
                    const int e = p.qlist[(size_t)h * p.cap_total + w_first + r];
                    qi = e / p.k;
                    slot = e - qi * p.k;
                } else {
                    qi = w_first + r;
                }
                lse2 = p.lse[(size_t)h * p.L + qi] * kLog2e;
                dlt = p.delta[(size_t)h * p.L + qi];
            }
            // stage the item's Q and dO rows together: consecutive threads take consecutive 16-byte pieces
            s_row[0][r] = qi;
            asm volatile("bar.sync 1, 128;" ::: "memory");
            constexpr int RP = 128 / CH;
            const int c16 = r % CH;
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                const __nv_bfloat16 *src = which ? p.dO : p.Q;
                uint8_t *dst = gbase + which * TILE_BYTES + (c16 >> 3) * SUB_BYTES;
                uint4 v[CH];
#pragma unroll
                for (int ps = 0; ps < CH; ++ps) {
                    const int rr = ps * RP + r / CH, q = s_row[0][rr];
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
        for (int jt = 0; jt < n_tiles; ++jt) {
            const int st = jt & 1;
            int valid = 128, t0;
            if (MODE != DKV) it.next(t0, valid);
            ok = mbar_wait(bar(T_FULL), jt & 1, abort_flag, p.status, BW_TFULL);
            if (MODE == DKV) ok = ok && mbar_wait(bar(Y_FULL + st), (jt >> 1) & 1, abort_flag, p.status, BW_YFULL);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
#pragma unroll 1
            for (int ch = 0; ch < 4; ++ch) {
                uint32_t s[32], dp[32];
                tmem_ld32(tmem + lane_off + ch * 32, s);
                tmem_ld32(tmem + lane_off + 128 + ch * 32, dp);
                tmem_wait_ld();
                uint32_t ups[16], uds[16];
#pragma unroll
                for (int x = 0; x < 32; x += 2) {
                    float l0 = lse2, l1 = lse2, d0 = dlt, d1 = dlt;
                    if (MODE == DKV) {
                        const float2 l = *reinterpret_cast<const float2 *>(&s_lse[st][ch * 32 + x]);
                        const float2 d = *reinterpret_cast<const float2 *>(&s_del[st][ch * 32 + x]);
                        l0 = l.x; l1 = l.y; d0 = d.x; d1 = d.y;
                    }
                    float p0 = ex2(fmaf(__uint_as_float(s[x]), c, -l0)), p1 = ex2(fmaf(__uint_as_float(s[x + 1]), c, -l1));
                    if (MODE != DKV) {
                        if (ch * 32 + x >= valid) p0 = 0.f;
                        if (ch * 32 + x + 1 >= valid) p1 = 0.f;
                    }
                    const float ds0 = p0 * (__uint_as_float(dp[x]) - d0), ds1 = p1 * (__uint_as_float(dp[x + 1]) - d1);
                    ups[x >> 1] = bf16x2(p0, p1);
                    uds[x >> 1] = bf16x2(ds0, ds1);
                }
                tmem_st16(tmem + lane_off + 128 + ch * 16, uds);          // dS over the T2 columns already read
                if (MODE == DKV) tmem_st16(tmem + lane_off + ch * 16, ups);   // P over the T1 columns already read
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar(D_FULL));
        }
        // ---- epilogue
        if (ok) {
            ok = mbar_wait(bar(ACC_FULL), 0, abort_flag, p.status, BW_ACCFULL);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            tc_fence_after();
#pragma unroll 1
            for (int ch = 0; ch < D / 32; ++ch) {
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
                if (MODE == DQ_ROUTED) {
                    if (qi >= 0) store_row(p.part + (((size_t)h * p.L + qi) * p.k + slot) * D + ch * 32);
                } else if (MODE == DQ_ANCHOR) {
                    if (qi >= 0) {
                        for (int s = 0; s < p.k; ++s) {
                            if (p.sel[((size_t)h * p.L + qi) * p.k + s] < 0) continue;
                            const uint4 *src = reinterpret_cast<const uint4 *>(p.part + (((size_t)h * p.L + qi) * p.k + s) * D + ch * 32);
#pragma unroll
                            for (int q4 = 0; q4 < 4; ++q4) {
                                const uint4 raw = __ldcg(src + q4);
                                const __nv_bfloat162 *b = reinterpret_cast<const __nv_bfloat162 *>(&raw);
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
    } else if (warp == 4) {
        // ------------------------------------------------------------ producer
        if (MODE != DKV) {
            if (lane == 0) {
                prefetch_tensormap(&tmK);
                prefetch_tensormap(&tmV);
                TileIter it(w_rng, w_nrng);
                int t0, valid, jt = 0;
                while (it.next(t0, valid)) {
                    const int st = jt & 1;
                    if (!mbar_wait(bar(Y_EMPTY + st), ((jt >> 1) & 1) ^ 1, abort_flag, p.status, BW_YEMPTY)) break;
                    mbar_expect_tx(bar(Y_FULL + st), 2 * TILE_BYTES);
#pragma unroll
                    for (int sub = 0; sub < SUB; ++sub) {
                        tma_load_2d(sY1 + st * TILE_BYTES + sub * SUB_BYTES, &tmK, sub * 64, h * p.L + t0, bar(Y_FULL + st));
                        tma_load_2d(sY2 + st * TILE_BYTES + sub * SUB_BYTES, &tmV, sub * 64, h * p.L + t0, bar(Y_FULL + st));
                    }
                    ++jt;
                }
                if (*abort_flag) {      // copies already issued must land before the shared memory is released
                    int dummy_flag = 0;
                    for (int b = 1; b <= 2; ++b)
                        if (jt - b >= 0) mbar_wait(bar(Y_FULL + ((jt - b) & 1)), ((jt - b) >> 1) & 1, &dummy_flag, p.status, BW_YFULL);
                }
            }
        } else {
            // the key tile itself: K -> X1, V -> X2
            if (lane == 0) {
                mbar_expect_tx(bar(X_FULL), 2 * TILE_BYTES);
#pragma unroll
                for (int sub = 0; sub < SUB; ++sub) {
                    tma_load_2d(sX + sub * SUB_BYTES, &tmK, sub * 64, h * p.L + w_t0, bar(X_FULL));
                    tma_load_2d(sX + TILE_BYTES + sub * SUB_BYTES, &tmV, sub * 64, h * p.L + w_t0, bar(X_FULL));
                }
            }
            // the queries that attend to this chunk, 128 at a time: Q rows -> Y1, dO rows -> Y2
            const int chunk = w_chunk;
            const int a1 = p.ranc_off[chunk + 1];
            int a = p.ranc_off[chunk], r0 = 0, r1 = 0;       // current row range [r0, r1)
            const int n_list = p.cnt[h * p.C + chunk];
            const int32_t *list = p.qlist + (size_t)h * p.cap_total + p.cap_off[chunk];
            int e0 = 0;                                        // next entry of the routed list
            bool ok = true;
            for (int jt = 0; ok && jt < n_tiles; ++jt) {
                const int st = jt & 1;
                if (r0 >= r1 && a < a1) {                      // next merged range of anchor query rows
                    int qc = p.ranc[a];
                    r0 = p.off[qc]; r1 = p.off[qc + 1];
                    for (++a; a < a1 && p.ranc[a] == qc + 1; ++a) { qc = p.ranc[a]; r1 = p.off[qc + 1]; }
                }
                int qrow[4];
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    const int i = m * 32 + lane;
                    qrow[m] = -1;
                    if (r0 < r1) { if (r0 + i < r1) qrow[m] = r0 + i; }
                    else if (e0 + i < n_list) qrow[m] = list[e0 + i] / p.k;
                }
                if (r0 < r1) r0 += 128; else e0 += 128;
                ok = mbar_wait(bar(Y_EMPTY + st), ((jt >> 1) & 1) ^ 1, abort_flag, p.status, BW_YEMPTY);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    const int i = m * 32 + lane, q = qrow[m];
                    s_row[st][i] = q;
                    // a column without a query gets lse = +inf: its P and dS come out as exact zeros
                    s_lse[st][i] = q >= 0 ? p.lse[(size_t)h * p.L + q] * kLog2e : INFINITY;
                    s_del[st][i] = q >= 0 ? p.delta[(size_t)h * p.L + q] : 0.f;
                }
                __syncwarp();
                constexpr int RP = 32 / CH;                    // rows per instruction
                const int c16 = lane % CH;
#pragma unroll 4
                for (int rb = 0; rb < 128; rb += RP) {
                    const int rr = rb + lane / CH, q = s_row[st][rr];
                    const size_t src = ((size_t)h * p.L + max(q, 0)) * D + c16 * 8;
                    const uint32_t dst = st * TILE_BYTES + (c16 >> 3) * SUB_BYTES + sw128_offset(rr, c16 & 7);
                    cp_async16(sY1 + dst, p.Q + src, q >= 0 ? 16u : 0u);
                    cp_async16(sY2 + dst, p.dO + src, q >= 0 ? 16u : 0u);
                }
                cp_async_wait_all();
                fence_proxy_async_smem();
                mbar_arrive(bar(Y_FULL + st));
            }
        }
    } else {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t IDESC_T = idesc_bf16_f32(128, 128, 0, 0);      // T = X Y^T, both K-major
            constexpr uint32_t IDESC_ACC = idesc_bf16_f32(128, D, 0, 1);      // ACC += (TMEM) Y, Y MN-major
            constexpr uint64_t STAGE = TILE_BYTES >> 4;
            const uint64_t x1 = smem_desc_sw128(sX, 16, 1024), x2 = smem_desc_sw128(sX + TILE_BYTES, 16, 1024);
            const uint64_t y1k = smem_desc_sw128(sY1, 16, 1024), y2k = smem_desc_sw128(sY2, 16, 1024);
            const uint64_t y1m = smem_desc_sw128(sY1, SUB_BYTES, 1024), y2m = smem_desc_sw128(sY2, SUB_BYTES, 1024);
            bool ok = mbar_wait(bar(X_FULL), 0, abort_flag, p.status, BW_XFULL);
            for (int jt = 0; ok && jt < n_tiles; ++jt) {
                const int st = jt & 1;
                const uint64_t so = st ? STAGE : 0;
                if (!(ok = mbar_wait(bar(Y_FULL + st), (jt >> 1) & 1, abort_flag, p.status, BW_YFULL))) break;
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t o = ((ks >> 2) * SUB_BYTES + (ks & 3) * 32) >> 4;
                    mma_ss(tmem, x1 + o, y1k + so + o, IDESC_T, ks > 0);
                }
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t o = ((ks >> 2) * SUB_BYTES + (ks & 3) * 32) >> 4;
                    mma_ss(tmem + 128, x2 + o, y2k + so + o, IDESC_T, ks > 0);
                }
                tc_commit(bar(T_FULL));
                if (!(ok = mbar_wait(bar(D_FULL), jt & 1, abort_flag, p.status, BW_DFULL))) break;
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) mma_ts(tmem + 256, tmem + 128 + ks * 8, y1m + so + ks * (2048 >> 4), IDESC_ACC, jt > 0 || ks > 0);
                if (MODE == DKV) {
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) mma_ts(tmem + 384, tmem + ks * 8, y2m + so + ks * (2048 >> 4), IDESC_ACC, jt > 0 || ks > 0);
                }
                tc_commit(bar(Y_EMPTY + st));
            }
            if (ok) tc_commit(bar(ACC_FULL));
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, 512);
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
    a.Q = Q; a.K = K; a.V = V; a.dO = dO; a.lse = lse; a.delta = delta; a.sel = sel;
    a.dQ = dQ; a.dK = dK; a.dV = dV;
    a.part = ws_ptr<__nv_bfloat16>(ws, p->ws.part_o);      // the forward's partial outputs are no longer needed
    a.ktiles = p->d_ktiles; a.off = p->d_off; a.ranc_off = p->d_ranc_off; a.ranc = p->d_ranc; a.cap_off = p->d_cap_off;
    a.cnt = ws_ptr<int>(ws, p->ws.cnt);
    a.qlist = ws_ptr<int32_t>(ws, p->ws.qlist);
    a.cap_total = (size_t)p->cap_off[p->C];
    a.status = ws_ptr<int>(ws, p->ws.status);
    a.H = p->H; a.L = p->L; a.C = p->C; a.k = p->k;
    a.scale = p->scale; a.scale_log2 = p->scale * kLog2e;
    const size_t smem = 6 * (size_t)128 * 128 * 2 + 1024;     // the d = 128 footprint: one CTA (512 TMEM columns) per SM
    static bool attr_done[2] = {false, false};
    if (!attr_done[D == 128]) {
        MOC_CUDA_TRY(cudaFuncSetAttribute(attend_bwd_tc_kernel<D, DQ_ROUTED>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        MOC_CUDA_TRY(cudaFuncSetAttribute(attend_bwd_tc_kernel<D, DQ_ANCHOR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        MOC_CUDA_TRY(cudaFuncSetAttribute(attend_bwd_tc_kernel<D, DKV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attr_done[D == 128] = true;
    }
    if (p->k > 0) {
        a.rng = p->d_chunk_rng;
        a.items = ws_ptr<WorkItem>(ws, p->ws.rtiles);
        a.n_items_dev = ws_ptr<int>(ws, p->ws.tile_off) + (size_t)p->H * p->C;
        const long long bound = (long long)p->H * (((long long)p->L * p->k + kQTileRows - 1) / kQTileRows + p->C);
        attend_bwd_tc_kernel<D, DQ_ROUTED><<<(unsigned)(2 * bound), kBwdThreads, smem, s>>>(tmK, tmV, a);
        MOC_LAUNCH_CHECK();
    }
    a.rng = p->d_anc_rng;
    a.items = p->d_qitems;
    a.n_items_dev = nullptr;
    attend_bwd_tc_kernel<D, DQ_ANCHOR><<<dim3((unsigned)(2 * p->qitems.size()), (unsigned)p->H), kBwdThreads, smem, s>>>(tmK, tmV, a);
    MOC_LAUNCH_CHECK();
    attend_bwd_tc_kernel<D, DKV><<<dim3((unsigned)p->ktiles.size(), (unsigned)p->H), kBwdThreads, smem, s>>>(tmK, tmV, a);
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
