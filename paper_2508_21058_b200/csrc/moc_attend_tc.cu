// Tensor-core sparse attention forward (tcgen05 MMA, TMEM accumulators, TMA-fed K/V).
//
// Two passes share one kernel:
//   routed pass (key-chunk stationary): work item = (head, chunk c, 128 entries of the list
//     of (query, slot) pairs that picked c).  The Q rows are gathered into shared memory,
//     the keys are exactly the tokens of chunk c, and each (query, slot) gets a partial
//     result (normalised output + log-sum-exp) in the workspace.
//   anchor pass (query-tile stationary): work item = (head, 128 consecutive rows of one
//     chunk); keys are the chunk's mandatory anchors (merged token ranges).  Its epilogue
//     merges the row's <= k routed partials by log-sum-exp and writes O and LSE.
//
// One CTA = 6 warps, two CTAs per SM so that one CTA's softmax overlaps the other's MMAs:
//   warps 0-3  one query row per thread (TMEM lane = row): load/gather Q into the
//              swizzled shared tile, online softmax straight from TMEM, P written back to
//              TMEM as packed bf16 (aliasing S), lazy rescale of O, epilogue;
//   warp 4     TMA producer: K and V tiles (128 keys) with 128-byte swizzle;
//   warp 5     one thread issues S = Q K^T (operands in shared memory) and O += P V
//              (P from TMEM, V as an MN-major shared-memory operand), accumulators in TMEM.
// Every mbarrier wait is bounded; a wait that runs out flags the workspace status word
// and the CTA drains and leaves.
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
    const int32_t *off;
    const int32_t *anc_off;
    const KeyRange *anc_rng;
    const QTile *qtiles;
    const int *gtile_off;   // [H*C + 1] running count of routed tiles over (head, chunk)
    const int *qoff;        // [H][C + 1]
    const int32_t *qlist;   // [H][L * k]
    int *status;
    int H, L, C, k;
    float scale_log2;       // softmax scale * log2(e)
};

constexpr int kBN = 128;               // keys per tile
constexpr int kThreads = 192;
constexpr int kTmemCols = 256;         // S/P: columns [0,128), O: [128, 128 + D)
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.0f;   // log2 units: O is rescaled only when the row max grows by more

enum WaitCode { W_QFULL = 1, W_KFULL, W_VFULL, W_SFULL, W_PFULL, W_PVDONE, W_KEMPTY, W_VEMPTY, W_EPILOGUE };

struct TileIter {
    const KeyRange *rng;
    int n, ri, t;
    __device__ TileIter(const KeyRange *r, int n_) : rng(r), n(n_), ri(0), t(n_ > 0 ? r[0].t0 : 0) {}
    __device__ bool next(int &t0, int &valid) {
        if (ri >= n) return false;
        const int end = rng[ri].t1;
        t0 = t;
        valid = min(kBN, end - t);
        t += kBN;
        if (t >= end) { ++ri; if (ri < n) t = rng[ri].t0; }
        return true;
    }
};

template <int D, bool ROUTED>
__global__ void __launch_bounds__(kThreads, 2) attend_tc_kernel(const __grid_constant__ CUtensorMap tmK,
                                                                const __grid_constant__ CUtensorMap tmV,
                                                                const AttendParams p) {
    constexpr int TILE_BYTES = 128 * D * 2;
    constexpr int SUB = D / 64;            // 64-column (128-byte) sub-tiles per row
    constexpr int SUB_BYTES = 128 * 128;   // one sub-tile: 128 rows of 128 bytes
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[6];
    __shared__ uint32_t tmem_slot;
    __shared__ int s_abort;
    __shared__ int w_valid, w_h, w_rows, w_first, w_nrng, w_ntiles;
    __shared__ KeyRange w_rng0;
    __shared__ const KeyRange *w_rng;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gbase = smem_raw + (sbase - smem_u32(smem_raw));
    const uint32_t sQ = sbase, sK = sbase + TILE_BYTES, sV = sbase + 2 * TILE_BYTES;
    const uint32_t q_full = smem_u32(&bars[0]), k_full = smem_u32(&bars[1]), v_full = smem_u32(&bars[2]),
                   s_full = smem_u32(&bars[3]), p_full = smem_u32(&bars[4]), pv_done = smem_u32(&bars[5]);

    if (threadIdx.x == 0) {
        s_abort = 0;
        int valid = (*(volatile int *)p.status == 0);
        if (ROUTED) {
            const int HC = p.H * p.C;
            const int tile = blockIdx.x;
            if (tile >= p.gtile_off[HC]) valid = 0;
            if (valid) {
                int lo = 0, hi = HC;   // largest hc with gtile_off[hc] <= tile
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (p.gtile_off[mid] <= tile) lo = mid; else hi = mid;
                }
                const int h = lo / p.C, c = lo % p.C;
                const int nth = tile - p.gtile_off[lo];
                const int e0 = p.qoff[h * (p.C + 1) + c] + nth * kQTileRows;
                w_h = h;
                w_first = e0;
                w_rows = min(kQTileRows, p.qoff[h * (p.C + 1) + c + 1] - e0);
                w_rng0 = KeyRange{p.off[c], p.off[c + 1]};
                w_rng = &w_rng0;
                w_nrng = 1;
                w_ntiles = (p.off[c + 1] - p.off[c] + kBN - 1) / kBN;
            }
        } else {
            const QTile qt = p.qtiles[blockIdx.x];
            w_h = blockIdx.y;
            w_first = qt.row0;
            w_rows = qt.rows;
            w_rng = p.anc_rng + p.anc_off[qt.chunk];
            w_nrng = p.anc_off[qt.chunk + 1] - p.anc_off[qt.chunk];
            int nt = 0;
            for (int r = 0; r < w_nrng; ++r) nt += (w_rng[r].t1 - w_rng[r].t0 + kBN - 1) / kBN;
            w_ntiles = nt;
        }
        w_valid = valid;
        mbar_init(q_full, 128);
        mbar_init(k_full, 1);
        mbar_init(v_full, 1);
        mbar_init(s_full, 1);
        mbar_init(p_full, 128);
        mbar_init(pv_done, 1);
        fence_barrier_init();
    }
    __syncthreads();
    if (!w_valid) return;
    if (warp == 4) {
        tmem_alloc(smem_u32(&tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    const uint32_t tmem = tmem_slot;
    const uint32_t tS = tmem, tP = tmem, tO = tmem + 128;
    const int h = w_h, rows = w_rows, first = w_first, n_tiles = w_ntiles;
    volatile int *abort_flag = &s_abort;

    if (warp < 4) {
        // ------------------------------------------------------------ softmax / epilogue threads
        const int r = threadIdx.x;
        const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
        int qi = -1, slot = 0;
        if (r < rows) {
            if (ROUTED) {
                const int e = p.qlist[(size_t)h * p.L * p.k + first + r];
                qi = e / p.k;
                slot = e - qi * p.k;
            } else {
                qi = first + r;
            }
        }
        {
            const uint4 *src = reinterpret_cast<const uint4 *>(p.Q + ((size_t)h * p.L + (qi >= 0 ? qi : 0)) * D);
#pragma unroll
            for (int c16 = 0; c16 < D / 8; ++c16) {
                uint4 v = make_uint4(0, 0, 0, 0);
                if (qi >= 0) v = __ldg(src + c16);
                *reinterpret_cast<uint4 *>(gbase + (c16 >> 3) * SUB_BYTES + sw128_offset(r, c16 & 7)) = v;
            }
        }
        fence_proxy_async_smem();
        mbar_arrive(q_full);

        float m_run = -INFINITY, l_run = 0.f;
        const float c = p.scale_log2;
        TileIter it(w_rng, w_nrng);
        int t0, valid, jt = 0;
        bool ok = true;
        while (it.next(t0, valid)) {
            const uint32_t par = jt & 1;
            ok = mbar_wait(s_full, par, abort_flag, p.status, W_SFULL);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            uint32_t v[32];
            // pass 1: row maximum over the valid columns
            float mx = -INFINITY;
#pragma unroll 1
            for (int ch = 0; ch * 32 < valid; ++ch) {
                tmem_ld32(tS + lane_off + ch * 32, v);
                tmem_wait_ld();
#pragma unroll
                for (int x = 0; x < 32; ++x) {
                    const float s = __uint_as_float(v[x]);
                    mx = fmaxf(mx, (ch * 32 + x < valid) ? s : -INFINITY);
                }
            }
            const float m_new = fmaxf(m_run, mx * c);
            float alpha = 1.f;
            if (jt == 0) {
                m_run = m_new;
            } else if (m_new - m_run > kRescaleThreshold) {
                alpha = exp2f(m_run - m_new);
                m_run = m_new;
            }
            if (__any_sync(0xffffffffu, alpha != 1.f)) {
                // PV of the previous tile has completed (its commit precedes this tile's S)
#pragma unroll 1
                for (int ch = 0; ch < D / 32; ++ch) {
                    tmem_ld32(tO + lane_off + ch * 32, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int x = 0; x < 32; ++x) v[x] = __float_as_uint(__uint_as_float(v[x]) * alpha);
                    tmem_st32(tO + lane_off + ch * 32, v);
                }
            }
            l_run *= alpha;
            // pass 2: P = exp2(s * c - m), packed bf16 into the P columns (aliasing S)
            const float neg_m = -m_run;
            float lsum = 0.f;
#pragma unroll 1
            for (int ch = 0; ch * 32 < valid; ++ch) {
                tmem_ld32(tS + lane_off + ch * 32, v);
                tmem_wait_ld();
                uint32_t u[16];
#pragma unroll
                for (int x = 0; x < 16; ++x) {
                    const int col = ch * 32 + 2 * x;
                    const float p0 = (col < valid) ? exp2f(fmaf(__uint_as_float(v[2 * x]), c, neg_m)) : 0.f;
                    const float p1 = (col + 1 < valid) ? exp2f(fmaf(__uint_as_float(v[2 * x + 1]), c, neg_m)) : 0.f;
                    lsum += p0 + p1;
                    __nv_bfloat162 b = __floats2bfloat162_rn(p0, p1);
                    u[x] = *reinterpret_cast<uint32_t *>(&b);
                }
                tmem_st16(tP + lane_off + ch * 16, u);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(p_full);
            l_run += lsum;
            ++jt;
        }
        // ---- epilogue
        if (ok) {
            ok = mbar_wait(pv_done, (uint32_t)((n_tiles - 1) & 1), abort_flag, p.status, W_EPILOGUE);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            tc_fence_after();
            const float inv_l = 1.f / l_run;
            const float lse_own = (m_run + log2f(l_run)) * kLn2;
            float w_own = inv_l, big = lse_own, wsum = 1.f;
            const float *pl = nullptr;
            const __nv_bfloat16 *po = nullptr;
            if (!ROUTED && qi >= 0 && p.k > 0) {
                pl = p.part_lse + ((size_t)h * p.L + qi) * p.k;
                po = p.part_o + ((size_t)h * p.L + qi) * p.k * D;
                for (int s = 0; s < p.k; ++s) big = fmaxf(big, pl[s]);
                wsum = __expf(lse_own - big);
                for (int s = 0; s < p.k; ++s) wsum += __expf(pl[s] - big);
                w_own = __expf(lse_own - big) / wsum * inv_l;
            }
            uint32_t v[32];
#pragma unroll 1
            for (int ch = 0; ch < D / 32; ++ch) {
                __syncwarp();
                tmem_ld32(tO + lane_off + ch * 32, v);
                tmem_wait_ld();
                float acc[32];
#pragma unroll
                for (int x = 0; x < 32; ++x) acc[x] = __uint_as_float(v[x]) * w_own;
                if (pl) {
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
                __nv_bfloat16 *dst = ROUTED ? p.part_o + (((size_t)h * p.L + qi) * p.k + slot) * D + ch * 32
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
    } else if (warp == 4) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tensormap(&tmK);
            prefetch_tensormap(&tmV);
            TileIter it(w_rng, w_nrng);
            int t0, valid, jt = 0;
            int k_last = -1, v_last = -1;   // last tile whose K / V copy was issued
            while (it.next(t0, valid)) {
                if (jt > 0 && !mbar_wait(s_full, (jt - 1) & 1, abort_flag, p.status, W_KEMPTY)) break;
                mbar_expect_tx(k_full, TILE_BYTES);
#pragma unroll
                for (int sub = 0; sub < SUB; ++sub) tma_load_2d(sK + sub * SUB_BYTES, &tmK, sub * 64, h * p.L + t0, k_full);
                k_last = jt;
                if (jt > 0 && !mbar_wait(pv_done, (jt - 1) & 1, abort_flag, p.status, W_VEMPTY)) break;
                mbar_expect_tx(v_full, TILE_BYTES);
#pragma unroll
                for (int sub = 0; sub < SUB; ++sub) tma_load_2d(sV + sub * SUB_BYTES, &tmV, sub * 64, h * p.L + t0, v_full);
                v_last = jt;
                ++jt;
            }
            if (*abort_flag) {
                // drain: copies already issued must land before the CTA's shared memory is released
                int dummy_flag = 0;
                if (k_last >= 0) mbar_wait(k_full, (uint32_t)(k_last & 1), &dummy_flag, p.status, W_KFULL);
                if (v_last >= 0) mbar_wait(v_full, (uint32_t)(v_last & 1), &dummy_flag, p.status, W_VFULL);
            }
        }
    } else {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t IDESC_PV = idesc_bf16_f32(128, D, 0, 1);
            bool ok = mbar_wait(q_full, 0, abort_flag, p.status, W_QFULL);
            TileIter it(w_rng, w_nrng);
            int t0, valid, jt = 0;
            while (ok && it.next(t0, valid)) {
                const uint32_t par = jt & 1;
                if (!mbar_wait(k_full, par, abort_flag, p.status, W_KFULL)) break;
                // S and P share columns: the previous tile's PV must have consumed P
                if (jt > 0 && !mbar_wait(pv_done, par ^ 1, abort_flag, p.status, W_PVDONE)) break;
                tc_fence_after();
                const int n_qk = max(16, (valid + 15) & ~15);
                const uint32_t idesc_qk = idesc_bf16_f32(128, n_qk, 0, 0);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t o = (ks >> 2) * SUB_BYTES + (ks & 3) * 32;
                    mma_ss(tS, smem_desc_sw128(sQ + o, 16, 1024), smem_desc_sw128(sK + o, 16, 1024), idesc_qk, ks > 0);
                }
                tc_commit(s_full);
                if (!mbar_wait(p_full, par, abort_flag, p.status, W_PFULL)) break;
                if (!mbar_wait(v_full, par, abort_flag, p.status, W_VFULL)) break;
                tc_fence_after();
                const int steps = (valid + 15) >> 4;
                for (int ks = 0; ks < steps; ++ks)
                    mma_ts(tO, tP + ks * 8, smem_desc_sw128(sV + ks * 2048, SUB_BYTES, 1024), IDESC_PV, (jt > 0 || ks > 0));
                tc_commit(pv_done);
                ++jt;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, kTmemCols);
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
    a.off = p->d_off; a.anc_off = p->d_anc_off; a.anc_rng = p->d_anc_rng; a.qtiles = p->d_qtiles;
    a.gtile_off = ws_ptr<int>(ws, p->ws.tile_off);
    a.qoff = ws_ptr<int>(ws, p->ws.qoff);
    a.qlist = ws_ptr<int32_t>(ws, p->ws.qlist);
    a.status = ws_ptr<int>(ws, p->ws.status);
    a.H = p->H; a.L = p->L; a.C = p->C; a.k = p->k;
    a.scale_log2 = p->scale * 1.4426950408889634f;
    const size_t smem = 3 * (size_t)128 * D * 2 + 1024;
    static bool attr_done[2] = {false, false};
    if (!attr_done[D == 128]) {
        MOC_CUDA_TRY(cudaFuncSetAttribute(attend_tc_kernel<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        MOC_CUDA_TRY(cudaFuncSetAttribute(attend_tc_kernel<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attr_done[D == 128] = true;
    }
    if (p->k > 0) {
        const long long bound = (long long)p->H * (((long long)p->L * p->k + kQTileRows - 1) / kQTileRows + p->C);
        attend_tc_kernel<D, true><<<(unsigned)bound, kThreads, smem, s>>>(tmK, tmV, a);
        MOC_LAUNCH_CHECK();
    }
    dim3 grid((unsigned)p->qtiles.size(), (unsigned)p->H);
    attend_tc_kernel<D, false><<<grid, kThreads, smem, s>>>(tmK, tmV, a);
    MOC_LAUNCH_CHECK();
    return MOC_OK;
}

int launch_attend_tc(const moc_plan *p, const __nv_bfloat16 *Q, const __nv_bfloat16 *K, const __nv_bfloat16 *V,
                     const int32_t *, __nv_bfloat16 *O, float *lse, void *ws, cudaStream_t s) {
    return p->d == 128 ? attend_tc_d<128>(p, Q, K, V, O, lse, ws, s) : attend_tc_d<64>(p, Q, K, V, O, lse, ws, s);
}

}  // namespace moc
