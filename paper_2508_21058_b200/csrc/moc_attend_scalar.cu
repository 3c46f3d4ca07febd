// Plain fp32 CUDA-core attention (forward and backward) over the selected key tokens.
// One warp owns one query (or, for dK/dV, one key token); within a batch of 32 partners
// each lane takes one and computes its full dot products from a shared-memory copy of
// the owner's row; the weighted accumulation then runs with lanes across the head dim.
// These kernels read the selection straight from sel_idx and the plan's anchor tables
// (forward, dQ) or from the chunk -> query lists (dK, dV).  They serve configurations
// outside the tensor-core kernel's reach and as its in-library cross-check.
#include "moc_common.cuh"

namespace moc {

template <int D>
__device__ __forceinline__ float dot_row(const float *__restrict__ own, const __nv_bfloat16 *__restrict__ row) {
    float s = 0.f;
    const uint4 *r = reinterpret_cast<const uint4 *>(row);
#pragma unroll
    for (int x = 0; x < D / 8; ++x) {
        uint4 v = __ldg(r + x);
        const __nv_bfloat162 *b = reinterpret_cast<const __nv_bfloat162 *>(&v);
#pragma unroll
        for (int y = 0; y < 4; ++y) {
            float2 f = __bfloat1622float2(b[y]);
            s = fmaf(own[x * 8 + 2 * y], f.x, s);
            s = fmaf(own[x * 8 + 2 * y + 1], f.y, s);
        }
    }
    return s;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// lanes across the head dim: lane owns elements [lane*E, lane*E+E), E = D/32
template <int D>
__device__ __forceinline__ void load_lane_elems(const __nv_bfloat16 *row, int lane, float *out) {
    constexpr int E = D / 32;
    if (E == 4) {
        uint2 v = __ldg(reinterpret_cast<const uint2 *>(row) + lane);
        const __nv_bfloat162 *b = reinterpret_cast<const __nv_bfloat162 *>(&v);
        float2 a = __bfloat1622float2(b[0]), c = __bfloat1622float2(b[1]);
        out[0] = a.x; out[1] = a.y; out[2] = c.x; out[3] = c.y;
    } else {
        unsigned v = __ldg(reinterpret_cast<const unsigned *>(row) + lane);
        float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&v));
        out[0] = a.x; out[1] = a.y;
    }
}
template <int D>
__device__ __forceinline__ void store_lane_elems(__nv_bfloat16 *row, int lane, const float *in) {
    constexpr int E = D / 32;
    if (E == 4) {
        __nv_bfloat162 a = __floats2bfloat162_rn(in[0], in[1]), b = __floats2bfloat162_rn(in[2], in[3]);
        uint2 v;
        v.x = *reinterpret_cast<unsigned *>(&a);
        v.y = *reinterpret_cast<unsigned *>(&b);
        reinterpret_cast<uint2 *>(row)[lane] = v;
    } else {
        __nv_bfloat162 a = __floats2bfloat162_rn(in[0], in[1]);
        reinterpret_cast<unsigned *>(row)[lane] = *reinterpret_cast<unsigned *>(&a);
    }
}

// Key ranges of query i: its chunk's merged anchor ranges, then its routed picks.
struct RangeIter {
    const KeyRange *anc; int n_anc; const int32_t *sel; int k; const int32_t *off; int pos;
    __device__ bool next(int &t0, int &t1) {
        while (pos < n_anc + k) {
            if (pos < n_anc) { t0 = anc[pos].t0; t1 = anc[pos].t1; ++pos; return true; }
            int j = sel[pos - n_anc]; ++pos;
            if (j >= 0) { t0 = off[j]; t1 = off[j + 1]; return true; }
        }
        return false;
    }
};

template <int D>
__global__ void __launch_bounds__(128) attend_scalar_kernel(const __nv_bfloat16 *__restrict__ Q, const __nv_bfloat16 *__restrict__ K,
                                                             const __nv_bfloat16 *__restrict__ V, const int32_t *__restrict__ sel,
                                                             __nv_bfloat16 *__restrict__ O, float *__restrict__ lse,
                                                             const int32_t *__restrict__ off, const int32_t *__restrict__ tok_chunk,
                                                             const int32_t *__restrict__ anc_off, const KeyRange *__restrict__ anc_rng,
                                                             int H, int L, int k, float scale) {
    constexpr int E = D / 32;
    __shared__ float qs[4][D];
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const size_t row = (size_t)blockIdx.x * 4 + warp;
    if (row >= (size_t)H * L) return;
    const int h = (int)(row / L), i = (int)(row % L);
    const __nv_bfloat16 *q = Q + row * D;
    for (int x = lane; x < D; x += 32) qs[warp][x] = __bfloat162float(q[x]);
    __syncwarp();
    const int c = tok_chunk[i];
    RangeIter it{anc_rng + anc_off[c], anc_off[c + 1] - anc_off[c], sel + row * k, k, off, 0};
    const __nv_bfloat16 *Kh = K + (size_t)h * L * D, *Vh = V + (size_t)h * L * D;
    float m = -INFINITY, l = 0.f, o[E];
#pragma unroll
    for (int e = 0; e < E; ++e) o[e] = 0.f;
    int t0, t1;
    while (it.next(t0, t1)) {
        for (int tb = t0; tb < t1; tb += 32) {
            const int t = tb + lane;
            const float s = (t < t1) ? scale * dot_row<D>(qs[warp], Kh + (size_t)t * D) : -INFINITY;
            const float mn = fmaxf(m, warp_max(s));
            const float alpha = __expf(m - mn);
            const float pr = (t < t1) ? __expf(s - mn) : 0.f;
            l = l * alpha + warp_sum(pr);
#pragma unroll
            for (int e = 0; e < E; ++e) o[e] *= alpha;
            const int nb = min(32, t1 - tb);
            for (int u = 0; u < nb; ++u) {
                const float pu = __shfl_sync(0xffffffffu, pr, u);
                float v[E];
                load_lane_elems<D>(Vh + (size_t)(tb + u) * D, lane, v);
#pragma unroll
                for (int e = 0; e < E; ++e) o[e] = fmaf(pu, v[e], o[e]);
            }
            m = mn;
        }
    }
    const float inv = 1.f / l;
#pragma unroll
    for (int e = 0; e < E; ++e) o[e] *= inv;
    store_lane_elems<D>(O + row * D, lane, o);
    if (lane == 0) lse[row] = m + __logf(l);
}

// delta_i = sum_x dO_ix O_ix
template <int D>
__global__ void __launch_bounds__(128) delta_kernel(const __nv_bfloat16 *__restrict__ O, const __nv_bfloat16 *__restrict__ dO,
                                                     float *__restrict__ delta, size_t n_rows) {
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const size_t row = (size_t)blockIdx.x * 4 + warp;
    if (row >= n_rows) return;
    float a[D / 32], b[D / 32], s = 0.f;
    load_lane_elems<D>(O + row * D, lane, a);
    load_lane_elems<D>(dO + row * D, lane, b);
#pragma unroll
    for (int e = 0; e < D / 32; ++e) s = fmaf(a[e], b[e], s);
    s = warp_sum(s);
    if (lane == 0) delta[row] = s;
}

template <int D>
__global__ void __launch_bounds__(128) dq_scalar_kernel(const __nv_bfloat16 *__restrict__ Q, const __nv_bfloat16 *__restrict__ K,
                                                         const __nv_bfloat16 *__restrict__ V, const __nv_bfloat16 *__restrict__ dO,
                                                         const float *__restrict__ lse, const float *__restrict__ delta,
                                                         const int32_t *__restrict__ sel, __nv_bfloat16 *__restrict__ dQ,
                                                         const int32_t *__restrict__ off, const int32_t *__restrict__ tok_chunk,
                                                         const int32_t *__restrict__ anc_off, const KeyRange *__restrict__ anc_rng,
                                                         int H, int L, int k, float scale) {
    constexpr int E = D / 32;
    __shared__ float qs[4][D], gs[4][D];
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const size_t row = (size_t)blockIdx.x * 4 + warp;
    if (row >= (size_t)H * L) return;
    const int h = (int)(row / L), i = (int)(row % L);
    for (int x = lane; x < D; x += 32) {
        qs[warp][x] = __bfloat162float(Q[row * D + x]);
        gs[warp][x] = __bfloat162float(dO[row * D + x]);
    }
    __syncwarp();
    const int c = tok_chunk[i];
    RangeIter it{anc_rng + anc_off[c], anc_off[c + 1] - anc_off[c], sel + row * k, k, off, 0};
    const __nv_bfloat16 *Kh = K + (size_t)h * L * D, *Vh = V + (size_t)h * L * D;
    const float li = lse[row], di = delta[row];
    float acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;
    int t0, t1;
    while (it.next(t0, t1)) {
        for (int tb = t0; tb < t1; tb += 32) {
            const int t = tb + lane;
            float ds = 0.f;
            if (t < t1) {
                const float s = scale * dot_row<D>(qs[warp], Kh + (size_t)t * D);
                const float pr = __expf(s - li);
                const float dp = dot_row<D>(gs[warp], Vh + (size_t)t * D);
                ds = pr * (dp - di) * scale;
            }
            const int nb = min(32, t1 - tb);
            for (int u = 0; u < nb; ++u) {
                const float du = __shfl_sync(0xffffffffu, ds, u);
                float kk[E];
                load_lane_elems<D>(Kh + (size_t)(tb + u) * D, lane, kk);
#pragma unroll
                for (int e = 0; e < E; ++e) acc[e] = fmaf(du, kk[e], acc[e]);
            }
        }
    }
    store_lane_elems<D>(dQ + row * D, lane, acc);
}

// One warp per key token t of head h: sums over the queries whose selection holds chunk
// c(t): every query of the chunks that have c(t) as an anchor, then the routed list.
template <int D>
__global__ void __launch_bounds__(128) dkv_scalar_kernel(const __nv_bfloat16 *__restrict__ Q, const __nv_bfloat16 *__restrict__ K,
                                                          const __nv_bfloat16 *__restrict__ V, const __nv_bfloat16 *__restrict__ dO,
                                                          const float *__restrict__ lse, const float *__restrict__ delta,
                                                          __nv_bfloat16 *__restrict__ dK, __nv_bfloat16 *__restrict__ dV,
                                                          const int32_t *__restrict__ off, const int32_t *__restrict__ tok_chunk,
                                                          const int32_t *__restrict__ ranc_off, const int32_t *__restrict__ ranc,
                                                          const int *__restrict__ cnt, const int32_t *__restrict__ cap_off,
                                                          const int32_t *__restrict__ qlist, size_t cap_total,
                                                          int H, int L, int C, int k, float scale) {
    constexpr int E = D / 32;
    __shared__ float ks[4][D], vs[4][D];
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const size_t row = (size_t)blockIdx.x * 4 + warp;
    if (row >= (size_t)H * L) return;
    const int h = (int)(row / L), t = (int)(row % L);
    for (int x = lane; x < D; x += 32) {
        ks[warp][x] = __bfloat162float(K[row * D + x]);
        vs[warp][x] = __bfloat162float(V[row * D + x]);
    }
    __syncwarp();
    const int j = tok_chunk[t];
    const __nv_bfloat16 *Qh = Q + (size_t)h * L * D, *Gh = dO + (size_t)h * L * D;
    const float *lh = lse + (size_t)h * L, *dh = delta + (size_t)h * L;
    float ak[E], av[E];
#pragma unroll
    for (int e = 0; e < E; ++e) { ak[e] = 0.f; av[e] = 0.f; }
    const int n_ra = ranc_off[j + 1] - ranc_off[j];
    const int q0 = cap_off[j], q1 = q0 + cnt[h * C + j];
    const int32_t *list = qlist + (size_t)h * cap_total;
    // segments: n_ra query-chunk ranges, then the routed list
    for (int seg = 0; seg <= n_ra; ++seg) {
        int b0, b1;
        if (seg < n_ra) { const int c = ranc[ranc_off[j] + seg]; b0 = off[c]; b1 = off[c + 1]; }
        else { b0 = q0; b1 = q1; }
        for (int bb = b0; bb < b1; bb += 32) {
            const int e_ = bb + lane;
            int i = -1;
            if (e_ < b1) i = (seg < n_ra) ? e_ : list[e_] / k;
            float pr = 0.f, ds = 0.f;
            if (i >= 0) {
                const float s = scale * dot_row<D>(ks[warp], Qh + (size_t)i * D);
                pr = __expf(s - lh[i]);
                const float dp = dot_row<D>(vs[warp], Gh + (size_t)i * D);
                ds = pr * (dp - dh[i]) * scale;
            }
            const int nb = min(32, b1 - bb);
            for (int u = 0; u < nb; ++u) {
                const float pu = __shfl_sync(0xffffffffu, pr, u), du = __shfl_sync(0xffffffffu, ds, u);
                const int iu = __shfl_sync(0xffffffffu, i, u);
                float qq[E], gg[E];
                load_lane_elems<D>(Qh + (size_t)iu * D, lane, qq);
                load_lane_elems<D>(Gh + (size_t)iu * D, lane, gg);
#pragma unroll
                for (int e = 0; e < E; ++e) { ak[e] = fmaf(du, qq[e], ak[e]); av[e] = fmaf(pu, gg[e], av[e]); }
            }
        }
    }
    store_lane_elems<D>(dK + row * D, lane, ak);
    store_lane_elems<D>(dV + row * D, lane, av);
}

template <int D>
static int attend_scalar_d(const moc_plan *p, const __nv_bfloat16 *Q, const __nv_bfloat16 *K, const __nv_bfloat16 *V,
                           const int32_t *sel, __nv_bfloat16 *O, float *lse, cudaStream_t s) {
    const size_t rows = (size_t)p->H * p->L;
    attend_scalar_kernel<D><<<(unsigned)((rows + 3) / 4), 128, 0, s>>>(Q, K, V, sel, O, lse, p->d_off, p->d_tok_chunk,
                                                                      p->d_anc_off, p->d_anc_rng, p->H, p->L, p->k, p->scale);
    MOC_LAUNCH_CHECK();
    return MOC_OK;
}

int launch_attend_scalar(const moc_plan *p, const __nv_bfloat16 *Q, const __nv_bfloat16 *K, const __nv_bfloat16 *V,
                         const int32_t *sel, __nv_bfloat16 *O, float *lse, void *, cudaStream_t s) {
    return p->d == 128 ? attend_scalar_d<128>(p, Q, K, V, sel, O, lse, s) : attend_scalar_d<64>(p, Q, K, V, sel, O, lse, s);
}

template <int D>
static int attend_bwd_scalar_d(const moc_plan *p, const __nv_bfloat16 *Q, const __nv_bfloat16 *K, const __nv_bfloat16 *V,
                               const __nv_bfloat16 *O, const float *lse, const __nv_bfloat16 *dO, const int32_t *sel,
                               __nv_bfloat16 *dQ, __nv_bfloat16 *dK, __nv_bfloat16 *dV, void *ws, cudaStream_t s) {
    const size_t rows = (size_t)p->H * p->L;
    const unsigned grid = (unsigned)((rows + 3) / 4);
    float *delta = ws_ptr<float>(ws, p->ws.delta);
    delta_kernel<D><<<grid, 128, 0, s>>>(O, dO, delta, rows);
    MOC_LAUNCH_CHECK();
    dq_scalar_kernel<D><<<grid, 128, 0, s>>>(Q, K, V, dO, lse, delta, sel, dQ, p->d_off, p->d_tok_chunk, p->d_anc_off,
                                             p->d_anc_rng, p->H, p->L, p->k, p->scale);
    MOC_LAUNCH_CHECK();
    dkv_scalar_kernel<D><<<grid, 128, 0, s>>>(Q, K, V, dO, lse, delta, dK, dV, p->d_off, p->d_tok_chunk, p->d_ranc_off,
                                              p->d_ranc, ws_ptr<int>(ws, p->ws.cnt), p->d_cap_off, ws_ptr<int32_t>(ws, p->ws.qlist),
                                              (size_t)p->cap_off[p->C],
                                              p->H, p->L, p->C, p->k, p->scale);
    MOC_LAUNCH_CHECK();
    return MOC_OK;
}

int launch_delta(const moc_plan *p, const __nv_bfloat16 *O, const __nv_bfloat16 *dO, float *delta, cudaStream_t s) {
    const size_t rows = (size_t)p->H * p->L;
    const unsigned grid = (unsigned)((rows + 3) / 4);
    if (p->d == 128) delta_kernel<128><<<grid, 128, 0, s>>>(O, dO, delta, rows);
    else delta_kernel<64><<<grid, 128, 0, s>>>(O, dO, delta, rows);
    MOC_LAUNCH_CHECK();
    return MOC_OK;
}

int launch_attend_bwd_scalar(const moc_plan *p, const __nv_bfloat16 *Q, const __nv_bfloat16 *K, const __nv_bfloat16 *V,
                             const __nv_bfloat16 *O, const float *lse, const __nv_bfloat16 *dO, const int32_t *sel,
                             __nv_bfloat16 *dQ, __nv_bfloat16 *dK, __nv_bfloat16 *dV, void *ws, cudaStream_t s) {
    return p->d == 128 ? attend_bwd_scalar_d<128>(p, Q, K, V, O, lse, dO, sel, dQ, dK, dV, ws, s)
                       : attend_bwd_scalar_d<64>(p, Q, K, V, O, lse, dO, sel, dQ, dK, dV, ws, s);
}

}  // namespace moc
