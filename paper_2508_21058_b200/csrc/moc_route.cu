// Routing: scores of every query against every chunk descriptor, causal chunk mask,
// anchors removed from the candidates, top-k per query (ties to the lower chunk index),
// and the inverse index (per head and chunk, the list of (query, slot) pairs that
// picked it) which the key-stationary attention pass consumes.
//
// route_kernel: one query per thread, 128 queries per block.  The Q tile is staged in
// shared memory with coalesced 128-bit loads; descriptors are visited in blocks of 32
// chunks held in shared memory as fp32 and read as warp-wide broadcasts; each thread
// keeps 32 fp32 accumulators and folds them into its running sorted top-k list.
#include <float.h>

#include "moc_common.cuh"

namespace moc {

constexpr int kRouteRows = 128;
constexpr int kRouteCB = 32;   // chunks per descriptor block (= bits of one anchor word)

template <int KMAX>
struct TopK {
    float s[KMAX];
    int j[KMAX];
    __device__ __forceinline__ void init() {
#pragma unroll(KMAX <= 8 ? KMAX : 1)
        for (int x = 0; x < KMAX; ++x) { s[x] = -INFINITY; j[x] = -1; }
    }
    // candidates arrive in ascending chunk index, so strict '>' keeps equal scores in index order
    __device__ __forceinline__ void push(float v, int idx, int k) {
        if (KMAX <= 8) {
            if (!(v > s[KMAX - 1])) return;
#pragma unroll
            for (int x = KMAX - 1; x >= 0; --x) {
                bool shift = (x > 0) && (v > s[x > 0 ? x - 1 : 0]);
                bool place = (v > s[x]) && !shift;
                float ns = shift ? s[x > 0 ? x - 1 : 0] : (place ? v : s[x]);
                int nj = shift ? j[x > 0 ? x - 1 : 0] : (place ? idx : j[x]);
                s[x] = ns; j[x] = nj;
            }
        } else {
            if (!(v > s[k - 1])) return;
            int x = k - 1;
            while (x > 0 && v > s[x - 1]) { s[x] = s[x - 1]; j[x] = j[x - 1]; --x; }
            s[x] = v; j[x] = idx;
        }
    }
};

template <int D, int KMAX>
__global__ void __launch_bounds__(kRouteRows) route_kernel(const __nv_bfloat16 *__restrict__ Q,
                                                            const float *__restrict__ desc, int32_t *__restrict__ sel,
                                                            int *__restrict__ cnt, float *__restrict__ part_lse,
                                                            const int32_t *__restrict__ tok_chunk,
                                                            const uint32_t *__restrict__ anc_bits, int words, int L,
                                                            int C, int k, int causal) {
    constexpr int QS = D + 8;   // padded row stride (bf16 elements): conflict-free 16-byte row reads
    extern __shared__ __align__(16) unsigned char smem[];
    __nv_bfloat16 *qs = reinterpret_cast<__nv_bfloat16 *>(smem);
    float *ds = reinterpret_cast<float *>(smem + sizeof(__nv_bfloat16) * kRouteRows * QS);
    int *hist = reinterpret_cast<int *>(ds + kRouteCB * D);
    const int h = blockIdx.y, r0 = blockIdx.x * kRouteRows;
    const int rows = min(kRouteRows, L - r0);
    const int tid = threadIdx.x;
    // stage the Q tile
    {
        constexpr int LANES = D / 8;
        const uint4 *src = reinterpret_cast<const uint4 *>(Q + ((size_t)h * L + r0) * D);
        for (int e = tid; e < rows * LANES; e += kRouteRows) {
            int r = e / LANES, l = e % LANES;
            *reinterpret_cast<uint4 *>(qs + r * QS + l * 8) = __ldg(src + e);
        }
    }
    for (int x = tid; x < C; x += kRouteRows) hist[x] = 0;
    const int i = r0 + tid;
    const bool live = tid < rows;
    const int ci = live ? tok_chunk[i] : 0;
    const int c_hi = causal ? tok_chunk[r0 + rows - 1] : C;   // exclusive bound on useful chunks for this tile
    TopK<KMAX> top;
    top.init();
    for (int jb = 0; jb < c_hi; jb += kRouteCB) {
        __syncthreads();
        const int nb = min(kRouteCB, C - jb);
        {
            const float4 *src = reinterpret_cast<const float4 *>(desc + ((size_t)h * C + jb) * D);
            for (int e = tid; e < nb * D / 4; e += kRouteRows) reinterpret_cast<float4 *>(ds)[e] = __ldg(src + e);
        }
        __syncthreads();
        float acc[kRouteCB];
#pragma unroll
        for (int c = 0; c < kRouteCB; ++c) acc[c] = 0.f;
#pragma unroll 1
        for (int x0 = 0; x0 < D; x0 += 8) {
            float q[8];
            {
                uint4 v = *reinterpret_cast<const uint4 *>(qs + tid * QS + x0);
                const __nv_bfloat162 *b = reinterpret_cast<const __nv_bfloat162 *>(&v);
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    float2 f = __bfloat1622float2(b[x]);
                    q[2 * x] = f.x; q[2 * x + 1] = f.y;
                }
            }
#pragma unroll
            for (int c = 0; c < kRouteCB; ++c) {
                float4 a = *reinterpret_cast<const float4 *>(ds + c * D + x0);
                float4 b = *reinterpret_cast<const float4 *>(ds + c * D + x0 + 4);
                acc[c] = fmaf(q[0], a.x, acc[c]); acc[c] = fmaf(q[1], a.y, acc[c]);
                acc[c] = fmaf(q[2], a.z, acc[c]); acc[c] = fmaf(q[3], a.w, acc[c]);
                acc[c] = fmaf(q[4], b.x, acc[c]); acc[c] = fmaf(q[5], b.y, acc[c]);
                acc[c] = fmaf(q[6], b.z, acc[c]); acc[c] = fmaf(q[7], b.w, acc[c]);
            }
        }
        if (live) {
            const uint32_t aw = anc_bits[(size_t)ci * words + jb / 32];
#pragma unroll
            for (int c = 0; c < kRouteCB; ++c) {
                const int j = jb + c;
                const bool cand = (c < nb) && !((aw >> c) & 1u) && (!causal || j < ci);
                if (cand) top.push(acc[c], j, k);
            }
        }
    }
    __syncthreads();
    if (live) {
        int32_t *out = sel + ((size_t)h * L + i) * k;
        float *pl = part_lse + ((size_t)h * L + i) * k;   // empty slots never get a routed partial
        if (KMAX <= 8) {
#pragma unroll
            for (int x = 0; x < (KMAX <= 8 ? KMAX : 1); ++x) {
                if (x < k) {
                    out[x] = top.j[x];
                    if (top.j[x] >= 0) atomicAdd(&hist[top.j[x]], 1);
                    else pl[x] = -INFINITY;
                }
            }
        } else {
            for (int x = 0; x < k; ++x) {
                const int j = top.j[x];
                out[x] = j;
                if (j >= 0) atomicAdd(&hist[j], 1);
                else pl[x] = -INFINITY;
            }
        }
    }
    __syncthreads();
    for (int x = tid; x < C; x += kRouteRows)
        if (hist[x]) atomicAdd(&cnt[h * C + x], hist[x]);
}

// Running totals over the H*C (head, chunk) pairs in one block: gcnt[i] = picks before pair i,
// gtile[i] = 128-row tiles before pair i (both with a final total entry), cursors zeroed;
// then qoff[h][c] = picks of head h before chunk c.  Flags the workspace as routed.
__global__ void __launch_bounds__(1024) route_scan_kernel(const int *__restrict__ cnt, int *__restrict__ gcnt,
                                                          int *__restrict__ gtile, int *__restrict__ qoff,
                                                          int *__restrict__ cursor, int *__restrict__ status, int H, int C) {
    __shared__ int sc[1024], st[1024];
    const int HC = H * C, t = threadIdx.x;
    const int per = (HC + 1023) / 1024;
    const int i0 = min(t * per, HC), i1 = min(i0 + per, HC);
    int a = 0, b = 0;
    for (int i = i0; i < i1; ++i) { a += cnt[i]; b += (cnt[i] + kQTileRows - 1) / kQTileRows; }
    sc[t] = a; st[t] = b;
    __syncthreads();
    for (int o = 1; o < 1024; o <<= 1) {   // inclusive scan
        int xa = 0, xb = 0;
        if (t >= o) { xa = sc[t - o]; xb = st[t - o]; }
        __syncthreads();
        sc[t] += xa; st[t] += xb;
        __syncthreads();
    }
    int ea = sc[t] - a, eb = st[t] - b;    // exclusive
    for (int i = i0; i < i1; ++i) {
        gcnt[i] = ea; gtile[i] = eb; cursor[i] = 0;
        ea += cnt[i]; eb += (cnt[i] + kQTileRows - 1) / kQTileRows;
    }
    if (t == 1023) { gcnt[HC] = sc[1023]; gtile[HC] = st[1023]; status[2] = 1; }
    __syncthreads();
    for (int idx = t; idx < H * (C + 1); idx += 1024) {
        const int h = idx / (C + 1), c = idx % (C + 1);
        qoff[idx] = gcnt[h * C + c] - gcnt[h * C];
    }
}

__global__ void route_scatter_kernel(const int32_t *__restrict__ sel, const int *__restrict__ qoff,
                                     int *__restrict__ cursor, int32_t *__restrict__ qlist, int L, int C, int k) {
    const int h = blockIdx.y;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= L) return;
    const int32_t *row = sel + ((size_t)h * L + i) * k;
    int32_t *list = qlist + (size_t)h * L * k;
    for (int s = 0; s < k; ++s) {
        const int j = row[s];
        if (j < 0) continue;
        const int pos = atomicAdd(&cursor[h * C + j], 1);
        list[qoff[h * (C + 1) + j] + pos] = i * k + s;
    }
}

__global__ void zero_i32_kernel2(int *p, size_t n) {
    size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    if (i < n) p[i] = 0;
}

template <int D>
static int launch_route_d(const moc_plan *p, const __nv_bfloat16 *Q, const float *desc, int32_t *sel, void *ws,
                          cudaStream_t s) {
    int *cnt = ws_ptr<int>(ws, p->ws.cnt);
    int *status = ws_ptr<int>(ws, p->ws.status);
    const size_t n = (size_t)p->H * p->C;
    zero_i32_kernel2<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(cnt, n);
    MOC_LAUNCH_CHECK();
    zero_i32_kernel2<<<1, kStatusWords, 0, s>>>(status, kStatusWords);
    MOC_LAUNCH_CHECK();
    if (p->k > 0) {
        const size_t smem = sizeof(__nv_bfloat16) * kRouteRows * (D + 8) + sizeof(float) * kRouteCB * D + sizeof(int) * p->C;
        dim3 grid((unsigned)((p->L + kRouteRows - 1) / kRouteRows), (unsigned)p->H);
        const int causal = (p->flags & MOC_FLAG_CAUSAL) ? 1 : 0;
#define MOC_ROUTE_CASE(KM)                                                                                          \
    do {                                                                                                            \
        MOC_CUDA_TRY(cudaFuncSetAttribute(route_kernel<D, KM>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
        route_kernel<D, KM><<<grid, kRouteRows, smem, s>>>(Q, desc, sel, cnt, ws_ptr<float>(ws, p->ws.part_lse), p->d_tok_chunk, p->d_anc_bits, p->words, \
                                                           p->L, p->C, p->k, causal);                               \
    } while (0)
        if (p->k <= 8) MOC_ROUTE_CASE(8);
        else if (p->k <= 64) MOC_ROUTE_CASE(64);
        else MOC_ROUTE_CASE(512);
#undef MOC_ROUTE_CASE
        MOC_LAUNCH_CHECK();
    }
    route_scan_kernel<<<1, 1024, 0, s>>>(cnt, ws_ptr<int>(ws, p->ws.gcnt), ws_ptr<int>(ws, p->ws.tile_off),
                                         ws_ptr<int>(ws, p->ws.qoff), ws_ptr<int>(ws, p->ws.cursor), status, p->H, p->C);
    MOC_LAUNCH_CHECK();
    if (p->k > 0) {
        dim3 grid((unsigned)((p->L + 255) / 256), (unsigned)p->H);
        route_scatter_kernel<<<grid, 256, 0, s>>>(sel, ws_ptr<int>(ws, p->ws.qoff), ws_ptr<int>(ws, p->ws.cursor),
                                                  ws_ptr<int32_t>(ws, p->ws.qlist), p->L, p->C, p->k);
        MOC_LAUNCH_CHECK();
    }
    return MOC_OK;
}

int launch_route(const moc_plan *p, const __nv_bfloat16 *Q, const float *desc, int32_t *sel, void *ws, cudaStream_t s) {
    return p->d == 128 ? launch_route_d<128>(p, Q, desc, sel, ws, s) : launch_route_d<64>(p, Q, desc, sel, ws, s);
}

}  // namespace moc
