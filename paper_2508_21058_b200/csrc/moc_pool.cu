// Chunk descriptors: desc[h][c][:] = mean of K[h][t][:] over the chunk's tokens.
//
// HBM-bound stream of K.  A work unit is (head, chunk, slice of kPoolSlice tokens); a
// block of 256 threads reads its slice with 128-bit loads (a token row of d bf16 is
// d/8 lanes wide, so one pass covers 256*8/d rows and every warp reads whole 128-byte
// lines), accumulates in fp32 registers, folds the row groups through shared memory
// and writes one partial sum.  The last block to finish a chunk (arrival counter)
// adds the partials in slice order and scales by 1/n, so the result does not depend
// on block scheduling.
// With few (head, chunk) pairs and no long chunk one block takes a whole chunk
// (chunk_pool_direct_kernel): no partial sums and no counters.
#include <mutex>

#include "moc_common.cuh"

namespace moc {

template <int D>
__global__ void __launch_bounds__(256) chunk_pool_kernel(const __nv_bfloat16 *__restrict__ K, float *__restrict__ desc,
                                                          float *__restrict__ part, int *__restrict__ done,
                                                          const int32_t *__restrict__ off,
                                                          const int32_t *__restrict__ unit_off,
                                                          const int32_t *__restrict__ unit_chunk, int L, int C,
                                                          int n_units) {
    constexpr int LANES = D / 8;          // 16-byte lanes per token row
    constexpr int ROWS = 256 / LANES;     // rows per pass
    __shared__ float red[ROWS][D + 4];
    __shared__ int is_last;
    const int h = blockIdx.y;
    const int lane = threadIdx.x % LANES, rg = threadIdx.x / LANES;
    for (int unit = blockIdx.x; unit < n_units; unit += gridDim.x) {
        const int c = unit_chunk[unit];
        const int slice = unit - unit_off[c];
        const int t0 = off[c] + slice * kPoolSlice;
        const int t1 = min(off[c + 1], t0 + kPoolSlice);
        float acc[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) acc[x] = 0.f;
        const uint4 *base = reinterpret_cast<const uint4 *>(K + ((size_t)h * L) * D) + lane;
        int t = t0 + rg;
        // 4 independent 16-byte loads in flight per thread
        for (; t + 3 * ROWS < t1; t += 4 * ROWS) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = __ldg(base + (size_t)(t + u * ROWS) * LANES);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const __nv_bfloat162 *b = reinterpret_cast<const __nv_bfloat162 *>(&v[u]);
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    float2 f = __bfloat1622float2(b[x]);
                    acc[2 * x] += f.x;
                    acc[2 * x + 1] += f.y;
                }
            }
        }
        for (; t < t1; t += ROWS) {
            uint4 v = __ldg(base + (size_t)t * LANES);
            const __nv_bfloat162 *b = reinterpret_cast<const __nv_bfloat162 *>(&v);
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                float2 f = __bfloat1622float2(b[x]);
                acc[2 * x] += f.x;
                acc[2 * x + 1] += f.y;
            }
        }
#pragma unroll
        for (int x = 0; x < 8; ++x) red[rg][lane * 8 + x] = acc[x];
        __syncthreads();
        float *mine = part + ((size_t)h * n_units + unit) * D;
        if (threadIdx.x < D) {
            float s = 0.f;
#pragma unroll
            for (int r = 0; r < ROWS; ++r) s += red[r][threadIdx.x];
            mine[threadIdx.x] = s;
            __threadfence();
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            const int n_slices = unit_off[c + 1] - unit_off[c];
            int prev = atomicAdd(&done[h * C + c], 1);
            is_last = (prev == n_slices - 1);
        }
        __syncthreads();
        if (is_last) {
            __threadfence();
            if (threadIdx.x < D) {
                const int u0 = unit_off[c], u1 = unit_off[c + 1];
                float s = 0.f;
                for (int u = u0; u < u1; ++u) s += __ldcg(part + ((size_t)h * n_units + u) * D + threadIdx.x);
                desc[((size_t)h * C + c) * D + threadIdx.x] = s / (float)(off[c + 1] - off[c]);
            }
        }
        __syncthreads();
    }
}

// The same stream with one block per (head, chunk): no partial sums, no arrival counters, so nothing has to be
// cleared first.  Used when every block is resident at once (few enough chunks) and no chunk is long.
template <int D>
__global__ void __launch_bounds__(256) chunk_pool_direct_kernel(const __nv_bfloat16 *__restrict__ K, float *__restrict__ desc,
                                                                 const int32_t *__restrict__ off, int L, int C) {
    constexpr int LANES = D / 8;          // 16-byte lanes per token row
    constexpr int ROWS = 256 / LANES;     // rows per pass
    __shared__ float red[ROWS][D + 4];
    const int c = blockIdx.x, h = blockIdx.y;
    const int lane = threadIdx.x % LANES, rg = threadIdx.x / LANES;
    const int t0 = off[c], t1 = off[c + 1];
    float acc[8];
#pragma unroll
    for (int x = 0; x < 8; ++x) acc[x] = 0.f;
    const uint4 *base = reinterpret_cast<const uint4 *>(K + ((size_t)h * L) * D) + lane;
    int t = t0 + rg;
    for (; t + 3 * ROWS < t1; t += 4 * ROWS) {          // 4 independent 16-byte loads in flight per thread
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = __ldg(base + (size_t)(t + u * ROWS) * LANES);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const __nv_bfloat162 *b = reinterpret_cast<const __nv_bfloat162 *>(&v[u]);
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                float2 f = __bfloat1622float2(b[x]);
                acc[2 * x] += f.x;
                acc[2 * x + 1] += f.y;
            }
        }
    }
    for (; t < t1; t += ROWS) {
        uint4 v = __ldg(base + (size_t)t * LANES);
        const __nv_bfloat162 *b = reinterpret_cast<const __nv_bfloat162 *>(&v);
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            float2 f = __bfloat1622float2(b[x]);
            acc[2 * x] += f.x;
            acc[2 * x + 1] += f.y;
        }
    }
#pragma unroll
    for (int x = 0; x < 8; ++x) red[rg][lane * 8 + x] = acc[x];
    __syncthreads();
    if (threadIdx.x < D) {
        float s = 0.f;
#pragma unroll
        for (int r = 0; r < ROWS; ++r) s += red[r][threadIdx.x];       // fixed order: the result does not depend on scheduling
        desc[((size_t)h * C + c) * D + threadIdx.x] = s / (float)(t1 - t0);
    }
}

__global__ void zero_i32_kernel(int *p, size_t n) {
    size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    if (i < n) p[i] = 0;
}

int launch_chunk_pool(const moc_plan *p, const __nv_bfloat16 *K, float *desc, void *ws, cudaStream_t s) {
    if (p->pool_direct) {
        dim3 grid((unsigned)p->C, (unsigned)p->H);
        if (p->d == 128) chunk_pool_direct_kernel<128><<<grid, 256, 0, s>>>(K, desc, p->d_off, p->L, p->C);
        else chunk_pool_direct_kernel<64><<<grid, 256, 0, s>>>(K, desc, p->d_off, p->L, p->C);
        MOC_LAUNCH_CHECK();
        return MOC_OK;
    }
    float *part = ws_ptr<float>(ws, p->ws.pool_part);
    int *done = ws_ptr<int>(ws, p->ws.pool_done);
    // the arrival counters live in caller-owned scratch whose contents are unknown
    size_t n = (size_t)p->H * p->C;
    zero_i32_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(done, n);
    MOC_LAUNCH_CHECK();
    dim3 grid((unsigned)std::min(p->n_pool_units, 65535), (unsigned)p->H);
    if (p->d == 128)
        chunk_pool_kernel<128><<<grid, 256, 0, s>>>(K, desc, part, done, p->d_off, p->d_pool_unit_off,
                                                    p->d_pool_unit_chunk, p->L, p->C, p->n_pool_units);
    else
        chunk_pool_kernel<64><<<grid, 256, 0, s>>>(K, desc, part, done, p->d_off, p->d_pool_unit_off,
                                                   p->d_pool_unit_chunk, p->L, p->C, p->n_pool_units);
    MOC_LAUNCH_CHECK();
    return MOC_OK;
}

}  // namespace moc

// ---------------------------------------------------------------------------------------------
// moc_chunk_pool_noalloc: the same descriptor kernel with its scratch (per-slice partial sums and
// per-chunk arrival counters) in a fixed array that is part of the library image, so the caller
// needs no workspace and the call allocates nothing.
namespace moc {

constexpr size_t kStaticPartBytes = 4u << 20;     // partial sums: H * units * d * 4 bytes must fit
constexpr size_t kStaticDoneBytes = 64u << 10;    // arrival counters: H * C * 4 bytes must fit
static __device__ __align__(256) unsigned char g_pool_scratch[kStaticPartBytes + kStaticDoneBytes];

constexpr int kMaxDevices = 64;
static std::mutex g_scratch_mu;
static unsigned char *g_scratch_addr[kMaxDevices] = {};

// Device address of the scratch array on `device`, which must be current.  In host code the array's
// name is only a handle; the address a kernel can use comes from cudaGetSymbolAddress, once per device.
// Called from moc_plan_create: the lookup is also what makes the driver load this module (and with it
// place the array) on the device, so it happens where allocating is allowed and never inside
// moc_chunk_pool_noalloc; the kernels' attributes are queried for the same reason (their code is loaded).
int pool_scratch_prepare(int device) {
    if (device < 0 || device >= kMaxDevices) return MOC_ERR_ARCH;
    std::lock_guard<std::mutex> g(g_scratch_mu);
    if (!g_scratch_addr[device]) {
        void *ptr = nullptr;
        MOC_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_pool_scratch));
        if (!ptr) return MOC_ERR_CUDA;
        cudaFuncAttributes fa;
        MOC_CUDA_TRY(cudaFuncGetAttributes(&fa, chunk_pool_kernel<128>));
        MOC_CUDA_TRY(cudaFuncGetAttributes(&fa, chunk_pool_kernel<64>));
        MOC_CUDA_TRY(cudaFuncGetAttributes(&fa, zero_i32_kernel));
        g_scratch_addr[device] = static_cast<unsigned char *>(ptr);
    }
    return MOC_OK;
}

static int pool_scratch_address(int device, unsigned char **out) {
    if (device < 0 || device >= kMaxDevices) return MOC_ERR_ARCH;
    std::lock_guard<std::mutex> g(g_scratch_mu);
    if (!g_scratch_addr[device]) return MOC_ERR_CUDA;      // no plan was ever created on this device
    *out = g_scratch_addr[device];
    return MOC_OK;
}

}  // namespace moc

extern "C" int moc_chunk_pool_noalloc(const moc_plan *p, const void *K, float *desc, void *stream) {
    using namespace moc;
    if (!p || !K || !desc) return MOC_ERR_NULL;
    if (!aligned(K, 16) || !aligned(desc, 16)) return MOC_ERR_ALIGN;
    int dev = -1;
    MOC_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != p->device) return MOC_ERR_ARCH;
    const size_t part_bytes = sizeof(float) * (size_t)p->H * p->n_pool_units * p->d;
    const size_t done_bytes = sizeof(int) * (size_t)p->H * p->C;
    if (part_bytes > kStaticPartBytes || done_bytes > kStaticDoneBytes) return MOC_ERR_TOO_LARGE;
    unsigned char *base = nullptr;
    if (int r = pool_scratch_address(dev, &base)) return r;
    float *part = reinterpret_cast<float *>(base);
    int *done = reinterpret_cast<int *>(base + kStaticPartBytes);
    cudaStream_t s = (cudaStream_t)stream;
    // the array keeps the previous call's contents: the counters must start at zero
    const size_t n = (size_t)p->H * p->C;
    zero_i32_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(done, n);
    MOC_LAUNCH_CHECK();
    dim3 grid((unsigned)std::min(p->n_pool_units, 65535), (unsigned)p->H);
    if (p->d == 128)
        chunk_pool_kernel<128><<<grid, 256, 0, s>>>(static_cast<const __nv_bfloat16 *>(K), desc, part, done, p->d_off,
                                                    p->d_pool_unit_off, p->d_pool_unit_chunk, p->L, p->C, p->n_pool_units);
    else
        chunk_pool_kernel<64><<<grid, 256, 0, s>>>(static_cast<const __nv_bfloat16 *>(K), desc, part, done, p->d_off,
                                                   p->d_pool_unit_off, p->d_pool_unit_chunk, p->L, p->C, p->n_pool_units);
    MOC_LAUNCH_CHECK();
    return MOC_OK;
}
