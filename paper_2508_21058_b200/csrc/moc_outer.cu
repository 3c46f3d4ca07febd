// Outer-loop context routing (the paper's appendix of that name): a coarse pre-selection of whole shots for
// one query block, ahead of the per-query routing.  High-level chunk = every token of a shot.
//   phi(Psi_s) = mean of the context features over the shot's tokens.  The features' chunk descriptors
//                (moc_chunk_pool) are already per-chunk means, so the shot mean is their token-weighted mean:
//                no second pass over the features;
//   x_g        = mean of the query features over the block [q0, q1): one streaming pass over the block
//                (256-token slices, partial sums reduced in slice order: deterministic);
//   s_s        = <x_g, phi(Psi_s)>, the M best among the shots that end before the block begins, equal scores to
//                the earlier shot.
// moc_outer_reduced_layout (host only) turns a selection into the chunk table of the reduced stream - every text
// chunk, the selected shots, the block's own shots - with the map from its tokens to the original ones, and
// moc_gather_tokens copies the kept rows of a [H][L][d] tensor, so the inner path can run on the reduced stream.
#include <vector>

#include "moc_common.cuh"

namespace moc {

template <int D>
__global__ void __launch_bounds__(256) block_sum_kernel(const __nv_bfloat16 *__restrict__ X, float *__restrict__ part, int L, int q0,
                                                        int q1, int n_slices) {
    constexpr int LANES = D / 8, ROWS = 256 / LANES;
    __shared__ float red[ROWS][D + 4];
    const int h = blockIdx.y, slice = blockIdx.x;
    const int lane = threadIdx.x % LANES, rg = threadIdx.x / LANES;
    const int t0 = q0 + slice * kPoolSlice, t1 = min(q1, t0 + kPoolSlice);
    float acc[8];
#pragma unroll
    for (int x = 0; x < 8; ++x) acc[x] = 0.f;
    const uint4 *base = reinterpret_cast<const uint4 *>(X + ((size_t)h * L) * D) + lane;
    for (int t = t0 + rg; t < t1; t += ROWS) {
        const uint4 v = __ldg(base + (size_t)t * LANES);
        const __nv_bfloat162 *b = reinterpret_cast<const __nv_bfloat162 *>(&v);
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const float2 f = __bfloat1622float2(b[x]);
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
        for (int r = 0; r < ROWS; ++r) s += red[r][threadIdx.x];
        part[((size_t)h * n_slices + slice) * D + threadIdx.x] = s;
    }
}

// one block of D threads per feature stream
template <int D>
__global__ void __launch_bounds__(D) outer_score_kernel(const float *__restrict__ part, const float *__restrict__ desc,
                                                        const int32_t *__restrict__ off, const KeyRange *__restrict__ shot_chunks,
                                                        float *__restrict__ shot_desc, float *__restrict__ scores,
                                                        int32_t *__restrict__ sel, int C, int S, int n_slices, int q0, int q1, int M) {
    __shared__ float red[D];
    extern __shared__ float s_score[];      // [S]
    const int h = blockIdx.x, x = threadIdx.x;
    float xg = 0.f;
    for (int u = 0; u < n_slices; ++u) xg += part[((size_t)h * n_slices + u) * D + x];
    xg /= (float)(q1 - q0);
    for (int s = 0; s < S; ++s) {
        const int c0 = shot_chunks[s].t0, c1 = shot_chunks[s].t1;
        float f = 0.f;
        for (int c = c0; c < c1; ++c) f += (float)(off[c + 1] - off[c]) * desc[((size_t)h * C + c) * D + x];
        f /= (float)(off[c1] - off[c0]);
        shot_desc[((size_t)h * S + s) * D + x] = f;
        red[x] = xg * f;
        __syncthreads();
        for (int o = D / 2; o > 0; o >>= 1) {       // fixed tree: the same sum whatever the schedule
            if (x < o) red[x] += red[x + o];
            __syncthreads();
        }
        if (x == 0) { s_score[s] = red[0]; scores[(size_t)h * S + s] = red[0]; }
        __syncthreads();
    }
    if (x == 0) {
        // candidates: the shots that end before the block begins; M rounds of "largest left", strict '>' so
        // that equal scores go to the earlier shot; a taken shot's score is overwritten
        for (int r = 0; r < M; ++r) {
            int best = -1;
            for (int s = 0; s < S; ++s) {
                if (off[shot_chunks[s].t1] > q0 || s_score[s] != s_score[s]) continue;     // NaN marks a taken shot
                if (best < 0 || s_score[s] > s_score[best]) best = s;
            }
            sel[(size_t)h * M + r] = best;
            if (best >= 0) s_score[best] = __int_as_float(0x7fc00000);
        }
    }
}

template <int D>
__global__ void __launch_bounds__(256) gather_rows_kernel(const __nv_bfloat16 *__restrict__ X, const int32_t *__restrict__ tok_map,
                                                          __nv_bfloat16 *__restrict__ out, int L, int n_out) {
    constexpr int LANES = D / 8;
    const int h = blockIdx.y;
    const size_t piece = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    if (piece >= (size_t)n_out * LANES) return;
    const int r = (int)(piece / LANES), lane = (int)(piece % LANES);
    const int t = tok_map[r];
    uint4 v = make_uint4(0, 0, 0, 0);
    if ((unsigned)t < (unsigned)L) v = __ldg(reinterpret_cast<const uint4 *>(X + ((size_t)h * L + t) * D) + lane);
    reinterpret_cast<uint4 *>(out + ((size_t)h * n_out + r) * D)[lane] = v;
}

}  // namespace moc

using namespace moc;

extern "C" int moc_outer_num_shots(const moc_plan *p, int32_t *n_shots) {
    if (!p || !n_shots) return MOC_ERR_NULL;
    *n_shots = (int32_t)p->shot_chunks.size();
    return MOC_OK;
}

extern "C" int moc_outer_route(const moc_plan *p, const void *Xq, const float *desc, int32_t q_tok0, int32_t q_tok1, int32_t top_m,
                               float *shot_desc, float *scores, int32_t *sel_shot, void *ws, void *stream) {
    moc::NvtxRange nvtx_range("moc_outer_route");
    if (!p) return MOC_ERR_NULL;
    int dev = -1;
    MOC_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != p->device) return MOC_ERR_ARCH;
    if (!Xq || !desc || !shot_desc || !scores || (top_m > 0 && !sel_shot)) return MOC_ERR_NULL;
    if (!aligned(Xq, 16) || !aligned(desc, 16) || !aligned(shot_desc, 4) || !aligned(scores, 4) || !aligned(sel_shot, 4)) return MOC_ERR_ALIGN;
    if (!ws) return MOC_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return MOC_ERR_ALIGN;
    const int S = (int)p->shot_chunks.size();
    if (q_tok0 < 0 || q_tok1 <= q_tok0 || q_tok1 > p->L || top_m < 0 || top_m > S) return MOC_ERR_SHAPE;
    cudaStream_t s = (cudaStream_t)stream;
    const int n_slices = (q_tok1 - q_tok0 + kPoolSlice - 1) / kPoolSlice;      // never more than the pooling units
    float *part = ws_ptr<float>(ws, p->ws.pool_part);
    const __nv_bfloat16 *X = static_cast<const __nv_bfloat16 *>(Xq);
    const dim3 grid((unsigned)n_slices, (unsigned)p->H);
    const size_t smem = sizeof(float) * (size_t)S;
    if (p->d == 128) {
        block_sum_kernel<128><<<grid, 256, 0, s>>>(X, part, p->L, q_tok0, q_tok1, n_slices);
        MOC_LAUNCH_CHECK();
        outer_score_kernel<128><<<(unsigned)p->H, 128, smem, s>>>(part, desc, p->d_off, p->d_shot_chunks, shot_desc, scores, sel_shot,
                                                                 p->C, S, n_slices, q_tok0, q_tok1, top_m);
    } else {
        block_sum_kernel<64><<<grid, 256, 0, s>>>(X, part, p->L, q_tok0, q_tok1, n_slices);
        MOC_LAUNCH_CHECK();
        outer_score_kernel<64><<<(unsigned)p->H, 64, smem, s>>>(part, desc, p->d_off, p->d_shot_chunks, shot_desc, scores, sel_shot,
                                                               p->C, S, n_slices, q_tok0, q_tok1, top_m);
    }
    MOC_LAUNCH_CHECK();
    return MOC_OK;
}

extern "C" int moc_outer_reduced_layout(const moc_plan *p, const int32_t *sel_shot, int32_t n_sel, int32_t q_tok0, int32_t q_tok1,
                                        int32_t *n_chunks, int32_t *n_tokens, int32_t *chunk_off, int32_t *chunk_shot,
                                        uint8_t *chunk_mod, int32_t *tok_map) {
    if (!p || (n_sel > 0 && !sel_shot) || !n_chunks || !n_tokens || !chunk_off || !chunk_shot || !chunk_mod || !tok_map) return MOC_ERR_NULL;
    const int S = (int)p->shot_chunks.size();
    if (q_tok0 < 0 || q_tok1 <= q_tok0 || q_tok1 > p->L || n_sel < 0) return MOC_ERR_SHAPE;
    std::vector<char> keep_shot(S, 0);
    for (int r = 0; r < n_sel; ++r) {
        if (sel_shot[r] == -1) continue;
        if (sel_shot[r] < 0 || sel_shot[r] >= S) return MOC_ERR_SHAPE;
        keep_shot[sel_shot[r]] = 1;
    }
    for (int s = 0; s < S; ++s) {        // the block's own shots
        const int t0 = p->off[p->shot_chunks[s].t0], t1 = p->off[p->shot_chunks[s].t1];
        if (t0 < q_tok1 && t1 > q_tok0) keep_shot[s] = 1;
    }
    int nc = 0, nt = 0;
    chunk_off[0] = 0;
    for (int s = 0; s < S; ++s)
        for (int c = p->shot_chunks[s].t0; c < p->shot_chunks[s].t1; ++c) {
            if (!keep_shot[s] && p->mod[c] != 1) continue;        // text chunks are mandatory, whatever their shot
            for (int t = p->off[c]; t < p->off[c + 1]; ++t) tok_map[nt++] = t;
            chunk_shot[nc] = p->shot[c];
            chunk_mod[nc] = p->mod[c];
            chunk_off[++nc] = nt;
        }
    *n_chunks = nc;
    *n_tokens = nt;
    return MOC_OK;
}

extern "C" int moc_gather_tokens(const moc_plan *p, const void *X, const int32_t *tok_map, int32_t n_out, void *out, void *stream) {
    moc::NvtxRange nvtx_range("moc_gather_tokens");
    if (!p) return MOC_ERR_NULL;
    int dev = -1;
    MOC_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != p->device) return MOC_ERR_ARCH;
    if (!X || !tok_map || !out) return MOC_ERR_NULL;
    if (!aligned(X, 16) || !aligned(out, 16) || !aligned(tok_map, 4)) return MOC_ERR_ALIGN;
    if (n_out < 1) return MOC_ERR_SHAPE;
    const size_t pieces = (size_t)n_out * (p->d / 8);
    const dim3 grid((unsigned)((pieces + 255) / 256), (unsigned)p->H);
    if (p->d == 128)
        gather_rows_kernel<128><<<grid, 256, 0, (cudaStream_t)stream>>>(static_cast<const __nv_bfloat16 *>(X), tok_map,
                                                                        static_cast<__nv_bfloat16 *>(out), p->L, n_out);
    else
        gather_rows_kernel<64><<<grid, 256, 0, (cudaStream_t)stream>>>(static_cast<const __nv_bfloat16 *>(X), tok_map,
                                                                       static_cast<__nv_bfloat16 *>(out), p->L, n_out);
    MOC_LAUNCH_CHECK();
    return MOC_OK;
}
