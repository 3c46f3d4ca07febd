// Context drop-off and drop-in (Sec. 3.1 of the paper): training-time edits of a routed selection.
//
// For every query row, on its k slots of sel_idx:
//   drop-off  p_drop = U p_max, U ~ Uniform[0, 1); floor(p_drop k) of the row's picks are removed (never more
//             than it has), each chosen uniformly among the picks still there;
//   drop-in   m ~ Poisson(lambda) chunks are added, each chosen uniformly among the chunks the row may route to
//             (not an anchor of its chunk, strictly earlier if causal) that are neither routed picks of the row
//             (kept or dropped) nor added already; they fill the free slots, lowest slot first, while there
//             is a free slot and a chunk left.
// One thread per row.  The draws come from Philox4x32-10 (Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as
// easy as 1, 2, 3", SC'11) keyed by the caller's seed with the counter (token, head, draw / 4, 0): draw 0 is U,
// draw 1 the Poisson variate (inversion against a table accumulated in double on the host), draw 2 + r the r-th
// removal, draw 2 + k + t the t-th addition; a draw is the top 24 bits of a word scaled to [0, 1), and every
// product that decides an integer is a single-precision product, so the result is a pure function of the seed.
// While a row is being edited a dropped pick j is kept as -2 - j (it still counts as "routed"); the row ends with
// -1 in every empty slot.  The chunk -> query lists are rebuilt afterwards by the caller (launch_lists_from_sel).
#include <math.h>

#include "moc_common.cuh"

namespace moc {

struct PoissonTable { float cdf[32]; };

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1,
                                              uint32_t (&out)[4]) {
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// the draws of one row, generated a block of four at a time
struct RowDraws {
    uint32_t tok, head, k0, k1, w[4];
    int blk;
    __device__ float uniform(int d) {
        if ((d >> 2) != blk) {
            blk = d >> 2;
            philox4x32_10(tok, head, (uint32_t)blk, 0u, k0, k1, w);
        }
        const uint32_t x = (d & 3) == 0 ? w[0] : (d & 3) == 1 ? w[1] : (d & 3) == 2 ? w[2] : w[3];
        return (float)(x >> 8) * (1.0f / 16777216.0f);
    }
};

__global__ void __launch_bounds__(128) context_drop_kernel(int32_t *__restrict__ sel, const int32_t *__restrict__ tok_chunk,
                                                           const uint32_t *__restrict__ anc_bits, PoissonTable tab, int H, int L,
                                                           int C, int k, int words, int causal, float p_max, uint32_t seed_lo,
                                                           uint32_t seed_hi) {
    const size_t r = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    if (r >= (size_t)H * L) return;
    const int h = (int)(r / L), i = (int)(r % L);
    int32_t *row = sel + r * k;
    const int ci = tok_chunk[i];
    RowDraws rng{(uint32_t)i, (uint32_t)h, seed_lo, seed_hi, {0u, 0u, 0u, 0u}, -1};
    int n_sel = 0;
    for (int s = 0; s < k; ++s) n_sel += row[s] >= 0;
    // ---- drop-off
    const float p_drop = rng.uniform(0) * p_max;
    int n_drop = min(n_sel, (int)(p_drop * (float)k));
    for (int d = 0; d < n_drop; ++d) {
        const int n_left = n_sel - d;
        int pos = min((int)(rng.uniform(2 + d) * (float)n_left), n_left - 1);
        for (int s = 0; s < k; ++s) {
            const int v = row[s];
            if (v < 0) continue;
            if (pos-- == 0) { row[s] = -2 - v; break; }
        }
    }
    // ---- drop-in
    const float u = rng.uniform(1);
    int m = 0;
    while (m < 31 && !(u < tab.cdf[m])) ++m;
    // candidate chunks of this row, 32 at a time: not an anchor, inside the stream, strictly earlier if causal
    const int lim = causal ? min(ci, C) : C;
    auto cand_word = [&](int w) -> uint32_t {
        const int n = lim - 32 * w;
        const uint32_t in = n <= 0 ? 0u : (n >= 32 ? 0xffffffffu : ((1u << n) - 1u));
        return ~anc_bits[(size_t)ci * words + w] & in;
    };
    // The additions are chosen first and written afterwards: a dropped pick stays in its slot (as -2 - j) while
    // they are drawn, because it must stay excluded even when an addition is about to take that slot.
    int added[31], n_added = 0, n_free = 0;
    for (int s = 0; s < k; ++s) n_free += row[s] < 0;
    for (int t = 0; t < m && n_added < n_free; ++t) {
        // eligible chunks, word by word: the candidates minus what the row holds (picks kept or dropped) and
        // what has been added already
        auto eligible_word = [&](int w) -> uint32_t {
            uint32_t cw = cand_word(w);
            for (int s = 0; s < k; ++s) {
                const int v = row[s], j = v >= 0 ? v : (v <= -2 ? -2 - v : -1);
                if (j >= 0 && (j >> 5) == w) cw &= ~(1u << (j & 31));
            }
            for (int a = 0; a < n_added; ++a)
                if ((added[a] >> 5) == w) cw &= ~(1u << (added[a] & 31));
            return cw;
        };
        int n_left = 0;
        for (int w = 0; w < words; ++w) n_left += __popc(eligible_word(w));
        if (n_left == 0) break;
        int pos = min((int)(rng.uniform(2 + k + t) * (float)n_left), n_left - 1);
        for (int w = 0; w < words; ++w) {
            uint32_t cw = eligible_word(w);
            const int n = __popc(cw);
            if (pos >= n) { pos -= n; continue; }
            for (; pos > 0; --pos) cw &= cw - 1;          // drop the lowest pos set bits
            added[n_added++] = 32 * w + (__ffs(cw) - 1);
            break;
        }
    }
    for (int s = 0, a = 0; s < k; ++s) {                   // free slots, lowest first; the rest end as -1
        if (row[s] >= 0) continue;
        row[s] = a < n_added ? added[a++] : -1;
    }
}

int launch_context_drop(const moc_plan *p, int32_t *sel, float p_max, float lambda, uint64_t seed, cudaStream_t s) {
    if (p->k == 0) return MOC_OK;
    PoissonTable tab;
    double term = exp(-(double)lambda), acc = term;
    tab.cdf[0] = (float)acc;
    for (int j = 1; j < 32; ++j) {
        term = term * (double)lambda / (double)j;
        acc += term;
        tab.cdf[j] = (float)acc;
    }
    const size_t rows = (size_t)p->H * p->L;
    context_drop_kernel<<<(unsigned)((rows + 127) / 128), 128, 0, s>>>(sel, p->d_tok_chunk, p->d_anc_bits, tab, p->H, p->L, p->C, p->k,
                                                                      p->words, (p->flags & MOC_FLAG_CAUSAL) ? 1 : 0, p_max,
                                                                      (uint32_t)seed, (uint32_t)(seed >> 32));
    MOC_LAUNCH_CHECK();
    return MOC_OK;
}

}  // namespace moc
