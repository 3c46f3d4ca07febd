// Plan object (validated problem + derived chunk tables on the device), workspace layout,
// argument checking and the C entry points.
#include <math.h>
#include <algorithm>
#include <string.h>
#include <mutex>
#include <new>
#include <string>

#include "moc_common.cuh"

namespace moc {

std::atomic<long long> g_launches{0};
static std::mutex g_err_mu;
static std::string g_err = "";

void set_cuda_error(cudaError_t e, const char *where) {
    std::lock_guard<std::mutex> g(g_err_mu);
    g_err = std::string(cudaGetErrorName(e)) + ": " + cudaGetErrorString(e) + " (" + where + ")";
    (void)cudaGetLastError();
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Sec. 3.2: text chunks are anchors of every query; so are the chunks of the query's shot
// inside the window around its own chunk.
static bool is_anchor(const moc_plan *p, int c, int j) {
    if (p->mod[j] == 1) return true;
    if (p->shot[j] != p->shot[c]) return false;
    if (j < c && p->win_back != MOC_WHOLE_SHOT && c - j > p->win_back) return false;
    if (j > c && p->win_fwd != MOC_WHOLE_SHOT && j - c > p->win_fwd) return false;
    return true;
}

// Workspace layout.  The routed partial outputs ([heads][L][k][d] bf16, k times the size of O) are held for
// one group of Hg heads at a time; attention and its backward run group by group.  If all heads fit the plan's
// budget there is one group and one buffer; otherwise two buffers of Hg heads each (consecutive groups
// alternate, so that one group's routed items can run while the previous group's anchor items still merge),
// Hg the largest even split of the heads for which both stay within the budget (at least one head).
void layout_workspace(moc_plan *p) {
    WsLayout &w = p->ws;
    const size_t H = p->H, L = p->L, d = p->d, C = p->C, k = p->k;
    const size_t per_head = sizeof(__nv_bfloat16) * ((L + 127) / 128 * 128) * k * d;      // whole blocks of 128 queries
    size_t groups = 1, buffers = 1;
    p->heads_per_group = (int)H;
    if (per_head * H > p->partials_budget) {
        const size_t hg = std::max<size_t>(1, p->partials_budget / (2 * per_head));
        groups = (H + hg - 1) / hg;
        p->heads_per_group = (int)((H + groups - 1) / groups);
        groups = (H + p->heads_per_group - 1) / p->heads_per_group;
        buffers = groups > 1 ? 2 : 1;
    }
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    w.status = take(sizeof(int32_t) * kStatusWords);
    w.cnt = take(sizeof(int32_t) * H * C);
    w.tile_off = take(sizeof(int32_t) * (H * C + 1));
    w.rtiles = take(sizeof(WorkItem) * H * ((L * (k ? k : 1) + kQTileRows - 1) / kQTileRows + C));
    w.qlist = take(sizeof(int32_t) * H * (size_t)std::max(p->cap_off[C], 1));
    w.desc3 = take(sizeof(__nv_bfloat16) * H * 3 * (size_t)p->c_pad * d);
    w.pool_part = take(sizeof(float) * H * (size_t)p->n_pool_units * d);
    w.pool_done = take(sizeof(int32_t) * H * C);
    w.queue = take(sizeof(int32_t) * (kQueueHeader + 6 * groups));
    w.part_o = take(per_head * (size_t)p->heads_per_group * buffers);
    w.part_lse = take(sizeof(float) * H * L * (k ? k : 1));
    w.fwd_end = o;
    w.delta = take(sizeof(float) * H * L);
    w.bwd_end = o;
}

// FNV-1a over the problem: a workspace routed by one plan is not accepted by a plan of another problem
static uint32_t plan_cookie(const moc_plan *p) {
    uint32_t hsh = 2166136261u;
    auto mix = [&](const void *data, size_t n) {
        const unsigned char *b = static_cast<const unsigned char *>(data);
        for (size_t i = 0; i < n; ++i) { hsh ^= b[i]; hsh *= 16777619u; }
    };
    const int32_t hdr[] = {p->H, p->L, p->d, p->C, p->k, p->win_back, p->win_fwd, (int32_t)(p->flags & MOC_FLAG_CAUSAL)};
    mix(hdr, sizeof hdr);
    mix(p->off.data(), p->off.size() * 4);
    mix(p->shot.data(), p->shot.size() * 4);
    mix(p->mod.data(), p->mod.size());
    return hsh ? hsh : 1u;
}

}  // namespace moc

using namespace moc;

extern "C" int moc_plan_create(const moc_problem *pr, moc_plan **out) {
    if (!pr || !out) return MOC_ERR_NULL;
    *out = nullptr;
    if (!pr->chunk_off || !pr->chunk_shot || !pr->chunk_mod) return MOC_ERR_NULL;
    if (pr->n_heads < 1 || pr->n_tokens < 1 || pr->n_chunks < 1 || pr->n_chunks > pr->n_tokens) return MOC_ERR_SHAPE;
    // heads index grid.y; head * L + token is a 32-bit row coordinate of the tensor maps
    if (pr->n_heads > 65535 || (double)pr->n_heads * pr->n_tokens >= 2147483647.0) return MOC_ERR_SHAPE;
    if (pr->head_dim != 64 && pr->head_dim != 128) return MOC_ERR_SHAPE;
    if (pr->top_k < 0 || pr->top_k > 512) return MOC_ERR_SHAPE;
    if (pr->win_back < MOC_WHOLE_SHOT || pr->win_fwd < MOC_WHOLE_SHOT) return MOC_ERR_SHAPE;
    if ((double)pr->n_tokens * (pr->top_k ? pr->top_k : 1) >= 2147483647.0) return MOC_ERR_SHAPE;
    if ((double)pr->n_heads * pr->n_chunks >= 1e8) return MOC_ERR_SHAPE;
    if (pr->flags & ~MOC_FLAG_CAUSAL) return MOC_ERR_SHAPE;
    if (!(pr->softmax_scale >= 0.f) || isinf(pr->softmax_scale)) return MOC_ERR_SHAPE;
    const int C = pr->n_chunks, L = pr->n_tokens;
    if (pr->chunk_off[0] != 0 || pr->chunk_off[C] != L) return MOC_ERR_CHUNK_TABLE;
    for (int c = 0; c < C; ++c) {
        if (pr->chunk_off[c + 1] <= pr->chunk_off[c]) return MOC_ERR_CHUNK_TABLE;
        if (pr->chunk_mod[c] > 1) return MOC_ERR_CHUNK_TABLE;
        if (c > 0 && pr->chunk_shot[c] < pr->chunk_shot[c - 1]) return MOC_ERR_CHUNK_TABLE;
    }
    int dev = 0;
    MOC_CUDA_TRY(cudaGetDevice(&dev));
    cudaDeviceProp prop;
    MOC_CUDA_TRY(cudaGetDeviceProperties(&prop, dev));
    if (prop.major != 10) return MOC_ERR_ARCH;

    moc_plan *p = new (std::nothrow) moc_plan();
    if (!p) return MOC_ERR_CUDA;
    p->H = pr->n_heads; p->L = L; p->d = pr->head_dim; p->C = C; p->k = pr->top_k;
    p->win_back = pr->win_back; p->win_fwd = pr->win_fwd; p->flags = pr->flags;
    p->scale = pr->softmax_scale > 0.f ? pr->softmax_scale : 1.0f / sqrtf((float)pr->head_dim);
    p->device = dev; p->n_sm = prop.multiProcessorCount;
    p->off.assign(pr->chunk_off, pr->chunk_off + C + 1);
    p->shot.assign(pr->chunk_shot, pr->chunk_shot + C);
    p->mod.assign(pr->chunk_mod, pr->chunk_mod + C);

    // anchor bitmaps, merged anchor key ranges, reverse anchors
    p->words = (C + 31) / 32;
    std::vector<uint32_t> bits((size_t)C * p->words, 0u);
    std::vector<std::vector<int32_t>> rev(C);
    p->anc_off.assign(C + 1, 0);
    p->anc_tokens.assign(C, 0);
    for (int c = 0; c < C; ++c) {
        for (int j = 0; j < C; ++j) {
            if (!is_anchor(p, c, j)) continue;
            bits[(size_t)c * p->words + j / 32] |= 1u << (j % 32);
            rev[j].push_back(c);
            p->anc_tokens[c] += p->off[j + 1] - p->off[j];
            if ((int)p->anc_rng.size() > p->anc_off[c] && p->anc_rng.back().t1 == p->off[j])
                p->anc_rng.back().t1 = p->off[j + 1];
            else
                p->anc_rng.push_back(KeyRange{p->off[j], p->off[j + 1]});
        }
        p->anc_off[c + 1] = (int32_t)p->anc_rng.size();
    }
    p->ranc_off.assign(C + 1, 0);
    for (int j = 0; j < C; ++j) {
        p->ranc.insert(p->ranc.end(), rev[j].begin(), rev[j].end());
        p->ranc_off[j + 1] = (int32_t)p->ranc.size();
    }
    // query tiles (never straddle a chunk) and pool work units
    std::vector<int32_t> tok_chunk(L), unit_chunk;
    std::vector<KeyRange> chunk_rng(C);
    for (int c = 0; c < C; ++c) chunk_rng[c] = KeyRange{p->off[c], p->off[c + 1]};
    p->pool_unit_off.assign(C + 1, 0);
    for (int c = 0; c < C; ++c) {
        for (int t = p->off[c]; t < p->off[c + 1]; ++t) tok_chunk[t] = c;
        int anc_tiles = 0;
        for (int a = p->anc_off[c]; a < p->anc_off[c + 1]; ++a) anc_tiles += (p->anc_rng[a].t1 - p->anc_rng[a].t0 + 127) / 128;
        for (int r = p->off[c]; r < p->off[c + 1]; r += kQTileRows)
            p->qitems.push_back(WorkItem{0, r, std::min(kQTileRows, p->off[c + 1] - r), anc_tiles, p->anc_off[c],
                                         p->anc_off[c + 1] - p->anc_off[c], p->anc_rng[p->anc_off[c]].t0,
                                         p->anc_rng[p->anc_off[c]].t1});
        int units = (p->off[c + 1] - p->off[c] + kPoolSlice - 1) / kPoolSlice;
        p->pool_unit_off[c + 1] = p->pool_unit_off[c] + units;
        for (int u = 0; u < units; ++u) unit_chunk.push_back(c);
    }
    p->n_pool_units = p->pool_unit_off[C];
    {
        int longest = 0;
        for (int c = 0; c < C; ++c) longest = std::max(longest, p->off[c + 1] - p->off[c]);
        p->pool_direct = (int64_t)p->H * C <= 8LL * p->n_sm && C <= 65535 && longest <= 4096;
    }
    // Key tiles of the backward's key-stationary pass.  A tile's block streams every query that attends its chunk:
    // the rows of the chunks that have it as an anchor (known here) and the routed list.  Tiles of chunks whose
    // anchor rows are far above the average (a caption, which every query attends) go first, for all heads, so
    // that the longest blocks start at once instead of forming the tail of the launch.
    {
        std::vector<int64_t> anc_rows(C, 0);
        int64_t total = 0, tiles = 0;
        for (int c = 0; c < C; ++c) {
            for (int a = p->ranc_off[c]; a < p->ranc_off[c + 1]; ++a) anc_rows[c] += p->off[p->ranc[a] + 1] - p->off[p->ranc[a]];
            const int nt = (p->off[c + 1] - p->off[c] + 127) / 128;
            total += anc_rows[c] * nt;
            tiles += nt;
        }
        const int64_t mean_rows = total / std::max<int64_t>(tiles, 1);
        for (int pass = 0; pass < 2; ++pass) {
            for (int c = 0; c < C; ++c) {
                const bool is_long = anc_rows[c] > 4 * mean_rows;
                if (is_long != (pass == 0)) continue;
                for (int t = p->off[c]; t < p->off[c + 1]; t += 128) p->ktiles.push_back(KTile{c, t, std::min(128, p->off[c + 1] - t), 0});
            }
            if (pass == 0) p->n_long_ktiles = (int)p->ktiles.size();
        }
    }
    // Query-list capacities: chunk c can be picked by at most the rows after it (causal) or by
    // every row (non-causal); the lists sit back to back at these fixed offsets, so routing can
    // append to them without a counting pass.
    p->cap_off.assign(C + 1, 0);
    for (int c = 0; c < C; ++c) {
        const int64_t cap = p->k == 0 ? 0 : ((p->flags & MOC_FLAG_CAUSAL) ? L - p->off[c + 1] : L);
        const int64_t next = (int64_t)p->cap_off[c] + cap;
        if (next >= 2147483647LL) { delete p; return MOC_ERR_SHAPE; }
        p->cap_off[c + 1] = (int32_t)next;
    }
    // score columns: the chunks that are not text; per query chunk its candidate columns (not an anchor, strictly
    // earlier if causal), whether they form a prefix of the columns (they do under the causal rule: everything
    // before the own shot's window), and how far any query up to that chunk can reach
    std::vector<int32_t> col_chunk, col_of(C, -1);
    for (int j = 0; j < C; ++j)
        if (p->mod[j] != 1) { col_of[j] = (int32_t)col_chunk.size(); col_chunk.push_back(j); }
    p->ncol = (int)col_chunk.size();
    p->cwords = std::max(1, (p->ncol + 31) / 32);
    p->c_pad = std::max(16, (p->ncol + 15) / 16 * 16);
    std::vector<uint32_t> cand_c((size_t)C * p->cwords, 0u);
    std::vector<int32_t> lim(C, 0), reach(C, 0);
    p->prefix_mode = 1;
    for (int c = 0; c < C; ++c) {
        int n_cand = 0, top = 0;
        for (int j = 0; j < C; ++j) {
            if (is_anchor(p, c, j) || ((p->flags & MOC_FLAG_CAUSAL) && j >= c)) continue;
            const int col = col_of[j];          // a non-anchor is never text
            cand_c[(size_t)c * p->cwords + col / 32] |= 1u << (col % 32);
            ++n_cand;
            top = col + 1;
        }
        lim[c] = top == n_cand ? n_cand : -1;
        if (lim[c] < 0) p->prefix_mode = 0;
        reach[c] = std::max(top, c ? reach[c - 1] : 0);
    }
    for (int c = 0; c < C; ++c) {
        if (c == 0 || p->shot[c] != p->shot[c - 1]) p->shot_chunks.push_back(KeyRange{c, c});
        p->shot_chunks.back().t1 = c + 1;
    }
    p->partials_budget = (size_t)6 << 30;
    p->wait_us = 0;
    p->cookie = plan_cookie(p);
    layout_workspace(p);
    // the fixed scratch of moc_chunk_pool_noalloc: its address is looked up here, where allocating is allowed
    if (int r = pool_scratch_prepare(dev)) { delete p; return r; }

    // one device blob
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    size_t o_off = take(4 * (C + 1)), o_shot = take(4 * C), o_mod = take(C), o_tok = take(4 * (size_t)L);
    size_t o_bits = take(4 * bits.size()), o_aoff = take(4 * (C + 1)), o_arng = take(sizeof(KeyRange) * p->anc_rng.size());
    size_t o_roff = take(4 * (C + 1)), o_ranc = take(4 * p->ranc.size()), o_qt = take(sizeof(WorkItem) * p->qitems.size());
    size_t o_puo = take(4 * (C + 1)), o_puc = take(4 * unit_chunk.size()), o_cap = take(4 * (C + 1)), o_crng = take(sizeof(KeyRange) * C), o_kt = take(sizeof(KTile) * p->ktiles.size());
    size_t o_shots = take(sizeof(KeyRange) * p->shot_chunks.size());
    size_t o_candc = take(4 * cand_c.size()), o_lim = take(4 * C), o_reach = take(4 * C), o_colc = take(4 * std::max<size_t>(col_chunk.size(), 1));
    cudaError_t e = cudaMalloc(&p->d_blob, o);
    if (e != cudaSuccess) { set_cuda_error(e, "cudaMalloc(plan tables)"); delete p; return MOC_ERR_CUDA; }
    char *b = static_cast<char *>(p->d_blob);
    auto up = [&](size_t at, const void *src, size_t bytes) {
        return bytes ? cudaMemcpy(b + at, src, bytes, cudaMemcpyHostToDevice) : cudaSuccess;
    };
    cudaError_t es[] = {up(o_off, p->off.data(), 4 * (C + 1)), up(o_shot, p->shot.data(), 4 * C), up(o_mod, p->mod.data(), C),
                        up(o_tok, tok_chunk.data(), 4 * (size_t)L), up(o_bits, bits.data(), 4 * bits.size()),
                        up(o_aoff, p->anc_off.data(), 4 * (C + 1)), up(o_arng, p->anc_rng.data(), sizeof(KeyRange) * p->anc_rng.size()),
                        up(o_roff, p->ranc_off.data(), 4 * (C + 1)), up(o_ranc, p->ranc.data(), 4 * p->ranc.size()),
                        up(o_qt, p->qitems.data(), sizeof(WorkItem) * p->qitems.size()),
                        up(o_puo, p->pool_unit_off.data(), 4 * (C + 1)), up(o_puc, unit_chunk.data(), 4 * unit_chunk.size()),
                        up(o_cap, p->cap_off.data(), 4 * (C + 1)), up(o_crng, chunk_rng.data(), sizeof(KeyRange) * C),
                        up(o_kt, p->ktiles.data(), sizeof(KTile) * p->ktiles.size()),
                        up(o_candc, cand_c.data(), 4 * cand_c.size()), up(o_lim, lim.data(), 4 * C), up(o_reach, reach.data(), 4 * C),
                        up(o_colc, col_chunk.data(), 4 * col_chunk.size()),
                        up(o_shots, p->shot_chunks.data(), sizeof(KeyRange) * p->shot_chunks.size())};
    for (cudaError_t x : es)
        if (x != cudaSuccess) { set_cuda_error(x, "cudaMemcpy(plan tables)"); cudaFree(p->d_blob); delete p; return MOC_ERR_CUDA; }
    p->d_off = (int32_t *)(b + o_off); p->d_shot = (int32_t *)(b + o_shot); p->d_mod = (uint8_t *)(b + o_mod);
    p->d_tok_chunk = (int32_t *)(b + o_tok); p->d_anc_bits = (uint32_t *)(b + o_bits);
    p->d_anc_off = (int32_t *)(b + o_aoff); p->d_anc_rng = (KeyRange *)(b + o_arng);
    p->d_ranc_off = (int32_t *)(b + o_roff); p->d_ranc = (int32_t *)(b + o_ranc); p->d_qitems = (WorkItem *)(b + o_qt);
    p->d_pool_unit_off = (int32_t *)(b + o_puo); p->d_pool_unit_chunk = (int32_t *)(b + o_puc);
    p->d_cap_off = (int32_t *)(b + o_cap);
    p->d_chunk_rng = (KeyRange *)(b + o_crng);
    p->d_ktiles = (KTile *)(b + o_kt);
    p->d_cand_c = (uint32_t *)(b + o_candc); p->d_lim = (int32_t *)(b + o_lim); p->d_reach = (int32_t *)(b + o_reach);
    p->d_col_chunk = (int32_t *)(b + o_colc);
    p->d_shot_chunks = (KeyRange *)(b + o_shots);
    *out = p;
    return MOC_OK;
}

extern "C" int moc_plan_destroy(moc_plan *p) {
    if (!p) return MOC_ERR_NULL;
    if (p->d_blob) cudaFree(p->d_blob);
    delete p;
    return MOC_OK;
}

extern "C" int moc_plan_set_workspace_budget(moc_plan *p, size_t max_bytes) {
    if (!p) return MOC_ERR_NULL;
    const size_t per_head = sizeof(__nv_bfloat16) * (((size_t)p->L + 127) / 128 * 128) * p->k * p->d;
    const size_t old = p->partials_budget;
    // the smallest workspace there is: one head at a time (two buffers of one head, or one if there is one head)
    p->partials_budget = p->H > 1 ? 2 * per_head : per_head;
    layout_workspace(p);
    const size_t rest = p->ws.fwd_end - p->partials_budget;
    if (p->ws.fwd_end > max_bytes) {
        p->partials_budget = old;
        layout_workspace(p);
        return MOC_ERR_TOO_LARGE;
    }
    p->partials_budget = std::max(p->partials_budget, max_bytes - rest - 65536);
    layout_workspace(p);
    if (p->ws.fwd_end > max_bytes) return MOC_ERR_TOO_LARGE;       // cannot happen: the partials only shrank
    return MOC_OK;
}

extern "C" int moc_workspace_bytes(const moc_plan *p, int with_bwd, size_t *bytes) {
    if (!p || !bytes) return MOC_ERR_NULL;
    *bytes = with_bwd ? p->ws.bwd_end : p->ws.fwd_end;
    return MOC_OK;
}

static int check_dev_ptrs(std::initializer_list<const void *> ptrs, size_t a) {
    for (const void *q : ptrs) {
        if (!q) return MOC_ERR_NULL;
        if (!aligned(q, a)) return MOC_ERR_ALIGN;
    }
    return MOC_OK;
}

static int enter(const moc_plan *p) {
    if (!p) return MOC_ERR_NULL;
    int dev = -1;
    MOC_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != p->device) return MOC_ERR_ARCH;
    return MOC_OK;
}

extern "C" int moc_chunk_pool(const moc_plan *p, const void *K, float *desc, void *ws, void *stream) {
    moc::NvtxRange nvtx_range("moc_chunk_pool");
    if (int r = enter(p)) return r;
    if (int r = check_dev_ptrs({K, desc}, 16)) return r;
    if (!ws) return MOC_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return MOC_ERR_ALIGN;
    return launch_chunk_pool(p, (const __nv_bfloat16 *)K, desc, ws, (cudaStream_t)stream);
}

extern "C" int moc_route(const moc_plan *p, const void *Q, const float *desc, int32_t *sel_idx, void *ws, void *stream) {
    moc::NvtxRange nvtx_range("moc_route");
    if (int r = enter(p)) return r;
    if (int r = check_dev_ptrs({Q, desc}, 16)) return r;
    if (p->k > 0) { if (int r = check_dev_ptrs({sel_idx}, 4)) return r; }
    if (!ws) return MOC_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return MOC_ERR_ALIGN;
    return launch_route(p, (const __nv_bfloat16 *)Q, desc, sel_idx, ws, (cudaStream_t)stream);
}

extern "C" int moc_lists_from_sel(const moc_plan *p, int32_t *sel_idx, void *ws, void *stream) {
    moc::NvtxRange nvtx_range("moc_lists_from_sel");
    if (int r = enter(p)) return r;
    if (p->k > 0) { if (int r = check_dev_ptrs({sel_idx}, 4)) return r; }
    if (!ws) return MOC_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return MOC_ERR_ALIGN;
    return launch_lists_from_sel(p, sel_idx, ws, (cudaStream_t)stream);
}

extern "C" int moc_context_drop(const moc_plan *p, int32_t *sel_idx, float p_max, float lambda, uint64_t seed, void *ws,
                                void *stream) {
    moc::NvtxRange nvtx_range("moc_context_drop");
    if (int r = enter(p)) return r;
    if (!(p_max >= 0.f && p_max <= 1.f) || !(lambda >= 0.f && lambda <= 8.f)) return MOC_ERR_SHAPE;
    if (p->k > 0) { if (int r = check_dev_ptrs({sel_idx}, 4)) return r; }
    if (!ws) return MOC_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return MOC_ERR_ALIGN;
    if (int r = launch_context_drop(p, sel_idx, p_max, lambda, seed, (cudaStream_t)stream)) return r;
    return launch_lists_from_sel(p, sel_idx, ws, (cudaStream_t)stream);
}

extern "C" int moc_attend(const moc_plan *p, const void *Q, const void *K, const void *V, const int32_t *sel_idx,
                          void *O, float *lse, void *ws, void *stream) {
    moc::NvtxRange nvtx_range("moc_attend");
    if (int r = enter(p)) return r;
    if (int r = check_dev_ptrs({Q, K, V, O}, 16)) return r;
    if (int r = check_dev_ptrs({lse}, 4)) return r;
    if (p->k > 0) { if (int r = check_dev_ptrs({sel_idx}, 4)) return r; }
    if (!ws) return MOC_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return MOC_ERR_ALIGN;
    auto q = (const __nv_bfloat16 *)Q, k = (const __nv_bfloat16 *)K, v = (const __nv_bfloat16 *)V;
    if (p->flags & kPrivFlagCudaCoreAttend)
        return launch_attend_scalar(p, q, k, v, sel_idx, (__nv_bfloat16 *)O, lse, ws, (cudaStream_t)stream);
    return launch_attend_tc(p, q, k, v, sel_idx, (__nv_bfloat16 *)O, lse, ws, (cudaStream_t)stream);
}

extern "C" int moc_attend_bwd(const moc_plan *p, const void *Q, const void *K, const void *V, const void *O,
                              const float *lse, const void *dO, const int32_t *sel_idx, void *dQ, void *dK, void *dV,
                              void *ws, void *stream) {
    moc::NvtxRange nvtx_range("moc_attend_bwd");
    if (int r = enter(p)) return r;
    if (int r = check_dev_ptrs({Q, K, V, O, dO, dQ, dK, dV}, 16)) return r;
    if (int r = check_dev_ptrs({lse}, 4)) return r;
    if (p->k > 0) { if (int r = check_dev_ptrs({sel_idx}, 4)) return r; }
    if (!ws) return MOC_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return MOC_ERR_ALIGN;
    auto bwd = (p->flags & kPrivFlagCudaCoreAttend) ? launch_attend_bwd_scalar : launch_attend_bwd_tc;
    return bwd(p, (const __nv_bfloat16 *)Q, (const __nv_bfloat16 *)K, (const __nv_bfloat16 *)V, (const __nv_bfloat16 *)O, lse,
               (const __nv_bfloat16 *)dO, sel_idx, (__nv_bfloat16 *)dQ, (__nv_bfloat16 *)dK, (__nv_bfloat16 *)dV, ws,
               (cudaStream_t)stream);
}

extern "C" int moc_selected_pairs(const moc_plan *p, const void *ws, void *stream, int64_t *pairs) {
    if (int r = enter(p)) return r;
    if (!pairs) return MOC_ERR_NULL;
    if (!ws) return MOC_ERR_WORKSPACE;
    std::vector<int32_t> cnt((size_t)p->H * p->C);
    MOC_CUDA_TRY(cudaMemcpyAsync(cnt.data(), ws_ptr<int32_t>(ws, p->ws.cnt), cnt.size() * 4, cudaMemcpyDeviceToHost,
                                 (cudaStream_t)stream));
    MOC_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    int64_t per_head = 0;
    for (int c = 0; c < p->C; ++c) per_head += p->anc_tokens[c] * (int64_t)(p->off[c + 1] - p->off[c]);
    int64_t total = per_head * p->H;
    for (int h = 0; h < p->H; ++h)
        for (int c = 0; c < p->C; ++c) total += (int64_t)cnt[(size_t)h * p->C + c] * (p->off[c + 1] - p->off[c]);
    *pairs = total;
    return MOC_OK;
}

extern "C" int moc_get_status(const moc_plan *p, const void *ws, void *stream, int *device_status, int *detail) {
    if (int r = enter(p)) return r;
    if (!device_status) return MOC_ERR_NULL;
    if (!ws) return MOC_ERR_WORKSPACE;
    int32_t st[2] = {0, 0};
    MOC_CUDA_TRY(cudaMemcpyAsync(st, ws_ptr<int32_t>(ws, p->ws.status), sizeof st, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    MOC_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    *device_status = st[0];
    if (detail) *detail = st[1];
    return MOC_OK;
}

extern "C" int moc_debug_use_cuda_core_attention(moc_plan *p, int on) {
    if (!p) return MOC_ERR_NULL;
    p->flags = on ? (p->flags | kPrivFlagCudaCoreAttend) : (p->flags & ~kPrivFlagCudaCoreAttend);
    return MOC_OK;
}

extern "C" int moc_debug_set_wait_limit_us(moc_plan *p, unsigned us) {
    if (!p) return MOC_ERR_NULL;
    p->wait_us = us;
    return MOC_OK;
}

extern "C" int64_t moc_launch_count(void) { return (int64_t)g_launches.load(); }

extern "C" const char *moc_strerror(int s) {
    switch (s) {
        case MOC_OK: return "ok";
        case MOC_ERR_NULL: return "a required pointer is NULL";
        case MOC_ERR_SHAPE: return "unsupported shape or parameter";
        case MOC_ERR_CHUNK_TABLE: return "invalid chunk table";
        case MOC_ERR_ALIGN: return "misaligned device pointer";
        case MOC_ERR_WORKSPACE: return "workspace missing, or it does not hold this plan's routing";
        case MOC_ERR_ARCH: return "device is not sm_100 or differs from the plan's device";
        case MOC_ERR_CUDA: return "CUDA runtime error";
        case MOC_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case MOC_ERR_TOO_LARGE: return "problem exceeds the fixed scratch of the no-allocation entry point, or the workspace budget";
        case MOC_ERR_INDEX: return "debug build: an index taken from the workspace was out of range";
        default: return "unknown status";
    }
}

extern "C" const char *moc_last_cuda_error(void) {
    static thread_local std::string copy;
    std::lock_guard<std::mutex> g(g_err_mu);
    copy = g_err;
    return copy.c_str();
}
