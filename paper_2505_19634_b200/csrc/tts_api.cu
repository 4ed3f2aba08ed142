// C-ABI layer: argument checks, context and workspace management, kernel launches, and the
// host-only helpers (answer aggregation, greedy search).  See include/tts.h for the contract.
#include <math.h>
#include <algorithm>
#include <new>
#include <vector>
#include <stdlib.h>
#include <string.h>

#include "attn_plan.cuh"
#include "tts_internal.cuh"

using namespace tts;

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int cuda_fail(Ctx* c, cudaError_t e) {
    if (c) c->last_cuda_error = (int)e;
    return TTS_ERR_CUDA;
}

// Row-block size and tile length the chosen kernel works with.
struct Plan { int impl, rb_rows, tile_tokens, grid, copies, copies_pre; };

Plan make_plan(const Ctx* c, int nr, int n_branches) {
    Plan pl;
    int impl = c->cfg.attn_impl;
    if (impl == TTS_ATTN_AUTO) impl = umma_available() && nr >= kUmmaMinRows ? TTS_ATTN_TCGEN05 : TTS_ATTN_SIMT;
    // few rows per KV head: KV tokens on the MMA M dimension; many (draft trees): query rows on M
    if (impl == TTS_ATTN_TCGEN05)
        impl = nr <= kUmmaTMaxRows ? TTS_ATTN_TCGEN05_TOKEN_MAJOR : TTS_ATTN_TCGEN05_ROW_MAJOR;
    pl.impl = impl;
    if (impl == TTS_ATTN_TCGEN05_TOKEN_MAJOR) {
        pl.rb_rows = umma_t_rows(nr); pl.tile_tokens = kUmmaTileTokens; pl.grid = c->n_sms;
        pl.copies = pl.copies_pre = kUmmaTGroups;
    } else if (impl == TTS_ATTN_TCGEN05_ROW_MAJOR) {
        pl.rb_rows = kUmmaRows; pl.tile_tokens = kUmmaTileTokens; pl.grid = c->n_sms;
        pl.copies = nr <= kUmmaRows ? umma_copies(nr) : 1; pl.copies_pre = 1;
    } else {
        pl.rb_rows = simt_rb_rows(nr); pl.tile_tokens = kSimtTileTokens; pl.grid = c->n_sms * 3;
        pl.copies = pl.copies_pre = 1;
    }
    if (c->cfg.max_ctas > 0 && pl.grid > c->cfg.max_ctas) pl.grid = c->cfg.max_ctas;
    return pl;
}

void free_workspace(Ctx* c) {
    cudaFree(c->part_o_pre); cudaFree(c->part_ml_pre); cudaFree(c->part_o_priv); cudaFree(c->part_ml_priv);
    cudaFree(c->group_desc); c->group_desc = nullptr;
    cudaFree(c->plan_cta); cudaFree(c->plan_pieces); c->plan_cta = nullptr; c->plan_pieces = nullptr;
    c->part_o_pre = c->part_o_priv = nullptr; c->part_ml_pre = c->part_ml_priv = nullptr;
    c->pre_rows = c->priv_rows = 0;
}

// Partial-result rows one call needs: every piece reserves min(rb_rows, rows of its segment kind).
void workspace_rows(int N, int Hkv, int nr, int rb_rows, int copies, int copies_pre, int grid, size_t* pre, size_t* priv) {
    const long n_rb_pre = ((long)N * nr + rb_rows - 1) / rb_rows;
    const long n_rb_priv = (nr + rb_rows - 1) / rb_rows;
    const long pre_stride = copies_pre * ((long)N * nr < rb_rows ? (long)N * nr : rb_rows);
    const long priv_stride = (long)copies * (nr < rb_rows ? nr : rb_rows);
    *pre = (size_t)(Hkv * n_rb_pre + grid) * pre_stride;
    *priv = (size_t)((long)N * Hkv * n_rb_priv + grid) * priv_stride;
}

// Workspace for the largest problem the config allows, whichever kernel a call ends up using.
cudaError_t alloc_workspace(Ctx* c) {
    const tts_config& f = c->cfg;
    const int G = f.n_q_heads / f.n_kv_heads;
    const int nr = f.max_rows_per_branch * G;
    size_t pre = 0, priv = 0;
    // every (row block, copies of private pieces, copies of prefix pieces) a call may run with; a call
    // may carry fewer rows than the maximum and the row-major kernel then replicates them more often
    struct Cand { int rb, copies, copies_pre, nr_cap; };
    const Cand cand[] = {{8, 1, 1, nr},  {16, 1, 1, nr}, {32, 1, 1, nr},                         // CUDA cores
                         {32, kUmmaTGroups, kUmmaTGroups, nr}, {64, kUmmaTGroups, kUmmaTGroups, nr},   // token-major
                         {kUmmaRows, 1, 1, nr}, {kUmmaRows, 2, 1, kUmmaRows / 2}, {kUmmaRows, 4, 1, kUmmaRows / 4}};
    for (const Cand& k : cand) {
        size_t a, b;
        workspace_rows(f.max_branches, f.n_kv_heads, nr < k.nr_cap ? nr : k.nr_cap, k.rb, k.copies, k.copies_pre,
                       c->n_sms * 3, &a, &b);
        pre = a > pre ? a : pre; priv = b > priv ? b : priv;
    }
    // several prefix sets per call (token-major kernel): up to one more prefix row block per set and KV head
    pre += (size_t)kMaxPrefixSets * f.n_kv_heads * umma_t_rows(nr);
    cudaError_t e;
    if ((e = cudaMalloc(&c->part_o_pre, pre * kHeadDim * sizeof(float))) != cudaSuccess) return e;
    if ((e = cudaMalloc(&c->part_ml_pre, pre * sizeof(float2))) != cudaSuccess) return e;
    if ((e = cudaMalloc(&c->part_o_priv, priv * kHeadDim * sizeof(float))) != cudaSuccess) return e;
    if ((e = cudaMalloc(&c->part_ml_priv, priv * sizeof(float2))) != cudaSuccess) return e;
    c->pre_rows = pre; c->priv_rows = priv;
    if ((e = cudaMalloc(&c->group_desc, (size_t)f.max_branches * f.n_kv_heads * 64)) != cudaSuccess) return e;   // a GroupDesc is at most 64 bytes
    // plan of the token-major kernel (row blocks of 32 rows): one piece per segment and one more per CTA
    const size_t rb = (size_t)umma_t_rows(nr);
    const size_t n_seg = (size_t)f.max_branches * f.n_kv_heads * ((nr + rb - 1) / rb) +
                         (size_t)f.n_kv_heads * (((size_t)f.max_branches * nr + rb - 1) / rb);
    c->plan_pieces_cap = n_seg + (size_t)kMaxPrefixSets * f.n_kv_heads + (size_t)c->n_sms;
    if ((e = cudaMalloc(&c->plan_cta, (size_t)c->n_sms * sizeof(CtaPlan))) != cudaSuccess) return e;
    return cudaMalloc(&c->plan_pieces, c->plan_pieces_cap * sizeof(PieceDesc));
}

// Checks the arguments that describe the schedule of an attention call and fills the parameters that
// depend on them (everything but q, K/V and out).  With several prefix sets the parameters describe the call
// as a whole (p.P, p.n_pre and p.tiles_pre are then those of the first set and only the plan uses the rest).
int attn_setup(Ctx* c, const int32_t* block_table, const PrefixSets& sets, const int32_t* branch_lens,
               const int32_t* tree_parents, int n_branches, int rows, AttnParams* out_p, Plan* out_pl) {
    if (!c || !block_table || !branch_lens) return TTS_ERR_INVALID;
    const tts_config& f = c->cfg;
    if (n_branches < 1 || n_branches > f.max_branches) return TTS_ERR_INVALID;
    if (rows < 1 || rows > f.max_rows_per_branch) return TTS_ERR_INVALID;
    if (rows > kMaxTreeRows) return TTS_ERR_UNSUPPORTED;
    if (sets.n_sets < 1 || sets.n_sets > kMaxPrefixSets || sets.first_branch[0] != 0 || sets.first_branch[sets.n_sets] != n_branches)
        return TTS_ERR_INVALID;
    int max_set = 0;
    for (int s = 0; s < sets.n_sets; ++s) {
        const int prefix_len = sets.prefix_len[s], size = sets.first_branch[s + 1] - sets.first_branch[s];
        if (size < 1) return TTS_ERR_INVALID;
        if (prefix_len < 0 || prefix_len % f.page_size != 0) return TTS_ERR_INVALID;
        if (prefix_len / f.page_size > f.max_blocks_per_branch) return TTS_ERR_INVALID;
        max_set = size > max_set ? size : max_set;
    }
    if ((reinterpret_cast<uintptr_t>(block_table) & 3u) || (reinterpret_cast<uintptr_t>(branch_lens) & 3u)) return TTS_ERR_INVALID;

    const int G = f.n_q_heads / f.n_kv_heads;
    const int nr = rows * G;
    const Plan pl = make_plan(c, nr, n_branches);
    const int pre_stride = pl.copies_pre * (max_set * nr < pl.rb_rows ? max_set * nr : pl.rb_rows);
    {
        // prefix partial results: one slot per prefix segment of every set and one more per CTA
        long n_pre_seg = 0;
        for (int s = 0; s < sets.n_sets; ++s)
            if (sets.prefix_len[s] > 0)
                n_pre_seg += (long)f.n_kv_heads * (((long)(sets.first_branch[s + 1] - sets.first_branch[s]) * nr + pl.rb_rows - 1) / pl.rb_rows);
        size_t need_pre, need_priv;
        workspace_rows(n_branches, f.n_kv_heads, nr, pl.rb_rows, pl.copies, pl.copies_pre, pl.grid, &need_pre, &need_priv);
        need_pre = (size_t)(n_pre_seg + pl.grid) * pre_stride;
        if (need_pre > c->pre_rows || need_priv > c->priv_rows) return TTS_ERR_INVALID;
    }
    AttnParams& p = *out_p;
    memset(&p, 0, sizeof p);
    p.block_table = block_table; p.branch_lens = branch_lens; p.tree_parents = tree_parents;
    p.part_o_pre = c->part_o_pre; p.part_ml_pre = c->part_ml_pre;
    p.part_o_priv = c->part_o_priv; p.part_ml_priv = c->part_ml_priv;
    p.status = c->d_status;
    // the token-major kernel and its merge kernel run from the plan tables
    if (pl.impl == TTS_ATTN_TCGEN05_TOKEN_MAJOR) { p.group_desc = c->group_desc; p.plan_cta = c->plan_cta; p.plan_pieces = c->plan_pieces; }
    p.N = n_branches; p.R = rows; p.Hq = f.n_q_heads; p.Hkv = f.n_kv_heads; p.G = G; p.nr = nr;
    p.P = sets.prefix_len[0]; p.max_blocks = f.max_blocks_per_branch; p.num_pages = f.num_pages;
    p.rb_rows = pl.rb_rows;
    p.pre_stride = pre_stride;
    p.priv_stride = pl.copies * (nr < pl.rb_rows ? nr : pl.rb_rows);
    p.copies = pl.copies; p.copies_pre = pl.copies_pre;
    p.n_rb_pre = ceil_div(n_branches * nr, pl.rb_rows);
    p.n_rb_priv = ceil_div(nr, pl.rb_rows);
    p.n_pre = p.P > 0 ? f.n_kv_heads * p.n_rb_pre : 0;
    if ((long long)n_branches * f.n_kv_heads * f.n_kv_heads * p.n_rb_pre >= (1ll << 31)) return TTS_ERR_UNSUPPORTED;
    p.tile_tokens = pl.tile_tokens;
    p.tiles_pre = ceil_div(p.P, pl.tile_tokens);
    p.grid = pl.grid;
    p.out_dtype = f.out_dtype; p.debug = f.debug_bounds;
    const float scale = f.softmax_scale > 0.f ? f.softmax_scale : 1.0f / sqrtf((float)f.head_dim);
    p.scale_log2 = scale * 1.4426950408889634f;
    *out_pl = pl;
    return TTS_OK;
}

PrefixSets one_set(int prefix_len, int n_branches) {
    PrefixSets sets;
    memset(&sets, 0, sizeof sets);
    sets.n_sets = 1; sets.first_branch[1] = n_branches; sets.prefix_len[0] = prefix_len;
    return sets;
}

// group_sizes / group_prefix_len (host arrays) as prefix sets; false when they are not a valid description
bool sets_from_groups(const int32_t* group_sizes, const int32_t* group_prefix_len, int n_groups, int n_branches, PrefixSets* sets) {
    if (!group_sizes || !group_prefix_len || n_groups < 1 || n_groups > kMaxPrefixSets) return false;
    memset(sets, 0, sizeof *sets);
    sets->n_sets = n_groups;
    long first = 0;
    for (int g = 0; g < n_groups; ++g) {
        if (group_sizes[g] < 1) return false;
        sets->first_branch[g] = (int)first;
        sets->prefix_len[g] = group_prefix_len[g];
        first += group_sizes[g];
        if (first > n_branches) return false;
    }
    sets->first_branch[n_groups] = (int)first;
    return first == n_branches;
}

bool same_sets(const PrefixSets& a, const PrefixSets& b) {
    return a.n_sets == b.n_sets && memcmp(a.first_branch, b.first_branch, sizeof(int) * (a.n_sets + 1)) == 0 &&
           memcmp(a.prefix_len, b.prefix_len, sizeof(int) * a.n_sets) == 0;
}

// Does the plan in the context's tables, built by tts_attn_plan, describe this call?
bool plan_matches(const Ctx* c, const int32_t* block_table, const PrefixSets& sets, const int32_t* branch_lens, int n_branches, int rows) {
    return c->plan_explicit && c->plan_key.block_table == block_table && c->plan_key.branch_lens == branch_lens &&
           c->plan_key.n_branches == n_branches && c->plan_key.rows == rows && same_sets(c->plan_key.sets, sets);
}

int attn_common(Ctx* c, const void* q, const void* k_pages, const void* v_pages,
                const int32_t* block_table, const PrefixSets& sets, const int32_t* branch_lens,
                const int32_t* tree_parents, int n_branches, int rows, void* out) {
    if (!c || !q || !k_pages || !v_pages || !out) return TTS_ERR_INVALID;
    if (!aligned16(q) || !aligned16(k_pages) || !aligned16(v_pages) || !aligned16(out)) return TTS_ERR_INVALID;
    AttnParams p;
    Plan pl;
    const int rc = attn_setup(c, block_table, sets, branch_lens, tree_parents, n_branches, rows, &p, &pl);
    if (rc != TTS_OK) return rc;
    if (sets.n_sets > 1 && pl.impl != TTS_ATTN_TCGEN05_TOKEN_MAJOR) {
        // the other kernels take one prefix per launch: set by set, on the rows, table rows and lengths of each
        const size_t row_elts = (size_t)rows * c->cfg.n_q_heads * kHeadDim;
        const size_t out_elt = c->cfg.out_dtype == TTS_OUT_FP32 ? 4 : 2;
        for (int s = 0; s < sets.n_sets; ++s) {
            const int b0 = sets.first_branch[s], n = sets.first_branch[s + 1] - b0;
            const int rc_s = attn_common(c, static_cast<const char*>(q) + b0 * row_elts * 2, k_pages, v_pages,
                                         block_table + (size_t)b0 * c->cfg.max_blocks_per_branch, one_set(sets.prefix_len[s], n),
                                         branch_lens + b0, tree_parents ? tree_parents + (size_t)b0 * rows : nullptr, n, rows,
                                         static_cast<char*>(out) + b0 * row_elts * out_elt);
            if (rc_s != TTS_OK) return rc_s;
        }
        return TTS_OK;
    }
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k_pages = static_cast<const __nv_bfloat16*>(k_pages);
    p.v_pages = static_cast<const __nv_bfloat16*>(v_pages);
    p.out = out;
    cudaError_t e;

    if (pl.impl == TTS_ATTN_TCGEN05_TOKEN_MAJOR && !plan_matches(c, block_table, sets, branch_lens, n_branches, rows)) {
        // no plan from tts_attn_plan for these arguments: build one for this call alone
        c->plan_explicit = 0;
        e = launch_attn_plan(p, sets, c->stream);
        if (e != cudaSuccess) return cuda_fail(c, e);
        c->launches += 1;
    }
    const bool prof = c->profiling && c->prof_ev && c->prof_n < kProfMaxCalls;
    cudaEvent_t* ev = prof ? c->prof_ev + 3 * c->prof_n : nullptr;
    // inside a stream capture the events become event-record nodes of the graph: every replay records them
    cudaStreamCaptureStatus capture = cudaStreamCaptureStatusNone;
    if (prof) cudaStreamIsCapturing(c->stream, &capture);
    auto record = [&](cudaEvent_t event) {
        if (capture == cudaStreamCaptureStatusActive) cudaEventRecordWithFlags(event, c->stream, cudaEventRecordExternal);
        else cudaEventRecord(event, c->stream);
    };
    if (prof) record(ev[0]);
    if (pl.impl == TTS_ATTN_TCGEN05_TOKEN_MAJOR) {
        e = launch_attn_umma_t(c, p, c->stream);
    } else if (pl.impl == TTS_ATTN_TCGEN05_ROW_MAJOR) {
        if (!umma_available()) return TTS_ERR_UNSUPPORTED;
        e = launch_attn_umma(c, p, c->stream);
    } else {
        e = launch_attn_simt(p, c->stream);
    }
    if (e != cudaSuccess) return cuda_fail(c, e);
    c->launches += 1;
    if (prof) record(ev[1]);
    e = launch_attn_combine(p, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e);
    c->launches += 1;
    if (prof) { record(ev[2]); c->prof_n += 1; }
    return TTS_OK;
}

int plan_common(Ctx* c, const int32_t* block_table, const PrefixSets& sets, const int32_t* branch_lens, int n_branches, int rows) {
    AttnParams p;
    Plan pl;
    const int rc = attn_setup(c, block_table, sets, branch_lens, nullptr, n_branches, rows, &p, &pl);
    if (rc != TTS_OK) return rc;
    c->plan_explicit = 0;
    if (pl.impl != TTS_ATTN_TCGEN05_TOKEN_MAJOR) return TTS_OK;      // the other kernels derive their schedule themselves
    const cudaError_t e = launch_attn_plan(p, sets, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e);
    c->launches += 1;
    c->plan_key.block_table = block_table; c->plan_key.branch_lens = branch_lens;
    c->plan_key.n_branches = n_branches; c->plan_key.rows = rows; c->plan_key.sets = sets;
    c->plan_explicit = 1;
    return TTS_OK;
}

}  // namespace

extern "C" {

int tts_create(const tts_config* cfg, tts_ctx** out) {
    if (!cfg || !out) return TTS_ERR_INVALID;
    *out = nullptr;
    if (cfg->head_dim != kHeadDim || cfg->page_size != kPage) return TTS_ERR_UNSUPPORTED;
    if (cfg->n_q_heads < 1 || cfg->n_kv_heads < 1 || cfg->n_q_heads % cfg->n_kv_heads != 0) return TTS_ERR_INVALID;
    if (cfg->max_branches < 1 || cfg->max_branches > kMaxBranches) return TTS_ERR_INVALID;
    if (cfg->max_rows_per_branch < 1 || cfg->max_rows_per_branch > kMaxTreeRows) return TTS_ERR_INVALID;
    if (cfg->max_blocks_per_branch < 1 || cfg->num_pages < 1) return TTS_ERR_INVALID;
    if (cfg->out_dtype != TTS_OUT_BF16 && cfg->out_dtype != TTS_OUT_FP32) return TTS_ERR_UNSUPPORTED;
    if (cfg->attn_impl < TTS_ATTN_AUTO || cfg->attn_impl > TTS_ATTN_TCGEN05_ROW_MAJOR) return TTS_ERR_UNSUPPORTED;
    if (!(cfg->softmax_scale >= 0.f) || cfg->max_ctas < 0) return TTS_ERR_INVALID;

    Ctx* c = new (std::nothrow) Ctx();
    if (!c) return TTS_ERR_INVALID;
    memset(c, 0, sizeof *c);
    c->cfg = *cfg;
    cudaError_t e = cudaGetDevice(&c->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->n_sms, cudaDevAttrMultiProcessorCount, c->device);
    if (e == cudaSuccess) e = cudaMalloc(&c->d_status, sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(c->d_status, 0, sizeof(int32_t));
    if (e == cudaSuccess) e = alloc_workspace(c);
    if (e != cudaSuccess) {
        free_workspace(c);
        cudaFree(c->d_status);
        delete c;
        return TTS_ERR_CUDA;
    }
    *out = reinterpret_cast<tts_ctx*>(c);
    return TTS_OK;
}

int tts_destroy(tts_ctx* ctx) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c) return TTS_ERR_INVALID;
    free_workspace(c);
    cudaFree(c->d_status);
    cudaFree(c->stage);
    if (c->host_ev) {
        for (int i = 0; i < kHostEvents; ++i) if (c->host_ev[i]) cudaEventDestroy(c->host_ev[i]);
        free(c->host_ev);
    }
    if (c->h2d_stream) cudaStreamDestroy(c->h2d_stream);
    if (c->d2h_stream) cudaStreamDestroy(c->d2h_stream);
    if (c->prof_ev) {
        for (int i = 0; i < 3 * kProfMaxCalls; ++i) if (c->prof_ev[i]) cudaEventDestroy(c->prof_ev[i]);
        free(c->prof_ev);
    }
    umma_release(c);
    delete c;
    return TTS_OK;
}

int tts_set_stream(tts_ctx* ctx, void* cuda_stream) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c) return TTS_ERR_INVALID;
    c->stream = static_cast<cudaStream_t>(cuda_stream);
    return TTS_OK;
}

int tts_verify_attn(tts_ctx* ctx, const void* q, const void* k_pages, const void* v_pages,
                    const int32_t* block_table, int prefix_len, const int32_t* branch_lens,
                    int n_branches, int gamma, int mask_kind, void* out) {
    if (mask_kind == TTS_MASK_TREE) return TTS_ERR_UNSUPPORTED;     // needs parents: tts_verify_attn_tree
    if (mask_kind != TTS_MASK_CAUSAL) return TTS_ERR_UNSUPPORTED;
    if (gamma < 0) return TTS_ERR_INVALID;
    return attn_common(reinterpret_cast<Ctx*>(ctx), q, k_pages, v_pages, block_table, one_set(prefix_len, n_branches),
                       branch_lens, nullptr, n_branches, gamma + 1, out);
}

int tts_verify_attn_groups(tts_ctx* ctx, const void* q, const void* k_pages, const void* v_pages,
                           const int32_t* block_table, const int32_t* group_sizes, const int32_t* group_prefix_len,
                           int n_groups, const int32_t* branch_lens, int n_branches, int gamma, void* out) {
    PrefixSets sets;
    if (gamma < 0 || !sets_from_groups(group_sizes, group_prefix_len, n_groups, n_branches, &sets)) return TTS_ERR_INVALID;
    return attn_common(reinterpret_cast<Ctx*>(ctx), q, k_pages, v_pages, block_table, sets, branch_lens, nullptr,
                       n_branches, gamma + 1, out);
}

int tts_verify_attn_tree(tts_ctx* ctx, const void* q, const void* k_pages, const void* v_pages,
                         const int32_t* block_table, int prefix_len, const int32_t* branch_lens,
                         const int32_t* tree_parents, int n_branches, int n_nodes, void* out) {
    if (!tree_parents) return TTS_ERR_INVALID;
    return attn_common(reinterpret_cast<Ctx*>(ctx), q, k_pages, v_pages, block_table, one_set(prefix_len, n_branches),
                       branch_lens, tree_parents, n_branches, n_nodes, out);
}

int tts_attn_plan(tts_ctx* ctx, const int32_t* block_table, int prefix_len, const int32_t* branch_lens,
                  int n_branches, int rows_per_branch) {
    return plan_common(reinterpret_cast<Ctx*>(ctx), block_table, one_set(prefix_len, n_branches), branch_lens, n_branches,
                       rows_per_branch);
}

int tts_attn_plan_groups(tts_ctx* ctx, const int32_t* block_table, const int32_t* group_sizes,
                         const int32_t* group_prefix_len, int n_groups, const int32_t* branch_lens, int n_branches,
                         int rows_per_branch) {
    PrefixSets sets;
    if (!sets_from_groups(group_sizes, group_prefix_len, n_groups, n_branches, &sets)) return TTS_ERR_INVALID;
    return plan_common(reinterpret_cast<Ctx*>(ctx), block_table, sets, branch_lens, n_branches, rows_per_branch);
}

int tts_attn_plan_drop(tts_ctx* ctx) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c) return TTS_ERR_INVALID;
    c->plan_explicit = 0;
    return TTS_OK;
}

int tts_accept(tts_ctx* ctx, const float* p_target, const float* q_draft, const int32_t* draft_tokens,
               const float* uniforms, int n_branches, int gamma, int vocab, int32_t* accepted_len,
               int32_t* next_token) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c || !p_target || !uniforms || !accepted_len || !next_token) return TTS_ERR_INVALID;
    if (gamma < 0 || n_branches < 1) return TTS_ERR_INVALID;
    if (gamma > 0 && (!q_draft || !draft_tokens)) return TTS_ERR_INVALID;
    if (vocab < 4 || vocab % 4 != 0 || vocab > 524288) return TTS_ERR_INVALID;
    if (!aligned16(p_target) || (q_draft && !aligned16(q_draft))) return TTS_ERR_INVALID;
    cudaError_t e = launch_accept(p_target, q_draft, draft_tokens, uniforms, n_branches, gamma, vocab,
                                  accepted_len, next_token, c->d_status, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e);
    c->launches += 1;
    return TTS_OK;
}

int tts_accept_logits(tts_ctx* ctx, const void* target_logits, const void* draft_logits, int logits_dtype,
                      const int32_t* draft_tokens, const float* uniforms, int n_branches, int gamma, int vocab,
                      int32_t* accepted_len, int32_t* next_token) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c || !target_logits || !uniforms || !accepted_len || !next_token) return TTS_ERR_INVALID;
    if (logits_dtype != TTS_LOGITS_BF16 && logits_dtype != TTS_LOGITS_FP32) return TTS_ERR_UNSUPPORTED;
    if (gamma < 0 || n_branches < 1) return TTS_ERR_INVALID;
    if (gamma > 0 && (!draft_logits || !draft_tokens)) return TTS_ERR_INVALID;
    if (vocab < 4 || vocab % 4 != 0 || vocab > 524288) return TTS_ERR_INVALID;
    if (!aligned16(target_logits) || (draft_logits && !aligned16(draft_logits))) return TTS_ERR_INVALID;
    cudaError_t e = launch_accept_logits(target_logits, draft_logits, logits_dtype, draft_tokens, uniforms, n_branches,
                                         gamma, vocab, accepted_len, next_token, c->d_status, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e);
    c->launches += 1;
    return TTS_OK;
}

int tts_accept_tree(tts_ctx* ctx, const float* p_target, const float* q_draft, const int32_t* draft_tokens,
                    const int32_t* tree_parents, const float* uniforms, int n_branches, int n_nodes, int vocab,
                    int32_t* accepted_len, int32_t* last_node, int32_t* next_token) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c || !p_target || !uniforms || !accepted_len || !last_node || !next_token) return TTS_ERR_INVALID;
    if (n_nodes < 0 || n_nodes > kMaxTreeRows || n_branches < 1) return TTS_ERR_INVALID;
    if (n_nodes > 0 && (!q_draft || !draft_tokens || !tree_parents)) return TTS_ERR_INVALID;
    if (vocab < 4 || vocab % 4 != 0 || vocab > 524288) return TTS_ERR_INVALID;
    if (!aligned16(p_target) || (q_draft && !aligned16(q_draft))) return TTS_ERR_INVALID;
    cudaError_t e = launch_accept_tree(p_target, q_draft, draft_tokens, tree_parents, uniforms, n_branches, n_nodes,
                                       vocab, accepted_len, last_node, next_token, c->d_status, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e);
    c->launches += 1;
    return TTS_OK;
}

int tts_kv_append(tts_ctx* ctx, const void* k_new, const void* v_new, void* k_pages, void* v_pages,
                  const int32_t* block_table, int prefix_len, const int32_t* branch_lens, int n_branches, int rows) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c || !k_new || !v_new || !k_pages || !v_pages || !block_table || !branch_lens) return TTS_ERR_INVALID;
    const tts_config& f = c->cfg;
    if (n_branches < 1 || n_branches > f.max_branches || rows < 1 || rows > f.max_rows_per_branch) return TTS_ERR_INVALID;
    if (prefix_len < 0 || prefix_len % f.page_size != 0 || prefix_len / f.page_size > f.max_blocks_per_branch)
        return TTS_ERR_INVALID;
    if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_pages) || !aligned16(v_pages)) return TTS_ERR_INVALID;
    cudaError_t e = launch_kv_append(k_new, v_new, k_pages, v_pages, block_table, f.max_blocks_per_branch, f.num_pages,
                                     prefix_len, branch_lens, n_branches, rows, f.n_kv_heads, c->d_status, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e);
    c->launches += 1;
    return TTS_OK;
}

int tts_kv_rollback(tts_ctx* ctx, int32_t* branch_lens, const int32_t* accepted_len, int n_branches, int gamma) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c || !branch_lens || !accepted_len) return TTS_ERR_INVALID;
    if (n_branches < 1 || n_branches > c->cfg.max_branches || gamma < 0) return TTS_ERR_INVALID;
    if (c->plan_explicit && c->plan_key.branch_lens == branch_lens) c->plan_explicit = 0;   // the lengths change
    cudaError_t e = launch_kv_rollback(branch_lens, accepted_len, n_branches, gamma, c->d_status, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e);
    c->launches += 1;
    return TTS_OK;
}

// Answer aggregation.  The branches are ordered by (answer, branch index); every run of equal answers
// is one candidate whose score is its number of branches or the sum of their weights (added in branch
// order, fp64); the best score wins and equal scores go to the run that starts at the lowest branch.
static int aggregate_votes(const int64_t* answers, const float* weights, int n, int64_t* winner, int* votes) {
    if (!answers || !winner || n < 1) return TTS_ERR_INVALID;
    std::vector<int> order(n);
    for (int i = 0; i < n; ++i) order[i] = i;
    std::sort(order.begin(), order.end(), [&](int a, int b) {
        return answers[a] != answers[b] ? answers[a] < answers[b] : a < b;
    });
    int win_first = -1, win_count = 0;
    double win_score = 0.0;
    for (int lo = 0; lo < n;) {
        int hi = lo;
        double score = 0.0;
        while (hi < n && answers[order[hi]] == answers[order[lo]]) {
            score += weights ? (double)weights[order[hi]] : 1.0;
            ++hi;
        }
        const int first = order[lo];                      // lowest branch index of the run
        if (win_first < 0 || score > win_score || (score == win_score && first < win_first)) {
            win_first = first; win_score = score; win_count = hi - lo;
        }
        lo = hi;
    }
    *winner = answers[win_first];
    if (votes) *votes = win_count;
    return TTS_OK;
}

int tts_majority_vote(const int64_t* answers, const float* weights, int n, int64_t* winner, int* votes) {
    return aggregate_votes(answers, weights, n, winner, votes);
}

int tts_confidence_max(const int64_t* answers, const float* weights, int n, int64_t* winner, int* votes) {
    if (!answers || !weights || !winner || n < 1) return TTS_ERR_INVALID;
    const float* top = std::max_element(weights, weights + n);      // the first of equal maxima
    *winner = answers[top - weights];
    if (votes) *votes = (int)std::count(answers, answers + n, *winner);
    return TTS_OK;
}

// (B, gamma) search.  A configuration is a point of the lattice B = 1, 2, 4, .. <= max_branches,
// gamma = 0 .. max_gamma; the caller's task function scores it (negative = not available).
namespace {

struct SearchBox { int max_branches, max_gamma, max_steps; };

bool search_box(const tts_search_limits* lim, SearchBox* box) {
    box->max_branches = lim ? lim->max_branches : 64;
    box->max_gamma = lim ? lim->max_gamma : 7;
    box->max_steps = lim && lim->max_steps > 0 ? lim->max_steps : 64;
    return box->max_branches >= 1 && box->max_branches <= (1 << 20) && box->max_gamma >= 0 && box->max_gamma <= 4096;
}

struct Move { int branch_factor, gamma_step; };
// Candidate moves in order of preference among equals: more branches first, then a longer draft.
const Move kMoves[] = {{2, 0}, {1, 1}};

}  // namespace

int tts_greedy_search(tts_task_fn tts_task, void* user, const tts_search_limits* limits, int* best_branches,
                      int* best_gamma, double* best_acc, int* steps, int* evaluations) {
    SearchBox box;
    if (!tts_task || !best_branches || !best_gamma || !search_box(limits, &box)) return TTS_ERR_INVALID;
    int at_b = 1, at_g = 0, n_steps = 0, n_eval = 1;
    double at_acc = tts_task(at_b, at_g, user);
    while (n_steps < box.max_steps) {
        ++n_steps;
        int to_b = 0, to_g = 0;
        double to_acc = -1.0;
        for (const Move& mv : kMoves) {
            const int b = at_b * mv.branch_factor, g = at_g + mv.gamma_step;
            if (b > box.max_branches || g > box.max_gamma) continue;      // outside the lattice: not evaluated
            const double a = tts_task(b, g, user);
            ++n_eval;
            if (a >= 0.0 && a > to_acc) { to_b = b; to_g = g; to_acc = a; }
        }
        if (!(to_acc > at_acc)) break;                                    // no neighbour improves: local optimum
        at_b = to_b; at_g = to_g; at_acc = to_acc;
    }
    *best_branches = at_b; *best_gamma = at_g;
    if (best_acc) *best_acc = at_acc;
    if (steps) *steps = n_steps;
    if (evaluations) *evaluations = n_eval;
    return TTS_OK;
}

int tts_grid_search(tts_task_fn tts_task, void* user, const tts_search_limits* limits, int* best_branches,
                    int* best_gamma, double* best_acc, int* evaluations) {
    SearchBox box;
    if (!tts_task || !best_branches || !best_gamma || !search_box(limits, &box)) return TTS_ERR_INVALID;
    int win_b = 1, win_g = 0, n_eval = 0;
    double win_acc = -1.0;
    for (int b = 1; b <= box.max_branches; b *= 2)
        for (int g = 0; g <= box.max_gamma; ++g) {
            const double a = tts_task(b, g, user);
            ++n_eval;
            if (a >= 0.0 && a > win_acc) { win_b = b; win_g = g; win_acc = a; }   // first of equal optima in (B, gamma) order
        }
    *best_branches = win_b; *best_gamma = win_g;
    if (best_acc) *best_acc = win_acc;
    if (evaluations) *evaluations = n_eval;
    return TTS_OK;
}

int tts_last_status(tts_ctx* ctx, int* device_status) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c || !device_status) return TTS_ERR_INVALID;
    int32_t h = 0;
    cudaError_t e = cudaMemcpyAsync(&h, c->d_status, sizeof h, cudaMemcpyDeviceToHost, c->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->d_status, 0, sizeof h, c->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e);
    *device_status = h;
    return TTS_OK;
}

int tts_debug_wait_timeout(tts_ctx* ctx, int64_t limit_ns) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c || limit_ns < 1000 || limit_ns > 1000ll * 1000 * 1000) return TTS_ERR_INVALID;
    const cudaError_t e = launch_wait_probe(c->d_status, limit_ns, nullptr, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e);
    c->launches += 1;
    return TTS_OK;
}

int tts_profile_enable(tts_ctx* ctx, int on) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c) return TTS_ERR_INVALID;
    if (on && !c->prof_ev) {
        c->prof_ev = static_cast<cudaEvent_t*>(calloc(3 * kProfMaxCalls, sizeof(cudaEvent_t)));
        if (!c->prof_ev) return TTS_ERR_INVALID;
        for (int i = 0; i < 3 * kProfMaxCalls; ++i) {
            cudaError_t e = cudaEventCreate(&c->prof_ev[i]);
            if (e != cudaSuccess) return cuda_fail(c, e);
        }
    }
    c->profiling = on ? 1 : 0;
    c->prof_n = 0;
    return TTS_OK;
}

int tts_profile_read(tts_ctx* ctx, float* attn_main_us, float* attn_merge_us, int* n_calls) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c || !attn_main_us || !attn_merge_us || !n_calls) return TTS_ERR_INVALID;
    cudaError_t e = cudaStreamSynchronize(c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e);
    double a = 0.0, b = 0.0;
    for (int i = 0; i < c->prof_n; ++i) {
        float ms = 0.f;
        cudaEventElapsedTime(&ms, c->prof_ev[3 * i], c->prof_ev[3 * i + 1]); a += ms;
        cudaEventElapsedTime(&ms, c->prof_ev[3 * i + 1], c->prof_ev[3 * i + 2]); b += ms;
    }
    *n_calls = c->prof_n;
    *attn_main_us = c->prof_n ? (float)(a * 1e3 / c->prof_n) : 0.f;
    *attn_merge_us = c->prof_n ? (float)(b * 1e3 / c->prof_n) : 0.f;
    c->prof_n = 0;
    return TTS_OK;
}

int tts_last_cuda_error(tts_ctx* ctx) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    return c ? c->last_cuda_error : 0;
}

int64_t tts_launch_count(tts_ctx* ctx) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    return c ? c->launches : 0;
}

const char* tts_strerror(int status) {
    switch (status) {
        case TTS_OK: return "ok";
        case TTS_ERR_INVALID: return "invalid argument";
        case TTS_ERR_UNSUPPORTED: return "unsupported configuration";
        case TTS_ERR_CUDA: return "CUDA call failed";
        case TTS_ERR_DEVICE_BOUNDS: return "device-side bounds check failed";
        case TTS_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        case TTS_ERR_SCRATCH: return "problem exceeds the fixed scratch array of the no-allocation entry point";
        default: return "unknown status";
    }
}

}  // extern "C"

namespace {

// The end-to-end step from host buffers.  dist_elt: bytes per element of the two distribution tensors (4: fp32
// probabilities or logits, 2: bf16 logits); logits_dtype < 0: they are probabilities.
int step_host(tts_ctx* ctx, int n_layers, const void* q_host, const void* const* k_pools,
              const void* const* v_pools, const int32_t* block_table_host, int prefix_len,
              const int32_t* branch_lens_host, int n_branches, int gamma,
              const void* p_target_host, const void* q_draft_host, int logits_dtype,
              const int32_t* draft_tokens_host, const float* uniforms_host, int vocab,
              void* out_host, int32_t* accepted_len_host, int32_t* next_token_host) {
    const size_t dist_elt = logits_dtype == TTS_LOGITS_BF16 ? 2 : 4;
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c || n_layers < 1 || !q_host || !k_pools || !v_pools || !block_table_host || !branch_lens_host ||
        !p_target_host || !uniforms_host || !out_host || !accepted_len_host || !next_token_host)
        return TTS_ERR_INVALID;
    if (gamma < 0 || (gamma > 0 && (!q_draft_host || !draft_tokens_host))) return TTS_ERR_INVALID;
    if (n_branches < 1 || n_branches > c->cfg.max_branches || gamma + 1 > c->cfg.max_rows_per_branch)
        return TTS_ERR_INVALID;
    if (vocab < 4 || vocab % 4 != 0) return TTS_ERR_INVALID;
    const tts_config& f = c->cfg;
    const size_t out_elt = f.out_dtype == TTS_OUT_FP32 ? 4 : 2;
    const size_t q_layer = (size_t)n_branches * (gamma + 1) * f.n_q_heads * kHeadDim * 2;
    const size_t o_layer = (size_t)n_branches * (gamma + 1) * f.n_q_heads * kHeadDim * out_elt;
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    const size_t bt_b = up((size_t)n_branches * f.max_blocks_per_branch * 4), bl_b = up((size_t)n_branches * 4);
    const size_t pt_b = up((size_t)n_branches * (gamma + 1) * vocab * dist_elt);
    const size_t qd_b = up((size_t)n_branches * gamma * vocab * dist_elt);
    const size_t dt_b = up((size_t)n_branches * gamma * 4), un_b = up((size_t)n_branches * (gamma + 1) * 4);
    const size_t res_b = up((size_t)n_branches * 4);
    const size_t need = up(q_layer) * n_layers + up(o_layer) * n_layers + bt_b + bl_b + pt_b + qd_b + dt_b +
                        un_b + 2 * res_b;
    cudaError_t e;
    if (c->stage_bytes < need) {
        cudaFree(c->stage); c->stage = nullptr; c->stage_bytes = 0;
        if ((e = cudaMalloc(&c->stage, need)) != cudaSuccess) return cuda_fail(c, e);
        c->stage_bytes = need;
    }
    char* base = static_cast<char*>(c->stage);
    char* d_q = base;               base += up(q_layer) * n_layers;
    char* d_o = base;               base += up(o_layer) * n_layers;
    int32_t* d_bt = (int32_t*)base; base += bt_b;
    int32_t* d_bl = (int32_t*)base; base += bl_b;
    char* d_pt = base;              base += pt_b;
    char* d_qd = base;              base += qd_b;
    int32_t* d_dt = (int32_t*)base; base += dt_b;
    float* d_un = (float*)base;     base += un_b;
    int32_t* d_al = (int32_t*)base; base += res_b;
    int32_t* d_nt = (int32_t*)base;

    // Two more streams carry the copies that need not wait for the kernels: the queries of later layers and
    // the accept inputs go host-to-device while the first layers run, the outputs of finished layers go back
    // while later layers run.  Events order them against the context's stream, chunk of layers by chunk.
    // an error return must not leave copies from or to the caller's host buffers in flight
    auto drain = [&]() {
        cudaStreamSynchronize(c->stream);
        if (c->h2d_stream) cudaStreamSynchronize(c->h2d_stream);
        if (c->d2h_stream) cudaStreamSynchronize(c->d2h_stream);
    };
#define TTS_CK(x) do { e = (x); if (e != cudaSuccess) { drain(); return cuda_fail(c, e); } } while (0)
    if (!c->host_ev) {
        TTS_CK(cudaStreamCreateWithFlags(&c->h2d_stream, cudaStreamNonBlocking));
        TTS_CK(cudaStreamCreateWithFlags(&c->d2h_stream, cudaStreamNonBlocking));
        c->host_ev = static_cast<cudaEvent_t*>(calloc(kHostEvents, sizeof(cudaEvent_t)));
        if (!c->host_ev) return TTS_ERR_INVALID;
        for (int i = 0; i < kHostEvents; ++i) TTS_CK(cudaEventCreateWithFlags(&c->host_ev[i], cudaEventDisableTiming));
    }
    cudaStream_t st = c->stream, up_st = c->h2d_stream, down_st = c->d2h_stream;
    cudaEvent_t* ev_q = c->host_ev;                         // queries of chunk i are on the device
    cudaEvent_t* ev_o = c->host_ev + kHostChunks;           // outputs of chunk i are computed
    cudaEvent_t ev_start = c->host_ev[2 * kHostChunks], ev_acc = c->host_ev[2 * kHostChunks + 1];
    const int per_chunk = (n_layers + kHostChunks - 1) / kHostChunks < 4 ? (n_layers < 4 ? n_layers : 4)
                                                                         : (n_layers + kHostChunks - 1) / kHostChunks;
    const int n_chunks = (n_layers + per_chunk - 1) / per_chunk;
    // the staging buffers may still be read by work queued on the context's stream before this call
    TTS_CK(cudaEventRecord(ev_start, st));
    TTS_CK(cudaStreamWaitEvent(up_st, ev_start, 0));
    TTS_CK(cudaStreamWaitEvent(down_st, ev_start, 0));
    TTS_CK(cudaMemcpyAsync(d_bt, block_table_host, (size_t)n_branches * f.max_blocks_per_branch * 4, cudaMemcpyHostToDevice, st));
    TTS_CK(cudaMemcpyAsync(d_bl, branch_lens_host, (size_t)n_branches * 4, cudaMemcpyHostToDevice, st));
    auto copy_q = [&](int l0, int l1, cudaStream_t s2) -> cudaError_t {
        if (up(q_layer) == q_layer)                         // contiguous on both sides: one copy
            return cudaMemcpyAsync(d_q + q_layer * l0, (const char*)q_host + q_layer * l0, q_layer * (l1 - l0), cudaMemcpyHostToDevice, s2);
        for (int l = l0; l < l1; ++l) {
            cudaError_t e2 = cudaMemcpyAsync(d_q + up(q_layer) * l, (const char*)q_host + q_layer * l, q_layer, cudaMemcpyHostToDevice, s2);
            if (e2 != cudaSuccess) return e2;
        }
        return cudaSuccess;
    };
    auto copy_o = [&](int l0, int l1, cudaStream_t s2) -> cudaError_t {
        if (up(o_layer) == o_layer)
            return cudaMemcpyAsync((char*)out_host + o_layer * l0, d_o + o_layer * l0, o_layer * (l1 - l0), cudaMemcpyDeviceToHost, s2);
        for (int l = l0; l < l1; ++l) {
            cudaError_t e2 = cudaMemcpyAsync((char*)out_host + o_layer * l, d_o + up(o_layer) * l, o_layer, cudaMemcpyDeviceToHost, s2);
            if (e2 != cudaSuccess) return e2;
        }
        return cudaSuccess;
    };
    // host-to-device: the first chunk of queries on the context's stream, the rest and the accept inputs beside it
    TTS_CK(copy_q(0, per_chunk < n_layers ? per_chunk : n_layers, st));
    for (int ch = 1; ch < n_chunks; ++ch) {
        const int l0 = ch * per_chunk, l1 = l0 + per_chunk < n_layers ? l0 + per_chunk : n_layers;
        TTS_CK(copy_q(l0, l1, up_st));
        TTS_CK(cudaEventRecord(ev_q[ch], up_st));
    }
    // Probabilities in pinned (device-mapped) host memory are not copied: the accept kernel reads, straight from the
    // host, the 2 gamma scalars of its tests and the one row pair of its draw, a quarter of the two tensors, instead
    // of all of them crossing the link behind the queries.  (The logits variant reads its rows twice: it copies.)
    const void* p_dev = nullptr; const void* q_dev = nullptr;
    bool zero_copy = false;
    if (logits_dtype < 0) {
        void* a = nullptr; void* b = nullptr;
        zero_copy = cudaHostGetDevicePointer(&a, const_cast<void*>(p_target_host), 0) == cudaSuccess &&
                    (gamma == 0 || cudaHostGetDevicePointer(&b, const_cast<void*>(q_draft_host), 0) == cudaSuccess);
        if (!zero_copy) (void)cudaGetLastError();            // pageable memory: not an error of this call
        zero_copy = zero_copy && aligned16(a) && (gamma == 0 || aligned16(b));
        p_dev = a; q_dev = b;
    }
    if (!zero_copy)
        TTS_CK(cudaMemcpyAsync(d_pt, p_target_host, (size_t)n_branches * (gamma + 1) * vocab * dist_elt, cudaMemcpyHostToDevice, up_st));
    if (gamma > 0) {
        if (!zero_copy)
            TTS_CK(cudaMemcpyAsync(d_qd, q_draft_host, (size_t)n_branches * gamma * vocab * dist_elt, cudaMemcpyHostToDevice, up_st));
        TTS_CK(cudaMemcpyAsync(d_dt, draft_tokens_host, (size_t)n_branches * gamma * 4, cudaMemcpyHostToDevice, up_st));
    }
    TTS_CK(cudaMemcpyAsync(d_un, uniforms_host, (size_t)n_branches * (gamma + 1) * 4, cudaMemcpyHostToDevice, up_st));
    TTS_CK(cudaEventRecord(ev_acc, up_st));
    // one schedule serves all layers
    {
        const int rc = tts_attn_plan(ctx, d_bt, prefix_len, d_bl, n_branches, gamma + 1);
        if (rc != TTS_OK) { drain(); return rc; }
    }
    // the layers, chunk by chunk; every finished chunk's outputs go back beside the next chunk's kernels
    for (int ch = 0; ch < n_chunks; ++ch) {
        const int l0 = ch * per_chunk, l1 = l0 + per_chunk < n_layers ? l0 + per_chunk : n_layers;
        if (ch > 0) TTS_CK(cudaStreamWaitEvent(st, ev_q[ch], 0));
        for (int l = l0; l < l1; ++l) {
            int rc = tts_verify_attn(ctx, d_q + up(q_layer) * l, k_pools[l], v_pools[l], d_bt, prefix_len, d_bl,
                                     n_branches, gamma, TTS_MASK_CAUSAL, d_o + up(o_layer) * l);
            if (rc != TTS_OK) { drain(); return rc; }
        }
        TTS_CK(cudaEventRecord(ev_o[ch], st));
        TTS_CK(cudaStreamWaitEvent(down_st, ev_o[ch], 0));
        TTS_CK(copy_o(l0, l1, down_st));
    }
    TTS_CK(cudaStreamWaitEvent(st, ev_acc, 0));
    int rc = logits_dtype < 0
                 ? tts_accept(ctx, zero_copy ? (const float*)p_dev : (const float*)d_pt,
                              gamma > 0 ? (zero_copy ? (const float*)q_dev : (const float*)d_qd) : nullptr, gamma > 0 ? d_dt : nullptr, d_un,
                              n_branches, gamma, vocab, d_al, d_nt)
                 : tts_accept_logits(ctx, d_pt, gamma > 0 ? d_qd : nullptr, logits_dtype, gamma > 0 ? d_dt : nullptr, d_un,
                                     n_branches, gamma, vocab, d_al, d_nt);
    if (rc != TTS_OK) { drain(); return rc; }
    TTS_CK(cudaMemcpyAsync(accepted_len_host, d_al, (size_t)n_branches * 4, cudaMemcpyDeviceToHost, st));
    TTS_CK(cudaMemcpyAsync(next_token_host, d_nt, (size_t)n_branches * 4, cudaMemcpyDeviceToHost, st));
    c->plan_explicit = 0;                                   // the staging buffers' contents change with the next call
    TTS_CK(cudaStreamSynchronize(st));
    TTS_CK(cudaStreamSynchronize(down_st));
    TTS_CK(cudaStreamSynchronize(up_st));
#undef TTS_CK
    return TTS_OK;
}

}  // namespace

extern "C" {

int tts_verify_step_host(tts_ctx* ctx, int n_layers, const void* q_host, const void* const* k_pools,
                         const void* const* v_pools, const int32_t* block_table_host, int prefix_len,
                         const int32_t* branch_lens_host, int n_branches, int gamma,
                         const float* p_target_host, const float* q_draft_host,
                         const int32_t* draft_tokens_host, const float* uniforms_host, int vocab,
                         void* out_host, int32_t* accepted_len_host, int32_t* next_token_host) {
    return step_host(ctx, n_layers, q_host, k_pools, v_pools, block_table_host, prefix_len, branch_lens_host, n_branches,
                     gamma, p_target_host, q_draft_host, -1, draft_tokens_host, uniforms_host, vocab, out_host,
                     accepted_len_host, next_token_host);
}

int tts_verify_step_host_logits(tts_ctx* ctx, int n_layers, const void* q_host, const void* const* k_pools,
                                const void* const* v_pools, const int32_t* block_table_host, int prefix_len,
                                const int32_t* branch_lens_host, int n_branches, int gamma,
                                const void* target_logits_host, const void* draft_logits_host, int logits_dtype,
                                const int32_t* draft_tokens_host, const float* uniforms_host, int vocab,
                                void* out_host, int32_t* accepted_len_host, int32_t* next_token_host) {
    if (logits_dtype != TTS_LOGITS_BF16 && logits_dtype != TTS_LOGITS_FP32) return TTS_ERR_UNSUPPORTED;
    return step_host(ctx, n_layers, q_host, k_pools, v_pools, block_table_host, prefix_len, branch_lens_host, n_branches,
                     gamma, target_logits_host, draft_logits_host, logits_dtype, draft_tokens_host, uniforms_host, vocab,
                     out_host, accepted_len_host, next_token_host);
}

}  // extern "C"
