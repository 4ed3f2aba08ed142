// Internal declarations shared by the kernels and the C-ABI layer (not installed).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "tts.h"

namespace tts {

constexpr int kHeadDim = 128;
constexpr int kPage = 16;
constexpr int kMaxTreeRows = 64;      // rows per branch that may carry an explicit visibility mask
constexpr int kMaxBranches = 1024;

// Work decomposition of one attention call.
//
// A *segment* is (KV head, block of <= rb_rows stacked query rows, run of KV tokens):
//   prefix segments   s = kvh * n_rb_pre + rb            rows = all branches' rows, stacked
//                                                          (b, i, g) -> b*nr + i*G + g; every row
//                                                          sees every prefix token (no mask)
//   private segments  (b, kvh, rb)                         rows = (i, g) -> i*G + g
// Each segment is cut into tiles of tile_tokens KV tokens; all tiles of all segments form one
// global list, and CTA c of a persistent grid owns the contiguous run [c*tpc, (c+1)*tpc) of it
// (tpc = ceil(total / grid)).  The list goes group by group, a group being the n_rb_priv private
// segments of one (branch, KV head), idx = b*Hkv + kvh; the prefix segments are spread evenly
// between the groups (segments [pre_before(idx), pre_before(idx+1)) follow group idx), so that no
// CTA gets more than a few of these short segments.  The run of one CTA inside one segment is a
// *piece*; it produces one partial result (running max m, sum l, unnormalised O) per row.  Because
// segments of either kind and CTAs both advance along the list, (segment index within its kind +
// CTA) is a unique index for every piece, so no scan over pieces is needed to place them in the
// workspace.
struct CtaPlan;
struct PieceDesc;

// Sets of branches that share a prefix each (several questions in one call): set s holds the branches
// [first_branch[s], first_branch[s + 1]) and its prefix is prefix_len[s] tokens long.
constexpr int kMaxPrefixSets = 64;
struct PrefixSets {
    int n_sets;
    int first_branch[kMaxPrefixSets + 1];
    int prefix_len[kMaxPrefixSets];
};
struct AttnParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k_pages;
    const __nv_bfloat16* v_pages;
    const int32_t* block_table;
    const int32_t* branch_lens;
    const int32_t* tree_parents;   // null for causal
    void* out;
    float* part_o_pre;    // [n_pre + grid][pre_stride][128]
    float2* part_ml_pre;  // [n_pre + grid][pre_stride]      (m in log2 units, l)
    float* part_o_priv;   // [N*Hkv*n_rb_priv + grid][priv_stride][128]
    float2* part_ml_priv;
    int32_t* status;      // device status word
    void* group_desc;     // [N*Hkv] GroupDesc (attn_merge.cuh) for the merge kernel: part of the plan, or null
    const CtaPlan* plan_cta;        // [grid] the plan the token-major kernel runs from (attn_plan.cuh)
    const PieceDesc* plan_pieces;
    int N, R, Hq, Hkv, G, nr;      // nr = R*G rows per (branch, kv head)
    int P;                          // prefix tokens
    int max_blocks, num_pages;
    int rb_rows;                    // rows per row block
    int pre_stride, priv_stride;    // rows reserved per piece: copies_pre * min(rb_rows, N*nr) / copies * min(rb_rows, nr)
    int copies;                     // tcgen05 paths: independent key-subset copies of a private piece's rows,
    int copies_pre;                 //   and of a prefix piece's rows (each copy is a partial result of its own)
    int n_rb_pre, n_rb_priv;        // row blocks per prefix kv head / per (branch, kv head)
    int n_pre;                      // prefix segments (0 when P == 0)
    int tiles_pre;                  // tiles per prefix segment
    int tile_tokens;
    int grid;                       // CTAs of the main kernel
    int out_dtype, debug;
    float scale_log2;               // softmax scale * log2(e)
};

struct SegInfo {
    int kind;        // 0 prefix, 1 private
    int idx;         // group b*Hkv + kvh the segment belongs to (private) or follows (prefix)
    int kvh, rb, b;  // b = -1 for prefix
    int n_rows;      // valid rows in this row block
    int row0;        // first stacked row of the block (prefix: in [0, N*nr); private: in [0, nr))
    int tile_begin;  // global index of the segment's first tile
    int n_tiles;
    int tok_begin;   // logical token of the segment's first key (0 for prefix, P for private)
    int n_tokens;    // keys in the segment (P or L_b)
};

__host__ __device__ inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// cum[b] = tiles of branches < b (per private segment of that branch), cum[N] = sum.
// Must be called by all threads of the block; cum lives in shared memory (N+1 ints).
__device__ inline void build_branch_tile_prefix(const AttnParams& p, int* cum) {
    for (int b = threadIdx.x; b < p.N; b += blockDim.x) {
        int L = p.branch_lens[b];
        L = L < 0 ? 0 : L;
        cum[b + 1] = ceil_div(L, p.tile_tokens);
    }
    __syncthreads();
    if (threadIdx.x < 32) {                                  // inclusive scan by the first warp, 32 at a time
        const int lane = threadIdx.x;
        int carry = 0;
        for (int base = 0; base < p.N; base += 32) {
            int v = base + lane < p.N ? cum[base + lane + 1] : 0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int n = __shfl_up_sync(0xffffffffu, v, o);
                if (lane >= o) v += n;
            }
            if (base + lane < p.N) cum[base + lane + 1] = carry + v;
            carry += __shfl_sync(0xffffffffu, v, 31);
        }
        if (lane == 0) cum[0] = 0;
    }
    __syncthreads();
}

__device__ __forceinline__ int branch_len(const AttnParams& p, const int* cum, int b) {
    (void)cum;
    return p.branch_lens[b];
}

// a / b and a % b for 0 <= a < 2^31 with a quotient below 2^22, 0 < b: float estimate, corrected
// exactly (integer division by a run-time divisor is an expensive instruction sequence)
__device__ __forceinline__ void fast_divmod(int a, int b, int& q, int& r) {
    q = __float2int_rz(__fdividef((float)a, (float)b));
    r = a - q * b;
    while (r < 0) { --q; r += b; }
    while (r >= b) { ++q; r -= b; }
}
__device__ __forceinline__ int fast_div(int a, int b) { int q, r; fast_divmod(a, b, q, r); return q; }

// prefix segments placed before group idx (idx in [0, N*Hkv]); the host rejects calls whose
// N * Hkv * n_pre does not fit 31 bits
__device__ inline int pre_before(const AttnParams& p, int idx) { return fast_div(idx * p.n_pre, p.N * p.Hkv); }

// global index of the first tile of group idx (idx == N*Hkv gives the total)
__device__ inline int group_tile_begin(const AttnParams& p, const int* cum, int idx) {
    int b, kvh;
    fast_divmod(idx, p.Hkv, b, kvh);
    const int tb = b < p.N ? cum[b + 1] - cum[b] : 0;
    return p.n_rb_priv * (p.Hkv * cum[b] + kvh * tb) + p.tiles_pre * pre_before(p, idx);
}

__device__ inline int total_tiles(const AttnParams& p, const int* cum) {
    return group_tile_begin(p, cum, p.N * p.Hkv);
}

__device__ inline SegInfo prefix_segment(const AttnParams& p, int s, int tile_begin, int idx) {
    SegInfo g;
    g.kind = 0; g.b = -1; g.idx = idx;
    g.kvh = s / p.n_rb_pre; g.rb = s % p.n_rb_pre;
    g.row0 = g.rb * p.rb_rows;
    g.n_rows = min(p.rb_rows, p.N * p.nr - g.row0);
    g.tile_begin = tile_begin; g.n_tiles = p.tiles_pre;
    g.tok_begin = 0; g.n_tokens = p.P;
    return g;
}

// Segment that contains global tile g (0 <= g < total), given the group idx it falls into (the
// largest one whose first tile is <= g).
__device__ inline SegInfo segment_in_group(const AttnParams& p, const int* cum, int idx, int g) {
    int b, kvh;
    fast_divmod(idx, p.Hkv, b, kvh);
    const int begin = group_tile_begin(p, cum, idx);
    const int tb = cum[b + 1] - cum[b];
    const int priv_tiles = p.n_rb_priv * tb;
    const int within = g - begin;
    if (within >= priv_tiles) {                 // one of the prefix segments that follow the group
        const int k = fast_div(within - priv_tiles, p.tiles_pre);
        return prefix_segment(p, pre_before(p, idx) + k, begin + priv_tiles + k * p.tiles_pre, idx);
    }
    SegInfo s;
    s.kind = 1; s.b = b; s.kvh = kvh; s.idx = idx;
    s.rb = fast_div(within, tb);
    s.row0 = s.rb * p.rb_rows;
    s.n_rows = min(p.rb_rows, p.nr - s.row0);
    s.tile_begin = begin + s.rb * tb; s.n_tiles = tb;
    s.tok_begin = p.P; s.n_tokens = branch_len(p, cum, b);
    return s;
}

// Segment that contains global tile g (0 <= g < total): binary search by one thread.
__device__ inline SegInfo segment_of_tile(const AttnParams& p, const int* cum, int g) {
    int lo = 0, hi = p.N * p.Hkv - 1;          // largest group whose first tile is <= g
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (group_tile_begin(p, cum, mid) <= g) lo = mid; else hi = mid - 1;
    }
    return segment_in_group(p, cum, lo, g);
}

// The segment after s in the tile list (the caller knows there is one): the next row block of the
// same group, else the next prefix segment that follows the group, else the next non-empty group.
__device__ inline SegInfo next_segment(const AttnParams& p, const int* cum, const SegInfo& s) {
    const int end = s.tile_begin + s.n_tiles;
    if (s.kind == 1 && s.rb + 1 < p.n_rb_priv) {
        SegInfo n = s;
        n.rb = s.rb + 1; n.row0 = n.rb * p.rb_rows; n.n_rows = min(p.rb_rows, p.nr - n.row0);
        n.tile_begin = end;
        return n;
    }
    int idx = s.idx;
    const int k_next = s.kind == 1 ? pre_before(p, idx) : s.kvh * p.n_rb_pre + s.rb + 1;
    if (k_next < pre_before(p, idx + 1)) return prefix_segment(p, k_next, end, idx);
    for (++idx; idx < p.N * p.Hkv - 1; ++idx) {           // skip groups without tiles
        const int b = idx / p.Hkv;
        if (cum[b + 1] - cum[b] > 0 || pre_before(p, idx + 1) > pre_before(p, idx)) break;
    }
    const int b = idx / p.Hkv;
    if (cum[b + 1] - cum[b] == 0) return prefix_segment(p, pre_before(p, idx), end, idx);
    SegInfo n;
    n.kind = 1; n.idx = idx; n.b = b; n.kvh = idx - b * p.Hkv; n.rb = 0;
    n.row0 = 0; n.n_rows = min(p.rb_rows, p.nr);
    n.tile_begin = end; n.n_tiles = cum[b + 1] - cum[b];
    n.tok_begin = p.P; n.n_tokens = branch_len(p, cum, b);
    return n;
}

// First tile of prefix segment s: it follows the first group idx with pre_before(idx + 1) > s.
__device__ inline int prefix_segment_tile_begin(const AttnParams& p, const int* cum, int s) {
    // (s + 1) * groups + n_pre - 1 <= groups * n_pre + n_pre < 2^32: the host rejects groups * n_pre >= 2^31
    const unsigned int n_groups = (unsigned int)(p.N * p.Hkv);
    const int idx = (int)(((unsigned int)(s + 1) * n_groups + (unsigned int)p.n_pre - 1u) / (unsigned int)p.n_pre) - 1;
    const int b = idx / p.Hkv;
    const int tb = cum[b + 1] - cum[b];
    return group_tile_begin(p, cum, idx) + p.n_rb_priv * tb + (s - pre_before(p, idx)) * p.tiles_pre;
}

__device__ inline int segment_index(const AttnParams& p, const SegInfo& s) {
    return s.kind == 0 ? s.kvh * p.n_rb_pre + s.rb
                       : p.n_pre + (s.b * p.Hkv + s.kvh) * p.n_rb_priv + s.rb;
}

// Where the piece (segment s, CTA c) keeps its partial result.
__device__ inline void piece_slot(const AttnParams& p, const SegInfo& s, int cta, float*& o,
                                  float2*& ml) {
    if (s.kind == 0) {
        const size_t id = (size_t)(s.kvh * p.n_rb_pre + s.rb) + cta;
        o = p.part_o_pre + id * p.pre_stride * kHeadDim;
        ml = p.part_ml_pre + id * p.pre_stride;
    } else {
        const size_t id = (size_t)((s.b * p.Hkv + s.kvh) * p.n_rb_priv + s.rb) + cta;
        o = p.part_o_priv + id * p.priv_stride * kHeadDim;
        ml = p.part_ml_priv + id * p.priv_stride;
    }
}

// Physical page of logical block `blk` of a block-table row.  With the debug checks on, a block
// beyond the row or a page outside the pool raises TTS_ERR_DEVICE_BOUNDS and page 0 is read instead
// (valid memory; the result of the call is then meaningless, the access is not out of range).
__device__ __forceinline__ int checked_page(const AttnParams& p, const int32_t* bt_row, int blk) {
    if (!p.debug) return bt_row[blk];
    int page = blk >= 0 && blk < p.max_blocks ? bt_row[blk] : -1;
    if (page < 0 || page >= p.num_pages) {
        atomicMin(p.status, (int)TTS_ERR_DEVICE_BOUNDS);
        page = 0;
    }
    return page;
}

// 64-bit visibility mask of query position i over the last R private tokens of its branch:
// bit a set <=> row i sees token (L - R + a).  Causal: bits 0..i.  Tree: i and its ancestors.
__device__ inline unsigned long long row_visibility(const AttnParams& p, int b, int i) {
    if (p.tree_parents == nullptr) return i >= 63 ? ~0ull : ((2ull << i) - 1ull);
    unsigned long long m = 0;
    int a = i;
    for (int guard = 0; a >= 0 && guard < kMaxTreeRows; ++guard) {
        m |= 1ull << a;
        int par = p.tree_parents[b * p.R + a];
        a = par < a ? par : -1;               // malformed parents end the walk
    }
    return m;
}

struct Ctx {
    tts_config cfg;
    int device;
    int n_sms;
    cudaStream_t stream;
    int last_cuda_error;
    long long launches;
    int32_t* d_status;
    // split-KV workspace
    float* part_o_pre; float2* part_ml_pre; float* part_o_priv; float2* part_ml_priv;
    size_t pre_rows, priv_rows;       // allocated partial rows (each 128 fp32 + one float2)
    void* group_desc;                 // one merge descriptor per (branch, KV head)
    // plan of the token-major kernel (attn_plan.cuh): one record per CTA, the list of all pieces
    CtaPlan* plan_cta; PieceDesc* plan_pieces; size_t plan_pieces_cap;
    // the arguments the plan in the tables was built from by tts_attn_plan (valid while plan_explicit is set)
    struct { const int32_t* block_table; const int32_t* branch_lens; int n_branches, rows; PrefixSets sets; } plan_key;
    int plan_explicit;
    // staging for the host entry point
    void* stage; size_t stage_bytes;
    cudaStream_t h2d_stream, d2h_stream;   // copies of the host entry point that overlap the kernels (created on first use)
    cudaEvent_t* host_ev;                  // kHostEvents events ordering them against the context's stream
    void* tmap_cache;                  // opaque: tensor maps keyed by pool pointer
    // profiling aid
    int profiling, prof_n;
    cudaEvent_t* prof_ev;              // 3 events per recorded call
};
constexpr int kProfMaxCalls = 4096;
constexpr int kHostChunks = 16;       // the host entry point moves queries and outputs in at most this many chunks of layers
constexpr int kHostEvents = 2 * kHostChunks + 2;

// kernel launchers (each returns the cudaError_t of its launch)
cudaError_t launch_attn_simt(const AttnParams& p, cudaStream_t st);
cudaError_t launch_attn_combine(const AttnParams& p, cudaStream_t st);
cudaError_t launch_accept(const float* p_target, const float* q_draft, const int32_t* draft_tokens,
                          const float* uniforms, int n_branches, int gamma, int vocab,
                          int32_t* accepted_len, int32_t* next_token, int32_t* status,
                          cudaStream_t st);
cudaError_t launch_accept_logits(const void* target_logits, const void* draft_logits, int logits_dtype,
                                 const int32_t* draft_tokens, const float* uniforms, int n_branches, int gamma, int vocab,
                                 int32_t* accepted_len, int32_t* next_token, int32_t* status, cudaStream_t st);
cudaError_t launch_accept_tree(const float* p_target, const float* q_draft, const int32_t* draft_tokens,
                               const int32_t* tree_parents, const float* uniforms, int n_branches, int n_nodes, int vocab,
                               int32_t* accepted_len, int32_t* last_node, int32_t* next_token, int32_t* status,
                               cudaStream_t st);
cudaError_t launch_kv_append(const void* k_new, const void* v_new, void* k_pages, void* v_pages,
                             const int32_t* block_table, int max_blocks, int num_pages, int prefix_len,
                             const int32_t* branch_lens, int N, int R, int Hkv, int32_t* status, cudaStream_t st);
cudaError_t launch_kv_rollback(int32_t* branch_lens, const int32_t* accepted_len, int N, int gamma, int32_t* status,
                               cudaStream_t st);
cudaError_t launch_wait_probe(int32_t* status, long long limit_ns, int* gave_up, cudaStream_t st);
int simt_rb_rows(int nr);
constexpr int kSimtTileTokens = 64;

// tcgen05 path
constexpr int kUmmaRows = 128;         // MMA tile height = rows per row block
constexpr int kUmmaTileTokens = 128;
constexpr int kUmmaMinRows = 9;        // below this many stacked rows per KV head the CUDA-core kernel runs
bool umma_available();
int umma_copies(int nr);              // replication factor of a private piece's rows along the MMA M dimension
cudaError_t launch_attn_umma(Ctx* c, const AttnParams& p, cudaStream_t st);
// token-major tcgen05 kernel (KV tokens on the MMA M dimension): row blocks of 32 or 64 stacked rows
constexpr int kUmmaTMaxRows = 64;
constexpr int kUmmaTGroups = 1;        // partial results a piece leaves per row
int umma_t_rows(int nr);
cudaError_t launch_attn_umma_t(Ctx* c, const AttnParams& p, cudaStream_t st);
void umma_release(Ctx* c);

}  // namespace tts
