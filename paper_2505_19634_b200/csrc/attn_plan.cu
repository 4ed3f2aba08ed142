// Builds the plan tables (attn_plan.cuh): the pieces of every CTA of the token-major kernel, the pages
// of each CTA's first two tiles, and the merge descriptors of every (branch, KV head).  One CTA; thread c
// walks the run of CTA c of the main kernel through the segment list of tts_internal.cuh.
//
// A call may carry several sets of branches, each set sharing a prefix of its own (several questions in
// flight).  Every set is scheduled by the single-prefix rules applied to it alone; the tile lists of the
// sets are laid end to end and cut into equal runs as one list.
#include "attn_merge.cuh"
#include "attn_plan.cuh"
#include "tts_internal.cuh"

namespace tts {

namespace {

constexpr int kPlanThreads = 1024;
static_assert(sizeof(GroupDesc) <= 64, "the context reserves 64 bytes per merge descriptor");

// Where the pages of one of a CTA's first two tiles are listed: block-table row, first block, number of
// pages, KV head.
struct FirstTile { int bt_row, blk0, n_pages, kvh; };

// The parameters of set s alone: its branches, prefix and segment counts.
__device__ AttnParams set_params(const AttnParams& p, const PrefixSets& sets, int s) {
    AttnParams q = p;
    const int b0 = sets.first_branch[s];
    q.N = sets.first_branch[s + 1] - b0;
    q.P = sets.prefix_len[s];
    q.branch_lens = p.branch_lens + b0;
    q.block_table = p.block_table + (size_t)b0 * p.max_blocks;
    q.n_rb_pre = ceil_div(q.N * p.nr, p.rb_rows);
    q.n_pre = q.P > 0 ? p.Hkv * q.n_rb_pre : 0;
    q.tiles_pre = ceil_div(q.P, p.tile_tokens);
    return q;
}

// Walks the part [l_begin, l_end) of set s's tile list that falls into the run of CTA c.  With out ==
// nullptr only counts the pieces; otherwise appends them at out[n0 ..] and notes the CTA's first two tiles
// (u = tiles of the run before this call).
__device__ int walk_set(const AttnParams& ps, const int* cum, const SetOffsets so, int l_begin, int l_end, int c,
                        PieceDesc* out, CtaPlan* hdr, FirstTile* first2, int n0, int& u) {
    SegInfo seg = segment_of_tile(ps, cum, l_begin);
    int n = 0;
    for (;;) {
        const int t_first = max(0, l_begin - seg.tile_begin);
        const int t_last = min(seg.n_tiles, l_end - seg.tile_begin);
        if (out) {
            PieceDesc d;
            d.kind = seg.kind; d.b = so.first_branch + (seg.kind == 0 ? 0 : seg.b); d.kvh = seg.kvh;
            d.row0 = seg.row0; d.n_rows = seg.n_rows;
            d.bt_row = d.b;
            d.tok_begin = seg.tok_begin; d.seg_tokens = seg.n_tokens;
            d.tile0 = t_first; d.n_tiles = t_last - t_first;
            d.slot = (seg.kind == 0 ? so.pre_slot_base + seg.kvh * ps.n_rb_pre + seg.rb
                                    : ((so.first_branch + seg.b) * ps.Hkv + seg.kvh) * ps.n_rb_priv + seg.rb) + c;
            d.pad = 0;
            out[n0 + n] = d;
            if (n0 + n < kPlanInline) hdr->first_pieces[n0 + n] = d;
            for (int t = t_first; t < t_last && u < 2; ++t, ++u) {
                const int tok0 = t * ps.tile_tokens;
                first2[u].bt_row = d.bt_row; first2[u].blk0 = (seg.tok_begin + tok0) / kPage;
                first2[u].n_pages = min(8, ceil_div(min(ps.tile_tokens, seg.n_tokens - tok0), kPage));
                first2[u].kvh = seg.kvh;
            }
        }
        ++n;
        if (seg.tile_begin + t_last >= l_end) break;
        seg = next_segment(ps, cum, seg);
    }
    return n;
}

// The run [g_begin, g_end) of CTA c over the sets' concatenated tile lists.
__device__ int walk_run(const AttnParams& p, const PrefixSets& sets, const int* cum_all, const int* tile_off,
                        const int* pre_base, int tpc, int c, PieceDesc* out, CtaPlan* hdr, FirstTile* first2) {
    const int total = tile_off[sets.n_sets];
    const int g_begin = c * tpc, g_end = min(total, g_begin + tpc);
    if (hdr) {
        hdr->n_tiles = max(0, g_end - g_begin);
        first2[0].n_pages = first2[1].n_pages = 0;
    }
    int n = 0, u = 0;
    for (int s = 0; s < sets.n_sets && g_begin < g_end; ++s) {
        if (tile_off[s + 1] <= g_begin || tile_off[s] >= g_end) continue;
        const AttnParams ps = set_params(p, sets, s);
        const SetOffsets so{sets.first_branch[s], tile_off[s], pre_base[s]};
        n += walk_set(ps, cum_all + sets.first_branch[s] + s, so, max(g_begin, tile_off[s]) - tile_off[s],
                      min(g_end, tile_off[s + 1]) - tile_off[s], c, out, hdr, first2, n, u);
    }
    return n;
}

__global__ void __launch_bounds__(kPlanThreads) attn_plan_kernel(const AttnParams p, const PrefixSets sets, CtaPlan* cta,
                                                                 PieceDesc* pieces, GroupDesc* groups) {
    extern __shared__ int sm[];
    int* cum_all = sm;                                     // set s: N_s + 1 ints at offset first_branch[s] + s
    int* tile_off = cum_all + p.N + sets.n_sets;           // n_sets + 1: tiles of the sets before set s
    int* pre_base = tile_off + sets.n_sets + 1;            // n_sets: prefix partial-result slots before set s
    int* first = pre_base + sets.n_sets;                   // grid + 1 ints: index of every CTA's first piece
    FirstTile* first2 = reinterpret_cast<FirstTile*>(first + p.grid + 1);   // 2 per CTA
    for (int s = 0; s < sets.n_sets; ++s)                  // block-wide; a handful of sets
        build_branch_tile_prefix(set_params(p, sets, s), cum_all + sets.first_branch[s] + s);
    if (threadIdx.x == 0) {
        int t = 0, slots = 0;
        for (int s = 0; s < sets.n_sets; ++s) {
            const AttnParams ps = set_params(p, sets, s);
            tile_off[s] = t; pre_base[s] = slots;
            t += total_tiles(ps, cum_all + sets.first_branch[s] + s);
            slots += ps.n_pre;
        }
        tile_off[sets.n_sets] = t;
    }
    __syncthreads();
    const int tpc = ceil_div(tile_off[sets.n_sets], p.grid);
    for (int c = threadIdx.x; c < p.grid; c += blockDim.x)
        first[c + 1] = walk_run(p, sets, cum_all, tile_off, pre_base, tpc, c, nullptr, nullptr, nullptr);
    __syncthreads();
    if (threadIdx.x < 32) {                                // inclusive scan of the counts by the first warp, 32 at a time
        const int lane = threadIdx.x;
        int carry = 0;
        for (int base = 0; base < p.grid; base += 32) {
            int v = base + lane < p.grid ? first[base + lane + 1] : 0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int n = __shfl_up_sync(0xffffffffu, v, o);
                if (lane >= o) v += n;
            }
            if (base + lane < p.grid) first[base + lane + 1] = carry + v;
            carry += __shfl_sync(0xffffffffu, v, 31);
        }
        if (lane == 0) first[0] = 0;
    }
    __syncthreads();
    for (int c = threadIdx.x; c < p.grid; c += blockDim.x) {
        cta[c].piece_begin = first[c];
        cta[c].n_pieces = walk_run(p, sets, cum_all, tile_off, pre_base, tpc, c, pieces + first[c], cta + c, first2 + 2 * c);
    }
    __syncthreads();
    // the pages of every CTA's first two tiles: one thread per page, all loads independent
    for (int i = threadIdx.x; i < p.grid * 16; i += blockDim.x) {
        const int c = i >> 4, j = i & 7;
        const FirstTile ft = first2[2 * c + ((i >> 3) & 1)];
        int page_head = -1;
        if (j < ft.n_pages) page_head = checked_page(p, p.block_table + (size_t)ft.bt_row * p.max_blocks, ft.blk0 + j) * p.Hkv + ft.kvh;
        cta[c].first_pages[i & 15] = page_head;
    }
    // the merge descriptor of every (branch, KV head)
    constexpr int kEntries = kMaxPrivBlocks + kMaxPreBlocks;
    if (groups)
        for (int s = 0; s < sets.n_sets; ++s) {
            const AttnParams ps = set_params(p, sets, s);
            const SetOffsets so{sets.first_branch[s], tile_off[s], pre_base[s]};
            for (int i = threadIdx.x; i < ps.N * p.Hkv * kEntries; i += blockDim.x) {
                const int grp = i / kEntries;
                group_describe_entry(ps, cum_all + sets.first_branch[s] + s, tpc, grp / p.Hkv, grp % p.Hkv, i % kEntries,
                                     groups[so.first_branch * p.Hkv + grp], so);
            }
        }
}

}  // namespace

cudaError_t launch_attn_plan(const AttnParams& main_params, const PrefixSets& sets, cudaStream_t st) {
    AttnParams p = main_params;
    const size_t smem = (size_t)(p.N + sets.n_sets + 2 * sets.n_sets + 1 + p.grid + 1) * sizeof(int) +
                        (size_t)p.grid * 2 * sizeof(FirstTile);
    attn_plan_kernel<<<1, kPlanThreads, smem, st>>>(p, sets, const_cast<CtaPlan*>(p.plan_cta),
                                                    const_cast<PieceDesc*>(p.plan_pieces), static_cast<GroupDesc*>(p.group_desc));
    return cudaGetLastError();
}

}  // namespace tts
