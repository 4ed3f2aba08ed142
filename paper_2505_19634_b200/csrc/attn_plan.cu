// Builds the plan tables (attn_plan.cuh): the pieces of every CTA of the token-major kernel, the pages
// of each CTA's first two tiles, and the merge descriptors of every (branch, KV head).  One CTA; thread c
// walks the run of CTA c of the main kernel through the segment list of tts_internal.cuh.
#include "attn_merge.cuh"
#include "attn_plan.cuh"
#include "tts_internal.cuh"

namespace tts {

namespace {

constexpr int kPlanThreads = 1024;

// Where the pages of one of a CTA's first two tiles are listed: block-table row, first block, number of
// pages, KV head (-1 pages: no such tile).
struct FirstTile { int bt_row, blk0, n_pages, kvh; };

// Walks the run of CTA c.  With out == nullptr only counts its pieces.
__device__ int walk_run(const AttnParams& p, const int* cum, int total, int tpc, int c, PieceDesc* out, CtaPlan* hdr, FirstTile* first2) {
    const int g_begin = c * tpc, g_end = min(total, g_begin + tpc);
    if (hdr) {
        hdr->n_tiles = max(0, g_end - g_begin);
        first2[0].n_pages = first2[1].n_pages = 0;
    }
    if (g_begin >= g_end) return 0;
    SegInfo seg = segment_of_tile(p, cum, g_begin);
    int n = 0, u = 0;                                      // pieces, tiles so far
    for (;;) {
        const int t_first = max(0, g_begin - seg.tile_begin);
        const int t_last = min(seg.n_tiles, g_end - seg.tile_begin);
        if (out) {
            PieceDesc d;
            d.kind = seg.kind; d.b = seg.kind == 0 ? 0 : seg.b; d.kvh = seg.kvh;
            d.row0 = seg.row0; d.n_rows = seg.n_rows;
            d.bt_row = seg.kind == 0 ? 0 : seg.b;
            d.tok_begin = seg.tok_begin; d.seg_tokens = seg.n_tokens;
            d.tile0 = t_first; d.n_tiles = t_last - t_first;
            d.slot = (seg.kind == 0 ? seg.kvh * p.n_rb_pre + seg.rb : (seg.b * p.Hkv + seg.kvh) * p.n_rb_priv + seg.rb) + c;
            d.pad = 0;
            out[n] = d;
            if (n < kPlanInline) hdr->first_pieces[n] = d;
            for (int t = t_first; t < t_last && u < 2; ++t, ++u) {
                const int tok0 = t * p.tile_tokens;
                first2[u].bt_row = d.bt_row; first2[u].blk0 = (seg.tok_begin + tok0) / kPage;
                first2[u].n_pages = min(8, ceil_div(min(p.tile_tokens, seg.n_tokens - tok0), kPage));
                first2[u].kvh = seg.kvh;
            }
        }
        ++n;
        if (seg.tile_begin + t_last >= g_end) break;
        seg = next_segment(p, cum, seg);
    }
    return n;
}

__global__ void __launch_bounds__(kPlanThreads) attn_plan_kernel(const AttnParams p, CtaPlan* cta, PieceDesc* pieces, GroupDesc* groups) {
    extern __shared__ int sm[];
    int* cum = sm;                                         // N + 1 ints
    int* first = sm + p.N + 1;                             // grid + 1 ints: index of every CTA's first piece
    FirstTile* first2 = reinterpret_cast<FirstTile*>(first + p.grid + 1);   // 2 per CTA
    build_branch_tile_prefix(p, cum);
    const int total = total_tiles(p, cum);
    const int tpc = ceil_div(total, p.grid);
    for (int c = threadIdx.x; c < p.grid; c += blockDim.x) first[c + 1] = walk_run(p, cum, total, tpc, c, nullptr, nullptr, nullptr);
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
        cta[c].n_pieces = walk_run(p, cum, total, tpc, c, pieces + first[c], cta + c, first2 + 2 * c);
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
    constexpr int kEntries = kMaxPrivBlocks + kMaxPreBlocks;
    if (groups)
        for (int i = threadIdx.x; i < p.N * p.Hkv * kEntries; i += blockDim.x) {
            const int grp = i / kEntries;
            group_describe_entry(p, cum, tpc, grp / p.Hkv, grp % p.Hkv, i % kEntries, groups[grp]);
        }
}

}  // namespace

cudaError_t launch_attn_plan(const AttnParams& main_params, cudaStream_t st) {
    AttnParams p = main_params;
    p.lens_smem = 0;
    const size_t smem = (size_t)(p.N + 1 + p.grid + 1) * sizeof(int) + (size_t)p.grid * 2 * sizeof(FirstTile);
    attn_plan_kernel<<<1, kPlanThreads, smem, st>>>(p, const_cast<CtaPlan*>(p.plan_cta), const_cast<PieceDesc*>(p.plan_pieces),
                                                    static_cast<GroupDesc*>(p.group_desc));
    return cudaGetLastError();
}

}  // namespace tts
