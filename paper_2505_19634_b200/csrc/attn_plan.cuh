// The schedule of an attention call as tables in device memory ("plan"), built once by a small
// kernel and then read by every launch that works on the same block table and branch lengths: the
// 64 layers of a verify step share one plan, so the per-layer kernels start from a table read
// instead of rebuilding the work decomposition of tts_internal.cuh.
#pragma once
#include "tts_internal.cuh"

namespace tts {

// One piece: the part of a segment that falls into one CTA's run of the tile list.
struct __align__(16) PieceDesc {
    int kind;        // 0 prefix, 1 private
    int b;           // private: the branch; prefix: first branch of the rows stacked in the segment
    int kvh;
    int row0;        // first stacked row of the segment's row block
    int n_rows;      // valid rows of the row block
    int bt_row;      // row of the block table that lists the segment's pages
    int tok_begin;   // logical token (within that row) of the segment's first key
    int seg_tokens;  // keys in the segment
    int tile0;       // first tile of the piece inside its segment
    int n_tiles;     // tiles of the piece
    int slot;        // the piece's partial result: rows [slot * stride, ..) of the workspace of its kind
    int pad;
};
static_assert(sizeof(PieceDesc) == 48, "PieceDesc is copied as three 16-byte words");

// Per CTA, one 512-byte record that the CTA copies to shared memory with a single coalesced read: where
// its pieces are, the pages of its first two tiles (their loads are the first thing the CTA issues, so they
// must not wait for a dependent read of the block table), and a copy of its first pieces.
constexpr int kPlanInline = 8;         // pieces of a CTA held in its record; further ones are read from the global list
struct __align__(16) CtaPlan {
    int piece_begin, n_pieces; // the CTA's pieces are plan_pieces[piece_begin .. piece_begin + n_pieces)
    int n_tiles;               // all tiles of the CTA's run
    int pad0;
    int first_pages[16];       // page * Hkv + kvh for the (up to) 8 pages of tiles 0 and 1; -1 = no such page
    int pad1[12];
    PieceDesc first_pieces[kPlanInline];
};
static_assert(sizeof(CtaPlan) == 512, "CtaPlan is copied as 32 x 16 bytes");

// Builds the tables for the schedule that `p` and the prefix sets describe (p.plan_cta, p.plan_pieces,
// p.group_desc must point to the context's tables).  One launch of one CTA.
cudaError_t launch_attn_plan(const AttnParams& p, const PrefixSets& sets, cudaStream_t st);

}  // namespace tts
