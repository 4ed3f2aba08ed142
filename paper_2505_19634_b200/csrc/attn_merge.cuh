// Group-wise merge of the split-KV partial results: a group (b, kvh) is the nr output rows of one
// branch and KV head.  Its rows belong to at most kMaxPrivBlocks private segments (row blocks) and to
// at most kMaxPreBlocks prefix segments (the stacked rows b*nr .. b*nr+nr-1 cut by row blocks); every
// such segment was computed in `n` pieces by consecutive CTAs, piece c of it leaving its rows at
// partial row (first + c) * stride + (row within the block).  For kernels that leave one partial
// result per piece and row (no replicated rows).
#pragma once
#include "tts_internal.cuh"

namespace tts {

constexpr int kMaxPrivBlocks = 2, kMaxPreBlocks = 3;     // nr <= 2 row blocks
struct GroupDesc {
    int group;                                           // b * Hkv + kvh
    int pre_row0;                                        // stacked row of the group's first row among the rows that share its prefix
    int pre_rb0;                                         // first prefix row block of the group's stacked rows
    int priv_first[kMaxPrivBlocks], priv_n[kMaxPrivBlocks];
    int pre_first[kMaxPreBlocks], pre_n[kMaxPreBlocks];
};

// Where a set of branches that share one prefix (p describes them alone: N, P, branch_lens and the
// segment counts are theirs) sits within a call that carries several such sets: its first branch, the tiles
// of the sets before it in the tile list, and the prefix partial-result slots they take.
struct SetOffsets { int first_branch, tile_off, pre_slot_base; };

// One entry of the descriptor of group (b, kvh), b counted within its set, so that the entries can be
// computed by different threads: e < kMaxPrivBlocks is private row block e, the others prefix row block
// e - kMaxPrivBlocks of the group's stacked rows (tpc = tiles per CTA of the kernel that produced the pieces).
__device__ inline void group_describe_entry(const AttnParams& p, const int* cum, int tpc, int b, int kvh, int e, GroupDesc& d,
                                            const SetOffsets so = SetOffsets{0, 0, 0}) {
    const int group = b * p.Hkv + kvh;
    if (e < kMaxPrivBlocks) {
        const int rb = e, tiles_b = cum[b + 1] - cum[b];
        d.priv_first[rb] = 0; d.priv_n[rb] = 0;
        if (rb < p.n_rb_priv && tiles_b > 0) {
            const int tb = so.tile_off + group_tile_begin(p, cum, group) + rb * tiles_b, c0 = fast_div(tb, tpc);
            d.priv_first[rb] = (so.first_branch * p.Hkv + group) * p.n_rb_priv + rb + c0;
            d.priv_n[rb] = fast_div(tb + tiles_b - 1, tpc) - c0 + 1;
        }
    } else {
        const int k = e - kMaxPrivBlocks;
        const int rb0 = fast_div(b * p.nr, p.rb_rows), rb_last = fast_div(b * p.nr + p.nr - 1, p.rb_rows);
        if (k == 0) { d.group = so.first_branch * p.Hkv + group; d.pre_row0 = b * p.nr; d.pre_rb0 = rb0; }
        d.pre_first[k] = 0; d.pre_n[k] = 0;
        if (p.n_pre > 0 && rb0 + k <= rb_last) {
            const int seg = kvh * p.n_rb_pre + rb0 + k;
            const int tb = so.tile_off + prefix_segment_tile_begin(p, cum, seg), c0 = fast_div(tb, tpc);
            d.pre_first[k] = so.pre_slot_base + seg + c0;
            d.pre_n[k] = fast_div(tb + p.tiles_pre - 1, tpc) - c0 + 1;
        }
    }
}

// Merge of the rows of one group from a descriptor, by a whole thread block: half a warp per output
// row, eight head dims per lane.  All loads of a row (up to kMergeBatch partial results at a time)
// are issued before the first is used; no lane waits for another.
constexpr int kMergeBatch = 8;
__device__ inline void merge_group(const AttnParams& p, const GroupDesc& d, int tid, int n_threads) {
    const int b = d.group / p.Hkv, kvh = d.group - b * p.Hkv;
    const int sub = tid & 15;                                            // dims [8 sub, 8 sub + 8)
    for (int r = tid >> 4; r < p.nr; r += n_threads >> 4) {
        const int i = r / p.G, gq = r - i * p.G;
        const int rb = r / p.rb_rows, r_in = r - rb * p.rb_rows;         // private row block, row within it
        const int pr = d.pre_row0 + r;
        const int k = pr / p.rb_rows - d.pre_rb0, pr_in = pr % p.rb_rows;   // prefix row block (relative), row within it
        const int n_pre = d.pre_n[k], np = n_pre + d.priv_n[rb];
        float m_run = -INFINITY, l_run = 0.f;
        float acc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = 0.f;
        for (int base = 0; base < np; base += kMergeBatch) {
            float2 ml[kMergeBatch];
            float4 o[kMergeBatch][2];
#pragma unroll
            for (int j = 0; j < kMergeBatch; ++j) {
                ml[j] = make_float2(-INFINITY, 0.f);
                o[j][0] = o[j][1] = make_float4(0.f, 0.f, 0.f, 0.f);
                const int e = base + j;
                if (e < np) {
                    const bool pre = e < n_pre;
                    const size_t row = pre ? (size_t)(d.pre_first[k] + e) * p.pre_stride + pr_in
                                           : (size_t)(d.priv_first[rb] + e - n_pre) * p.priv_stride + r_in;
                    ml[j] = (pre ? p.part_ml_pre : p.part_ml_priv)[row];
                    const float4* src = reinterpret_cast<const float4*>((pre ? p.part_o_pre : p.part_o_priv) + row * kHeadDim) + 2 * sub;
                    o[j][0] = src[0]; o[j][1] = src[1];
                }
            }
            float m_new = m_run;
#pragma unroll
            for (int j = 0; j < kMergeBatch; ++j)
                if (ml[j].y > 0.f) m_new = fmaxf(m_new, ml[j].x);       // l == 0: the piece saw no visible key for this row
            const float a = (m_run == -INFINITY || m_new == -INFINITY) ? 0.f : exp2f(m_run - m_new);
            l_run *= a;
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] *= a;
#pragma unroll
            for (int j = 0; j < kMergeBatch; ++j) {
                if (ml[j].y > 0.f) {
                    const float w = exp2f(ml[j].x - m_new);
                    l_run = fmaf(ml[j].y, w, l_run);
                    acc[0] = fmaf(o[j][0].x, w, acc[0]); acc[1] = fmaf(o[j][0].y, w, acc[1]);
                    acc[2] = fmaf(o[j][0].z, w, acc[2]); acc[3] = fmaf(o[j][0].w, w, acc[3]);
                    acc[4] = fmaf(o[j][1].x, w, acc[4]); acc[5] = fmaf(o[j][1].y, w, acc[5]);
                    acc[6] = fmaf(o[j][1].z, w, acc[6]); acc[7] = fmaf(o[j][1].w, w, acc[7]);
                }
            }
            m_run = m_new;
        }
        const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] *= inv;
        const size_t out_row = (size_t)(b * p.R + i) * p.Hq + kvh * p.G + gq;
        if (p.out_dtype == TTS_OUT_FP32) {
            float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.out) + out_row * kHeadDim) + 2 * sub;
            dst[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
            dst[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
        } else {
            __nv_bfloat162 h[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) h[e] = __floats2bfloat162_rn(acc[2 * e], acc[2 * e + 1]);
            *(reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.out) + out_row * kHeadDim) + sub) = *reinterpret_cast<uint4*>(h);
        }
    }
}

}  // namespace tts
