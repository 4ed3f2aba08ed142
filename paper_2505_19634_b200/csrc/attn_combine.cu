// Merge of the split-KV partial results: for every output row, the log-sum-exp combination of
// the pieces of its prefix segment and of its private segment, normalisation and the cast to
// the output type.  One warp per output row, four head dims per lane.
#include "attn_merge.cuh"
#include "tts_internal.cuh"

namespace tts {

namespace {

constexpr int kRowsPerBlock = 4;

__global__ void __launch_bounds__(kRowsPerBlock * 32) attn_combine_kernel(const AttnParams p) {
    extern __shared__ int cum[];                                         // N + 1 ints
    build_branch_tile_prefix(p, cum);
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * kRowsPerBlock + (threadIdx.x >> 5);     // (b, i, h) flattened
    if (row >= p.N * p.R * p.Hq) return;
    const int h = row % p.Hq, i = (row / p.Hq) % p.R, b = row / (p.Hq * p.R);
    const int kvh = h / p.G, gq = h % p.G;
    const int tiles_b = cum[b + 1] - cum[b];
    const int total = total_tiles(p, cum);
    const int tpc = ceil_div(total, p.grid);

    // The row's partial results: `n_copies` stacked blocks of `rows_in_block` rows per piece, row r of
    // every block belongs to this output row; first the pieces of its prefix segment, then those of its
    // private segment.  Lanes fetch the (m, l) of up to 32 partials at once; the O rows are then loaded
    // back to back (their addresses do not depend on the weights).
    struct Part { const float* o; const float2* ml; int stride, seg, r0, rows_in_block, n_copies, c0, n; };
    Part part[2];
    int n_kinds = 0;
    const int r_priv = i * p.G + gq;
    if (p.n_pre > 0) {
        const int pr = b * p.nr + r_priv;
        const int rb = pr / p.rb_rows, r = pr % p.rb_rows;
        const int seg = kvh * p.n_rb_pre + rb;
        const int t_begin = prefix_segment_tile_begin(p, cum, seg);
        const int c0 = t_begin / tpc, c1 = (t_begin + p.tiles_pre - 1) / tpc;
        part[n_kinds++] = Part{p.part_o_pre, p.part_ml_pre, p.pre_stride, seg, r, min(p.rb_rows, p.N * p.nr - rb * p.rb_rows),
                               p.copies_pre, c0, (c1 - c0 + 1) * p.copies_pre};
    }
    if (tiles_b > 0) {
        const int rb = r_priv / p.rb_rows, r = r_priv % p.rb_rows;
        const int seg = (b * p.Hkv + kvh) * p.n_rb_priv + rb;
        const int t_begin = group_tile_begin(p, cum, b * p.Hkv + kvh) + rb * tiles_b;
        const int c0 = t_begin / tpc, c1 = (t_begin + tiles_b - 1) / tpc;
        part[n_kinds++] = Part{p.part_o_priv, p.part_ml_priv, p.priv_stride, seg, r, min(p.rb_rows, p.nr - rb * p.rb_rows),
                               p.copies, c0, (c1 - c0 + 1) * p.copies};
    }
    const int np = (n_kinds > 0 ? part[0].n : 0) + (n_kinds > 1 ? part[1].n : 0);

    float m_run = -INFINITY, l_run = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int base = 0; base < np; base += 32) {
        int j = base + lane;
        const float* o_row = p.part_o_priv;                  // any valid address for lanes without a partial
        float2 ml = make_float2(-INFINITY, 0.f);
        if (j < np) {
            const Part& k = (n_kinds > 1 && j >= part[0].n) ? part[1] : part[0];
            if (n_kinds > 1 && j >= part[0].n) j -= part[0].n;
            const int c = k.c0 + j / k.n_copies, r = (j % k.n_copies) * k.rows_in_block + k.r0;
            const size_t row = (size_t)(k.seg + c) * k.stride + r;
            o_row = k.o + row * kHeadDim;
            ml = k.ml[row];
        }
        const bool live = ml.y > 0.f;                       // else the piece saw no visible key for this row
        float m_new = live ? ml.x : -INFINITY;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m_new = fmaxf(m_new, __shfl_xor_sync(0xffffffffu, m_new, o));
        m_new = fmaxf(m_new, m_run);
        const float a = (m_run == -INFINITY || m_new == -INFINITY) ? 0.f : exp2f(m_run - m_new);
        const float w = live ? exp2f(ml.x - m_new) : 0.f;
        float lw = ml.y * w;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) lw += __shfl_xor_sync(0xffffffffu, lw, o);
        l_run = l_run * a + lw;
        acc.x *= a; acc.y *= a; acc.z *= a; acc.w *= a;
        m_run = m_new;
        const int cnt = min(32, np - base);
        const unsigned long long o_addr = reinterpret_cast<unsigned long long>(o_row);
#pragma unroll 4
        for (int jj = 0; jj < cnt; ++jj) {
            const float wj = __shfl_sync(0xffffffffu, w, jj);
            const float4 o = *(reinterpret_cast<const float4*>(__shfl_sync(0xffffffffu, o_addr, jj)) + lane);
            if (wj > 0.f) {
                acc.x = fmaf(o.x, wj, acc.x); acc.y = fmaf(o.y, wj, acc.y);
                acc.z = fmaf(o.z, wj, acc.z); acc.w = fmaf(o.w, wj, acc.w);
            }
        }
    }

    const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
    acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    if (p.out_dtype == TTS_OUT_FP32) {
        *reinterpret_cast<float4*>(static_cast<float*>(p.out) + (size_t)row * kHeadDim + lane * 4) = acc;
    } else {
        __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
        uint2 pk;
        pk.x = *reinterpret_cast<unsigned*>(&lo);
        pk.y = *reinterpret_cast<unsigned*>(&hi);
        *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(p.out) + (size_t)row * kHeadDim + lane * 4) = pk;
    }
}

// The same merge for the common layout (one partial result per piece and row, at most two row blocks
// per branch and KV head), arranged for latency, which is all this kernel costs: one CTA per group
// (branch, KV head), half a warp per output row; five threads work out where the group's partial
// results lie, then every thread issues all loads of its row before it uses the first.
__global__ void __launch_bounds__(512) attn_combine_groups_kernel(const AttnParams p) {
    extern __shared__ int cum[];                                         // N + 1 ints
    __shared__ GroupDesc desc;
    static_assert(sizeof(GroupDesc) % sizeof(int) == 0, "GroupDesc is copied word by word");
    if (p.group_desc) {                                                  // the main kernel has worked it out
        if (threadIdx.x < sizeof(GroupDesc) / sizeof(int))
            reinterpret_cast<int*>(&desc)[threadIdx.x] = reinterpret_cast<const int*>(static_cast<const GroupDesc*>(p.group_desc) + blockIdx.x)[threadIdx.x];
    } else {
        build_branch_tile_prefix(p, cum);
        const int b = blockIdx.x / p.Hkv, kvh = blockIdx.x - b * p.Hkv;
        if (threadIdx.x < kMaxPrivBlocks + kMaxPreBlocks)
            group_describe_entry(p, cum, ceil_div(total_tiles(p, cum), p.grid), b, kvh, threadIdx.x, desc);
    }
    __syncthreads();
    merge_group(p, desc, threadIdx.x, blockDim.x);
}

}  // namespace

cudaError_t launch_attn_combine(const AttnParams& main_params, cudaStream_t st) {
    AttnParams p = main_params;
    if (p.copies == 1 && p.copies_pre == 1 && p.n_rb_priv <= kMaxPrivBlocks && p.nr <= 2 * p.rb_rows) {
        const int threads = min(512, (p.nr * 16 + 31) / 32 * 32);        // 128 registers each: a row's loads are all in flight at once
        attn_combine_groups_kernel<<<p.N * p.Hkv, threads, (p.N + 1) * sizeof(int), st>>>(p);
        return cudaGetLastError();
    }
    const int rows = p.N * p.R * p.Hq;
    attn_combine_kernel<<<ceil_div(rows, kRowsPerBlock), kRowsPerBlock * 32, (p.N + 1) * sizeof(int), st>>>(p);
    return cudaGetLastError();
}

}  // namespace tts
