// Merge of the split-KV partial results: for every output row, the log-sum-exp combination of
// the pieces of its prefix segment and of its private segment, normalisation and the cast to
// the output type.  One warp per output row, four head dims per lane.
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

    float m_run = -INFINITY, l_run = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);

    // rows of one piece: `n_copies` stacked blocks of `rows_in_block` rows; row r of every block
    // belongs to this output row
    auto merge = [&](const float* o_base, const float2* ml_base, int stride, int seg_local, int r0,
                     int rows_in_block, int n_copies, int t_begin, int n_tiles) {
        if (n_tiles <= 0) return;
        const int c0 = t_begin / tpc, c1 = (t_begin + n_tiles - 1) / tpc;
        for (int cc = c0 * n_copies; cc < (c1 + 1) * n_copies; ++cc) {
            const int c = cc / n_copies, r = (cc % n_copies) * rows_in_block + r0;
            const size_t id = (size_t)seg_local + c;
            const float2 ml = ml_base[id * stride + r];
            if (!(ml.y > 0.f)) continue;                  // piece saw no visible key for this row
            const float4 o = *reinterpret_cast<const float4*>(
                o_base + (id * stride + r) * kHeadDim + lane * 4);
            const float m_new = fmaxf(m_run, ml.x);
            const float a = (m_run == -INFINITY) ? 0.f : exp2f(m_run - m_new);
            const float w = exp2f(ml.x - m_new);
            acc.x = acc.x * a + o.x * w; acc.y = acc.y * a + o.y * w;
            acc.z = acc.z * a + o.z * w; acc.w = acc.w * a + o.w * w;
            l_run = l_run * a + ml.y * w;
            m_run = m_new;
        }
    };

    const int r_priv = i * p.G + gq;
    if (p.n_pre > 0) {
        const int pr = b * p.nr + r_priv;
        const int rb = pr / p.rb_rows, r = pr % p.rb_rows;
        const int seg = kvh * p.n_rb_pre + rb;
        merge(p.part_o_pre, p.part_ml_pre, p.pre_stride, seg, r, min(p.rb_rows, p.N * p.nr - rb * p.rb_rows), p.copies_pre,
              prefix_segment_tile_begin(p, cum, seg), p.tiles_pre);
    }
    {
        const int rb = r_priv / p.rb_rows, r = r_priv % p.rb_rows;
        const int seg = (b * p.Hkv + kvh) * p.n_rb_priv + rb;
        merge(p.part_o_priv, p.part_ml_priv, p.priv_stride, seg, r, min(p.rb_rows, p.nr - rb * p.rb_rows), p.copies,
              group_tile_begin(p, cum, b * p.Hkv + kvh) + rb * tiles_b, tiles_b);
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

}  // namespace

cudaError_t launch_attn_combine(const AttnParams& p, cudaStream_t st) {
    const int rows = p.N * p.R * p.Hq;
    attn_combine_kernel<<<ceil_div(rows, kRowsPerBlock), kRowsPerBlock * 32, (p.N + 1) * sizeof(int), st>>>(p);
    return cudaGetLastError();
}

}  // namespace tts
