// CUDA-core verify attention: the path used when the stacked query rows per KV head are too few
// for tensor-core tiles to pay, and the reference point for the tcgen05 kernel.
//
// Persistent grid over the global tile list (see tts_internal.cuh).  One CTA = 128 threads works
// on one piece at a time: RB query rows (fp32 in shared memory) against tiles of 64 KV tokens
// staged in shared memory with 16-byte loads, scores on CUDA cores, fp32 online softmax with
// warp-shuffle reductions, P.V on CUDA cores, partial (m, l, O) to the workspace.
#include "tts_internal.cuh"

namespace tts {

namespace {

constexpr int kThreads = 128;
constexpr int kTile = kSimtTileTokens;       // 64 tokens
constexpr int kKStride = kHeadDim + 8;       // bf16 elements per K row in smem (272 B: conflict-free 16-B reads)

__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 t = __bfloat1622float2(h[i]);
        f[2 * i] = t.x; f[2 * i + 1] = t.y;
    }
}

template <int RB>
struct SimtSmem {
    float q[RB][kHeadDim];
    __nv_bfloat16 k[kTile][kKStride];
    __nv_bfloat16 v[kTile][kHeadDim];
    float s[kTile][RB];                // scores, then probabilities, token-major
    unsigned long long vis[RB];
    float m[RB], l[RB], alpha[RB];
};

template <int RB>
__global__ void __launch_bounds__(kThreads) attn_simt_kernel(const AttnParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SimtSmem<RB>& sm = *reinterpret_cast<SimtSmem<RB>*>(smem_raw);
    int* cum = reinterpret_cast<int*>(smem_raw + sizeof(SimtSmem<RB>));

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    build_branch_tile_prefix(p, cum);
    const int total = total_tiles(p, cum);
    const int tpc = ceil_div(total, p.grid);
    int g = blockIdx.x * tpc;
    const int g_end = min(total, g + tpc);

    while (g < g_end) {
        const SegInfo seg = segment_of_tile(p, cum, g);
        const int t_first = g - seg.tile_begin;                                   // first tile of the piece
        const int t_last = min(seg.n_tiles, g_end - seg.tile_begin);              // one past the last
        const int L = seg.n_tokens;
        const int bt_row = seg.kind == 0 ? 0 : seg.b;
        const int32_t* bt = p.block_table + (size_t)bt_row * p.max_blocks;

        // ---- stage the query rows of this piece (zero rows beyond n_rows) ----
        for (int idx = tid; idx < RB * (kHeadDim / 8); idx += kThreads) {
            const int r = idx / (kHeadDim / 8), part = idx % (kHeadDim / 8);
            float f[8];
            if (r < seg.n_rows) {
                int row = seg.row0 + r, b = seg.b;
                if (seg.kind == 0) { b = row / p.nr; row = row % p.nr; }
                const int i = row / p.G, gq = row % p.G;
                const __nv_bfloat16* src =
                    p.q + (((size_t)b * p.R + i) * p.Hq + seg.kvh * p.G + gq) * kHeadDim + part * 8;
                unpack8(*reinterpret_cast<const uint4*>(src), f);
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) f[e] = 0.f;
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) sm.q[r][part * 8 + e] = f[e];
        }
        if (tid < RB) {
            unsigned long long vis = ~0ull;
            if (seg.kind == 1 && tid < seg.n_rows) vis = row_visibility(p, seg.b, (seg.row0 + tid) / p.G);
            sm.vis[tid] = vis;
            sm.m[tid] = -INFINITY; sm.l[tid] = 0.f;
        }
        float acc[RB];
#pragma unroll
        for (int r = 0; r < RB; ++r) acc[r] = 0.f;
        __syncthreads();

        for (int tile = t_first; tile < t_last; ++tile) {
            const int tok0 = tile * kTile;                       // token offset inside the segment
            const int n_valid = min(kTile, L - tok0);
            // ---- stage K and V (16-byte loads; tokens past the end become zeros) ----
            for (int idx = tid; idx < kTile * (kHeadDim / 8); idx += kThreads) {
                const int t = idx / (kHeadDim / 8), part = idx % (kHeadDim / 8);
                uint4 kv = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
                if (t < n_valid) {
                    const int tok = seg.tok_begin + tok0 + t;
                    const int page = checked_page(p, bt, tok / kPage);
                    const size_t off = (((size_t)page * p.Hkv + seg.kvh) * kPage + tok % kPage) * kHeadDim + part * 8;
                    kv = *reinterpret_cast<const uint4*>(p.k_pages + off);
                    vv = *reinterpret_cast<const uint4*>(p.v_pages + off);
                }
                *reinterpret_cast<uint4*>(&sm.k[t][part * 8]) = kv;
                *reinterpret_cast<uint4*>(&sm.v[t][part * 8]) = vv;
            }
            __syncthreads();

            // ---- scores: thread = (token, half of the rows) ----
            {
                constexpr int HR = RB / 2;
                const int t = tid & (kTile - 1), r0 = (tid >> 6) * HR;
                float dot[HR];
#pragma unroll
                for (int r = 0; r < HR; ++r) dot[r] = 0.f;
#pragma unroll 4
                for (int part = 0; part < kHeadDim / 8; ++part) {
                    float kf[8];
                    unpack8(*reinterpret_cast<const uint4*>(&sm.k[t][part * 8]), kf);
#pragma unroll
                    for (int r = 0; r < HR; ++r) {
                        const float4 qa = *reinterpret_cast<const float4*>(&sm.q[r0 + r][part * 8]);
                        const float4 qb = *reinterpret_cast<const float4*>(&sm.q[r0 + r][part * 8 + 4]);
                        dot[r] = fmaf(qa.x, kf[0], dot[r]); dot[r] = fmaf(qa.y, kf[1], dot[r]);
                        dot[r] = fmaf(qa.z, kf[2], dot[r]); dot[r] = fmaf(qa.w, kf[3], dot[r]);
                        dot[r] = fmaf(qb.x, kf[4], dot[r]); dot[r] = fmaf(qb.y, kf[5], dot[r]);
                        dot[r] = fmaf(qb.z, kf[6], dot[r]); dot[r] = fmaf(qb.w, kf[7], dot[r]);
                    }
                }
#pragma unroll
                for (int r = 0; r < HR; ++r) sm.s[t][r0 + r] = dot[r] * p.scale_log2;
            }
            __syncthreads();

            // ---- online softmax, one warp per row, two tokens per lane ----
            for (int r = warp; r < RB; r += kThreads / 32) {
                const unsigned long long vis = sm.vis[r];
                float sc[2];
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    const int t = lane + 32 * k;
                    const int j = tok0 + t;
                    bool ok = t < n_valid;
                    if (seg.kind == 1 && j >= L - p.R) ok = ok && ((vis >> (j - (L - p.R))) & 1ull);
                    sc[k] = ok ? sm.s[t][r] : -INFINITY;
                }
                float mx = fmaxf(sc[0], sc[1]);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                const float m_old = sm.m[r];
                const float m_new = fmaxf(m_old, mx);
                float pr[2], sum = 0.f;
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    pr[k] = (sc[k] == -INFINITY) ? 0.f : exp2f(sc[k] - m_new);
                    sum += pr[k];
                    sm.s[lane + 32 * k][r] = pr[k];
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
                if (lane == 0) {
                    const float a = (m_old == -INFINITY) ? 0.f : exp2f(m_old - m_new);
                    sm.alpha[r] = (m_new == -INFINITY) ? 1.f : a;
                    sm.l[r] = sm.l[r] * a + sum;
                    sm.m[r] = m_new;
                }
            }
            __syncthreads();

            // ---- O = O * alpha + P V : thread = one of the 128 output dims ----
#pragma unroll
            for (int r = 0; r < RB; ++r) acc[r] *= sm.alpha[r];
#pragma unroll 2
            for (int t = 0; t < kTile; ++t) {
                const float v = __bfloat162float(sm.v[t][tid]);
#pragma unroll
                for (int r4 = 0; r4 < RB; r4 += 4) {
                    const float4 pw = *reinterpret_cast<const float4*>(&sm.s[t][r4]);
                    acc[r4] = fmaf(pw.x, v, acc[r4]);
                    acc[r4 + 1] = fmaf(pw.y, v, acc[r4 + 1]);
                    acc[r4 + 2] = fmaf(pw.z, v, acc[r4 + 2]);
                    acc[r4 + 3] = fmaf(pw.w, v, acc[r4 + 3]);
                }
            }
            __syncthreads();
        }

        // ---- partial result of the piece ----
        float* po; float2* pml;
        piece_slot(p, seg, blockIdx.x, po, pml);
#pragma unroll
        for (int r = 0; r < RB; ++r)
            if (r < seg.n_rows) po[(size_t)r * kHeadDim + tid] = acc[r];
        if (tid < seg.n_rows) pml[tid] = make_float2(sm.m[tid], sm.l[tid]);
        __syncthreads();
        g = seg.tile_begin + t_last;
    }
}

template <int RB>
cudaError_t launch_rb(const AttnParams& p, cudaStream_t st) {
    const size_t smem = sizeof(SimtSmem<RB>) + (size_t)(p.N + 1) * sizeof(int);
    cudaError_t e = cudaFuncSetAttribute(attn_simt_kernel<RB>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)(sizeof(SimtSmem<RB>) + (kMaxBranches + 1) * sizeof(int)));
    if (e != cudaSuccess) return e;
    attn_simt_kernel<RB><<<p.grid, kThreads, smem, st>>>(p);
    return cudaGetLastError();
}

}  // namespace

int simt_rb_rows(int nr) { return nr <= 8 ? 8 : (nr <= 16 ? 16 : 32); }

cudaError_t launch_attn_simt(const AttnParams& p, cudaStream_t st) {
    switch (p.rb_rows) {
        case 8: return launch_rb<8>(p, st);
        case 16: return launch_rb<16>(p, st);
        case 32: return launch_rb<32>(p, st);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace tts
