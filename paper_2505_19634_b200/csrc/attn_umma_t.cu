// Token-major tensor-core verify attention for sm_100a: the kernel for FEW query rows per KV head
// (at most 64 stacked rows per row block; a chain of gamma+1 positions times the GQA group).
//
// With 20 or 40 query rows a row-major score tile would leave most of the 128-row MMA idle, so
// the KV tokens go on the MMA M dimension instead and both contractions are computed transposed:
//     S^T[128 tokens x NB rows] = K[128 x 128] . Q^T        (A = K tile, B = Q block, both K-major)
//     O^T[128 dims   x NB rows] = V^T[128 x 128] . P^T      (A = V tile as MN-major, B = P^T K-major)
// NB is 32 or 64.  The operands K and V are the TMA-staged page tiles themselves; Q and P^T are
// small (NB x 256 bytes), which leaves room for a ring of 5-6 operand tiles (32 KiB each) in shared
// memory, the depth that hides HBM latency at 4 KiB page granularity.
//
// One persistent CTA per SM walks its run of the global tile list (tts_internal.cuh):
//   warp 4*CG   producer: per tile arms the "full" barrier of the next ring slot with the byte count
//               and issues the TMA boxes of the K tile, then of the V tile (8 pages x 2 boxes each)
//   warp 4*CG+1 MMA issuer (one thread): S^T into one of two TMEM buffers, O^T (+)= V^T P^T once the
//               softmax warps have published P^T; tcgen05.commit frees ring slots and P buffers
//   warps 0..4*CG-1  softmax: thread = (TMEM lane = KV token, column group).  The NB rows are cut
//               into chunks of 4; column group cg owns chunks cg, cg+CG, ... and a thread holds the
//               scores of its token for the rows of its chunks (chunks past the piece's last row are
//               skipped).  The running reference m of every row lives in shared memory and only
//               moves when some score exceeds it by more than 2^8 (consensus through a reducing
//               named barrier; the exact row maximum is then found with warp redux + shared memory
//               and O^T is rescaled in TMEM).  The result is exact either way: l is accumulated
//               against the same reference.  Row sums are kept per thread and reduced once per piece.
//
// Every wait is bounded.  A wait that runs out raises TTS_ERR_DEVICE_TIMEOUT; the softmax warps only
// leave their loops on the result of a block-wide reduction, so no thread is left behind at a named
// barrier; in-flight copies are awaited (bounded) and TMEM is released before the CTA returns.
#include <cuda.h>

#include "tts_internal.cuh"
#include "umma_ptx.cuh"

namespace tts {

namespace {

using namespace ptx;

constexpr int kTileT = kUmmaTileTokens;              // 128 tokens = MMA M
constexpr int kSlotBytes = kTileT * kHeadDim * 2;    // one K or V tile: 32 KiB
constexpr int kHalfT = kTileT * 128;                 // one 64-element block of a 128-row operand: 16 KiB
constexpr float kLazy = 8.f;                         // the reference moves when exceeded by 2^8

template <int NB>
struct Lay {
    static constexpr int kSlots = NB == 32 ? 6 : 5;
    static constexpr int kQBytes = NB * 256;         // two 64-dim K-blocks of NB rows x 128 B
    static constexpr int kPBytes = NB * 256;         // two 64-token K-blocks of NB rows x 128 B
    static constexpr int kOffQ = 0;
    static constexpr int kOffP = kQBytes;            // two buffers
    static constexpr int kOffRing = kOffP + 2 * kPBytes;
    static constexpr int kOffBar = kOffRing + kSlots * kSlotBytes;
    static constexpr int kOffMisc = kOffBar + 24 * 8;            // 2 * kSlots + 9 barriers
    static constexpr int kOffMref = kOffMisc + 64;               // float[NB]
    static constexpr int kOffRed = kOffMref + NB * 4;            // float[4][NB]
    static constexpr int kOffVis = kOffRed + 4 * NB * 4;         // u64[64]
    static constexpr int kOffCum = kOffVis + 64 * 8;             // int[N + 1]
    static constexpr int kFixedBytes = kOffCum + 1024;           // + slack for the manual 1024-B alignment
    static constexpr uint32_t kTmemCols = NB == 32 ? 128 : 256;  // 2 S^T buffers + O^T, power of two
    // barrier indices
    static constexpr int FULL = 0, EMPTY = kSlots, S_FULL = 2 * kSlots, S_FREE = S_FULL + 2, P_FULL = S_FREE + 2,
                         P_FREE = P_FULL + 2, Q_FULL = P_FREE + 2;
};

// reducing / plain named barrier 1 over the NT softmax threads
template <int NT>
__device__ __forceinline__ bool bar_red_or(bool pred) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "barrier.cta.red.or.pred p, 1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out) : "r"((uint32_t)pred), "n"(NT) : "memory");
    return out != 0;
}
template <int NT>
__device__ __forceinline__ void bar_sync_softmax() { asm volatile("barrier.cta.sync 1, %0;" ::"n"(NT) : "memory"); }

__device__ __forceinline__ float warp_max_f32(float v) {
    int i = __float_as_int(v);
    i ^= (i >> 31) & 0x7fffffff;                                 // order-preserving map to signed int
    i = __reduce_max_sync(0xffffffffu, i);
    i ^= (i >> 31) & 0x7fffffff;
    return __int_as_float(i);
}
__device__ __forceinline__ float warp_sum_f32(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ void tmem_ld4(uint32_t taddr, float* v) {       // 4 consecutive columns of this thread's lane
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st4(uint32_t taddr, const float* v) {
    const uint32_t* r = reinterpret_cast<const uint32_t*>(v);
    asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1, %2, %3, %4};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}

// Q block of a piece -> shared memory as the K-major B operand (zero rows beyond n_rows), and, for
// private segments under a tree mask, the visibility word of every query position.
template <int NB, int NT>
__device__ __forceinline__ void stage_q(const AttnParams& p, const SegInfo& seg, unsigned char* smem, int tid) {
    using L = Lay<NB>;
    for (int idx = tid; idx < NB * 16; idx += NT) {
        const int r = idx >> 4, c = idx & 15;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (r < seg.n_rows) {
            int row = seg.row0 + r, b = seg.b;
            if (seg.kind == 0) { b = row / p.nr; row = row % p.nr; }
            const int i = row / p.G, gq = row % p.G;
            const __nv_bfloat16* src = p.q + (((size_t)b * p.R + i) * p.Hq + seg.kvh * p.G + gq) * kHeadDim;
            v = __ldg(reinterpret_cast<const uint4*>(src) + c);
        }
        *reinterpret_cast<uint4*>(smem + L::kOffQ + (c >> 3) * (NB * 128) + r * 128 + (((c & 7) ^ (r & 7)) << 4)) = v;
    }
    if (seg.kind == 1 && p.tree_parents != nullptr && tid < p.R)
        reinterpret_cast<unsigned long long*>(smem + L::kOffVis)[tid] = row_visibility(p, seg.b, tid);
}

template <int NB, int CG>
__global__ void __launch_bounds__(128 * CG + 64, 1)
attn_umma_t_kernel(const AttnParams p, const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v) {
    using L = Lay<NB>;
    constexpr int NS = L::kSlots;
    constexpr int NT = 128 * CG;                           // softmax threads
    constexpr int NCK = NB / 4 / CG;                       // 4-row chunks per thread
    constexpr int kProducerWarp = 4 * CG, kMmaWarp = 4 * CG + 1;
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + L::kOffBar;
    auto bar = [&](int i) { return bar0 + 8u * i; };
    volatile int* misc = reinterpret_cast<volatile int*>(smem + L::kOffMisc);   // [0] abort flag, [1] tmem base
    int* cum = reinterpret_cast<int*>(smem + L::kOffCum);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const Abort ab{misc, p.status};

    build_branch_tile_prefix(p, cum);
    const int total = total_tiles(p, cum);
    const int tpc = ceil_div(total, p.grid);
    const int g_begin = blockIdx.x * tpc;
    const int g_end = min(total, g_begin + tpc);
    if (g_begin >= g_end) return;                          // uniform: nothing to do for this CTA

    if (tid == 0) {
        misc[0] = 0;
        for (int i = 0; i < NS; ++i) { mbar_init(bar(L::FULL + i), 1); mbar_init(bar(L::EMPTY + i), 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(L::S_FULL + i), 1); mbar_init(bar(L::S_FREE + i), NT);
            mbar_init(bar(L::P_FULL + i), NT); mbar_init(bar(L::P_FREE + i), 1);
        }
        mbar_init(bar(L::Q_FULL), NT);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + L::kOffMisc + 4), "r"(L::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = (uint32_t)misc[1];
    const uint32_t tmem_s[2] = {tmem, tmem + (uint32_t)NB};
    const uint32_t tmem_o = tmem + 2u * NB;

    if (warp == kProducerWarp) {
        // =========================== producer ===========================
        int u = 0;                                          // operand tiles issued by this CTA (K, V, K, V, ...)
        int g = g_begin;
        bool alive = true;
        while (g < g_end && alive) {
            const SegInfo seg = segment_of_tile(p, cum, g);
            const int t_first = g - seg.tile_begin, t_last = min(seg.n_tiles, g_end - seg.tile_begin);
            const int32_t* bt = p.block_table + (size_t)(seg.kind == 0 ? 0 : seg.b) * p.max_blocks;
            for (int t = t_first; t < t_last && alive; ++t) {
                const int tok0 = t * kTileT;
                const int n_pages = ceil_div(min(kTileT, seg.n_tokens - tok0), kPage);
                int page = 0;
                if (lane < n_pages) {
                    page = bt[(seg.tok_begin + tok0) / kPage + lane];
                    if (p.debug && (page < 0 || page >= p.num_pages)) {
                        atomicMin(p.status, (int)TTS_ERR_DEVICE_BOUNDS);
                        page = 0;
                    }
                }
                const int y = (page * p.Hkv + seg.kvh) * kPage;
#pragma unroll
                for (int op = 0; op < 2 && alive; ++op, ++u) {
                    const int slot = u % NS;
                    if (lane == 0) {
                        alive = mbar_wait(bar(L::EMPTY + slot), ((u / NS) & 1) ^ 1, ab);
                        if (alive) mbar_arrive_expect_tx(bar(L::FULL + slot), (uint32_t)n_pages * 4096u);
                    }
                    alive = __shfl_sync(0xffffffffu, alive, 0);
                    if (alive && lane < n_pages) {
                        const uint32_t dst = sbase + L::kOffRing + slot * kSlotBytes + lane * 2048;
                        const CUtensorMap* tm = op == 0 ? &tm_k : &tm_v;
                        tma_load_2d(dst, tm, 0, y, bar(L::FULL + slot));
                        tma_load_2d(dst + kHalfT, tm, 64, y, bar(L::FULL + slot));
                    }
                }
            }
            g = seg.tile_begin + t_last;
        }
        // Copies this warp started must have landed before the CTA may exit: the consumers wait on
        // the same phases in the normal case; after an abort wait for them here (bounded).
        if (*ab.flag && lane == 0) {
            for (int back = 1; back <= NS && back <= u; ++back) {
                const int j = u - back;
                const Abort quiet{misc + 2, p.status};       // do not re-raise; misc[2] is scratch
                misc[2] = 0;
                mbar_wait(bar(L::FULL + j % NS), (j / NS) & 1, quiet);
            }
        }
    } else if (warp == kMmaWarp) {
        // =========================== MMA issuer ===========================
        if (lane == 0) {
            constexpr uint32_t idesc_qk = instr_desc(kTileT, NB, false, false);
            constexpr uint32_t idesc_pv = instr_desc(kTileT, NB, true, false);
            int it = 0, piece = 0;
            int g = g_begin;
            bool alive = true;
            auto issue_qk = [&](int j) -> bool {
                const int u = 2 * j, slot = u % NS, sb = j & 1;
                if (!mbar_wait(bar(L::FULL + slot), (u / NS) & 1, ab)) return false;
                if (!mbar_wait(bar(L::S_FREE + sb), ((j >> 1) & 1) ^ 1, ab)) return false;
                tc_fence_after();
                const uint32_t ka = sbase + L::kOffRing + slot * kSlotBytes, qa = sbase + L::kOffQ;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    umma_bf16(tmem_s[sb], smem_desc(ka + (ks >> 2) * kHalfT + (ks & 3) * 32, 16, 1024),
                              smem_desc(qa + (ks >> 2) * (NB * 128) + (ks & 3) * 32, 16, 1024), idesc_qk, ks > 0);
                umma_commit(bar(L::EMPTY + slot));
                umma_commit(bar(L::S_FULL + sb));
                return true;
            };
            while (g < g_end && alive) {
                const SegInfo seg = segment_of_tile(p, cum, g);
                const int t_first = g - seg.tile_begin, t_last = min(seg.n_tiles, g_end - seg.tile_begin);
                const int n = t_last - t_first;
                alive = mbar_wait(bar(L::Q_FULL), piece & 1, ab);
                if (!alive) break;
                tc_fence_after();
                alive = issue_qk(it);
                for (int j = 0; j < n && alive; ++j) {
                    if (j + 1 < n) { alive = issue_qk(it + j + 1); if (!alive) break; }
                    const int cur = it + j, u = 2 * cur + 1, slot = u % NS, pb = cur & 1;
                    alive = mbar_wait(bar(L::P_FULL + pb), (cur >> 1) & 1, ab) && mbar_wait(bar(L::FULL + slot), (u / NS) & 1, ab);
                    if (!alive) break;
                    tc_fence_after();
                    const uint32_t va = sbase + L::kOffRing + slot * kSlotBytes, pa = sbase + L::kOffP + pb * L::kPBytes;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)          // 16 tokens per step: V rows ks*16.., P^T 32-byte column step
                        umma_bf16(tmem_o, smem_desc(va + ks * 2048, kHalfT, 1024),
                                  smem_desc(pa + (ks >> 2) * (NB * 128) + (ks & 3) * 32, 16, 1024), idesc_pv,
                                  (j > 0 || ks > 0) ? 1u : 0u);
                    umma_commit(bar(L::EMPTY + slot));
                    umma_commit(bar(L::P_FREE + pb));
                }
                it += n; ++piece;
                g = seg.tile_begin + t_last;
            }
        }
    } else {
        // =========================== softmax warps ===========================
        // A wait that fails only clears `ok`; loops are left on block-wide reductions of !ok so that
        // all softmax threads leave together.
        float* mref = reinterpret_cast<float*>(smem + L::kOffMref);
        float* red = reinterpret_cast<float*>(smem + L::kOffRed);
        const unsigned long long* vis = reinterpret_cast<const unsigned long long*>(smem + L::kOffVis);
        const int quarter = warp & 3, cg = warp >> 2;       // TMEM lane quarter of this warp, column group
        const int tok = quarter * 32 + lane;                 // this thread's token in the tile; its dim in O^T
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        auto row_of = [&](int k) { return 4 * (cg + CG * k); };    // first row of this thread's k-th chunk
        int it = 0;
        bool ok = true;
        SegInfo seg = segment_of_tile(p, cum, g_begin);
        stage_q<NB, NT>(p, seg, smem, tid);
        fence_proxy_async();
        mbar_arrive(bar(L::Q_FULL));

        for (;;) {
            const int t_first = g_begin > seg.tile_begin ? g_begin - seg.tile_begin : 0;
            const int t_last = min(seg.n_tiles, g_end - seg.tile_begin);
            const int Ltok = seg.n_tokens;
            const int tail0 = seg.kind == 1 ? Ltok - p.R : Ltok;     // first token that needs the row mask
            const int n_rows = seg.n_rows;                            // chunks starting at or past it are skipped
            float l_part[NCK][4];
#pragma unroll
            for (int k = 0; k < NCK; ++k)
#pragma unroll
                for (int e = 0; e < 4; ++e) l_part[k][e] = 0.f;
            if (tid < NB) mref[tid] = -INFINITY;
            bar_sync_softmax<NT>();

            for (int t = t_first; t < t_last; ++t, ++it) {
                const int sb = it & 1, pb = it & 1;
                const int tok0 = t * kTileT;
                const bool need_mask = tok0 + kTileT > tail0;        // uniform: tile touches masked / missing tokens
                ok = ok && mbar_wait(bar(L::S_FULL + sb), (it >> 1) & 1, ab);
                float s[NCK][4];                                      // raw scores of this token
#pragma unroll
                for (int k = 0; k < NCK; ++k)
#pragma unroll
                    for (int e = 0; e < 4; ++e) s[k][e] = 0.f;
                if (ok) {
                    tc_fence_after();
#pragma unroll
                    for (int k = 0; k < NCK; ++k)
                        if (row_of(k) < n_rows) tmem_ld4(tmem_s[sb] + lane_base + (uint32_t)row_of(k), s[k]);
                    tmem_wait_ld();
                }
                tc_fence_before();
                mbar_arrive(bar(L::S_FREE + sb));            // the scores are in registers: S^T may be overwritten

                unsigned long long rowmask = ~0ull;         // bit r: this thread's token is visible to row r
                if (need_mask) {
                    const int j = tok0 + tok;
                    if (j >= Ltok) rowmask = 0ull;
                    else if (j >= tail0) {
                        // token a of the last R: visible to query position i = (row0 + r) / G iff i >= a
                        // (causal) or a is i or an ancestor of i (tree)
                        const int a = j - tail0;
                        if (p.tree_parents == nullptr) {
                            const int sh = a * p.G - seg.row0;
                            rowmask = sh <= 0 ? ~0ull : (sh >= 64 ? 0ull : ~0ull << sh);
                        } else {
                            rowmask = 0ull;
                            for (int r = 0; r < NB; ++r) {
                                const int i = (seg.row0 + r) / p.G;
                                if (i < p.R && ((vis[i] >> a) & 1ull)) rowmask |= 1ull << r;
                            }
                        }
                    }
                }
                // d = score * scale - reference (log2 units); masked entries are -inf
                float d[NCK][4];
                auto compute_d = [&]() -> float {
                    float mx = -INFINITY;
#pragma unroll
                    for (int k = 0; k < NCK; ++k) {
                        if (row_of(k) < n_rows) {
                            const float4 m4 = *reinterpret_cast<const float4*>(mref + row_of(k));
                            const float mm[4] = {m4.x, m4.y, m4.z, m4.w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                float v = fmaf(s[k][e], p.scale_log2, -mm[e]);      // +inf while the reference is -inf
                                if (need_mask && !((rowmask >> (row_of(k) + e)) & 1ull)) v = -INFINITY;
                                d[k][e] = v;
                                mx = fmaxf(mx, v);
                            }
                        }
                    }
                    return mx;
                };
                const float dmax = compute_d();
                if (bar_red_or<NT>(dmax > kLazy || !ok)) {
                    // ---- rare: move the reference of every row to the running maximum ----
                    if (bar_red_or<NT>(!ok)) goto done;
#pragma unroll
                    for (int k = 0; k < NCK; ++k) {
                        if (row_of(k) < n_rows) {
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                float v = s[k][e] * p.scale_log2;
                                if (need_mask && !((rowmask >> (row_of(k) + e)) & 1ull)) v = -INFINITY;
                                const float wm = warp_max_f32(v);
                                if (lane == 0) red[quarter * NB + row_of(k) + e] = wm;
                            }
                        }
                    }
                    bar_sync_softmax<NT>();
                    float fac[NCK][4];
                    bool any_scale = false;
#pragma unroll
                    for (int k = 0; k < NCK; ++k) {
                        if (row_of(k) < n_rows) {
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const int r = row_of(k) + e;
                                const float tm = fmaxf(fmaxf(red[r], red[NB + r]), fmaxf(red[2 * NB + r], red[3 * NB + r]));
                                const float old = mref[r];
                                const float nm = fmaxf(old, tm);
                                fac[k][e] = (old == -INFINITY) ? 0.f : ex2(old - nm);   // nothing accumulated yet under -inf
                                l_part[k][e] *= fac[k][e];
                                if (old == -INFINITY) fac[k][e] = 1.f;                   // O^T of such a row is still all zeros
                                any_scale |= (old != -INFINITY) && (nm != old);
                            }
                        }
                    }
                    // whether any row of any column group moved is a block-wide question
                    if (t > t_first && bar_red_or<NT>(any_scale)) {
                        ok = ok && mbar_wait(bar(L::P_FREE + ((it - 1) & 1)), ((it - 1) >> 1) & 1, ab);   // P.V of the previous tile done
                        if (bar_red_or<NT>(!ok)) goto done;
                        tc_fence_after();
#pragma unroll
                        for (int k = 0; k < NCK; ++k) {
                            if (row_of(k) < n_rows) {
                                float o[4];
                                tmem_ld4(tmem_o + lane_base + (uint32_t)row_of(k), o);
                                tmem_wait_ld();
#pragma unroll
                                for (int e = 0; e < 4; ++e) o[e] *= fac[k][e];
                                tmem_st4(tmem_o + lane_base + (uint32_t)row_of(k), o);
                            }
                        }
                        tmem_wait_st();
                        tc_fence_before();
                    }
                    bar_sync_softmax<NT>();                  // everyone has read the old references
                    if (tid < NB && (tid & ~3) < n_rows)
                        mref[tid] = fmaxf(mref[tid], fmaxf(fmaxf(red[tid], red[NB + tid]), fmaxf(red[2 * NB + tid], red[3 * NB + tid])));
                    bar_sync_softmax<NT>();
                    compute_d();
                }

                // ---- probabilities of this token for its rows -> P^T ----
                ok = ok && mbar_wait(bar(L::P_FREE + pb), ((it >> 1) & 1) ^ 1, ab);      // P.V two tiles back done
                {
                    unsigned char* pbase = smem + L::kOffP + pb * L::kPBytes + (tok >> 6) * (NB * 128) + (tok & 7) * 2;
                    const int chunk = (tok & 63) >> 3;
#pragma unroll
                    for (int k = 0; k < NCK; ++k) {
                        if (row_of(k) < n_rows) {
                            float e4[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                e4[e] = ex2(d[k][e]);                 // masked entries: ex2(-inf) = 0
                                l_part[k][e] += e4[e];
                            }
                            if (ok) {
                                __nv_bfloat162 h0 = __floats2bfloat162_rn(e4[0], e4[1]), h1 = __floats2bfloat162_rn(e4[2], e4[3]);
                                const uint32_t w0 = *reinterpret_cast<uint32_t*>(&h0), w1 = *reinterpret_cast<uint32_t*>(&h1);
                                const int r = row_of(k);              // multiple of 4: r & 7 is 0 or 4
                                unsigned char* q0 = pbase + r * 128;
                                *reinterpret_cast<unsigned short*>(q0 + ((chunk ^ (r & 7)) << 4)) = (unsigned short)(w0 & 0xffffu);
                                *reinterpret_cast<unsigned short*>(q0 + 128 + ((chunk ^ ((r + 1) & 7)) << 4)) = (unsigned short)(w0 >> 16);
                                *reinterpret_cast<unsigned short*>(q0 + 256 + ((chunk ^ ((r + 2) & 7)) << 4)) = (unsigned short)(w1 & 0xffffu);
                                *reinterpret_cast<unsigned short*>(q0 + 384 + ((chunk ^ ((r + 3) & 7)) << 4)) = (unsigned short)(w1 >> 16);
                            }
                        }
                    }
                }
                // last tile of a segment: V rows past the last valid token must be zero (they may hold
                // anything, and 0 x NaN is NaN)
                if (need_mask) {
                    const int n_valid = min(kTileT, Ltok - tok0);
                    if (n_valid < kTileT) {
                        const int uv = 2 * it + 1, slot = uv % NS;
                        ok = ok && mbar_wait(bar(L::FULL + slot), (uv / NS) & 1, ab);
                        if (ok) {
                            unsigned char* vb = smem + L::kOffRing + slot * kSlotBytes;
                            for (int idx = tid; idx < (kTileT - n_valid) * 16; idx += NT) {
                                const int row = n_valid + (idx >> 4), c = idx & 15;
                                *reinterpret_cast<uint4*>(vb + (c >> 3) * kHalfT + row * 128 + ((c & 7) << 4)) = make_uint4(0, 0, 0, 0);
                            }
                        }
                    }
                }
                fence_proxy_async();
                mbar_arrive(bar(L::P_FULL + pb));
            }

            // ---- piece epilogue ----
            const int g_next = seg.tile_begin + t_last;
            const bool have_next = g_next < g_end;
            SegInfo next = seg;
            if (have_next) {
                // all S^T of this piece have been seen, so its Q is no longer read: stage the next one now
                next = segment_of_tile(p, cum, g_next);
                stage_q<NB, NT>(p, next, smem, tid);
                fence_proxy_async();
                mbar_arrive(bar(L::Q_FULL));
            }
            ok = ok && mbar_wait(bar(L::P_FREE + ((it - 1) & 1)), ((it - 1) >> 1) & 1, ab);      // last P.V done
            if (bar_red_or<NT>(!ok)) goto done;
            tc_fence_after();
            {
                float* po; float2* pml;
                piece_slot(p, seg, blockIdx.x, po, pml);
#pragma unroll
                for (int k = 0; k < NCK; ++k) {
                    if (row_of(k) < n_rows) {
                        float o[4];
                        tmem_ld4(tmem_o + lane_base + (uint32_t)row_of(k), o);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int r = row_of(k) + e;
                            if (r < n_rows) po[(size_t)r * kHeadDim + tok] = o[e];
                            const float ws = warp_sum_f32(l_part[k][e]);
                            if (lane == 0) red[quarter * NB + r] = ws;
                        }
                    }
                }
                bar_sync_softmax<NT>();
                if (tid < n_rows)
                    pml[tid] = make_float2(mref[tid], (red[tid] + red[NB + tid]) + (red[2 * NB + tid] + red[3 * NB + tid]));
                tc_fence_before();
                bar_sync_softmax<NT>();
            }
            if (!have_next) break;
            seg = next;
        }
    }
done:
    // ---- teardown: everyone arrives here, normally or after an abort ----
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(L::kTmemCols) : "memory");
    }
}

template <int NB, int CG>
cudaError_t launch_nb(Ctx* c, const AttnParams& p, const CUtensorMap& mk, const CUtensorMap& mv, cudaStream_t st) {
    const int smem = Lay<NB>::kFixedBytes + (p.N + 1) * (int)sizeof(int);
    static bool attr_set[64] = {};                          // the attribute is per device
    if (c->device < 0 || c->device >= 64 || !attr_set[c->device]) {
        cudaError_t err = cudaFuncSetAttribute(attn_umma_t_kernel<NB, CG>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               Lay<NB>::kFixedBytes + (kMaxBranches + 1) * (int)sizeof(int));
        if (err != cudaSuccess) return err;
        if (c->device >= 0 && c->device < 64) attr_set[c->device] = true;
    }
    attn_umma_t_kernel<NB, CG><<<p.grid, 128 * CG + 64, smem, st>>>(p, mk, mv);
    return cudaGetLastError();
}

}  // namespace

int umma_t_rows(int nr) { return nr <= 32 ? 32 : 64; }

cudaError_t launch_attn_umma_t(Ctx* c, const AttnParams& p, cudaStream_t st) {
    cudaError_t err = cudaSuccess;
    const CUtensorMap* mk = umma_pool_map(c, p.k_pages, &err);
    if (!mk) return err;
    const CUtensorMap mk_copy = *mk;                       // the cache may reallocate on the next insert
    const CUtensorMap* mv = umma_pool_map(c, p.v_pages, &err);
    if (!mv) return err;
    if (p.rb_rows == 32) return launch_nb<32, 2>(c, p, mk_copy, *mv, st);
    if (p.rb_rows == 64) return launch_nb<64, 2>(c, p, mk_copy, *mv, st);
    return cudaErrorInvalidValue;
}

}  // namespace tts
