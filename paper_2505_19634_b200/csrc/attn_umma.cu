// Tensor-core verify attention for sm_100a: tcgen05.mma with TMEM accumulators, K/V page tiles
// staged by TMA, fp32 online softmax between the two contractions.
//
// One persistent CTA per SM walks its run of the global tile list (tts_internal.cuh).  A tile is
// 128 KV tokens of one KV head = 8 pages gathered through the block table, each page-head tile
// (16 tokens x 128 dims, 4 KiB contiguous) arriving as one 128-byte-swizzled 5-D TMA box.
//
//   warps 8, 9  producers, one for the K tiles (ring of 3 slots x 32 KiB) and one for the V tiles (ring
//               of 2): per tile the warp arms the slot's "full" barrier with the byte count and issues
//               one TMA box per page.  K tiles are wanted a whole softmax step before their V tiles.
//   warp 10     MMA issuer (one thread): S = Q K^T into one of two TMEM buffers, then
//               O (+)= P V once the softmax warps have published P; frees ring slots with
//               tcgen05.commit
//   warps 0-7   softmax: two threads per query row (TMEM lane), each on one half of the tile's 128 key
//               columns.  A thread reads its 64 scores once, the pair agrees on the row maximum
//               through shared memory, and each writes its probabilities as packed bf16 pairs over
//               the first half of its own score columns: the second contraction takes P from TMEM as
//               its A operand, so there is no P buffer in shared memory and a tile's exponentials
//               do not wait for the previous tile's second contraction.  O is rescaled in TMEM only
//               when the max moved by more than 2^8 (the final result is exact either way, l carries
//               the same reference; only then does a warp wait for the previous contraction); each
//               thread keeps the sum of its own columns; the piece's partial (m, l, O) is written at
//               the end.
//
// This is the kernel for many query rows per KV head (draft trees: nodes x GQA group rows); with few rows
// most of the 128-row tile is padding and the token-major kernel (attn_umma_t.cu) is the one to use.
//
// Every wait is bounded: when a limit runs out the CTA raises TTS_ERR_DEVICE_TIMEOUT in the
// status word, all roles leave their loops, in-flight copies are awaited (bounded) and TMEM is
// released before the CTA returns.
#include <cuda.h>

#include <vector>

#include "tts_internal.cuh"
#include "umma_ptx.cuh"

namespace tts {

namespace {

using namespace ptx;

constexpr int kTile = kUmmaTileTokens;            // 128 tokens
constexpr int kRows = kUmmaRows;                   // 128 = MMA M
constexpr int kSoftmaxThreads = 256;                 // 8 warps: (TMEM lane quarter, column half)
constexpr int kThreadsUmma = kSoftmaxThreads + 96;
constexpr int kProducerWarp = kSoftmaxThreads / 32, kMmaWarp = kProducerWarp + 2;   // producers: K, then V
constexpr int kHalfBytes = kRows * 128;            // one 64-element K-block of a 128-row operand: 16 KiB
constexpr int kOperandBytes = 2 * kHalfBytes;      // 32 KiB
constexpr int kRingK = 3, kRingV = 2;                 // K tiles are wanted a whole softmax step before their V tiles
constexpr uint32_t kTmemCols = 512;

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int kOffQ = 0;
constexpr int kOffK = kOffQ + kOperandBytes;
constexpr int kOffV = kOffK + kRingK * kOperandBytes;
constexpr int kOffBar = kOffV + kRingV * kOperandBytes;
constexpr int kNumBars = 16;
constexpr int kOffMisc = kOffBar + kNumBars * 8;
constexpr int kOffXch = kOffMisc + 64;                         // float[5][128]: row maxima of two tiles x two halves, row sums
constexpr int kOffCum = kOffXch + 5 * kRows * 4;
constexpr int kUmmaMaxBranches = 1024;
constexpr int kSmemBytes = kOffCum + (kUmmaMaxBranches + 1) * 4 + 1024;   // + slack for manual alignment

// PV_DONE: two barriers, tile j completes PV_DONE + (j & 1), so that a waiter's parity follows from the tile index alone
// even when it has not waited for every tile
enum Bar { K_FULL = 0, K_EMPTY = 3, V_FULL = 6, V_EMPTY = 8, S_FULL = 10, PV_DONE = 12, P_FULL = 14, Q_FULL = 15 };
static_assert(kRingK == 3 && kRingV == 2 && kNumBars == 16, "barrier numbering");

// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = 128; B either K-major or MN-major.
__host__ __device__ constexpr uint32_t instr_desc(bool b_mn_major) { return ptx::instr_desc(128, 128, false, b_mn_major); }
// byte offset of the 16-byte chunk holding elements [8*chunk, 8*chunk+8) of `row` in a 128-row,
// 128-element-wide K-major operand with 128-byte swizzle
__device__ __forceinline__ uint32_t kmajor_chunk_off(int row, int chunk) {
    return (uint32_t)((chunk >> 3) * kHalfBytes + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

// One mbarrier arrival for the whole warp, after every lane's preceding work (arrivals of single threads
// on one barrier serialise, so the barriers count warps).
__device__ __forceinline__ void warp_arrive(uint32_t bar, int lane) {
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
}

struct PieceWalk {                    // every role iterates the CTA's pieces the same way
    int g, g_end;
};

__global__ void __launch_bounds__(kThreadsUmma, 1)
attn_umma_kernel(const AttnParams p, const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v) {
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + kOffBar;
    auto bar = [&](int i) { return bar0 + 8u * i; };
    volatile int* misc = reinterpret_cast<volatile int*>(smem + kOffMisc);   // [0] abort flag, [1] tmem base
    int* cum = reinterpret_cast<int*>(smem + kOffCum);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const Abort ab{misc, p.status};

    build_branch_tile_prefix(p, cum);
    const int total = total_tiles(p, cum);
    const int tpc = ceil_div(total, p.grid);
    const int g_begin = blockIdx.x * tpc;
    const int g_end = min(total, g_begin + tpc);
    if (g_begin >= g_end) return;                          // uniform: nothing to do for this CTA

    // ---- set-up: zero the V ring (nothing non-finite may ever meet a zero weight), barriers, TMEM ----
    for (int i = tid; i < kRingV * kOperandBytes / 16; i += kThreadsUmma)
        *reinterpret_cast<uint4*>(smem + kOffV + i * 16) = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
        misc[0] = 0;
        for (int i = 0; i < kRingK; ++i) { mbar_init(bar(K_FULL + i), 1); mbar_init(bar(K_EMPTY + i), 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(V_FULL + i), 1); mbar_init(bar(V_EMPTY + i), 1);
            mbar_init(bar(S_FULL + i), 1);
        }
        mbar_init(bar(P_FULL), kSoftmaxThreads / 32); mbar_init(bar(PV_DONE), 1); mbar_init(bar(PV_DONE + 1), 1); mbar_init(bar(Q_FULL), kSoftmaxThreads / 32);   // the softmax warps arrive once per warp
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + kOffMisc + 4), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = (uint32_t)misc[1];
    const uint32_t tmem_s[2] = {tmem, tmem + 128u};
    const uint32_t tmem_o = tmem + 256u;

    if (warp == kProducerWarp || warp == kProducerWarp + 1) {
        // =========================== producers: one warp for the K tiles, one for the V tiles ===========================
        const int op = warp - kProducerWarp;               // 0: K, 1: V
        const int ring_n = op == 0 ? kRingK : kRingV;
        const int full0 = op == 0 ? K_FULL : V_FULL, empty0 = op == 0 ? K_EMPTY : V_EMPTY;
        const uint32_t ring_base = sbase + (op == 0 ? kOffK : kOffV);
        const CUtensorMap* tm = op == 0 ? &tm_k : &tm_v;
        int it = 0;                                         // tiles issued by this warp
        int slot = 0, round = 0;                            // it % ring_n, (it / ring_n) & 1
        int g = g_begin;
        bool alive = true;
        const uint64_t stream_once = l2_policy_evict_first();
        SegInfo seg = segment_of_tile(p, cum, g);           // the first piece by search, the following ones by stepping
        for (bool first_piece = true; g < g_end && alive; first_piece = false) {
            if (!first_piece) seg = next_segment(p, cum, seg);
            const int t_first = g - seg.tile_begin, t_last = min(seg.n_tiles, g_end - seg.tile_begin);
            const int32_t* bt = p.block_table + (size_t)(seg.kind == 0 ? 0 : seg.b) * p.max_blocks;
            for (int t = t_first; t < t_last && alive; ++t, ++it) {
                const int tok0 = t * kTile;
                const int n_pages = ceil_div(min(kTile, seg.n_tokens - tok0), kPage);
                int page = 0;
                if (lane < n_pages) page = checked_page(p, bt, (seg.tok_begin + tok0) / kPage + lane);
                // one box per page-head tile (4 KiB), laid out [token half][dim half][8 tokens][128 bytes], so the
                // pages of a tile form one MMA operand with 2 KiB between its 8-token groups
                const int page_head = page * p.Hkv + seg.kvh;
                if (lane == 0) {
                    alive = mbar_wait(bar(empty0 + slot), round ^ 1, ab);
                    if (alive) mbar_arrive_expect_tx(bar(full0 + slot), (uint32_t)n_pages * 4096u);
                }
                alive = __shfl_sync(0xffffffffu, alive, 0);
                if (!alive) break;
                if (lane < n_pages)
                    tma_load_page(ring_base + slot * kOperandBytes + lane * 4096, tm, page_head, bar(full0 + slot), stream_once);
                if (++slot == ring_n) { slot = 0; round ^= 1; }
            }
            g = seg.tile_begin + t_last;
        }
        // Copies this warp started must have landed before the CTA may exit: the consumers wait on
        // the same phases in the normal case; after an abort wait for them here (bounded).
        if (*ab.flag && lane == 0) {
            for (int back = 1; back <= ring_n && back <= it; ++back) {
                const int j = it - back;
                const Abort quiet{misc + 2 + op, p.status};  // do not re-raise; misc[2], misc[3] are scratch
                misc[2 + op] = 0;
                mbar_wait(bar(full0 + j % ring_n), (j / ring_n) & 1, quiet);
            }
        }
    } else if (warp == kMmaWarp) {
        // =========================== MMA issuer ===========================
        if (lane == 0) {
            constexpr uint32_t idesc_qk = instr_desc(false), idesc_pv = instr_desc(true);
            int it = 0, piece = 0;
            int g = g_begin;
            bool alive = true;
            auto issue_qk = [&](int j) -> bool {
                const int slot = j % kRingK, sb = j & 1;
                if (!mbar_wait(bar(K_FULL + slot), (j / kRingK) & 1, ab)) return false;
                // S buffer sb last held the probabilities of tile j - 2, read by that tile's second contraction,
                // which was issued before this one: the tensor pipe keeps the order
                tc_fence_after();
                const uint32_t qa = sbase + kOffQ, ka = sbase + kOffK + slot * kOperandBytes;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)               // Q: two 64-dim blocks of 128 rows; K: dim halves 1 KiB apart inside a page
                    umma_bf16(tmem_s[sb], smem_desc(qa + (ks >> 2) * kHalfBytes + (ks & 3) * 32, 16, 1024),
                              smem_desc(ka + (ks >> 2) * 1024 + (ks & 3) * 32, 16, 2048), idesc_qk, ks > 0);
                umma_commit(bar(K_EMPTY + slot));
                umma_commit(bar(S_FULL + sb));
                return true;
            };
            SegInfo seg = segment_of_tile(p, cum, g);
            for (bool first_piece = true; g < g_end && alive; first_piece = false) {
                if (!first_piece) seg = next_segment(p, cum, seg);
                const int t_first = g - seg.tile_begin, t_last = min(seg.n_tiles, g_end - seg.tile_begin);
                const int n = t_last - t_first;
                alive = mbar_wait(bar(Q_FULL), piece & 1, ab);
                if (!alive) break;
                tc_fence_after();
                alive = issue_qk(it);
                for (int j = 0; j < n && alive; ++j) {
                    if (j + 1 < n) { alive = issue_qk(it + j + 1); if (!alive) break; }
                    const int cur = it + j, slot = cur % kRingV;
                    alive = mbar_wait(bar(P_FULL), cur & 1, ab) && mbar_wait(bar(V_FULL + slot), (cur / kRingV) & 1, ab);
                    if (!alive) break;
                    tc_fence_after();
                    const uint32_t va = sbase + kOffV + slot * kOperandBytes;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        // P: the A operand straight from TMEM, 16 tokens = 8 columns of packed bf16 pairs per step; the
                        // two halves of a row sit at columns 0 and 64 of the tile's score buffer (see the softmax warps)
                        const uint32_t pa = tmem_s[cur & 1] + (uint32_t)((ks >> 2) * 64 + (ks & 3) * 8);
                        const uint32_t boff = ks * 4096;                                    // V: one page (16 tokens) per step
                        umma_bf16_tmem_a(tmem_o, pa, smem_desc(va + boff, 1024, 2048), idesc_pv, (j > 0 || ks > 0) ? 1u : 0u);
                    }
                    umma_commit(bar(V_EMPTY + slot));
                    umma_commit(bar(PV_DONE + (cur & 1)));
                }
                it += n; ++piece;
                g = seg.tile_begin + t_last;
            }
        }
    } else {
        // =========================== softmax warps ===========================
        const int quarter = warp & 3, half = warp >> 2;     // TMEM lane quarter of this warp; column half of this thread
        const int L = quarter * 32 + lane;                  // TMEM lane = row of the MMA tile
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        constexpr int W = kTile / 2;                        // S columns (keys) this thread looks at
        const int col0 = half * W;
        float* xch = reinterpret_cast<float*>(smem + kOffXch);   // [2 tile parities][2 halves][128 rows]
        int it = 0;
        int g = g_begin;
        bool alive = true;
        SegInfo seg = segment_of_tile(p, cum, g);
        for (bool first_piece = true; g < g_end && alive; first_piece = false) {
            if (!first_piece) seg = next_segment(p, cum, seg);
            const int t_first = g - seg.tile_begin, t_last = min(seg.n_tiles, g_end - seg.tile_begin);
            const bool valid = L < seg.n_rows;

            // ---- stage Q (each thread half of its row, zero rows past the block), per-row mask ----
            unsigned long long vis = ~0ull;
            {
                const __nv_bfloat16* src = nullptr;
                if (valid) {
                    int row = seg.row0 + L, b = seg.b;
                    if (seg.kind == 0) { b = row / p.nr; row = row % p.nr; }
                    const int i = row / p.G, gq = row % p.G;
                    src = p.q + (((size_t)b * p.R + i) * p.Hq + seg.kvh * p.G + gq) * kHeadDim;
                    if (seg.kind == 1) vis = row_visibility(p, b, i);
                }
#pragma unroll
                for (int c = 8 * half; c < 8 * half + 8; ++c) {
                    uint4 v = make_uint4(0, 0, 0, 0);
                    if (valid) v = __ldg(reinterpret_cast<const uint4*>(src) + c);
                    *reinterpret_cast<uint4*>(smem + kOffQ + kmajor_chunk_off(L, c)) = v;
                }
            }
            fence_proxy_async();
            warp_arrive(bar(Q_FULL), lane);

            float m_ref = -INFINITY, l_sum = 0.f;           // reference max (log2 units); sum over this thread's columns
            const int Ltok = seg.n_tokens;
            const int tail0 = seg.kind == 1 ? Ltok - p.R : Ltok;     // first token that needs the row mask

            for (int t = t_first; t < t_last && alive; ++t, ++it) {
                const int sb = it & 1;
                const int tok0 = t * kTile;
                const bool need_mask = tok0 + kTile > tail0;        // uniform: tile touches masked / missing tokens
                alive = __all_sync(0xffffffffu, mbar_wait(bar(S_FULL + sb), (it >> 1) & 1, ab));
                if (!alive) break;
                tc_fence_after();

                // this thread's 64 scores, read once; masked ones become -inf
                float sv[W];
                tmem_ld32(tmem_s[sb] + lane_base + (uint32_t)col0, reinterpret_cast<uint32_t*>(sv));
                tmem_ld32(tmem_s[sb] + lane_base + (uint32_t)col0 + 32u, reinterpret_cast<uint32_t*>(sv) + 32);
                tmem_wait_ld();
                if (need_mask) {
#pragma unroll
                    for (int c = 0; c < W; ++c) {
                        const int j = tok0 + col0 + c;
                        const bool ok = j < Ltok && (j < tail0 || ((vis >> (j - tail0)) & 1ull));
                        if (!ok) sv[c] = -INFINITY;
                    }
                }
                float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};     // four independent chains
#pragma unroll
                for (int c = 0; c < W; ++c) mx4[c & 3] = fmaxf(mx4[c & 3], sv[c]);
                float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                // the row maximum over both halves
                float* x = xch + (it & 1) * 2 * kRows;
                x[half * kRows + L] = mx;
                asm volatile("barrier.cta.sync 1, %0;" ::"n"(kSoftmaxThreads) : "memory");
                mx = fmaxf(x[L], x[kRows + L]) * p.scale_log2;      // scale > 0; -inf stays -inf
                const bool move = mx > m_ref + 8.f || (m_ref == -INFINITY && mx > -INFINITY);
                const float m_new = move ? mx : m_ref;
                const float factor = (move && m_ref != -INFINITY) ? ex2(m_ref - m_new) : 1.f;

                if (t > t_first && __any_sync(0xffffffffu, factor != 1.f)) {     // this thread's half of its O row
                    // O is touched: the previous tile's second contraction must have finished
                    alive = __all_sync(0xffffffffu, mbar_wait(bar(PV_DONE + ((it - 1) & 1)), ((it - 1) >> 1) & 1, ab));
                    if (!alive) break;
                    tc_fence_after();
                    for (int ch = 0; ch < 2; ++ch) {
                        uint32_t ov[32];
                        tmem_ld32(tmem_o + lane_base + (uint32_t)(col0 + 32 * ch), ov);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) ov[c] = __float_as_uint(__uint_as_float(ov[c]) * factor);
                        tmem_st32(tmem_o + lane_base + (uint32_t)(col0 + 32 * ch), ov);
                    }
                    tmem_wait_st();
                }
                l_sum *= factor;
                m_ref = m_new;

                // probabilities -> bf16 pairs, written over the first 32 of this thread's own 64 score columns: the
                // second contraction takes P from TMEM as its A operand (row = lane, two tokens per 32-bit column)
                const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
                float l4[4] = {0.f, 0.f, 0.f, 0.f};
                uint32_t pw[W / 2];
#pragma unroll
                for (int c = 0; c < W; c += 2) {
                    const float e0 = ex2(fmaf(sv[c], p.scale_log2, neg_m));            // masked: ex2(-inf) = 0
                    const float e1 = ex2(fmaf(sv[c + 1], p.scale_log2, neg_m));
                    l4[(c >> 1) & 1] += e0; l4[2 + ((c >> 1) & 1)] += e1;
                    const __nv_bfloat162 h = __floats2bfloat162_rn(e0, e1);          // the even token in the low half
                    pw[c >> 1] = *reinterpret_cast<const uint32_t*>(&h);
                }
                l_sum += (l4[0] + l4[1]) + (l4[2] + l4[3]);
                tmem_st32(tmem_s[sb] + lane_base + (uint32_t)col0, pw);
                tmem_wait_st();
                tc_fence_before();

                // last tile of a private segment: zero the V rows of the loaded pages past the branch end
                if (need_mask) {
                    const int n_valid = min(kTile, Ltok - tok0);
                    const int n_loaded = ceil_div(n_valid, kPage) * kPage;
                    if (n_valid < n_loaded) {
                        const int slot = it % kRingV;
                        alive = __all_sync(0xffffffffu, mbar_wait(bar(V_FULL + slot), (it / kRingV) & 1, ab));
                        if (!alive) break;
                        for (int idx = tid; idx < (n_loaded - n_valid) * 16; idx += kSoftmaxThreads) {
                            const int row = n_valid + idx / 16, c = idx % 16;
                            // token `row` of the staged tile: page, token half, 8-token group row; both dim halves
                            *reinterpret_cast<uint4*>(smem + kOffV + slot * kOperandBytes + (row >> 4) * 4096 + ((row >> 3) & 1) * 2048 +
                                                      (c >> 3) * 1024 + (row & 7) * 128 + ((c & 7) << 4)) = make_uint4(0, 0, 0, 0);
                        }
                    }
                }
                fence_proxy_async();
                warp_arrive(bar(P_FULL), lane);
            }
            if (!alive) break;

            // ---- piece epilogue: partial (m, l, O) ----
            alive = __all_sync(0xffffffffu, mbar_wait(bar(PV_DONE + ((it - 1) & 1)), ((it - 1) >> 1) & 1, ab));
            if (!alive) break;
            tc_fence_after();
            float* po; float2* pml;
            piece_slot(p, seg, blockIdx.x, po, pml);
            float* lx = xch + 4 * kRows;                     // the two halves' sums of a row
            if (half == 1) lx[L] = l_sum;
            for (int ch = 0; ch < 2; ++ch) {
                uint32_t ov[32];
                tmem_ld32(tmem_o + lane_base + (uint32_t)(col0 + 32 * ch), ov);
                tmem_wait_ld();
                if (valid) {
                    float4* dst = reinterpret_cast<float4*>(po + (size_t)L * kHeadDim + col0 + 32 * ch);
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        dst[c] = make_float4(__uint_as_float(ov[4 * c]), __uint_as_float(ov[4 * c + 1]),
                                             __uint_as_float(ov[4 * c + 2]), __uint_as_float(ov[4 * c + 3]));
                }
            }
            asm volatile("barrier.cta.sync 1, %0;" ::"n"(kSoftmaxThreads) : "memory");
            if (valid && half == 0) pml[L] = make_float2(m_ref, l_sum + lx[L]);
            asm volatile("barrier.cta.sync 1, %0;" ::"n"(kSoftmaxThreads) : "memory");   // lx is free for the next piece
            tc_fence_before();
            g = seg.tile_begin + t_last;
        }
    }

    // ---- teardown: everyone arrives here, normally or after an abort ----
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

struct MapEntry { const void* ptr; long rows; int kind; CUtensorMap map; };
struct MapCache { std::vector<MapEntry> entries; };

}  // namespace

// Tensor maps over a page pool [num_pages][Hkv][16 tokens][128 dims] bf16, 128-byte swizzle.
//   kind 0: 2-D view, rows = num_pages * Hkv * 16 tokens of 128 dims; box = 64 dims x 16 tokens.
//   kind 1: 5-D view (64 dims, 8 tokens, 2 dim halves, 2 token halves, page-head); box = one whole
//           page-head tile (4 KiB), which lands as [token half][dim half][8 tokens][128 bytes]: the
//           8-token atoms of one dim half are then 2 KiB apart across the pages of a 128-token tile.
const CUtensorMap* umma_pool_map(Ctx* c, const void* pool, int kind, cudaError_t* err) {
    if (!c->tmap_cache) c->tmap_cache = new MapCache();
    MapCache* mc = static_cast<MapCache*>(c->tmap_cache);
    const long rows = (long)c->cfg.num_pages * c->cfg.n_kv_heads * kPage;
    for (auto& e : mc->entries)
        if (e.ptr == pool && e.rows == rows && e.kind == kind) return &e.map;
    EncodeTiledFn fn = encode_fn();
    if (!fn) { *err = cudaErrorNotSupported; return nullptr; }
    MapEntry e;
    e.ptr = pool; e.rows = rows; e.kind = kind;
    CUresult r;
    if (kind == 0) {
        const cuuint64_t dims[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)rows};
        const cuuint64_t strides[1] = {(cuuint64_t)kHeadDim * 2};
        const cuuint32_t box[2] = {64, (cuuint32_t)kPage};
        const cuuint32_t estr[2] = {1, 1};
        r = fn(&e.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(pool), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else {
        const cuuint64_t dims[5] = {64, 8, 2, 2, (cuuint64_t)(rows / kPage)};
        const cuuint64_t strides[4] = {256, 128, 2048, 4096};          // bytes, dimensions 1..4
        const cuuint32_t box[5] = {64, 8, 2, 2, 1};
        const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
        r = fn(&e.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(pool), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    if (r != CUDA_SUCCESS) { *err = cudaErrorInvalidValue; return nullptr; }
    if (mc->entries.size() >= 512) mc->entries.erase(mc->entries.begin());
    mc->entries.push_back(e);
    return &mc->entries.back().map;
}

bool umma_available() { return true; }

int umma_copies(int nr) { (void)nr; return 1; }

cudaError_t launch_attn_umma(Ctx* c, const AttnParams& p, cudaStream_t st) {
    if (p.N > kUmmaMaxBranches) return cudaErrorInvalidValue;
    cudaError_t err = cudaSuccess;
    const CUtensorMap* mk = umma_pool_map(c, p.k_pages, 1, &err);
    if (!mk) return err;
    const CUtensorMap mk_copy = *mk;                       // the cache may reallocate on the next insert
    const CUtensorMap* mv = umma_pool_map(c, p.v_pages, 1, &err);
    if (!mv) return err;
    static bool attr_set[64] = {};                          // the attribute is per device
    if (c->device < 0 || c->device >= 64 || !attr_set[c->device]) {
        err = cudaFuncSetAttribute(attn_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (err != cudaSuccess) return err;
        if (c->device >= 0 && c->device < 64) attr_set[c->device] = true;
    }
    attn_umma_kernel<<<p.grid, kThreadsUmma, kSmemBytes, st>>>(p, mk_copy, *mv);
    return cudaGetLastError();
}

void umma_release(Ctx* c) {
    delete static_cast<MapCache*>(c->tmap_cache);
    c->tmap_cache = nullptr;
}

}  // namespace tts
