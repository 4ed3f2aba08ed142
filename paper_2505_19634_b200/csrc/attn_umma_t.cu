// Token-major tensor-core verify attention for sm_100a: the kernel for FEW query rows per KV head
// (at most 64 stacked rows per row block; a chain of gamma+1 positions times the GQA group).
//
// With 20 or 40 query rows a row-major score tile would leave most of the 128-row MMA idle, so
// the KV tokens go on the MMA M dimension instead and both contractions are computed transposed:
//     S^T[128 tokens x NB rows] = K[128 x 128] . Q^T        (A = K tile, B = Q block, both K-major)
//     O^T[128 dims   x NB rows] = V^T[128 x 128] . P^T      (A = V tile as MN-major, B = P^T K-major)
// NB is 32 (the code is generic in it).  The operands K and V are the TMA-staged page tiles themselves; Q and P^T are
// small (NB x 256 bytes), which leaves room for a ring of 5-6 operand tiles (32 KiB each) in shared
// memory, the depth that hides HBM latency at 4 KiB page granularity.
//
// One persistent CTA per SM works through its pieces (the parts of the segments of tts_internal.cuh that
// fall into its run of the tile list), which it reads from the plan tables of attn_plan.cuh: the schedule
// is worked out once per verify step, not in each of its 64 launches.  Two tiles (256 tokens) per step: the latency chain of a step (MMA -> TMEM load -> consensus -> exp -> P^T
// -> MMA) is paid once for both tiles, and every thread works on two independent tokens.
//
//   producer warps   one for K, one for V, each with its own ring of slots (K tiles are consumed as soon
//                    as they land, V tiles wait for the softmax of their step, so one FIFO would block
//                    behind its oldest V tile): per tile the warp arms the "full" barrier of the next slot
//                    with the byte count and issues one 5-D TMA box per page-head tile (4 KiB), laid out
//                    so that the 8 pages of a tile form one MMA operand
//   MMA warp         one thread: S^T of the step's tiles into one of two pairs of TMEM buffers (the
//                    next step's scores are computed while the softmax warps work on this one's),
//                    O^T (+)= V^T P^T once P^T has been published; tcgen05.commit frees ring slots,
//                    P buffers and, at the end of a piece, the Q block
//   softmax warps    4*CG warps: thread = (TMEM lane = KV token of either tile, column group).  The NB
//                    rows are cut into chunks of 4; column group cg owns chunks cg, cg+CG, ... and a
//                    thread holds the scores of its tokens for the rows of its chunks (chunks past the
//                    piece's last row are skipped).  The running reference m of every row lives in
//                    shared memory and only moves when some score exceeds it by more than 2^16
//                    (consensus through a reducing named barrier; the exact row maximum is then found
//                    with warp redux + shared memory and O^T is rescaled in TMEM).  The result is
//                    exact either way: l is accumulated against the same reference.  Row sums are kept
//                    per thread and reduced once per piece.  The Q block of the next piece is
//                    prefetched into registers and stored during the last step of the current piece
//                    (its scores being complete, Q is no longer read), so that the next piece's first
//                    scores are computed while this piece finishes.
//   epilogue warps   4 warps: thread = TMEM lane = head dim.  O^T is double-buffered by piece parity, so
//                    the softmax warps go straight on to the next piece while these warps wait for the
//                    piece's last accumulation, read O^T and write the piece's partial (m, l, O).
//
// Every wait is bounded.  A wait that runs out raises TTS_ERR_DEVICE_TIMEOUT; the softmax warps only
// leave their loops on the result of a block-wide reduction, so no thread is left behind at a named
// barrier; in-flight copies are awaited (bounded) and TMEM is released before the CTA returns.
#include <cuda.h>

#include <type_traits>

#include "attn_plan.cuh"
#include "tts_internal.cuh"
#include "umma_ptx.cuh"

namespace tts {

namespace {

using namespace ptx;

constexpr int kTileT = kUmmaTileTokens;              // 128 tokens = MMA M
constexpr int kSlotBytes = kTileT * kHeadDim * 2;    // one K or V tile: 32 KiB
constexpr float kLazy = 16.f;                        // the reference moves when exceeded by 2^16

template <int NB>
struct Lay {
    static constexpr int kSlots = NB == 32 ? 6 : 5;
    static constexpr int kSlotsK = 2, kSlotsV = kSlots - kSlotsK;   // ring of K tiles, ring of V tiles
    static constexpr int kQBytes = NB * 256;         // two 64-dim K-blocks of NB rows x 128 B
    static constexpr int kPBytes = NB * 256;         // two 64-token K-blocks of NB rows x 128 B
    static constexpr int kOffQ = 0;
    static constexpr int kOffP = kQBytes;            // one buffer per tile of a step
    static constexpr int kOffRing = kOffP + 2 * kPBytes;
    static constexpr int kOffBar = kOffRing + kSlots * kSlotBytes;
    static constexpr int kOffMisc = kOffBar + 32 * 8;            // 2 * kSlots + 15 barriers
    static constexpr int kOffMref = kOffMisc + 64;               // float[NB]
    static constexpr int kOffRed = kOffMref + NB * 4;            // float[4][NB]
    static constexpr int kOffVis = kOffRed + 4 * NB * 4;         // u64[64]
    static constexpr int kOffLsum = kOffVis + 64 * 8;            // float[2][4][NB]: row sums of a finished piece
    static constexpr int kOffMout = kOffLsum + 2 * 4 * NB * 4;   // float[2][NB]: its row references
    static constexpr int kOffPlan = kOffMout + 2 * NB * 4;       // CtaPlan: this CTA's record of the plan
    static constexpr int kBytes = kOffPlan + (int)sizeof(CtaPlan) + 1024;   // + slack for the manual 1024-B alignment
    static_assert(kOffPlan % 16 == 0, "the plan record is copied in 16-byte words");
    static constexpr uint32_t kTmemCols = NB == 32 ? 256 : 512;  // 2 pairs of S^T buffers + 2 O^T, power of two
    // barrier indices
    static constexpr int FULL = 0, EMPTY = kSlots, S_FULL = 2 * kSlots, S_FREE = S_FULL + 2, P_FULL = S_FREE + 2,
                         P_FREE = P_FULL + 1, Q_FULL = P_FREE + 1, O_FULL = Q_FULL + 1, O_FREE = O_FULL + 2,
                         L_FULL = O_FREE + 2, L_FREE = L_FULL + 2;
};

// reducing / plain named barrier `id` over NT threads
template <int NT>
__device__ __forceinline__ bool bar_red_or(int id, bool pred) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "barrier.cta.red.or.pred p, %2, %3, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out) : "r"((uint32_t)pred), "r"(id), "n"(NT) : "memory");
    return out != 0;
}
template <int NT>
__device__ __forceinline__ void bar_sync_id(int id) { asm volatile("barrier.cta.sync %0, %1;" ::"r"(id), "n"(NT) : "memory"); }

// One mbarrier arrival for the whole warp, after every lane's preceding work (arrivals of single
// threads on one barrier serialise, so the barriers count warps).
__device__ __forceinline__ void warp_arrive(uint32_t bar, int lane) {
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
}

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

// The Q block of a piece, fetched by the NT threads of group 0 (QPT 16-byte chunks each) and later
// stored as the K-major B operand (zero rows beyond n_rows).
template <int NB, int NT>
struct QFetch {
    static constexpr int QPT = NB * 16 / NT;
    uint4 v[QPT];
    __device__ __forceinline__ void load(const AttnParams& p, const PieceDesc& seg, int t) {
#pragma unroll
        for (int k = 0; k < QPT; ++k) {
            const int idx = t + k * NT, r = idx >> 4, c = idx & 15;
            v[k] = make_uint4(0, 0, 0, 0);
            if (r < seg.n_rows) {
                int row = seg.row0 + r, b = seg.b, i, gq;
                if (seg.kind == 0) { int db; fast_divmod(row, p.nr, db, row); b += db; }
                fast_divmod(row, p.G, i, gq);
                const __nv_bfloat16* src = p.q + (((size_t)b * p.R + i) * p.Hq + seg.kvh * p.G + gq) * kHeadDim;
                v[k] = __ldg(reinterpret_cast<const uint4*>(src) + c);
            }
        }
    }
    __device__ __forceinline__ void store(unsigned char* q_smem, int t) const {
#pragma unroll
        for (int k = 0; k < QPT; ++k) {
            const int idx = t + k * NT, r = idx >> 4, c = idx & 15;
            *reinterpret_cast<uint4*>(q_smem + (c >> 3) * (NB * 128) + r * 128 + (((c & 7) ^ (r & 7)) << 4)) = v[k];
        }
    }
};

// Byte offset of token `row` (dim half 0) inside a staged K or V tile: pages of 4 KiB, each
// [token half][dim half][8 tokens][128 bytes].
__device__ __forceinline__ int tile_row_off(int row) { return (row >> 4) * 4096 + ((row >> 3) & 1) * 2048 + (row & 7) * 128; }

// This CTA's part of the plan: its record (a copy in shared memory) and, for a CTA with more pieces than
// the record holds, the global list.
struct PlanView {
    const CtaPlan* rec;
    const PieceDesc* rest;      // plan_pieces + piece_begin
    __device__ __forceinline__ PieceDesc piece(int i) const { return i < kPlanInline ? rec->first_pieces[i] : rest[i]; }
    __device__ __forceinline__ int tiles(int i) const { return i < kPlanInline ? rec->first_pieces[i].n_tiles : rest[i].n_tiles; }
};

// Walks the steps (two tiles, one at the end of a piece with an odd count) of a CTA's pieces.
struct StepCursor {
    int piece, n_pieces;  // index of the current piece
    int t, n_t;           // first tile of the step within the piece, tiles of the piece
    bool valid, first;    // first: first step of its piece
    __device__ void init(const PlanView& pv) {
        piece = 0; n_pieces = pv.rec->n_pieces; valid = n_pieces > 0; first = true;
        t = 0; n_t = valid ? pv.tiles(0) : 0;
    }
    __device__ int nt() const { return min(2, n_t - t); }
    __device__ bool last() const { return t + 2 >= n_t; }            // last step of its piece
    __device__ void advance(const PlanView& pv) {
        t += 2; first = false;
        if (t < n_t) return;
        if (++piece >= n_pieces) { valid = false; return; }
        n_t = pv.tiles(piece); t = 0; first = true;
    }
};

template <int NB, int CG>
__global__ void __launch_bounds__(128 * CG + 224, 1)
attn_umma_t_kernel(const AttnParams p, const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v) {
    using L = Lay<NB>;
    constexpr int NS = L::kSlots;
    constexpr int NT = 128 * CG;                           // softmax threads
    constexpr int NCK = NB / 4 / CG;                       // 4-row chunks per thread
    constexpr int NK = L::kSlotsK, NV = L::kSlotsV;
    constexpr int kEpilogueWarp = 4 * CG;                  // 4 warps, a multiple of 4 from the start: warp & 3 = TMEM quarter
    constexpr int kProducerWarp = kEpilogueWarp + 4, kMmaWarp = kProducerWarp + 2;   // producers: K, then V
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + L::kOffBar;
    auto bar = [&](int i) { return bar0 + 8u * i; };
    volatile int* misc = reinterpret_cast<volatile int*>(smem + L::kOffMisc);   // [0] abort flag, [1] tmem base
    const CtaPlan* rec = reinterpret_cast<const CtaPlan*>(smem + L::kOffPlan);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const Abort ab{misc, p.status};

    // ---- first of all, the loads of the CTA's first two tiles: each producer warp sets up the barriers of its
    // own ring, takes the tiles' pages straight from the plan in global memory and issues the copies; the data
    // is then on its way while the rest of the set-up runs ----
    int n_early = 0;                                       // tiles already issued (producer warps)
    if (warp == kProducerWarp || warp == kProducerWarp + 1) {
        const int op = warp - kProducerWarp;
        const int ring0 = op == 0 ? 0 : NK, ring_n = op == 0 ? NK : NV;
        static_assert(NK >= 2 && NV >= 2, "the first two tiles go to slots 0 and 1 of either ring");
        if (lane == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(op == 0 ? &tm_k : &tm_v) : "memory");
        int ph = -1;
        if (lane < 16) ph = __ldg(&p.plan_cta[blockIdx.x].first_pages[lane]);
        if (lane == 0) {
            for (int i = 0; i < ring_n; ++i) { mbar_init(bar(L::FULL + ring0 + i), 1); mbar_init(bar(L::EMPTY + ring0 + i), 1); }
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncwarp();
        const unsigned have = __ballot_sync(0xffffffffu, ph >= 0);
        const uint64_t stream_once = l2_policy_evict_first();
        const CUtensorMap* tm = op == 0 ? &tm_k : &tm_v;
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int n_pages = __popc((have >> (8 * u)) & 0xffu);      // uniform
            const int my = __shfl_sync(0xffffffffu, ph, 8 * u + (lane & 7));
            if (n_pages > 0) {
                if (lane == 0) mbar_arrive_expect_tx(bar(L::FULL + ring0 + u), (uint32_t)n_pages * 4096u);
                __syncwarp();
                if (lane < n_pages)
                    tma_load_page(sbase + L::kOffRing + (ring0 + u) * kSlotBytes + lane * 4096, tm, my, bar(L::FULL + ring0 + u), stream_once);
                ++n_early;
            }
        }
    }
    // ---- set-up: the other barriers, TMEM, tensor-map prefetch, and this CTA's record of the plan (one coalesced read) ----
    if (tid >= 32 && tid < 64)
        reinterpret_cast<uint4*>(smem + L::kOffPlan)[tid - 32] = __ldg(reinterpret_cast<const uint4*>(p.plan_cta + blockIdx.x) + (tid - 32));
    if (tid == 0) {
        misc[0] = 0;
        for (int i = 0; i < 2; ++i) { mbar_init(bar(L::S_FULL + i), 1); mbar_init(bar(L::S_FREE + i), 4 * CG); }
        mbar_init(bar(L::P_FULL), 4 * CG); mbar_init(bar(L::P_FREE), 1);     // softmax warps arrive once per warp
        mbar_init(bar(L::Q_FULL), 4 * CG);
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(L::O_FULL + i), 1); mbar_init(bar(L::O_FREE + i), 4);
            mbar_init(bar(L::L_FULL + i), 4 * CG); mbar_init(bar(L::L_FREE + i), 4);
        }
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
    const PlanView pv{rec, p.plan_pieces + rec->piece_begin};
    const int n_pieces = rec->n_pieces;
    const bool has_work = n_pieces > 0;                    // uniform
    // S^T of tile i of step ss at columns [(2 (ss & 1) + i) NB, +NB); O^T of piece pc at [(4 + (pc & 1)) NB, +NB)
    const uint32_t tmem_o0 = tmem + 4u * NB;
    if (!has_work) {
        // nothing to do for this CTA
    } else if (warp == kProducerWarp || warp == kProducerWarp + 1) {
        // =========================== producers ===========================
        const int op = warp - kProducerWarp;                // 0: K tiles into slots [0, NK), 1: V tiles into [NK, NS)
        const int ring0 = op == 0 ? 0 : NK, ring_n = op == 0 ? NK : NV;
        const CUtensorMap* tm = op == 0 ? &tm_k : &tm_v;
        int u = 0;                                          // tiles of this operand issued by this CTA
        int ring_pos = 0, ring_round = 0;                   // u % ring_n, (u / ring_n) & 1, kept without dividing
        bool alive = true;
        const uint64_t stream_once = l2_policy_evict_first();
        for (int pi = 0; pi < n_pieces && alive; ++pi) {
            const PieceDesc pc = pv.piece(pi);
            const int32_t* bt = p.block_table + (size_t)pc.bt_row * p.max_blocks;
            for (int i = 0; i < pc.n_tiles && alive; ++i, ++u) {
                const int tok0 = (pc.tile0 + i) * kTileT;
                const int n_pages = ceil_div(min(kTileT, pc.seg_tokens - tok0), kPage);
                if (u < n_early) {                             // issued at the start of the kernel
                    if (++ring_pos == ring_n) { ring_pos = 0; ring_round ^= 1; }
                    continue;
                }
                int page_head = 0;                             // page * Hkv + kvh: the TMA coordinate of a page-head tile
                if (lane < n_pages)
                    page_head = u < 2 ? rec->first_pages[u * 8 + lane]
                                      : checked_page(p, bt, (pc.tok_begin + tok0) / kPage + lane) * p.Hkv + pc.kvh;
                const int slot = ring0 + ring_pos;
                if (lane == 0) {
                    alive = mbar_wait(bar(L::EMPTY + slot), ring_round ^ 1, ab);
                    if (alive) mbar_arrive_expect_tx(bar(L::FULL + slot), (uint32_t)n_pages * 4096u);
                }
                alive = __shfl_sync(0xffffffffu, alive, 0);
                if (alive && lane < n_pages)
                    tma_load_page(sbase + L::kOffRing + slot * kSlotBytes + lane * 4096, tm, page_head,
                                  bar(L::FULL + slot), stream_once);
                if (++ring_pos == ring_n) { ring_pos = 0; ring_round ^= 1; }
            }
        }
        // Copies this warp started must have landed before the CTA may exit: the consumers wait on
        // the same phases in the normal case; after an abort wait for them here (bounded).
        if (*ab.flag && lane == 0) {
            for (int back = 1; back <= ring_n && back <= u; ++back) {
                const int j = u - back;
                const Abort quiet{misc + 2 + op, p.status};  // do not re-raise; misc[2], misc[3] are scratch
                misc[2 + op] = 0;
                mbar_wait(bar(L::FULL + ring0 + j % ring_n), (j / ring_n) & 1, quiet);
            }
        }
    } else if (warp == kMmaWarp) {
        // =========================== MMA issuer ===========================
        if (lane == 0) {
            constexpr uint32_t idesc_qk = instr_desc(kTileT, NB, false, false);
            constexpr uint32_t idesc_pv = instr_desc(kTileT, NB, true, false);
            bool alive = true;
            int n_q = 0, n_p = 0, u_k = 0, u_v = 0;           // steps scored / accumulated, K / V tiles consumed
            // scores of the step under `c`
            auto issue_qk = [&](const StepCursor& c) -> bool {
                const int set = n_q & 1;
                if (c.first) {                                // a new piece: its Q block must have been staged
                    if (!mbar_wait(bar(L::Q_FULL), c.piece & 1, ab)) return false;
                }
                if (!mbar_wait(bar(L::S_FREE + set), ((n_q >> 1) & 1) ^ 1, ab)) return false;
                const int nt = c.nt();
                for (int i = 0; i < nt; ++i, ++u_k) {
                    const int slot = u_k % NK;
                    if (!mbar_wait(bar(L::FULL + slot), (u_k / NK) & 1, ab)) return false;
                    tc_fence_after();
                    const uint32_t ka = sbase + L::kOffRing + slot * kSlotBytes, qa = sbase + L::kOffQ;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        umma_bf16(tmem + (uint32_t)((2 * set + i) * NB), smem_desc(ka + (ks >> 2) * 1024 + (ks & 3) * 32, 16, 2048),
                                  smem_desc(qa + (ks >> 2) * (NB * 128) + (ks & 3) * 32, 16, 1024), idesc_qk, ks > 0);
                    umma_commit(bar(L::EMPTY + slot));
                }
                umma_commit(bar(L::S_FULL + set));
                ++n_q;
                return true;
            };
            auto issue_pv = [&](const StepCursor& c) -> bool {
                const int ob = c.piece & 1;
                if (c.first) {                                // the epilogue of two pieces ago has read this O^T buffer
                    if (!mbar_wait(bar(L::O_FREE + ob), ((c.piece >> 1) & 1) ^ 1, ab)) return false;
                }
                if (!mbar_wait(bar(L::P_FULL), n_p & 1, ab)) return false;
                const int nt = c.nt();
                for (int i = 0; i < nt; ++i, ++u_v) {
                    const int slot = NK + u_v % NV;
                    if (!mbar_wait(bar(L::FULL + slot), (u_v / NV) & 1, ab)) return false;
                    tc_fence_after();
                    const uint32_t va = sbase + L::kOffRing + slot * kSlotBytes, pa = sbase + L::kOffP + i * L::kPBytes;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)          // one page (16 tokens) per step; P^T 32-byte column step
                        umma_bf16(tmem_o0 + (uint32_t)(ob * NB), smem_desc(va + ks * 4096, 1024, 2048),
                                  smem_desc(pa + (ks >> 2) * (NB * 128) + (ks & 3) * 32, 16, 1024), idesc_pv,
                                  (!c.first || i > 0 || ks > 0) ? 1u : 0u);
                    umma_commit(bar(L::EMPTY + slot));
                }
                umma_commit(bar(L::P_FREE));
                if (c.last()) umma_commit(bar(L::O_FULL + ob));   // the piece's O^T is complete
                ++n_p;
                return true;
            };
            // the scores run one step ahead of the accumulation, across piece boundaries too
            StepCursor cq, cp;
            cq.init(pv); cp = cq;
            alive = issue_qk(cq);
            cq.advance(pv);
            while (alive && cp.valid) {
                if (cq.valid) {
                    alive = issue_qk(cq);
                    if (!alive) break;
                    cq.advance(pv);
                }
                alive = issue_pv(cp);
                cp.advance(pv);
            }
        }
    } else if (warp >= kEpilogueWarp) {
        // =========================== epilogue warps ===========================
        const int et = tid - NT, quarter = warp & 3;
        const int dim = quarter * 32 + lane;                 // this thread's TMEM lane = head dim
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        const float* lsum = reinterpret_cast<const float*>(smem + L::kOffLsum);
        const float* mout = reinterpret_cast<const float*>(smem + L::kOffMout);
        bool alive = true;
        for (int pc = 0; pc < n_pieces && alive; ++pc) {
            const PieceDesc seg = pv.piece(pc);
            const int pb = pc & 1, n_rows = seg.n_rows;
            float* po; float2* pml;
            if (seg.kind == 0) {
                po = p.part_o_pre + (size_t)seg.slot * p.pre_stride * kHeadDim;
                pml = p.part_ml_pre + (size_t)seg.slot * p.pre_stride;
            } else {
                po = p.part_o_priv + (size_t)seg.slot * p.priv_stride * kHeadDim;
                pml = p.part_ml_priv + (size_t)seg.slot * p.priv_stride;
            }
            alive = mbar_wait(bar(L::L_FULL + pb), (pc >> 1) & 1, ab) && mbar_wait(bar(L::O_FULL + pb), (pc >> 1) & 1, ab);
            alive = __all_sync(0xffffffffu, alive);
            if (!alive) break;
            tc_fence_after();
            {   // all rows of this thread's head dim in one round trip to TMEM, then the stores
                float o[NB / 4][4];
#pragma unroll
                for (int k = 0; k < NB / 4; ++k)
                    if (4 * k < n_rows) tmem_ld4(tmem_o0 + (uint32_t)(pb * NB) + lane_base + (uint32_t)(4 * k), o[k]);
                tmem_wait_ld();
#pragma unroll
                for (int k = 0; k < NB / 4; ++k)
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (4 * k + e < n_rows) po[(size_t)(4 * k + e) * kHeadDim + dim] = o[k][e];
            }
            if (et < n_rows) {
                const float* ls = lsum + pb * 4 * NB + et;
                pml[et] = make_float2(mout[pb * NB + et], (ls[0] + ls[NB]) + (ls[2 * NB] + ls[3 * NB]));
            }
            tc_fence_before();
            warp_arrive(bar(L::O_FREE + pb), lane);
            warp_arrive(bar(L::L_FREE + pb), lane);
        }
    } else {
        // =========================== softmax warps ===========================
        // A wait that fails only clears `ok`; loops are left on block-wide reductions of !ok so that
        // all softmax threads leave together.
        float* mref = reinterpret_cast<float*>(smem + L::kOffMref);
        float* red = reinterpret_cast<float*>(smem + L::kOffRed);
        unsigned long long* vis = reinterpret_cast<unsigned long long*>(smem + L::kOffVis);
        const int quarter = warp & 3, cg = warp >> 2;       // TMEM lane quarter of this warp, column group
        const int tok = quarter * 32 + lane;                 // this thread's token in either tile; its dim in O^T
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        auto row_of = [&](int k) { return 4 * (cg + CG * k); };    // first row of this thread's k-th chunk
        // Where this thread's probabilities go.  P^T of a tile is the K-major B operand: two 64-token
        // blocks of NB rows x 128 bytes, 16-byte units XOR-swizzled with the row (r & 7).  The rows of
        // chunk k are 4 (cg + CG k) + e, e < 4; with an even CG their r & 7 is 4 (cg & 1) + e whatever k
        // is, so one address per e serves all chunks and both tiles with constant offsets.
        static_assert(CG % 2 == 0, "P^T store addresses assume an even number of column groups");
        uint32_t p_addr[4];
#pragma unroll
        for (int e = 0; e < 4; ++e)
            p_addr[e] = sbase + L::kOffP + (tok >> 6) * (NB * 128) + (4 * cg + e) * 128 +
                        (((((tok & 63) >> 3) ^ (4 * (cg & 1) + e))) << 4) + (tok & 7) * 2;
#pragma unroll
        for (int e = 0; e < 4; ++e) asm volatile("" : "+r"(p_addr[e]));      // kept in registers, not recomputed at every store
        auto store_p = [&](int i, int k, int e, unsigned short v) {   // row 4 (cg + CG k) + e of tile i
            asm volatile("st.shared.u16 [%0], %1;" ::"r"(p_addr[e] + (uint32_t)(i * L::kPBytes + k * (4 * CG * 128))), "h"(v) : "memory");
        };
        float* lsum = reinterpret_cast<float*>(smem + L::kOffLsum);
        float* mout = reinterpret_cast<float*>(smem + L::kOffMout);
        int ss = 0, u_v = 0, pc = 0;                          // steps, V tiles and pieces of this CTA so far
        bool ok = true;
        PieceDesc seg = pv.piece(0);
        QFetch<NB, NT> qf;
        qf.load(p, seg, tid);
        qf.store(smem + L::kOffQ, tid);
        fence_proxy_async();
        warp_arrive(bar(L::Q_FULL), lane);

        for (;;) {
            const int t_first = seg.tile0, t_last = seg.tile0 + seg.n_tiles;
            const int n_steps = ceil_div(seg.n_tiles, 2);
            const int Ltok = seg.seg_tokens;
            const int tail0 = seg.kind == 1 ? Ltok - p.R : Ltok;     // first token that needs the row mask
            const int n_rows = seg.n_rows;                            // chunks starting at or past it are skipped
            const uint32_t tmem_o = tmem_o0 + (uint32_t)((pc & 1) * NB);
            const bool have_next = pc + 1 < n_pieces;
            PieceDesc next = seg;
            if (have_next) {
                next = pv.piece(pc + 1);
                qf.load(p, next, tid);                                // in flight while this piece is computed
            }
            float l_part[NCK][4];
#pragma unroll
            for (int k = 0; k < NCK; ++k)
#pragma unroll
                for (int e = 0; e < 4; ++e) l_part[k][e] = 0.f;
            if (tid < NB) mref[tid] = -INFINITY;
            if (seg.kind == 1 && p.tree_parents != nullptr && tid < p.R) vis[tid] = row_visibility(p, seg.b, tid);
            bar_sync_id<NT>(1);

            for (int j = 0; j < n_steps; ++j, ++ss) {
                const int set = ss & 1;
                const int t = t_first + 2 * j;
                const int nt = min(2, t_last - t);                    // uniform: tiles of this step
                const bool need_mask = (t + nt) * kTileT > tail0;    // uniform: the step touches masked / missing tokens
                unsigned long long rowmask[2] = {~0ull, ~0ull};     // bit r: token i of this thread is visible to row r
                if (nt < 2) rowmask[1] = 0ull;
                if (need_mask) {
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        if (i >= nt) continue;
                        const int jt = (t + i) * kTileT + tok;
                        if (jt >= Ltok) rowmask[i] = 0ull;
                        else if (jt >= tail0) {
                            // token a of the last R: visible to query position i = (row0 + r) / G iff i >= a
                            // (causal) or a is i or an ancestor of i (tree)
                            const int a = jt - tail0;
                            if (p.tree_parents == nullptr) {
                                const int sh = a * p.G - seg.row0;
                                rowmask[i] = sh <= 0 ? ~0ull : (sh >= 64 ? 0ull : ~0ull << sh);
                            } else {
                                unsigned long long m = 0ull;
                                for (int r = 0; r < NB; ++r) {
                                    const int qi = (seg.row0 + r) / p.G;
                                    if (qi < p.R && ((vis[qi] >> a) & 1ull)) m |= 1ull << r;
                                }
                                rowmask[i] = m;
                            }
                        }
                    }
                }
                const bool masked = need_mask || nt < 2;             // uniform
                ok = ok && mbar_wait(bar(L::S_FULL + set), (ss >> 1) & 1, ab);
                if (ok) tc_fence_after();
                // d = score * scale - reference (log2 units), or the scaled score itself (raw); masked entries
                // are -inf.  The scores are read from TMEM each time (the rare second pass re-reads them), so
                // they do not occupy registers beside d.
                float d[2][NCK][4];
                // (with_mask: a step without masked tokens skips the tests; the columns of a missing second
                // tile hold stale scores, which the mask turns into -inf)
                auto compute_d = [&](bool raw, auto with_mask) -> float {
                    if (ok) {
#pragma unroll
                        for (int i = 0; i < 2; ++i)
#pragma unroll
                            for (int k = 0; k < NCK; ++k)
                                if (row_of(k) < n_rows) tmem_ld4(tmem + lane_base + (uint32_t)((2 * set + i) * NB + row_of(k)), d[i][k]);
                        tmem_wait_ld();
                    }
                    float mx = -INFINITY;
#pragma unroll
                    for (int k = 0; k < NCK; ++k) {
                        if (row_of(k) < n_rows) {
                            float4 m4 = make_float4(0.f, 0.f, 0.f, 0.f);
                            if (!raw) m4 = *reinterpret_cast<const float4*>(mref + row_of(k));
                            const float mm[4] = {m4.x, m4.y, m4.z, m4.w};
#pragma unroll
                            for (int i = 0; i < 2; ++i)
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    float v = fmaf(d[i][k][e], p.scale_log2, -mm[e]);      // +inf while the reference is -inf
                                    if (decltype(with_mask)::value && !((rowmask[i] >> (row_of(k) + e)) & 1ull)) v = -INFINITY;
                                    d[i][k][e] = v;
                                    mx = fmaxf(mx, v);
                                }
                        }
                    }
                    return mx;
                };
                float dmax;
                if (j == 0) {
                    // First step of a piece: the reference of every row is simply the score of the step's
                    // first token (of its two tiles); any reference within the lazy margin of the true
                    // maximum is as good, and the exact update below catches the rest.
                    compute_d(true, std::true_type{});
                    if (quarter == 0 && lane == 0) {
#pragma unroll
                        for (int k = 0; k < NCK; ++k) {
                            if (row_of(k) < n_rows) {
#pragma unroll
                                for (int e = 0; e < 4; ++e) mref[row_of(k) + e] = fmaxf(d[0][k][e], d[1][k][e]);
                            }
                        }
                    }
                    bar_sync_id<NT>(1);
                    dmax = -INFINITY;
#pragma unroll
                    for (int k = 0; k < NCK; ++k) {
                        if (row_of(k) < n_rows) {
                            const float4 m4 = *reinterpret_cast<const float4*>(mref + row_of(k));
                            const float mm[4] = {m4.x, m4.y, m4.z, m4.w};
#pragma unroll
                            for (int i = 0; i < 2; ++i)
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    // masked entries stay -inf; a row whose first token is masked has -inf as its
                                    // reference: +inf here, resolved by the exact update
                                    const float v = d[i][k][e] == -INFINITY ? -INFINITY : d[i][k][e] - mm[e];
                                    d[i][k][e] = v;
                                    dmax = fmaxf(dmax, v);
                                }
                        }
                    }
                } else {
                    dmax = masked ? compute_d(false, std::true_type{}) : compute_d(false, std::false_type{});
                }
                if (bar_red_or<NT>(1, dmax > kLazy || !ok)) {
                    // ---- rare: move the reference of every row to the running maximum ----
                    if (bar_red_or<NT>(1, !ok)) goto done;
                    compute_d(true, std::true_type{});
#pragma unroll
                    for (int k = 0; k < NCK; ++k) {
                        if (row_of(k) < n_rows) {
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float wm = warp_max_f32(fmaxf(d[0][k][e], d[1][k][e]));
                                if (lane == 0) red[quarter * NB + row_of(k) + e] = wm;
                            }
                        }
                    }
                    bar_sync_id<NT>(1);
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
                    if (j > 0 && bar_red_or<NT>(1, any_scale)) {
                        ok = ok && mbar_wait(bar(L::P_FREE), (ss & 1) ^ 1, ab);      // P.V of the previous step done
                        if (bar_red_or<NT>(1, !ok)) goto done;
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
                    bar_sync_id<NT>(1);                       // everyone has read the old references
                    if (tid < NB && (tid & ~3) < n_rows)
                        mref[tid] = fmaxf(mref[tid], fmaxf(fmaxf(red[tid], red[NB + tid]), fmaxf(red[2 * NB + tid], red[3 * NB + tid])));
                    bar_sync_id<NT>(1);
                    compute_d(false, std::true_type{});
                }
                tc_fence_before();
                warp_arrive(bar(L::S_FREE + set), lane);     // the scores have been consumed: S^T may be overwritten
                if (have_next && j == n_steps - 1) {
                    // the piece's last scores are complete, so its Q is no longer read: stage the next piece's
                    if (ok) qf.store(smem + L::kOffQ, tid);
                    fence_proxy_async();
                    warp_arrive(bar(L::Q_FULL), lane);
                }

                // ---- probabilities of this thread's tokens for its rows -> P^T of either tile ----
                ok = ok && mbar_wait(bar(L::P_FREE), (ss & 1) ^ 1, ab);      // P.V of the previous step done
                {
#pragma unroll
                    for (int i = 0; i < 2; ++i) {                  // a missing second tile gets zeros (nobody reads them)
#pragma unroll
                        for (int k = 0; k < NCK; ++k) {
                            if (row_of(k) < n_rows) {
                                float e4[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    e4[e] = ex2(d[i][k][e]);          // masked entries: ex2(-inf) = 0
                                    l_part[k][e] += e4[e];
                                }
#pragma unroll
                                for (int e = 0; e < 4; ++e) store_p(i, k, e, __bfloat16_as_ushort(__float2bfloat16_rn(e4[e])));
                            }
                        }
                    }
                }
                // last tile of a segment: V rows past the last valid token must be zero (they may hold
                // anything, and 0 x NaN is NaN)
                if (need_mask) {
                    for (int i = 0; i < nt; ++i) {
                        const int n_valid = min(kTileT, Ltok - (t + i) * kTileT);
                        if (n_valid < kTileT) {
                            const int uv = u_v + i, slot = NK + uv % NV;
                            ok = ok && mbar_wait(bar(L::FULL + slot), (uv / NV) & 1, ab);
                            if (ok) {
                                unsigned char* vb = smem + L::kOffRing + slot * kSlotBytes;
                                for (int idx = tid; idx < (kTileT - n_valid) * 16; idx += NT) {
                                    const int row = n_valid + (idx >> 4), c = idx & 15;
                                    *reinterpret_cast<uint4*>(vb + tile_row_off(row) + (c >> 3) * 1024 + ((c & 7) << 4)) = make_uint4(0, 0, 0, 0);
                                }
                            }
                        }
                    }
                }
                u_v += nt;
                fence_proxy_async();
                warp_arrive(bar(L::P_FULL), lane);
            }

            // ---- end of the piece: hand its row sums and references to the epilogue warps ----
            {
                const int pb = pc & 1;
                ok = ok && mbar_wait(bar(L::L_FREE + pb), ((pc >> 1) & 1) ^ 1, ab);      // read by the epilogue two pieces ago
                if (bar_red_or<NT>(1, !ok)) goto done;
#pragma unroll
                for (int k = 0; k < NCK; ++k) {
                    if (row_of(k) < n_rows) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float ws = warp_sum_f32(l_part[k][e]);
                            if (lane == 0) lsum[(pb * 4 + quarter) * NB + row_of(k) + e] = ws;
                        }
                    }
                }
                if (tid < NB) mout[pb * NB + tid] = mref[tid];            // the same thread resets mref[tid] below
                warp_arrive(bar(L::L_FULL + pb), lane);
            }
            ++pc;
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
    static bool attr_set[64] = {};                          // the attribute is per device
    if (c->device < 0 || c->device >= 64 || !attr_set[c->device]) {
        cudaError_t err = cudaFuncSetAttribute(attn_umma_t_kernel<NB, CG>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<NB>::kBytes);
        if (err != cudaSuccess) return err;
        if (c->device >= 0 && c->device < 64) attr_set[c->device] = true;
    }
    attn_umma_t_kernel<NB, CG><<<p.grid, 128 * CG + 224, Lay<NB>::kBytes, st>>>(p, mk, mv);
    return cudaGetLastError();
}

}  // namespace

// Row blocks of 32 also when a branch carries up to 64 rows per KV head (two blocks, the second reading
// the K/V tiles that the first left in L2): the 64-row instantiation holds twice the scores per thread
// and spills at the 128 registers that 15 warps allow, which cost more than the second pass.
int umma_t_rows(int nr) { (void)nr; return 32; }

cudaError_t launch_attn_umma_t(Ctx* c, const AttnParams& p, cudaStream_t st) {
    cudaError_t err = cudaSuccess;
    const CUtensorMap* mk = umma_pool_map(c, p.k_pages, 1, &err);
    if (!mk) return err;
    const CUtensorMap mk_copy = *mk;                       // the cache may reallocate on the next insert
    const CUtensorMap* mv = umma_pool_map(c, p.v_pages, 1, &err);
    if (!mv) return err;
    if (p.rb_rows == 32) return launch_nb<32, 2>(c, p, mk_copy, *mv, st);
    return cudaErrorInvalidValue;
}

}  // namespace tts
