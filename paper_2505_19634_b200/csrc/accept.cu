// Speculative-sampling accept / resample: one CTA per branch.
//
//  1. warp 0 gathers p_i(x_i), q_i(x_i) for the gamma draft tokens and applies the test
//     u_i * q <= p (single fp32 multiply) lane-parallel; a ballot gives the first rejection k.
//  2. all warps sweep the one row pair that matters -- max(0, p_k - q_k) after a rejection, or
//     p_gamma for the bonus token -- with 16-byte loads, 128 tokens per warp step, and leave one
//     fp64 sum per 128-token tile in shared memory.  This is the only pass over HBM.
//  3. warp 0 scans the tile sums (fp64), finds the tile where the running sum first exceeds
//     u_gamma * Z, re-reads those 128 weights and finishes the inverse CDF inside the tile.
#include "tts_internal.cuh"

namespace tts {

namespace {

constexpr int kAccThreads = 1024;
constexpr int kTileElems = 128;            // one warp step: 32 lanes x float4
constexpr int kMaxTiles = 4096;            // vocab <= 524288

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ double warp_incl_scan(double v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        double n = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += n;
    }
    return v;
}

// residual weight of one token; mode_residual: max(0, p - q) in fp32, else p
__device__ __forceinline__ float weight(float p, float q, bool residual) {
    if (!residual) return p;
    const float d = __fsub_rn(p, q);
    return d > 0.f ? d : 0.f;
}

// Where the weights of the final draw come from: four consecutive tokens at a time.  `Raw` is what one
// thread loads for them (all loads of a batch are issued before the first is used); weights() turns it into
// the four fp32 weights, max(0, p - q) for a residual draw and p otherwise.
struct ProbRows {                                   // rows of probabilities
    const float* pk; const float* qk;
    struct Raw { float4 p, q; };
    __device__ __forceinline__ Raw load(int x0, bool residual) const {
        Raw r;
        r.p = __ldg(reinterpret_cast<const float4*>(pk + x0));
        r.q = residual ? __ldg(reinterpret_cast<const float4*>(qk + x0)) : make_float4(0.f, 0.f, 0.f, 0.f);
        return r;
    }
    __device__ __forceinline__ void weights(const Raw& r, bool residual, float* w) const {
        w[0] = weight(r.p.x, r.q.x, residual); w[1] = weight(r.p.y, r.q.y, residual);
        w[2] = weight(r.p.z, r.q.z, residual); w[3] = weight(r.p.w, r.q.w, residual);
    }
};

// Probabilities from logits, every step one correctly rounded operation so that a host program can
// reproduce them bit for bit: d = l - max (fp32), y = d * log2(e) (fp32), n = round-to-nearest-even(y),
// f = y - n (exact), g = eight-term Taylor polynomial of 2^f by fp32 fused multiply-adds, e = g * 2^n (exact;
// 0 when y < -126), p = fp32((double) e * (1 / Z)) with Z the fp64 sum of the row's e.
__device__ __forceinline__ float exp_rel(float l, float m) {
    const float y = __fmul_rn(__fsub_rn(l, m), 1.44269504088896340736f);
    if (!(y >= -126.f)) return 0.f;
    const float n = rintf(y);
    const float f = __fsub_rn(y, n);
    float g = 1.52527338040598403e-5f;                                  // (ln 2)^k / k!, k = 7 .. 0
    g = __fmaf_rn(g, f, 1.54035303933816099e-4f);
    g = __fmaf_rn(g, f, 1.33335581464284434e-3f);
    g = __fmaf_rn(g, f, 9.61812910762847716e-3f);
    g = __fmaf_rn(g, f, 5.55041086648215800e-2f);
    g = __fmaf_rn(g, f, 2.40226506959100712e-1f);
    g = __fmaf_rn(g, f, 6.93147180559945309e-1f);
    g = __fmaf_rn(g, f, 1.0f);
    return __fmul_rn(g, __int_as_float(((int)n + 127) << 23));
}
__device__ __forceinline__ float prob_of(float l, float m, double inv_z) {
    return __double2float_rn(__dmul_rn((double)exp_rel(l, m), inv_z));
}

__device__ __forceinline__ float4 load4(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16* p) {
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
    return make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u),
                       __uint_as_float(v.y << 16), __uint_as_float(v.y & 0xffff0000u));
}

template <typename T>
struct LogitRows {                                  // rows of logits with their maxima and 1 / normalisers
    const T* lp; const T* lq;
    float mp, mq;
    double inv_p, inv_q;
    struct Raw { float4 p, q; };
    __device__ __forceinline__ Raw load(int x0, bool residual) const {
        Raw r;
        r.p = load4(lp + x0);
        r.q = residual ? load4(lq + x0) : make_float4(0.f, 0.f, 0.f, 0.f);
        return r;
    }
    __device__ __forceinline__ void weights(const Raw& r, bool residual, float* w) const {
        const float lpv[4] = {r.p.x, r.p.y, r.p.z, r.p.w}, lqv[4] = {r.q.x, r.q.y, r.q.z, r.q.w};
#pragma unroll
        for (int e = 0; e < 4; ++e)
            w[e] = weight(prob_of(lpv[e], mp, inv_p), residual ? prob_of(lqv[e], mq, inv_q) : 0.f, residual);
    }
};

// Steps 2 and 3 for one branch, by the whole CTA: the draw with u_final from norm(max(0, p - q)) (residual;
// from p if that is identically zero) or from p.  tile_sum, s_last_pos (-1) and s_redo (0) are shared scratch.
template <class Rows>
__device__ __forceinline__ void draw_token(const Rows& rows, bool residual,
                                           float u_final, int vocab, double* tile_sum, int* s_last_pos_p, int* s_redo_p,
                                           int32_t* next_token_out) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int& s_last_pos = *s_last_pos_p;
    int& s_redo = *s_redo_p;
    const int n_tiles = (vocab + kTileElems - 1) / kTileElems;

    double Z = 0.0;
    for (int attempt = 0; attempt < 2; ++attempt) {
        // ---- 2. one sweep: per-tile fp64 sums ----
        int last_pos = -1;
        // kSweepBatch tiles per warp and trip: their loads are all issued before the first is used (one SM has
        // to keep many loads in flight to pull its share of the bandwidth)
        constexpr int kSweepBatch = 4, kWarps = kAccThreads / 32;
        for (int j0 = warp; j0 < n_tiles; j0 += kWarps * kSweepBatch) {
            typename Rows::Raw raw[kSweepBatch];
#pragma unroll
            for (int k = 0; k < kSweepBatch; ++k) {
                const int x0 = (j0 + k * kWarps) * kTileElems + lane * 4;
                if (j0 + k * kWarps < n_tiles && x0 < vocab) raw[k] = rows.load(x0, residual);   // vocab % 4 == 0: four tokens in range
            }
#pragma unroll
            for (int k = 0; k < kSweepBatch; ++k) {
                const int j = j0 + k * kWarps;
                if (j >= n_tiles) break;                            // uniform over the warp
                const int x0 = j * kTileElems + lane * 4;
                double s = 0.0;
                if (x0 < vocab) {
                    float w[4];
                    rows.weights(raw[k], residual, w);
                    const float w0 = w[0], w1 = w[1], w2 = w[2], w3 = w[3];
                    s = (double)w0 + (double)w1 + (double)w2 + (double)w3;
                    if (w3 > 0.f) last_pos = max(last_pos, x0 + 3); else if (w2 > 0.f) last_pos = max(last_pos, x0 + 2);
                    else if (w1 > 0.f) last_pos = max(last_pos, x0 + 1); else if (w0 > 0.f) last_pos = max(last_pos, x0);
                }
                s = warp_sum(s);
                if (lane == 0) tile_sum[j] = s;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) last_pos = max(last_pos, __shfl_xor_sync(0xffffffffu, last_pos, o));
        if (lane == 0 && last_pos >= 0) atomicMax(&s_last_pos, last_pos);
        __syncthreads();

        // ---- 3a. warp 0: total mass ----
        if (warp == 0) {
            const int per = (n_tiles + 31) / 32;
            double c = 0.0;
            for (int j = lane * per; j < min(n_tiles, (lane + 1) * per); ++j) c += tile_sum[j];
            Z = warp_sum(c);
            if (lane == 0) s_redo = (residual && !(Z > 0.0)) ? 1 : 0;
        }
        __syncthreads();
        if (!s_redo) break;
        residual = false;                                        // residual identically 0: draw from p_k
        __syncthreads();
        if (tid == 0) s_last_pos = -1;
        __syncthreads();
    }

    // ---- 3b. warp 0: locate the crossing tile, then the token inside it ----
    if (warp == 0) {
        const double t = (double)u_final * Z;
        const int per = (n_tiles + 31) / 32;
        const int j0 = lane * per, j1 = min(n_tiles, (lane + 1) * per);
        double c = 0.0;
        for (int j = j0; j < j1; ++j) c += tile_sum[j];
        const double incl = warp_incl_scan(c, lane);
        const unsigned hit = __ballot_sync(0xffffffffu, incl > t);
        int chosen = -1;
        if (hit) {
            // The first lane whose inclusive sum exceeds t holds the crossing tile, unless re-adding its
            // tiles one by one rounds differently from the scan and leaves no crossing there: then the
            // crossing is the first tile with mass of the next lane, so the lanes of `hit` are tried in order.
            int tile = -1;
            double base = 0.0;
            for (unsigned h = hit; h != 0u && tile < 0; h &= h - 1u) {
                const int src = __ffs(h) - 1;
                if (lane == src) {
                    double run = incl - c;
                    for (int j = j0; j < j1; ++j) {
                        const double nxt = run + tile_sum[j];
                        if (nxt > t) { tile = j; base = run; break; }
                        run = nxt;
                    }
                }
                tile = __shfl_sync(0xffffffffu, tile, src);
                base = __shfl_sync(0xffffffffu, base, src);
            }
            if (tile >= 0) {
                const int x0 = tile * kTileElems + lane * 4;
                float w[4] = {0.f, 0.f, 0.f, 0.f};
                if (x0 < vocab) rows.weights(rows.load(x0, residual), residual, w);
                const double ls = (double)w[0] + (double)w[1] + (double)w[2] + (double)w[3];
                const double lincl = warp_incl_scan(ls, lane);
                const unsigned lhit = __ballot_sync(0xffffffffu, base + lincl > t);
                if (lhit) {
                    const int ls_src = __ffs(lhit) - 1;
                    int x = -1;
                    if (lane == ls_src) {
                        double run = base + (lincl - ls);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            run += (double)w[e];
                            if (x < 0 && run > t) x = x0 + e;
                        }
                        if (x < 0)                       // summation order left no crossing here
                            x = w[3] > 0.f ? x0 + 3 : (w[2] > 0.f ? x0 + 2 : (w[1] > 0.f ? x0 + 1 : x0));
                    }
                    chosen = __shfl_sync(0xffffffffu, x, ls_src);
                }
            }
        }
        if (lane == 0) {
            if (chosen < 0) chosen = s_last_pos >= 0 ? s_last_pos : vocab - 1;   // rounding left no crossing
            *next_token_out = chosen;
        }
    }
}

__global__ void __launch_bounds__(kAccThreads)
accept_kernel(const float* __restrict__ p_target, const float* __restrict__ q_draft,
              const int32_t* __restrict__ draft_tokens, const float* __restrict__ uniforms, int gamma,
              int vocab, int32_t* __restrict__ accepted_len, int32_t* __restrict__ next_token,
              int32_t* status) {
    __shared__ double tile_sum[kMaxTiles];
    __shared__ int s_k, s_last_pos, s_redo;

    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float* P = p_target + (size_t)b * (gamma + 1) * vocab;
    const float* Q = q_draft + (size_t)b * gamma * vocab;
    const float* U = uniforms + (size_t)b * (gamma + 1);

    // ---- 1. accept tests ----
    if (warp == 0) {
        int k = gamma;
        for (int base = 0; base < gamma && k == gamma; base += 32) {
            const int i = base + lane;
            bool reject = false;
            if (i < gamma) {
                int x = draft_tokens[(size_t)b * gamma + i];
                if (x < 0 || x >= vocab) { atomicMin(status, (int)TTS_ERR_DEVICE_BOUNDS); x = 0; }
                const float p = P[(size_t)i * vocab + x];
                const float q = Q[(size_t)i * vocab + x];
                const float uq = __fmul_rn(U[i], q);
                reject = !(p > 0.f && uq <= p);
            }
            const unsigned ballot = __ballot_sync(0xffffffffu, reject);
            if (ballot) k = base + __ffs(ballot) - 1;
        }
        if (lane == 0) { s_k = k; s_last_pos = -1; s_redo = 0; accepted_len[b] = k; }
    }
    __syncthreads();
    const int k = s_k;
    const float* pk = P + (size_t)k * vocab;
    const float* qk = Q + (size_t)(k < gamma ? k : 0) * vocab;
    draw_token(ProbRows{pk, qk}, k < gamma, U[gamma], vocab, tile_sum, &s_last_pos, &s_redo, next_token + b);
}

// Maximum and normaliser of one or two rows of logits, by the whole CTA: one pass for the maxima, one for the
// sums of exp_rel (fp64).  red is shared scratch of 64 doubles.  All threads return the same values.
template <typename T>
__device__ void rows_max_and_norm(const T* row_a, const T* row_b, int vocab, double* red, float* m_out, double* inv_out) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int kWarps = kAccThreads / 32;
    const int n_rows = row_b ? 2 : 1;
    float m[2] = {-INFINITY, -INFINITY};
    for (int x0 = tid * 4; x0 < vocab; x0 += kAccThreads * 4) {
        const float4 a = load4(row_a + x0);
        m[0] = fmaxf(m[0], fmaxf(fmaxf(a.x, a.y), fmaxf(a.z, a.w)));
        if (row_b) {
            const float4 c = load4(row_b + x0);
            m[1] = fmaxf(m[1], fmaxf(fmaxf(c.x, c.y), fmaxf(c.z, c.w)));
        }
    }
    float* redf = reinterpret_cast<float*>(red);
#pragma unroll
    for (int r = 0; r < 2; ++r) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m[r] = fmaxf(m[r], __shfl_xor_sync(0xffffffffu, m[r], o));
        if (lane == 0) redf[r * kWarps + warp] = m[r];
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        float v = redf[r * kWarps + lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
        m[r] = v;
    }
    __syncthreads();
    double z[2] = {0.0, 0.0};
    for (int x0 = tid * 4; x0 < vocab; x0 += kAccThreads * 4) {
        const float4 a = load4(row_a + x0);
        z[0] += ((double)exp_rel(a.x, m[0]) + (double)exp_rel(a.y, m[0])) + ((double)exp_rel(a.z, m[0]) + (double)exp_rel(a.w, m[0]));
        if (row_b) {
            const float4 c = load4(row_b + x0);
            z[1] += ((double)exp_rel(c.x, m[1]) + (double)exp_rel(c.y, m[1])) + ((double)exp_rel(c.z, m[1]) + (double)exp_rel(c.w, m[1]));
        }
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        z[r] = warp_sum(z[r]);
        if (lane == 0) red[r * kWarps + warp] = z[r];
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 2; ++r) z[r] = warp_sum(red[r * kWarps + lane]);
    __syncthreads();
    for (int r = 0; r < n_rows; ++r) { m_out[r] = m[r]; inv_out[r] = 1.0 / z[r]; }
}

// The accept rule fed with logits: the probabilities the tests and the final draw need are formed on the way
// (prob_of), position by position, so only the rows up to the first rejection are read.
template <typename T>
__global__ void __launch_bounds__(kAccThreads)
accept_logits_kernel(const T* __restrict__ target_logits, const T* __restrict__ draft_logits,
                     const int32_t* __restrict__ draft_tokens, const float* __restrict__ uniforms, int gamma,
                     int vocab, int32_t* __restrict__ accepted_len, int32_t* __restrict__ next_token,
                     int32_t* status) {
    __shared__ double tile_sum[kMaxTiles];
    __shared__ double red[64];
    __shared__ int s_last_pos, s_redo;
    static_assert(kAccThreads == 1024, "the block reductions assume 32 warps");

    const int b = blockIdx.x, tid = threadIdx.x;
    const T* P = target_logits + (size_t)b * (gamma + 1) * vocab;
    const T* Q = draft_logits + (size_t)b * gamma * vocab;
    const float* U = uniforms + (size_t)b * (gamma + 1);

    int k = gamma;
    float m[2] = {0.f, 0.f};
    double inv[2] = {1.0, 1.0};
    for (int i = 0; i < gamma; ++i) {
        const T* pi = P + (size_t)i * vocab;
        const T* qi = Q + (size_t)i * vocab;
        rows_max_and_norm(pi, qi, vocab, red, m, inv);
        int x = draft_tokens[(size_t)b * gamma + i];                     // the same for all threads
        if (x < 0 || x >= vocab) { if (tid == 0) atomicMin(status, (int)TTS_ERR_DEVICE_BOUNDS); x = 0; }
        const float p = prob_of((float)pi[x], m[0], inv[0]);
        const float q = prob_of((float)qi[x], m[1], inv[1]);
        const float uq = __fmul_rn(U[i], q);
        if (!(p > 0.f && uq <= p)) { k = i; break; }                     // uniform over the block
    }
    if (k == gamma) rows_max_and_norm<T>(P + (size_t)gamma * vocab, nullptr, vocab, red, m, inv);
    if (tid == 0) { accepted_len[b] = k; s_last_pos = -1; s_redo = 0; }
    __syncthreads();
    const LogitRows<T> rows{P + (size_t)k * vocab, Q + (size_t)(k < gamma ? k : 0) * vocab, m[0], m[1], inv[0], inv[1]};
    draw_token(rows, k < gamma, U[gamma], vocab, tile_sum, &s_last_pos, &s_redo, next_token + b);
}

// The same for a draft tree (n nodes per branch, at most kMaxTreeRows): node i passes iff
// p_par(i)(x_i) > 0 and u_i q_i(x_i) <= p_par(i)(x_i), p_par(i) being row 0 of p_target for a child of the
// last committed token and row 1 + parent otherwise; a node is accepted iff it and all its ancestors pass;
// the leaf whose path holds the most accepted nodes wins (ties: lowest leaf index).  The final draw uses
// the residual of the first failing node of that path, or row 1 + leaf if the whole path was accepted.
__global__ void __launch_bounds__(kAccThreads)
accept_tree_kernel(const float* __restrict__ p_target, const float* __restrict__ q_draft,
                   const int32_t* __restrict__ draft_tokens, const int32_t* __restrict__ tree_parents,
                   const float* __restrict__ uniforms, int n, int vocab, int32_t* __restrict__ accepted_len,
                   int32_t* __restrict__ last_node, int32_t* __restrict__ next_token, int32_t* status) {
    __shared__ double tile_sum[kMaxTiles];
    __shared__ int s_last_pos, s_redo, s_row, s_qrow;
    __shared__ signed char s_pass[kMaxTreeRows], s_par[kMaxTreeRows];

    const int b = blockIdx.x, tid = threadIdx.x;
    const float* P = p_target + (size_t)b * (n + 1) * vocab;
    const float* Q = q_draft + (size_t)b * n * vocab;
    const float* U = uniforms + (size_t)b * (n + 1);

    if (tid < n) {
        int par = tree_parents[(size_t)b * n + tid];
        if (par < -1 || par >= tid) { atomicMin(status, (int)TTS_ERR_DEVICE_BOUNDS); par = -1; }
        int x = draft_tokens[(size_t)b * n + tid];
        if (x < 0 || x >= vocab) { atomicMin(status, (int)TTS_ERR_DEVICE_BOUNDS); x = 0; }
        const float p = P[(size_t)(par + 1) * vocab + x];
        const float q = Q[(size_t)tid * vocab + x];
        const float uq = __fmul_rn(U[tid], q);
        s_pass[tid] = (p > 0.f && uq <= p) ? 1 : 0;
        s_par[tid] = (signed char)par;
    }
    __syncthreads();
    if (tid == 0) {
        // accepted nodes on the path to i, and whether the whole path to i is accepted (parents come first)
        signed char alen[kMaxTreeRows], whole[kMaxTreeRows], child[kMaxTreeRows];
        for (int i = 0; i < n; ++i) child[i] = 0;
        for (int i = 0; i < n; ++i) {
            const int par = s_par[i];
            const bool par_whole = par < 0 || whole[par];
            whole[i] = par_whole && s_pass[i];
            alen[i] = (par < 0 ? 0 : alen[par]) + (whole[i] ? 1 : 0);
            if (par >= 0) child[par] = 1;
        }
        int best = -1;
        for (int i = 0; i < n; ++i)
            if (!child[i] && (best < 0 || alen[i] > alen[best])) best = i;
        // walk the winning path up: the deepest accepted node and the failing node right after it
        int last = -1, fail = -1;
        for (int i = best; i >= 0; i = s_par[i]) {
            if (whole[i]) { last = i; break; }
            fail = i;
        }
        accepted_len[b] = best < 0 ? 0 : alen[best];
        last_node[b] = last;
        // n == 0: the bonus token of the committed prefix
        s_row = fail >= 0 ? s_par[fail] + 1 : best + 1;
        s_qrow = fail;
        s_last_pos = -1; s_redo = 0;
    }
    __syncthreads();
    const float* pk = P + (size_t)s_row * vocab;
    const float* qk = Q + (size_t)(s_qrow >= 0 ? s_qrow : 0) * vocab;
    draw_token(ProbRows{pk, qk}, s_qrow >= 0, U[n], vocab, tile_sum, &s_last_pos, &s_redo, next_token + b);
}

}  // namespace

cudaError_t launch_accept(const float* p_target, const float* q_draft, const int32_t* draft_tokens,
                          const float* uniforms, int n_branches, int gamma, int vocab,
                          int32_t* accepted_len, int32_t* next_token, int32_t* status,
                          cudaStream_t st) {
    accept_kernel<<<n_branches, kAccThreads, 0, st>>>(p_target, q_draft, draft_tokens, uniforms,
                                                      gamma, vocab, accepted_len, next_token, status);
    return cudaGetLastError();
}

cudaError_t launch_accept_logits(const void* target_logits, const void* draft_logits, int logits_dtype,
                                 const int32_t* draft_tokens, const float* uniforms, int n_branches, int gamma, int vocab,
                                 int32_t* accepted_len, int32_t* next_token, int32_t* status, cudaStream_t st) {
    if (logits_dtype == TTS_LOGITS_BF16)
        accept_logits_kernel<__nv_bfloat16><<<n_branches, kAccThreads, 0, st>>>(
            static_cast<const __nv_bfloat16*>(target_logits), static_cast<const __nv_bfloat16*>(draft_logits), draft_tokens,
            uniforms, gamma, vocab, accepted_len, next_token, status);
    else
        accept_logits_kernel<float><<<n_branches, kAccThreads, 0, st>>>(
            static_cast<const float*>(target_logits), static_cast<const float*>(draft_logits), draft_tokens, uniforms, gamma,
            vocab, accepted_len, next_token, status);
    return cudaGetLastError();
}

cudaError_t launch_accept_tree(const float* p_target, const float* q_draft, const int32_t* draft_tokens,
                               const int32_t* tree_parents, const float* uniforms, int n_branches, int n_nodes, int vocab,
                               int32_t* accepted_len, int32_t* last_node, int32_t* next_token, int32_t* status,
                               cudaStream_t st) {
    accept_tree_kernel<<<n_branches, kAccThreads, 0, st>>>(p_target, q_draft, draft_tokens, tree_parents, uniforms, n_nodes,
                                                           vocab, accepted_len, last_node, next_token, status);
    return cudaGetLastError();
}

}  // namespace tts
