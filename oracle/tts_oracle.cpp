// CPU oracle for the speculative-decoding verify step.  TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, obviously-correct restatement of what the verify step computes,
// used by the tests, by the smoke check and as the timed CPU baseline of the
// benchmark.  It shares no code with the CUDA path and the product never calls it.
//
// The paper (Section 3.2, "Sequence-wise Parallelism"; Section 2, "Speculative
// decoding") only says that the target model verifies gamma draft tokens in parallel,
// losslessly, for B concurrent branches of one question, with weights and KV caches
// streamed from HBM (Section 3.1).  The two computations below are therefore the
// textbook definitions the paper relies on:
//   * exact softmax attention with grouped KV heads over a paged KV cache whose
//     prompt prefix is shared by all branches (definition, written out directly), and
//   * the speculative-sampling accept / residual-resample rule of the works the paper
//     cites for lossless speculative decoding (taken step by step).
// All floating-point accumulation is fp64.  Decisions that the GPU must reproduce
// bit-for-bit (the accept test, the residual max(0, p - q)) are single fp32 operations.
//
// Build: g++ -O2 -std=c++17 -ffp-contract=off -shared -fPIC -pthread
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

namespace {

inline double bf16_to_double(uint16_t b) {
    uint32_t u = static_cast<uint32_t>(b) << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return static_cast<double>(f);
}

template <class F>
void parallel_for(long n, int n_threads, F fn) {
    if (n_threads <= 1 || n <= 1) {
        for (long i = 0; i < n; ++i) fn(i);
        return;
    }
    std::vector<std::thread> pool;
    int t_count = static_cast<int>(std::min<long>(n_threads, n));
    for (int t = 0; t < t_count; ++t)
        pool.emplace_back([=]() {
            for (long i = t; i < n; i += t_count) fn(i);
        });
    for (auto& th : pool) th.join();
}

}  // namespace

extern "C" {

// ---------------------------------------------------------------------------------
// Verify-step attention: the plain definition.
//
//   q            [N][R][Hq][D]              bf16 bits, R = gamma + 1
//   k_pages/v_pages [num_pages][Hkv][page][D] bf16 bits
//   block_table  [N][max_blocks]            physical page of logical page j of branch b;
//                                           logical order = shared prefix, then private
//   branch_lens  [N]                        private KV tokens, including the R in-flight ones
//   mask_kind 0  causal: row i sees prefix tokens [0,P) and private tokens j <= L_b - R + i
//   mask_kind 1  tree:   the last R private tokens are draft-tree nodes; row i sees the
//                prefix, private tokens j < L_b - R, and nodes a that are i or an ancestor
//                of i (tree_parents[b][i] in [-1, i), -1 = child of the committed context)
//   row_sel      optional n_sel triples (b, i, h): compute only those rows, out = [n_sel][D]
//   out          fp64 [N][R][Hq][D] (or [n_sel][D])
//   weight_sums  optional, one per computed row: sum of the softmax weights (must be 1)
//
// For query head h the KV head is h / (Hq / Hkv).  score = scale * <q, k>; weights =
// softmax over the allowed keys (two passes: max, then exp and sum); out = sum w * v.
// Returns 0, or -1 on inconsistent arguments.
// ---------------------------------------------------------------------------------
int oracle_verify_attn(const uint16_t* q, const uint16_t* k_pages, const uint16_t* v_pages,
                       const int32_t* block_table, int max_blocks, int prefix_len,
                       const int32_t* branch_lens, int n_branches, int gamma, int n_q_heads,
                       int n_kv_heads, int head_dim, int page_size, double scale, int mask_kind,
                       const int32_t* tree_parents, const int32_t* row_sel, int n_sel,
                       double* out, double* weight_sums, int n_threads) {
    const int R = gamma + 1;
    if (n_q_heads % n_kv_heads != 0 || prefix_len % page_size != 0) return -1;
    if (mask_kind == 1 && tree_parents == nullptr) return -1;
    for (int b = 0; b < n_branches; ++b)
        if (branch_lens[b] < R) return -1;
    const int G = n_q_heads / n_kv_heads;
    const long n_rows = row_sel ? n_sel : static_cast<long>(n_branches) * R * n_q_heads;

    parallel_for(n_rows, n_threads, [&](long row) {
        int b, i, h;
        if (row_sel) {
            b = row_sel[3 * row]; i = row_sel[3 * row + 1]; h = row_sel[3 * row + 2];
        } else {
            b = static_cast<int>(row / (static_cast<long>(R) * n_q_heads));
            i = static_cast<int>((row / n_q_heads) % R);
            h = static_cast<int>(row % n_q_heads);
        }
        const int kvh = h / G;
        const int L = branch_lens[b];
        const int total = prefix_len + L;          // logical tokens of this branch
        const uint16_t* qrow =
            q + ((static_cast<long>(b) * R + i) * n_q_heads + h) * head_dim;

        // which logical tokens may this row see?
        std::vector<char> allowed(total, 0);
        for (int t = 0; t < prefix_len; ++t) allowed[t] = 1;
        if (mask_kind == 0) {
            for (int j = 0; j <= L - R + i; ++j) allowed[prefix_len + j] = 1;
        } else {
            for (int j = 0; j < L - R; ++j) allowed[prefix_len + j] = 1;
            for (int a = i; a >= 0; a = tree_parents[static_cast<long>(b) * R + a])
                allowed[prefix_len + (L - R) + a] = 1;
        }

        auto kv_ptr = [&](const uint16_t* pages, int t) {
            long page = block_table[static_cast<long>(b) * max_blocks + t / page_size];
            int slot = t % page_size;
            return pages + ((page * n_kv_heads + kvh) * page_size + slot) * head_dim;
        };

        std::vector<double> score(total, 0.0);
        double mx = -std::numeric_limits<double>::infinity();
        for (int t = 0; t < total; ++t) {
            if (!allowed[t]) continue;
            const uint16_t* krow = kv_ptr(k_pages, t);
            double acc = 0.0;
            for (int d = 0; d < head_dim; ++d) acc += bf16_to_double(qrow[d]) * bf16_to_double(krow[d]);
            score[t] = scale * acc;
            mx = std::max(mx, score[t]);
        }
        double denom = 0.0;
        for (int t = 0; t < total; ++t)
            if (allowed[t]) {
                score[t] = std::exp(score[t] - mx);
                denom += score[t];
            }
        std::vector<double> acc(head_dim, 0.0);
        double wsum = 0.0;
        for (int t = 0; t < total; ++t) {
            if (!allowed[t]) continue;
            double w = score[t] / denom;
            wsum += w;
            const uint16_t* vrow = kv_ptr(v_pages, t);
            for (int d = 0; d < head_dim; ++d) acc[d] += w * bf16_to_double(vrow[d]);
        }
        double* o = out + row * head_dim;
        for (int d = 0; d < head_dim; ++d) o[d] = acc[d];
        if (weight_sums) weight_sums[row] = wsum;
    });
    return 0;
}

// ---------------------------------------------------------------------------------
// Speculative-sampling accept / resample, one chain of gamma draft tokens per branch.
//
//   p_target [N][gamma+1][V] fp32   target distribution at each of the gamma+1 positions
//   q_draft  [N][gamma][V]   fp32   draft distribution the draft token i was drawn from
//   draft_tokens [N][gamma]  int32
//   uniforms [N][gamma+1]    fp32   u_0..u_{gamma-1} decide the tests, u_gamma drives the one
//                                   final draw (residual resample or bonus token)
// Steps, per branch:
//   1. for i = 0..gamma-1: x = draft token i, p = p_i(x), q = q_i(x);
//      accept iff p > 0 and u_i * q <= p   (one fp32 multiply; same as u <= min(1, p/q));
//      stop at the first rejection, k = number accepted.
//   2. if k < gamma: r(x) = max(0, p_k(x) - q_k(x)) in fp32 (if every r is 0, r = p_k);
//      else            r(x) = p_gamma(x)  (bonus token).
//   3. Z = sum r (fp64, in index order); t = u_gamma * Z;
//      next = smallest x with C_x = sum_{x' <= x} r(x') > t; if rounding leaves none,
//      the last x with r(x) > 0.
// near_flags (optional, [N]): bit 0 = a test of step 1 had |u q - p| <= 1e-6 max(p, q);
//                             bit 1 = t within 1e-9 Z of the CDF boundary on either side
//                                     of the chosen token.
// ---------------------------------------------------------------------------------
int oracle_accept(const float* p_target, const float* q_draft, const int32_t* draft_tokens,
                  const float* uniforms, int n_branches, int gamma, int vocab,
                  int32_t* accepted_len, int32_t* next_token, int32_t* near_flags,
                  int n_threads) {
    if (n_branches < 0 || gamma < 0 || vocab <= 0) return -1;
    parallel_for(n_branches, n_threads, [&](long b) {
        const float* P = p_target + b * static_cast<long>(gamma + 1) * vocab;
        const float* Q = q_draft + b * static_cast<long>(gamma) * vocab;
        const int32_t* X = draft_tokens + b * static_cast<long>(gamma);
        const float* U = uniforms + b * static_cast<long>(gamma + 1);
        int flags = 0;
        int k = gamma;
        for (int i = 0; i < gamma; ++i) {
            const int x = X[i];
            const float p = P[static_cast<long>(i) * vocab + x];
            const float q = Q[static_cast<long>(i) * vocab + x];
            volatile float uq = U[i] * q;              // rounded to fp32 before the compare
            const float uqf = uq;
            if (std::fabs(static_cast<double>(uqf) - static_cast<double>(p)) <=
                1e-6 * std::max(static_cast<double>(p), static_cast<double>(q)))
                flags |= 1;
            const bool ok = (p > 0.0f) && (uqf <= p);
            if (!ok) { k = i; break; }
        }
        accepted_len[b] = k;

        const float* pk = P + static_cast<long>(k) * vocab;
        const float* qk = (k < gamma) ? Q + static_cast<long>(k) * vocab : nullptr;
        std::vector<float> r(vocab);
        double Z = 0.0;
        for (int x = 0; x < vocab; ++x) {
            float v;
            if (qk) {
                volatile float diff = pk[x] - qk[x];
                v = diff > 0.0f ? diff : 0.0f;
            } else {
                v = pk[x];
            }
            r[x] = v;
            Z += static_cast<double>(v);
        }
        if (qk && !(Z > 0.0)) {                      // p <= q everywhere (only by rounding)
            Z = 0.0;
            for (int x = 0; x < vocab; ++x) { r[x] = pk[x]; Z += static_cast<double>(pk[x]); }
        }
        const double t = static_cast<double>(U[gamma]) * Z;
        double C = 0.0, C_prev = 0.0;
        int chosen = -1, last_pos = -1;
        for (int x = 0; x < vocab; ++x) {
            if (r[x] > 0.0f) last_pos = x;
            C_prev = C;
            C += static_cast<double>(r[x]);
            if (C > t) { chosen = x; break; }
        }
        if (chosen < 0) { chosen = last_pos < 0 ? vocab - 1 : last_pos; flags |= 2; }
        else if (std::fabs(C - t) <= 1e-9 * Z || (chosen > 0 && std::fabs(t - C_prev) <= 1e-9 * Z))
            flags |= 2;
        next_token[b] = chosen;
        if (near_flags) near_flags[b] = flags;
    });
    return 0;
}

// ---------------------------------------------------------------------------------
// Probabilities from logits, for the accept rule fed with logits instead of probabilities (the
// softmax that sits between the target model's last layer and the accept test; Section 2,
// "Speculative decoding": the rule compares the target's and the draft's token distributions).
// The paper fixes no arithmetic for it; this is the reading, chosen so that the accept decisions
// can be reproduced bit for bit: every step is one correctly rounded fp32 operation (or one fp64
// sum), none of them left to a library exp.
//   per row l[0..V):  m = max_x l(x)
//     d = l(x) - m                       fp32 subtract
//     y = d * log2(e)                    fp32 multiply, log2(e) rounded to fp32
//     n = round-to-nearest-even(y),  f = y - n   (exact, |f| <= 1/2)
//     g = c0 + f (c1 + f (c2 + ... f c7))  eight-term Taylor polynomial of 2^f = exp(f ln 2), every
//                                          step one fp32 fused multiply-add, c_k = (ln 2)^k / k! in fp32
//     e(x) = g * 2^n   (exact scaling; 0 when y < -126: the value would be subnormal)
//   Z = sum_x e(x)   fp64, index order;   p(x) = fp32( (double) e(x) * (1 / Z) )   fp64 multiply, one rounding
// logits: fp32 [rows][V];  probs out: fp32 [rows][V].
// ---------------------------------------------------------------------------------
int oracle_softmax_rows(const float* logits, long rows, int vocab, float* probs, int n_threads) {
    if (rows < 0 || vocab <= 0) return -1;
    static const float kLog2e = 1.44269504088896340736f;
    // (ln 2)^k / k!, k = 0..7
    static const float kC[8] = {1.0f, 6.93147180559945309e-1f, 2.40226506959100712e-1f, 5.55041086648215800e-2f,
                                9.61812910762847716e-3f, 1.33335581464284434e-3f, 1.54035303933816099e-4f,
                                1.52527338040598403e-5f};
    parallel_for(rows, n_threads, [&](long r) {
        const float* l = logits + r * static_cast<long>(vocab);
        float* out = probs + r * static_cast<long>(vocab);
        float m = l[0];
        for (int x = 1; x < vocab; ++x) m = l[x] > m ? l[x] : m;
        std::vector<float> e(vocab);
        double Z = 0.0;
        for (int x = 0; x < vocab; ++x) {
            volatile float d = l[x] - m;
            volatile float y = d * kLog2e;
            float ex = 0.0f;
            if (y >= -126.0f) {
                const float n = std::nearbyintf(y);          // round to nearest even (default rounding mode)
                volatile float f = y - n;
                float g = kC[7];
                for (int k = 6; k >= 0; --k) g = std::fmaf(g, f, kC[k]);
                ex = std::ldexp(g, static_cast<int>(n));      // exact: g in [0.7, 1.5], n >= -126
            }
            e[x] = ex;
            Z += static_cast<double>(ex);
        }
        const double inv = 1.0 / Z;
        for (int x = 0; x < vocab; ++x) out[x] = static_cast<float>(static_cast<double>(e[x]) * inv);
    });
    return 0;
}

// ---------------------------------------------------------------------------------
// Answer aggregation over the N branches of one question (Section 3.2 "majority voting";
// Section 4.6 / Table "aggregation" for the confidence-weighted variants).
//   mode 0 "vote": winner = answer with the largest count (weights == NULL) or the largest
//                  sum of weights; ties go to the answer that occurs first.
//   mode 1 "max":  winner = answer of the single branch with the largest weight
//                  (ties: lowest branch index).  Needs weights.
// votes = number of branches that gave the winner; score = its count / weight sum / weight.
// ---------------------------------------------------------------------------------
int oracle_majority_vote(const int64_t* answers, const float* weights, int n, int mode,
                         int64_t* winner, int32_t* votes, double* score) {
    if (n <= 0 || (mode == 1 && !weights) || mode < 0 || mode > 1) return -1;
    int best = -1;
    double best_score = 0.0;
    if (mode == 1) {
        for (int i = 0; i < n; ++i)
            if (best < 0 || static_cast<double>(weights[i]) > best_score) {
                best = i; best_score = weights[i];
            }
    } else {
        for (int i = 0; i < n; ++i) {
            bool first = true;
            for (int j = 0; j < i; ++j) if (answers[j] == answers[i]) { first = false; break; }
            if (!first) continue;
            double s = 0.0;
            for (int j = i; j < n; ++j)
                if (answers[j] == answers[i]) s += weights ? static_cast<double>(weights[j]) : 1.0;
            if (best < 0 || s > best_score) { best = i; best_score = s; }
        }
    }
    int count = 0;
    for (int j = 0; j < n; ++j) if (answers[j] == answers[best]) ++count;
    *winner = answers[best];
    if (votes) *votes = count;
    if (score) *score = best_score;
    return 0;
}

// ---------------------------------------------------------------------------------
// Greedy search over (B, gamma) (Algorithm 1).  acc(B, gamma) is supplied as a dense
// table acc[log2 B][gamma] with (n_logb x n_gamma) entries; points outside it end the
// search in that direction.  Writes the chosen configuration, the number of loop
// iterations ("steps": one per accepted move plus the final one that fails to improve)
// and the number of tts_task evaluations (1 baseline + 2 per iteration).
// ---------------------------------------------------------------------------------
int oracle_greedy_search(const double* acc_table, int n_logb, int n_gamma, int* best_logb,
                         int* best_gamma, double* best_acc, int* n_steps, int* n_evals) {
    if (n_logb <= 0 || n_gamma <= 0) return -1;
    auto at = [&](int lb, int g) -> double {
        if (lb >= n_logb || g >= n_gamma) return -std::numeric_limits<double>::infinity();
        return acc_table[lb * n_gamma + g];
    };
    int lb = 0, g = 0, evals = 1, steps = 0;
    double acc = at(0, 0);
    for (;;) {
        double acc_b = at(lb + 1, g);
        double acc_g = at(lb, g + 1);
        evals += 2;
        ++steps;
        int nlb, ng; double nacc;
        if (acc_b >= acc_g) { nlb = lb + 1; ng = g; nacc = acc_b; }
        else                { nlb = lb; ng = g + 1; nacc = acc_g; }
        if (nacc > acc) { lb = nlb; g = ng; acc = nacc; }
        else break;
    }
    *best_logb = lb; *best_gamma = g; *best_acc = acc; *n_steps = steps; *n_evals = evals;
    return 0;
}

}  // extern "C"
