/*
 * tts.h -- C-ABI of the B200 (sm_100a) verify-step library.
 *
 * The verify step of batched speculative decoding for test-time scaling: the target model
 * scores N concurrent branches of one question (branch-wise parallelism, Section 3.2), each
 * carrying gamma draft tokens plus one bonus position (sequence-wise parallelism, Section 3.2;
 * the target checks all gamma drafts in one pass and the output distribution stays the
 * target's own, Section 2).  The library covers the two parts of that step that are not weight
 * GEMMs:
 *   (1) GQA attention of the N*(gamma+1) query positions over a paged KV cache (the cache is
 *       streamed from HBM at every step, Section 3.1) whose prompt prefix is shared by all
 *       branches, and
 *   (2) the speculative-sampling accept / residual-resample pass,
 * plus the host-side answer aggregation (majority voting, Section 3.2; confidence-weighted
 * variants, Section 4.6) and the greedy (B, gamma) search (Algorithm 1).
 *
 * Conventions
 *   - Every function returns a tts_status (0 = OK, negative = error); no exceptions, no
 *     process exit, no CPU fallback.
 *   - "device" pointers are CUDA device memory on the context's device, owned by the caller,
 *     16-byte aligned and densely packed in the stated layout.  The library never frees or
 *     retains them.  "host" pointers are ordinary process memory.
 *   - Device work is asynchronous on the context's stream; outputs are valid once the caller
 *     has synchronised that stream.
 *   - bf16 = 16-bit brain float, fp32 = IEEE binary32, i32 = int32_t.
 */
#ifndef TTS_H_
#define TTS_H_

#include <stdint.h>

#if defined(__GNUC__)
#define TTS_API __attribute__((visibility("default")))
#else
#define TTS_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    TTS_OK = 0,
    TTS_ERR_INVALID = -1,        /* null pointer, size out of range, misaligned, prefix_len % page != 0 */
    TTS_ERR_UNSUPPORTED = -2,    /* head_dim != 128, page_size != 16, unknown mask_kind / option */
    TTS_ERR_CUDA = -3,           /* a CUDA call failed; tts_last_cuda_error() has the code */
    TTS_ERR_DEVICE_BOUNDS = -4,  /* (via tts_last_status) a kernel saw a page id / token out of range */
    TTS_ERR_DEVICE_TIMEOUT = -5, /* (via tts_last_status) a bounded device-side wait ran out */
    TTS_ERR_SCRATCH = -6         /* tts_verify_attn_noalloc: the problem needs more than the fixed scratch array */
} tts_status;

enum { TTS_MASK_CAUSAL = 0, TTS_MASK_TREE = 1 };
enum { TTS_OUT_BF16 = 0, TTS_OUT_FP32 = 1 };
enum { TTS_LOGITS_BF16 = 0, TTS_LOGITS_FP32 = 1 };
/* Which attention kernel runs: AUTO picks tensor cores (tcgen05, TMEM accumulators) when the
 * stacked query rows per KV head make it worthwhile and CUDA cores otherwise.  TCGEN05 picks
 * between the two tensor-core kernels: TOKEN_MAJOR (KV tokens on the MMA M dimension, for at most
 * 64 rows per branch and KV head: chains of gamma+1 positions) and ROW_MAJOR (query rows on M, for
 * draft trees with many nodes).  The last two force one of them. */
enum { TTS_ATTN_AUTO = 0, TTS_ATTN_SIMT = 1, TTS_ATTN_TCGEN05 = 2, TTS_ATTN_TCGEN05_TOKEN_MAJOR = 3,
       TTS_ATTN_TCGEN05_ROW_MAJOR = 4 };

typedef struct tts_ctx tts_ctx;

typedef struct {
    int32_t n_q_heads;             /* Hq */
    int32_t n_kv_heads;            /* Hkv, divides Hq; query head h reads KV head h / (Hq/Hkv) */
    int32_t head_dim;              /* must be 128 */
    int32_t page_size;             /* must be 16 tokens */
    int32_t max_branches;          /* upper bound for n_branches (sizes the workspace) */
    int32_t max_rows_per_branch;   /* upper bound for gamma+1 (or tree nodes) */
    int32_t max_blocks_per_branch; /* row stride of block_table, in entries */
    int32_t num_pages;             /* pages in each K / V pool; page ids must be < num_pages */
    int32_t out_dtype;             /* TTS_OUT_BF16 (round to nearest even) or TTS_OUT_FP32 */
    int32_t attn_impl;             /* TTS_ATTN_* */
    float   softmax_scale;         /* 0 => 1/sqrt(head_dim) */
    int32_t debug_bounds;          /* != 0: the kernels range-check block indices and page ids and report
                                      through tts_last_status instead of reading out of range */
    int32_t max_ctas;              /* 0: the attention kernels size their grids from the SM count; > 0: upper
                                      bound on the CTAs of the main attention kernel.  It changes how the KV
                                      tokens are split between CTAs, not what is computed (tuning / tests) */
} tts_config;

/* Creates a context on the CURRENT CUDA device and allocates its workspace there (split-KV
 * partial results; a few MB to tens of MB depending on max_branches).  Host pointer out. */
TTS_API int tts_create(const tts_config* cfg, tts_ctx** out);
/* Frees the workspace.  The caller must have synchronised the stream first. */
TTS_API int tts_destroy(tts_ctx* ctx);
/* cuda_stream is a cudaStream_t passed as void*; NULL = the legacy default stream. */
TTS_API int tts_set_stream(tts_ctx* ctx, void* cuda_stream);

/*
 * Verify-step attention for one layer (Section 3.1: the KV cache is streamed from HBM; Section
 * 3.2: N branches x (gamma+1) positions are scored in one pass).  Exact softmax attention:
 *   out[b][i][h] = sum_t softmax_t(scale * <q[b][i][h], K[t][h/G]>) * V[t][h/G]
 * over the keys row i of branch b may see: all prefix tokens, and the private tokens
 * j <= L_b - (gamma+1) + i of that branch (TTS_MASK_CAUSAL, bottom-right aligned).
 *
 *   q, out       device  [n_branches][gamma+1][Hq][128]  bf16 (out: cfg.out_dtype)
 *   k_pages,     device  [num_pages][Hkv][16][128] bf16; slots no query may see (tail of a
 *   v_pages              branch's last page, unused pages) may hold anything, NaN included
 *   block_table  device  [n_branches][max_blocks_per_branch] i32: physical page of logical page
 *                        j of branch b, logical order = prefix pages then private pages.  The
 *                        first prefix_len/16 entries of every row must be equal (that equality
 *                        is the sharing); entries past a branch's last page are ignored.
 *   prefix_len   host    shared-prefix tokens, multiple of 16 (a ragged prompt tail belongs to
 *                        the private part); may be 0
 *   branch_lens  device  [n_branches] i32: private KV tokens of each branch INCLUDING the
 *                        gamma+1 in-flight positions, whose K/V are already in the pages;
 *                        precondition branch_lens[b] >= gamma+1
 *   mask_kind    TTS_MASK_CAUSAL (TTS_MASK_TREE: use tts_verify_attn_tree)
 * Errors: INVALID / UNSUPPORTED from host-side checks, CUDA on launch failure.  What lives on the
 * device cannot be checked by the host: branch_lens[b] >= gamma+1, prefix_len + branch_lens[b] <=
 * 16 * max_blocks_per_branch, and page ids in [0, num_pages) are preconditions.  With
 * cfg.debug_bounds != 0 the kernels test the last two: a block index past the table row or a page id
 * outside the pool raises TTS_ERR_DEVICE_BOUNDS (tts_last_status) and page 0 is read in its place;
 * without it such a call reads out of range.
 */
TTS_API int tts_verify_attn(tts_ctx* ctx, const void* q, const void* k_pages, const void* v_pages,
                    const int32_t* block_table, int prefix_len, const int32_t* branch_lens,
                    int n_branches, int gamma, int mask_kind, void* out);

/*
 * The schedule of the attention calls of one verify step, built once (Section 3.1: a step is one pass
 * through all layers over the same KV cache, so block_table and branch_lens are the same in every
 * layer's call; the target model of Appendix A.1 has 64 layers).  tts_attn_plan works out, on the device
 * and asynchronously on the context's stream, how the KV tokens of a call with these arguments are
 * divided among the thread blocks, and keeps the result in the context.  Every later tts_verify_attn /
 * tts_verify_attn_tree call with the SAME block_table and branch_lens pointers, prefix_len, n_branches
 * and rows per branch (gamma+1, or n_nodes) then starts from those tables instead of deriving the
 * schedule again in each launch.  The caller promises that the contents of block_table and branch_lens
 * do not change between tts_attn_plan and those calls; after changing them (tts_kv_rollback on the same
 * branch_lens drops the plan by itself) call tts_attn_plan again or tts_attn_plan_drop.  A call whose
 * arguments do not match the kept plan is still correct: it builds its own schedule first (one more small
 * launch) and drops the kept plan.  Arguments and errors as for tts_verify_attn.
 */
TTS_API int tts_attn_plan(tts_ctx* ctx, const int32_t* block_table, int prefix_len, const int32_t* branch_lens,
                  int n_branches, int rows_per_branch);
TTS_API int tts_attn_plan_drop(tts_ctx* ctx);

/*
 * Several questions in one call (the multi-request setting of the paper's appendix: #Req questions in
 * flight, each with B branches that share that question's prompt; Section 3.3: the forward pass turns
 * compute-bound as B * (gamma+1) * #Req grows).  The branches are numbered group by group: group g holds
 * group_sizes[g] consecutive branches whose block-table rows start with the same group_prefix_len[g] / 16
 * pages.  The result for every branch is what tts_verify_attn gives for its group alone; one launch
 * serves all groups, each shared prefix being read once per group.
 *   group_sizes, group_prefix_len   host  [n_groups] i32, sizes >= 1 summing to n_branches, prefix
 *                                         lengths multiples of 16 (0 allowed); n_groups <= 64
 *   everything else as for tts_verify_attn (causal mask).  tts_attn_plan_groups is tts_attn_plan for such
 *   calls; the kept plan also records the group arrays' contents.
 */
TTS_API int tts_verify_attn_groups(tts_ctx* ctx, const void* q, const void* k_pages, const void* v_pages,
                           const int32_t* block_table, const int32_t* group_sizes,
                           const int32_t* group_prefix_len, int n_groups, const int32_t* branch_lens,
                           int n_branches, int gamma, void* out);
TTS_API int tts_attn_plan_groups(tts_ctx* ctx, const int32_t* block_table, const int32_t* group_sizes,
                         const int32_t* group_prefix_len, int n_groups, const int32_t* branch_lens,
                         int n_branches, int rows_per_branch);

/*
 * Tree verification (draft token trees, as produced by tree drafters such as the EAGLE-3 draft
 * model used in Section 4.1): the last n_nodes private tokens of each branch are tree nodes;
 * row i sees the prefix, the private tokens before the tree, itself and its ancestors.
 *   tree_parents device [n_branches][n_nodes] i32, parent index in [-1, i); -1 = the node hangs
 *                off the committed context.  q/out are [n_branches][n_nodes][Hq][128].
 */
TTS_API int tts_verify_attn_tree(tts_ctx* ctx, const void* q, const void* k_pages, const void* v_pages,
                         const int32_t* block_table, int prefix_len, const int32_t* branch_lens,
                         const int32_t* tree_parents, int n_branches, int n_nodes, void* out);

/*
 * Verify-step attention without any allocation (the paper has no counterpart: this entry point exists
 * for the library's hosts, not for the method).  It is for callers that cannot obtain device memory
 * when they call: a server that gave the whole GPU to its own pool allocator at start-up, a plugin
 * inside a framework whose memory plan is frozen, code that must not trigger the implicit
 * synchronisation of a driver allocation.  They cannot use tts_create (it calls cudaMalloc), so this
 * function takes no context: shapes and the stream are arguments, and the split-KV partial results
 * go to a fixed 8 MiB array inside the library image (each GPU that loads the library holds it
 * until the process exits).  It computes exactly what tts_verify_attn computes with TTS_MASK_CAUSAL,
 * bf16 output and scale 1/sqrt(128), on the CUDA-core kernel; it calls no cudaMalloc / cudaFree.
 *   q, k_pages, v_pages, block_table, prefix_len, branch_lens, out: as for tts_verify_attn
 *   max_blocks_per_branch: row stride of block_table; n_q_heads, n_kv_heads: as in tts_config
 *   cuda_stream: cudaStream_t as void*, NULL = legacy default stream; the call is asynchronous on it
 * Limits and caveats:
 *   - a problem whose partial results exceed the array returns TTS_ERR_SCRATCH and launches nothing:
 *     (Hkv * ceil(N*nr/rb) + 128) * min(N*nr, rb) + (N * Hkv * ceil(nr/rb) + 128) * min(nr, rb) rows of 520
 *     bytes must fit 8 MiB, with nr = (gamma+1) * Hq/Hkv and rb = 8, 16 or 32 (the smallest >= nr, else 32);
 *     the 32B-shaped layer (N 16, Hkv 8, nr 20) fits;
 *   - the first call on a device looks up the array's address there (that device must be current);
 *     make that first call before any stream capture;
 *   - all calls share the one array, which keeps the previous call's contents (the status word in it
 *     is cleared on the stream at every call; nothing else needs clearing); two calls whose kernels
 *     may overlap on the GPU (different streams, no dependency) race on it - serialise them;
 *   - device-side preconditions (page ids in range, branch_lens >= gamma+1, prefix_len + branch_lens
 *     within the table row) are not checked, and the status word that the kernels keep in the array
 *     has no accessor: a caller cannot read it;
 *   - the array's address is looked up once per device and kept: after cudaDeviceReset on that device
 *     the kept address is stale and this entry point must not be called again in the process.
 */
TTS_API int tts_verify_attn_noalloc(const void* q, const void* k_pages, const void* v_pages,
                            const int32_t* block_table, int max_blocks_per_branch, int prefix_len,
                            const int32_t* branch_lens, int n_branches, int gamma, int n_q_heads,
                            int n_kv_heads, void* out, void* cuda_stream);

/*
 * Speculative-sampling accept / resample (the lossless verification rule of the works cited in
 * Section 2, "Speculative decoding").  Per branch b, with x_i = draft_tokens[b][i]:
 *   accept x_i iff p_i(x_i) > 0 and u_i * q_i(x_i) <= p_i(x_i)  (one fp32 multiply), i = 0.. ;
 *   accepted_len[b] = number accepted before the first rejection (0..gamma);
 *   next_token[b]  = inverse-CDF draw with u_gamma from norm(max(0, p_k - q_k)) after a rejection
 *                    at k (from p_k if that residual is identically 0), or from p_gamma (bonus
 *                    token) when all gamma were accepted: the smallest x whose running sum of
 *                    weights (fp64) exceeds u_gamma * total.
 *   p_target device [n_branches][gamma+1][vocab] fp32     q_draft device [n_branches][gamma][vocab] fp32
 *   draft_tokens device [n_branches][gamma] i32           uniforms device [n_branches][gamma+1] fp32 in [0,1)
 *   accepted_len, next_token device [n_branches] i32.     vocab % 4 == 0; gamma may be 0.
 */
TTS_API int tts_accept(tts_ctx* ctx, const float* p_target, const float* q_draft,
               const int32_t* draft_tokens, const float* uniforms, int n_branches, int gamma,
               int vocab, int32_t* accepted_len, int32_t* next_token);

/*
 * The same accept / resample rule fed with LOGITS (Section 2, "Speculative decoding": the rule compares
 * the target's and the draft's token distributions; this entry point takes them before the softmax, so
 * the fp32 probability tensors need not be materialised).  p_i = softmax(target_logits[b][i]) and q_i =
 * softmax(draft_logits[b][i]) are formed inside the kernel, then everything is as in tts_accept.  The
 * paper fixes no arithmetic for the softmax; the library's is stated step by step so that a host program
 * can reproduce every decision bit for bit.  Per row l, with m = max_x l(x) and every step one correctly
 * rounded operation:
 *     d = l(x) - m (fp32);  y = d * log2(e) (fp32);  n = round-to-nearest-even(y);  f = y - n (exact);
 *     g = sum_{k<8} (ln 2)^k / k! f^k by Horner's rule in fp32 fused multiply-adds, highest term first;
 *     e(x) = g * 2^n (exact; 0 when y < -126);  Z = sum_x e(x) in fp64;  p(x) = fp32((double) e(x) * (1 / Z)).
 * The fp64 sum is the only step whose result depends on the order of evaluation (relative 1e-16).  Callers
 * apply a sampling temperature by scaling the logits beforehand.  Logits must be finite or -inf (a token
 * that is ruled out), with at least one finite value per row.
 *   target_logits device [n_branches][gamma+1][vocab], draft_logits device [n_branches][gamma][vocab],
 *   both bf16 (TTS_LOGITS_BF16) or both fp32 (TTS_LOGITS_FP32), 16-byte aligned; the other arguments as
 *   for tts_accept.  Only the rows up to the first rejection are read (twice: maximum, then sum).
 */
TTS_API int tts_accept_logits(tts_ctx* ctx, const void* target_logits, const void* draft_logits, int logits_dtype,
                      const int32_t* draft_tokens, const float* uniforms, int n_branches, int gamma,
                      int vocab, int32_t* accepted_len, int32_t* next_token);

/*
 * Answer aggregation over the n branches of one question.  Host pointers, no GPU work.
 *   tts_majority_vote: winner = most frequent answer (weights == NULL, Section 3.2) or the answer
 *     with the largest weight sum ("vote" aggregation of Section 4.6); ties go to the answer whose
 *     first occurrence has the lowest branch index.  votes = branches that gave the winner.
 *   tts_confidence_max: answer of the single branch with the largest weight ("max" aggregation of
 *     Section 4.6; ties: lowest branch index); weights must not be NULL.
 */
TTS_API int tts_majority_vote(const int64_t* answers, const float* weights, int n, int64_t* winner,
                      int* votes);
TTS_API int tts_confidence_max(const int64_t* answers, const float* weights, int n, int64_t* winner,
                       int* votes);

/*
 * Search for the latency-optimal configuration (B, gamma) (Section 3.3, Algorithm 1; compared with
 * the exhaustive grid in Section 4.5).  Host only.  The configurations form a lattice: B = 1, 2, 4, ..
 * up to limits->max_branches, gamma = 0 .. limits->max_gamma.  tts_task(B, gamma, user) returns the
 * accuracy the caller reaches with that configuration inside its latency budget; a negative return
 * marks the point as unavailable.  limits == NULL means B <= 64, gamma <= 7 (the ranges of Section
 * 4.5) and at most 64 steps.
 *   tts_greedy_search: hill climbing from (1, 0).  Each step scores the two neighbours (2B, gamma) and
 *     (B, gamma+1) that lie inside the lattice, and moves to the better one if it beats the current
 *     point (equal neighbours: more branches); it stops at the first step that brings no improvement,
 *     or after limits->max_steps steps.  steps = steps taken including the last, unsuccessful one;
 *     evaluations = calls of tts_task.
 *   tts_grid_search: scores every lattice point, (log2 max_branches + 1) * (max_gamma + 1) calls, and
 *     returns the best (equal optima: the first in (B, gamma) order).
 * best_acc, steps and evaluations may be NULL.  TTS_ERR_INVALID for null callbacks or limits outside
 * 1 <= max_branches <= 2^20, 0 <= max_gamma <= 4096.
 */
typedef double (*tts_task_fn)(int n_branches, int gamma, void* user);
typedef struct {
    int32_t max_branches;   /* largest B tried (the lattice holds the powers of two up to it) */
    int32_t max_gamma;      /* largest draft length tried */
    int32_t max_steps;      /* greedy search: upper bound on steps; <= 0 means 64 */
} tts_search_limits;
TTS_API int tts_greedy_search(tts_task_fn tts_task, void* user, const tts_search_limits* limits,
                      int* best_branches, int* best_gamma, double* best_acc, int* steps, int* evaluations);
TTS_API int tts_grid_search(tts_task_fn tts_task, void* user, const tts_search_limits* limits,
                    int* best_branches, int* best_gamma, double* best_acc, int* evaluations);

/* Synchronises the stream and reads the device status word: TTS_OK, TTS_ERR_DEVICE_BOUNDS or
 * TTS_ERR_DEVICE_TIMEOUT, written to *device_status; clears it.  Host pointers. */
TTS_API int tts_last_status(tts_ctx* ctx, int* device_status);
/* cudaError_t of the last failed CUDA call seen by this context (0 if none). */
TTS_API int tts_last_cuda_error(tts_ctx* ctx);
/* Number of kernels this context has launched since creation (host counter). */
TTS_API int64_t tts_launch_count(tts_ctx* ctx);
/*
 * Profiling aid.  While enabled, every attention call records CUDA events on the context's stream
 * before its main kernel, between the main kernel and the merge kernel, and after the merge (at
 * most 4096 calls are kept).  tts_profile_read synchronises the stream, writes the mean duration
 * in microseconds of the main kernel and of the merge kernel over the recorded calls and their
 * number (host pointers), and forgets them.  Calls made while the stream is being captured into a
 * CUDA graph put the events into the graph: read after a replay, the durations are those of the
 * kernels inside that replay (without the gap that a stream launch adds between two events).
 */
TTS_API int tts_profile_enable(tts_ctx* ctx, int on);
TTS_API int tts_profile_read(tts_ctx* ctx, float* attn_main_us, float* attn_merge_us, int* n_calls);
/*
 * Diagnostics of the failure-detection path.  Every wait inside the tensor-core kernels (on a TMA copy,
 * on another warp role) is bounded: when its limit runs out the kernel raises TTS_ERR_DEVICE_TIMEOUT in
 * the device status word, lets go of what it holds and returns, so a lost signal never hangs the GPU.
 * tts_debug_wait_timeout runs a separate one-warp kernel on the context's stream that waits, through the
 * same routine, limit_ns nanoseconds (1 us .. 1 s) for a signal that is never sent.  Afterwards
 * tts_last_status reports TTS_ERR_DEVICE_TIMEOUT and the context works as before.
 */
TTS_API int tts_debug_wait_timeout(tts_ctx* ctx, int64_t limit_ns);
/* Static, NUL-terminated description of a tts_status. */
TTS_API const char* tts_strerror(int status);

/*
 * Accept test along the paths of a draft tree (tree verification with the tree drafts of the
 * speculative-decoding models used in Section 4.1; the paper does not spell the rule out, this is the
 * chain rule of tts_accept applied along every root-to-leaf path).  Per branch, n_nodes tree nodes:
 *   tree_parents device [n_branches][n_nodes] i32   parent of node i (an index < i), or -1 for a child
 *                                                   of the last committed token
 *   draft_tokens device [n_branches][n_nodes] i32   token x_i of node i
 *   p_target     device [n_branches][n_nodes+1][vocab] fp32   row 0: target distribution after the last
 *                                                   committed token; row 1 + i: after node i
 *   q_draft      device [n_branches][n_nodes][vocab] fp32     row i: the draft distribution x_i was drawn from
 *   uniforms     device [n_branches][n_nodes+1] fp32 in [0,1): u_i for node i, u_{n_nodes} for the final draw
 * Node i passes iff p(x_i) > 0 and u_i * q_i(x_i) <= p(x_i) (one fp32 multiply), p being row 0 if its
 * parent is -1 and row 1 + parent otherwise; a node is accepted iff it and all its ancestors pass.  The
 * leaf whose path holds the most accepted nodes wins (ties: lowest leaf index).
 *   accepted_len[b] = accepted nodes on the winning path;  last_node[b] = the deepest of them (-1: none);
 *   next_token[b]   = inverse-CDF draw with u_{n_nodes}, as in tts_accept, from norm(max(0, p - q_k)) for
 *                     the first node k of the winning path that failed (p: the row of k's parent), or from
 *                     row 1 + leaf when the whole path was accepted.
 * A chain (tree_parents[i] = i - 1) gives exactly tts_accept with gamma = n_nodes.  n_nodes <= 64;
 * vocab % 4 == 0.  Malformed parents or tokens raise TTS_ERR_DEVICE_BOUNDS and count as -1 / token 0.
 * The rule is not lossless across siblings (a sibling is not re-tested against the residual).
 */
TTS_API int tts_accept_tree(tts_ctx* ctx, const float* p_target, const float* q_draft, const int32_t* draft_tokens,
                            const int32_t* tree_parents, const float* uniforms, int n_branches, int n_nodes,
                            int vocab, int32_t* accepted_len, int32_t* last_node, int32_t* next_token);

/*
 * KV-cache bookkeeping either side of the verify step (Section 3.2, sequence-wise parallelism: the
 * target model scores the last committed token and the gamma drafts of every branch in one pass, so
 * their keys and values join the branch's cache before the attention, and the cache is cut back to
 * what was accepted afterwards).
 *   tts_kv_append: copies the keys and values of the `rows` newest positions of every branch into the
 *     paged pools, at private tokens branch_lens[b] - rows .. branch_lens[b] - 1 (branch_lens already
 *     counts them: these are the positions that tts_verify_attn treats as the causal tail).
 *       k_new, v_new device [n_branches][rows][n_kv_heads][128] bf16 (16-byte aligned), read only
 *       k_pages, v_pages, block_table, prefix_len, branch_lens as in tts_verify_attn; the pools are written.
 *     A branch shorter than `rows` or a page index outside [0, num_pages) writes nothing for that
 *     token and raises TTS_ERR_DEVICE_BOUNDS in the device status (tts_last_status).
 *   tts_kv_rollback: branch_lens[b] -= gamma - accepted_len[b] (device arrays, i32): the rejected drafts
 *     leave the cache; the pages stay with the branch.  accepted_len outside [0, gamma] changes nothing
 *     for that branch and raises TTS_ERR_DEVICE_BOUNDS.
 * Both are asynchronous on the context's stream; TTS_ERR_INVALID for null or misaligned pointers and
 * sizes outside the context's limits.
 */
TTS_API int tts_kv_append(tts_ctx* ctx, const void* k_new, const void* v_new, void* k_pages, void* v_pages,
                          const int32_t* block_table, int prefix_len, const int32_t* branch_lens,
                          int n_branches, int rows);
TTS_API int tts_kv_rollback(tts_ctx* ctx, int32_t* branch_lens, const int32_t* accepted_len, int n_branches,
                            int gamma);

/*
 * One whole verify step from HOST buffers (the end-to-end path): for each of n_layers layers,
 * copies that layer's q from pinned host memory, runs tts_verify_attn against that layer's
 * device-resident K/V pools (the KV cache is state that lives in HBM, like the weights) and
 * copies out back; then copies the probabilities, tokens and uniforms, runs tts_accept and
 * copies the two result arrays back.  Synchronises before returning.
 *   q_host, out_host   host  [n_layers][n_branches][gamma+1][Hq][128] bf16
 *   k_pools, v_pools   host arrays of n_layers DEVICE pointers
 *   block_table_host, branch_lens_host, p_target_host, q_draft_host, draft_tokens_host,
 *   uniforms_host, accepted_len_host, next_token_host: host copies in the device layouts above.
 * Staging buffers on the device are allocated inside the context on first use, and so are two
 * streams of its own on which the copies that need not wait for the kernels run beside them (the
 * queries of later layers and the accept inputs while the first layers run, the outputs of finished
 * layers while later ones run); the kernels run on the context's stream.  With pageable host memory
 * the copies do not overlap anything.  When p_target_host and q_draft_host are pinned memory that the
 * device can address (cudaHostAlloc / cudaHostRegister), they are not copied at all: the accept kernel
 * reads what it needs of them (its 2 gamma gathers and one row pair per branch) directly from the host.
 */
TTS_API int tts_verify_step_host(tts_ctx* ctx, int n_layers, const void* q_host, const void* const* k_pools,
                         const void* const* v_pools, const int32_t* block_table_host,
                         int prefix_len, const int32_t* branch_lens_host, int n_branches, int gamma,
                         const float* p_target_host, const float* q_draft_host,
                         const int32_t* draft_tokens_host, const float* uniforms_host, int vocab,
                         void* out_host, int32_t* accepted_len_host, int32_t* next_token_host);

/*
 * tts_verify_step_host with the accept pass fed with logits (tts_accept_logits): target_logits_host
 * [n_branches][gamma+1][vocab] and draft_logits_host [n_branches][gamma][vocab] in logits_dtype take the
 * place of the two probability tensors (half the bytes over the host link when they are bf16).
 */
TTS_API int tts_verify_step_host_logits(tts_ctx* ctx, int n_layers, const void* q_host, const void* const* k_pools,
                         const void* const* v_pools, const int32_t* block_table_host,
                         int prefix_len, const int32_t* branch_lens_host, int n_branches, int gamma,
                         const void* target_logits_host, const void* draft_logits_host, int logits_dtype,
                         const int32_t* draft_tokens_host, const float* uniforms_host, int vocab,
                         void* out_host, int32_t* accepted_len_host, int32_t* next_token_host);

#ifdef __cplusplus
}
#endif
#endif /* TTS_H_ */
