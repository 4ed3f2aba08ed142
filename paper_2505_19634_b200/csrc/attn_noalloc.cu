// tts_verify_attn_noalloc: verify-step attention for callers that must not allocate device memory.
//
// The regular entry point keeps its split-KV partial results in a workspace that tts_create obtains
// with cudaMalloc.  Some hosts of this library cannot do that: a serving process that has handed
// all device memory to its own pool allocator at start-up, a plugin running inside a framework that
// forbids driver allocations once its memory plan is frozen, or code between two points where an
// allocation would synchronise the device.  For them the same computation is offered with the
// scratch in a fixed array that is part of the library image: every GPU that loads the library
// holds kScratchBytes of it until the process exits, and a problem that needs more is refused.
//
// The CUDA-core attention kernel and the merge kernel run exactly as in the regular path; only the
// place their partial results go to differs.
#include <mutex>

#include <string.h>

#include "tts_internal.cuh"

namespace tts {

namespace {

constexpr size_t kScratchBytes = 8u << 20;               // partial results of one call
constexpr size_t kRowBytes = kHeadDim * sizeof(float) + sizeof(float2);   // one partial row: O, (m, l)
constexpr int kNoAllocGrid = 128;                        // CTAs of the main kernel (sets the number of pieces)
constexpr int kMaxDevices = 64;

// [status word, padded to 256 bytes][partial results].  File scope: in host code this name only
// stands for the symbol; the device address comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_scratch[256 + kScratchBytes];

std::mutex g_mu;
unsigned char* g_scratch_addr[kMaxDevices] = {};         // device address of g_scratch, per device

// First call on a device: resolves the array's address there (the device must be current).
cudaError_t scratch_of_current_device(unsigned char** addr, int* dev_out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_scratch);
        if (e != cudaSuccess) return e;
        if (!ptr) return cudaErrorInvalidSymbol;
        g_scratch_addr[dev] = static_cast<unsigned char*>(ptr);
    }
    *addr = g_scratch_addr[dev];
    *dev_out = dev;
    return cudaSuccess;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

}  // namespace tts

using namespace tts;

extern "C" int tts_verify_attn_noalloc(const void* q, const void* k_pages, const void* v_pages,
                                       const int32_t* block_table, int max_blocks_per_branch, int prefix_len,
                                       const int32_t* branch_lens, int n_branches, int gamma, int n_q_heads,
                                       int n_kv_heads, void* out, void* cuda_stream) {
    if (!q || !k_pages || !v_pages || !block_table || !branch_lens || !out) return TTS_ERR_INVALID;
    if (n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads != 0) return TTS_ERR_INVALID;
    if (n_branches < 1 || n_branches > kMaxBranches || gamma < 0 || gamma + 1 > kMaxTreeRows) return TTS_ERR_INVALID;
    if (prefix_len < 0 || prefix_len % kPage != 0 || max_blocks_per_branch < 1 ||
        prefix_len / kPage > max_blocks_per_branch)
        return TTS_ERR_INVALID;
    if (!aligned16(q) || !aligned16(k_pages) || !aligned16(v_pages) || !aligned16(out)) return TTS_ERR_INVALID;

    const int R = gamma + 1, G = n_q_heads / n_kv_heads, nr = R * G;
    const int rb = simt_rb_rows(nr);
    const long n_rb_pre = ((long)n_branches * nr + rb - 1) / rb, n_rb_priv = (nr + rb - 1) / rb;
    const long pre_stride = (long)n_branches * nr < rb ? (long)n_branches * nr : rb;
    const long priv_stride = nr < rb ? nr : rb;
    const size_t pre_rows = (size_t)(n_kv_heads * n_rb_pre + kNoAllocGrid) * pre_stride;
    const size_t priv_rows = (size_t)((long)n_branches * n_kv_heads * n_rb_priv + kNoAllocGrid) * priv_stride;
    if ((pre_rows + priv_rows) * kRowBytes > kScratchBytes) return TTS_ERR_SCRATCH;   // beyond the fixed array

    unsigned char* base = nullptr;
    int dev = 0;
    if (scratch_of_current_device(&base, &dev) != cudaSuccess) return TTS_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

    AttnParams p;
    memset(&p, 0, sizeof p);
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k_pages = static_cast<const __nv_bfloat16*>(k_pages);
    p.v_pages = static_cast<const __nv_bfloat16*>(v_pages);
    p.block_table = block_table; p.branch_lens = branch_lens; p.tree_parents = nullptr;
    p.out = out;
    p.status = reinterpret_cast<int32_t*>(base);
    unsigned char* cur = base + 256;                        // O rows are 512 bytes, (m, l) rows 8: all stay aligned
    p.part_o_pre = reinterpret_cast<float*>(cur);   cur += pre_rows * kHeadDim * sizeof(float);
    p.part_o_priv = reinterpret_cast<float*>(cur);  cur += priv_rows * kHeadDim * sizeof(float);
    p.part_ml_pre = reinterpret_cast<float2*>(cur); cur += pre_rows * sizeof(float2);
    p.part_ml_priv = reinterpret_cast<float2*>(cur);
    p.N = n_branches; p.R = R; p.Hq = n_q_heads; p.Hkv = n_kv_heads; p.G = G; p.nr = nr;
    p.P = prefix_len; p.max_blocks = max_blocks_per_branch; p.num_pages = 0;
    p.rb_rows = rb;
    p.pre_stride = (int)pre_stride; p.priv_stride = (int)priv_stride;
    p.copies = 1; p.copies_pre = 1;
    p.n_rb_pre = (int)n_rb_pre; p.n_rb_priv = (int)n_rb_priv;
    p.n_pre = prefix_len > 0 ? n_kv_heads * p.n_rb_pre : 0;
    if ((long long)n_branches * n_kv_heads * p.n_pre >= (1ll << 31)) return TTS_ERR_UNSUPPORTED;
    p.tile_tokens = kSimtTileTokens;
    p.tiles_pre = ceil_div(prefix_len, kSimtTileTokens);
    p.grid = kNoAllocGrid;
    p.out_dtype = TTS_OUT_BF16; p.debug = 0;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)kHeadDim);

    // The array keeps what the previous call left.  The partial results need no clearing (the merge
    // only reads pieces this call's main kernel writes); the status word must start at zero.
    if (cudaMemsetAsync(p.status, 0, sizeof(int32_t), st) != cudaSuccess) return TTS_ERR_CUDA;
    if (launch_attn_simt(p, st) != cudaSuccess) return TTS_ERR_CUDA;
    if (launch_attn_combine(p, st) != cudaSuccess) return TTS_ERR_CUDA;
    return TTS_OK;
}
