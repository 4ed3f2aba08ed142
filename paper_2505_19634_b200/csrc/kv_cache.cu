// KV-cache bookkeeping either side of the verify step: the keys and values of the newest positions
// of every branch go into the paged pools before the attention; after the accept test the branch
// lengths are cut back to what was accepted.  Pure data movement: one thread per 16 bytes.
#include "tts_internal.cuh"

namespace tts {

namespace {

// grid-stride over (K or V, branch, row, KV head, 16-byte chunk)
__global__ void kv_append_kernel(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new, uint4* k_pages,
                                 uint4* v_pages, const int32_t* __restrict__ block_table, int max_blocks, int num_pages,
                                 int prefix_len, const int32_t* __restrict__ branch_lens, int N, int R, int Hkv,
                                 int32_t* status) {
    constexpr int kChunks = kHeadDim * 2 / 16;                        // 16 chunks per token-head
    const long total = 2l * N * R * Hkv * kChunks;
    for (long w = blockIdx.x * (long)blockDim.x + threadIdx.x; w < total; w += (long)gridDim.x * blockDim.x) {
        const int c = (int)(w % kChunks);
        long rest = w / kChunks;
        const int h = (int)(rest % Hkv); rest /= Hkv;
        const int i = (int)(rest % R); rest /= R;
        const int b = (int)(rest % N);
        const bool is_v = rest / N != 0;
        const int L = branch_lens[b];
        if (L < R) { atomicMin(status, (int)TTS_ERR_DEVICE_BOUNDS); continue; }
        const int tok = prefix_len + L - R + i;                       // logical token of the branch
        if (tok / kPage >= max_blocks) { atomicMin(status, (int)TTS_ERR_DEVICE_BOUNDS); continue; }
        const int page = block_table[(size_t)b * max_blocks + tok / kPage];
        if (page < 0 || page >= num_pages) { atomicMin(status, (int)TTS_ERR_DEVICE_BOUNDS); continue; }
        const size_t src = (((size_t)b * R + i) * Hkv + h) * kChunks + c;
        const size_t dst = (((size_t)page * Hkv + h) * kPage + tok % kPage) * kChunks + c;
        if (is_v) v_pages[dst] = v_new[src]; else k_pages[dst] = k_new[src];
    }
}

__global__ void kv_rollback_kernel(int32_t* branch_lens, const int32_t* __restrict__ accepted_len, int N, int gamma,
                                   int32_t* status) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= N) return;
    const int a = accepted_len[b];
    if (a < 0 || a > gamma) { atomicMin(status, (int)TTS_ERR_DEVICE_BOUNDS); return; }
    branch_lens[b] -= gamma - a;
}

}  // namespace

cudaError_t launch_kv_append(const void* k_new, const void* v_new, void* k_pages, void* v_pages,
                             const int32_t* block_table, int max_blocks, int num_pages, int prefix_len,
                             const int32_t* branch_lens, int N, int R, int Hkv, int32_t* status, cudaStream_t st) {
    const long total = 2l * N * R * Hkv * (kHeadDim * 2 / 16);
    const int threads = 256;
    const int blocks = (int)((total + threads - 1) / threads < 4096 ? (total + threads - 1) / threads : 4096);
    kv_append_kernel<<<blocks, threads, 0, st>>>(static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new),
                                                 static_cast<uint4*>(k_pages), static_cast<uint4*>(v_pages), block_table,
                                                 max_blocks, num_pages, prefix_len, branch_lens, N, R, Hkv, status);
    return cudaGetLastError();
}

cudaError_t launch_kv_rollback(int32_t* branch_lens, const int32_t* accepted_len, int N, int gamma, int32_t* status,
                               cudaStream_t st) {
    kv_rollback_kernel<<<(N + 127) / 128, 128, 0, st>>>(branch_lens, accepted_len, N, gamma, status);
    return cudaGetLastError();
}

}  // namespace tts
