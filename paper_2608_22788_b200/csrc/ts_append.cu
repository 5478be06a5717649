// Append the K/V rows of the tokens scored in this step to the paged cache (runs before attention).
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/tailsieve.h"

namespace ts {

// One CTA per (sequence, new token); threads copy 16-byte vectors of all kv heads of K and V.
__global__ void __launch_bounds__(256)
ts_kv_append_kernel(const uint4 *__restrict__ new_k, const uint4 *__restrict__ new_v, uint16_t *k_pool, uint16_t *v_pool,
                    const int32_t *__restrict__ block_table, const int32_t *__restrict__ kv_lens, int q_len, int Hkv,
                    int D, int P, int max_pages, long long page_stride, long long token_stride, long long head_stride)
{
    const int s = blockIdx.x / q_len, t = blockIdx.x % q_len;
    const long long pos = (long long)kv_lens[s] - q_len + t;     // kv_lens already counts the new tokens
    if (pos < 0) return;                                         // fewer keys than new tokens: nothing to place
    const int page = block_table[(long long)s * max_pages + pos / P];
    const long long base = (long long)page * page_stride + (pos % P) * token_stride;
    const int vec_per_head = D / 8;
    const int nvec = Hkv * vec_per_head;
    const uint4 *src_k = new_k + (long long)blockIdx.x * nvec;
    const uint4 *src_v = new_v + (long long)blockIdx.x * nvec;
    for (int i = threadIdx.x; i < 2 * nvec; i += blockDim.x) {
        const bool is_v = i >= nvec;
        const int j = is_v ? i - nvec : i;
        const int g = j / vec_per_head, c = j % vec_per_head;
        uint16_t *dst = (is_v ? v_pool : k_pool) + base + (long long)g * head_stride + c * 8;
        *reinterpret_cast<uint4 *>(dst) = is_v ? src_v[j] : src_k[j];
    }
}

}  // namespace ts

extern "C" int ts_kv_append(const ts_attn_params *p, const void *new_k, const void *new_v, void *k_pool, void *v_pool,
                            const int32_t *block_table, const int32_t *kv_lens, void *stream)
{
    if (!p || !new_k || !new_v || !k_pool || !v_pool || !block_table || !kv_lens) return TS_ERR_INVALID_ARG;
    if (p->num_seqs < 0 || p->q_len < 1 || p->num_kv_heads < 1 || p->page_size < 1 || p->max_pages_per_seq < 1)
        return TS_ERR_INVALID_ARG;
    if (p->head_dim < 8 || p->head_dim % 8) return TS_ERR_UNSUPPORTED;
    if (p->kv_page_stride <= 0 || p->kv_token_stride <= 0 || p->kv_head_stride <= 0) return TS_ERR_INVALID_ARG;
    if (p->kv_page_stride % 8 || p->kv_token_stride % 8 || p->kv_head_stride % 8) return TS_ERR_INVALID_ARG;
    const uintptr_t bits = reinterpret_cast<uintptr_t>(new_k) | reinterpret_cast<uintptr_t>(new_v) |
                           reinterpret_cast<uintptr_t>(k_pool) | reinterpret_cast<uintptr_t>(v_pool);
    if (bits & 15u) return TS_ERR_INVALID_ARG;
    const long long rows = (long long)p->num_seqs * p->q_len;
    if (rows == 0) return TS_OK;
    if (rows > 0x7fffffffLL) return TS_ERR_UNSUPPORTED;
    ts::ts_kv_append_kernel<<<(unsigned)rows, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4 *>(new_k), static_cast<const uint4 *>(new_v), static_cast<uint16_t *>(k_pool),
        static_cast<uint16_t *>(v_pool), block_table, kv_lens, p->q_len, p->num_kv_heads, p->head_dim, p->page_size,
        p->max_pages_per_seq, p->kv_page_stride, p->kv_token_stride, p->kv_head_stride);
    return cudaGetLastError() == cudaSuccess ? TS_OK : TS_ERR_CUDA;
}
