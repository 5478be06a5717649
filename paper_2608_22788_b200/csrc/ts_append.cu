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

// Rotary embedding of the step's Q and K rows fused with the append.  One CTA per (sequence, new token):
// the D/2 (cos, sin) pairs of the token's position are computed once into shared memory and reused by
// every query and kv head; each thread then rotates 8 low-half and the 8 matching high-half dims at a time.
//
// The angle pos * inv_freq[d] reaches 1e5 rad at the longest contexts, where a float product is already
// off by several 1e-3 rad: it is formed in double (exact: 17-bit position x 24-bit significand), reduced
// by the nearest multiple of 2 pi there, and only the reduced angle goes through the float sincos.
__global__ void __launch_bounds__(128)
ts_rope_kv_append_kernel(const uint16_t *q_in, uint16_t *q_out, const uint16_t *__restrict__ new_k,
                         const uint4 *__restrict__ new_v, uint16_t *k_pool, uint16_t *v_pool,
                         const int32_t *__restrict__ block_table, const int32_t *__restrict__ kv_lens,
                         const float *__restrict__ inv_freq, int q_len, int Hq, int Hkv, int D, int P, int max_pages,
                         long long page_stride, long long token_stride, long long head_stride)
{
    __shared__ float cs[128], sn[128];                           // D/2 <= 128
    const int s = blockIdx.x / q_len, t = blockIdx.x % q_len;
    const long long pos = (long long)kv_lens[s] - q_len + t;     // kv_lens already counts the new tokens
    if (pos < 0) return;                                         // fewer keys than new tokens: nothing to place
    const int half = D / 2;
    for (int d = threadIdx.x; d < half; d += blockDim.x) {
        const double angle = (double)pos * (double)inv_freq[d];
        const double k = rint(angle * 0.15915494309189535);      // 1 / (2 pi)
        const double r = fma(-k, 1.2246467991473532e-16 * 2.0, fma(-k, 6.283185307179586, angle));
        float c, sv;
        sincosf((float)r, &sv, &c);
        cs[d] = c;
        sn[d] = sv;
    }
    __syncthreads();

    const int page = block_table[(long long)s * max_pages + pos / P];
    const long long kv_base = (long long)page * page_stride + (pos % P) * token_stride;
    const int vec_half = half / 8;                               // 16-byte vectors per half row
    const int q_items = Hq * vec_half, k_items = Hkv * vec_half, v_items = Hkv * (D / 8);
    const long long row = blockIdx.x;
    for (int i = threadIdx.x; i < q_items + k_items + v_items; i += blockDim.x) {
        if (i >= q_items + k_items) {                            // V: plain copy
            const int j = i - q_items - k_items;
            const int g = j / (D / 8), c = j % (D / 8);
            *reinterpret_cast<uint4 *>(v_pool + kv_base + (long long)g * head_stride + c * 8) =
                new_v[row * v_items + j];
            continue;
        }
        const bool is_k = i >= q_items;
        const int j = is_k ? i - q_items : i;
        const int h = j / vec_half, c = j % vec_half;
        const uint16_t *src = (is_k ? new_k + (row * Hkv + h) * D : q_in + (row * Hq + h) * D) + c * 8;
        uint16_t *dst = (is_k ? k_pool + kv_base + (long long)h * head_stride : q_out + (row * Hq + h) * D) + c * 8;
        const uint4 lo = *reinterpret_cast<const uint4 *>(src);
        const uint4 hi = *reinterpret_cast<const uint4 *>(src + half);
        const uint32_t lw[4] = {lo.x, lo.y, lo.z, lo.w}, hw[4] = {hi.x, hi.y, hi.z, hi.w};
        uint32_t ol[4], oh[4];
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            float rl[2], rh[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const float a = __uint_as_float(e ? (lw[w] & 0xffff0000u) : (lw[w] << 16));
                const float b = __uint_as_float(e ? (hw[w] & 0xffff0000u) : (hw[w] << 16));
                const float cc = cs[c * 8 + 2 * w + e], ss = sn[c * 8 + 2 * w + e];
                rl[e] = fmaf(a, cc, -b * ss);
                rh[e] = fmaf(b, cc, a * ss);
            }
            asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(ol[w]) : "f"(rl[1]), "f"(rl[0]));
            asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(oh[w]) : "f"(rh[1]), "f"(rh[0]));
        }
        *reinterpret_cast<uint4 *>(dst) = make_uint4(ol[0], ol[1], ol[2], ol[3]);
        *reinterpret_cast<uint4 *>(dst + half) = make_uint4(oh[0], oh[1], oh[2], oh[3]);
    }
}

}  // namespace ts

extern "C" int ts_rope_kv_append(const ts_attn_params *p, const void *q_in, void *q_out, const void *new_k,
                                 const void *new_v, void *k_pool, void *v_pool, const int32_t *block_table,
                                 const int32_t *kv_lens, const float *inv_freq, void *stream)
{
    if (!p || !q_in || !q_out || !new_k || !new_v || !k_pool || !v_pool || !block_table || !kv_lens || !inv_freq)
        return TS_ERR_INVALID_ARG;
    if (p->num_seqs < 0 || p->q_len < 1 || p->num_kv_heads < 1 || p->num_q_heads < 1 || p->page_size < 1 ||
        p->max_pages_per_seq < 1)
        return TS_ERR_INVALID_ARG;
    if (p->head_dim < 16 || p->head_dim % 16 || p->head_dim > 256) return TS_ERR_UNSUPPORTED;
    if (p->kv_page_stride <= 0 || p->kv_token_stride <= 0 || p->kv_head_stride <= 0) return TS_ERR_INVALID_ARG;
    if (p->kv_page_stride % 8 || p->kv_token_stride % 8 || p->kv_head_stride % 8) return TS_ERR_INVALID_ARG;
    const uintptr_t bits = reinterpret_cast<uintptr_t>(q_in) | reinterpret_cast<uintptr_t>(q_out) |
                           reinterpret_cast<uintptr_t>(new_k) | reinterpret_cast<uintptr_t>(new_v) |
                           reinterpret_cast<uintptr_t>(k_pool) | reinterpret_cast<uintptr_t>(v_pool);
    if (bits & 15u) return TS_ERR_INVALID_ARG;
    const long long rows = (long long)p->num_seqs * p->q_len;
    if (rows == 0) return TS_OK;
    if (rows > 0x7fffffffLL) return TS_ERR_UNSUPPORTED;
    ts::ts_rope_kv_append_kernel<<<(unsigned)rows, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint16_t *>(q_in), static_cast<uint16_t *>(q_out), static_cast<const uint16_t *>(new_k),
        static_cast<const uint4 *>(new_v), static_cast<uint16_t *>(k_pool), static_cast<uint16_t *>(v_pool), block_table,
        kv_lens, inv_freq, p->q_len, p->num_q_heads, p->num_kv_heads, p->head_dim, p->page_size, p->max_pages_per_seq,
        p->kv_page_stride, p->kv_token_stride, p->kv_head_stride);
    return cudaGetLastError() == cudaSuccess ? TS_OK : TS_ERR_CUDA;
}

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
