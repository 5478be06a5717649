// Greedy draft acceptance for sm_100a: a streaming per-row argmax over the vocabulary (HBM-bound,
// compare-only) followed by the longest-accepted-prefix rule.
//
// Kernel 1 cuts every logits row into `chunks` pieces so that even a handful of rows fills the
// GPU; each CTA reduces its piece to one 64-bit key = (order-preserving image of the bf16 value,
// ~index), whose maximum is "largest value, lowest index".  Kernel 2 (one CTA) reduces the keys of
// each row and applies the prefix rule.  No atomics: results are bit-reproducible.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <stdlib.h>

#include <mutex>

#include "../../include/tailsieve.h"
#include "ts_common.cuh"

namespace ts {

constexpr int kArgmaxThreads = 256;
constexpr int kMaxChunks = 64;

// Order-preserving map of a bf16 bit pattern to an unsigned key: larger value <-> larger key,
// -0 and +0 share a key, every NaN maps to 0 (below -inf), so NaN never wins.
__device__ __forceinline__ uint32_t bf16_key(uint32_t u)
{
    u &= 0xffffu;
    if ((u & 0x7fffu) > 0x7f80u) return 0u;          // NaN
    if (u == 0x8000u) u = 0u;                          // -0 -> +0
    const uint32_t ord = (u & 0x8000u) ? (~u & 0xffffu) : (u | 0x8000u);
    return ord + 1u;
}

__device__ __forceinline__ unsigned long long key_max(unsigned long long a, unsigned long long b)
{
    return a > b ? a : b;
}

__device__ __forceinline__ uint4 ld_stream_16B(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ void scan8(const uint4 &v, int idx0, uint32_t &best, int &best_idx)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t k0 = bf16_key(w[i]), k1 = bf16_key(w[i] >> 16);
        if (k0 > best) { best = k0; best_idx = idx0 + 2 * i; }
        if (k1 > best) { best = k1; best_idx = idx0 + 2 * i + 1; }
    }
}

// grid = (chunks, rows).  keys[row * chunks + chunk] = best key of the chunk.
__global__ void __launch_bounds__(kArgmaxThreads)
ts_argmax_chunk_kernel(const uint16_t *__restrict__ logits, long long row_stride, int vocab, int chunk_len,
                       unsigned long long *__restrict__ keys)
{
    grid_dependency_wait();
    const int chunk = blockIdx.x, row = blockIdx.y, chunks = gridDim.x;
    const uint16_t *base = logits + (long long)row * row_stride;
    const int begin = chunk * chunk_len;
    int end = begin + chunk_len;
    if (end > vocab) end = vocab;
    uint32_t best = 0u;
    int best_idx = begin < vocab ? begin : 0;
    // scalar head up to the first 16-byte boundary, 16-byte vectors, scalar tail; every thread
    // visits its elements in ascending index order, so "strictly greater" keeps the lowest index
    int head = 0, nvec = 0;
    if (end > begin) {
        const long long off = (long long)row * row_stride + begin;
        head = (int)((8 - (off & 7)) & 7);
        if (head > end - begin) head = end - begin;
        nvec = (end - begin - head) / 8;
    }
    for (int i = begin + threadIdx.x; i < begin + head; i += kArgmaxThreads) {
        const uint32_t k = bf16_key(base[i]);
        if (k > best) { best = k; best_idx = i; }
    }
    const int vbeg = begin + head;
    constexpr int UNROLL = 4;
    int v = threadIdx.x;
    for (; v + (UNROLL - 1) * kArgmaxThreads < nvec; v += UNROLL * kArgmaxThreads) {
        uint4 x[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) x[u] = ld_stream_16B(base + vbeg + (long long)(v + u * kArgmaxThreads) * 8);
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) scan8(x[u], vbeg + (v + u * kArgmaxThreads) * 8, best, best_idx);
    }
    for (; v < nvec; v += kArgmaxThreads) {
        const uint4 x = ld_stream_16B(base + vbeg + (long long)v * 8);
        scan8(x, vbeg + v * 8, best, best_idx);
    }
    for (int i = vbeg + nvec * 8 + threadIdx.x; i < end; i += kArgmaxThreads) {
        const uint32_t k = bf16_key(base[i]);
        if (k > best) { best = k; best_idx = i; }
    }
    unsigned long long key = ((unsigned long long)best << 32) | (unsigned long long)(0xffffffffu - (uint32_t)best_idx);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) key = key_max(key, __shfl_xor_sync(0xffffffffu, key, o));
    __shared__ unsigned long long wk[kArgmaxThreads / 32];
    if ((threadIdx.x & 31) == 0) wk[threadIdx.x >> 5] = key;
    __syncthreads();
    if (threadIdx.x < 32) {
        key = threadIdx.x < kArgmaxThreads / 32 ? wk[threadIdx.x] : 0ull;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) key = key_max(key, __shfl_xor_sync(0xffffffffu, key, o));
        if (threadIdx.x == 0) keys[(long long)row * chunks + chunk] = key;
    }
}

// Fast path (every row 16-byte aligned, vocab a multiple of 8): a CTA keeps its whole chunk in
// registers -- up to kVecPerThread 16-byte vectors per thread, all loads issued before the first
// use -- finds the chunk maximum with packed bf16x2 max instructions, then the first position equal
// to it with packed compares.  About 13 instructions per 16 bytes instead of ~80 for the generic
// key-per-element scan, which keeps the kernel bandwidth-bound.
// Eight vectors per thread: 52 registers, four CTAs per SM.  Sixteen (a 32768-element chunk, 79 registers,
// three CTAs per SM) measured 2 us slower per call at 144 and 272 rows, four to twelve the same as eight
// or slower: with more, shorter-lived CTAs on an SM their load and reduce phases interleave better.
constexpr int kVecPerThread = 8;
constexpr int kFastChunk = kArgmaxThreads * kVecPerThread * 8;      // elements per chunk (16384)

__global__ void __launch_bounds__(kArgmaxThreads)
ts_argmax_reg_kernel(const uint16_t *__restrict__ logits, long long row_stride, int vocab, int chunk_len,
                     unsigned long long *__restrict__ keys)
{
    grid_dependency_wait();
    const int chunk = blockIdx.x, row = blockIdx.y, chunks = gridDim.x;
    const int begin = chunk * chunk_len;
    int end = begin + chunk_len;
    if (end > vocab) end = vocab;
    const int nvec = end > begin ? (end - begin) >> 3 : 0;
    const uint4 *base = reinterpret_cast<const uint4 *>(logits + (long long)row * row_stride + begin);
    const uint32_t neg_inf2 = 0xff80ff80u;
    const uint32_t nan2 = 0x7fc07fc0u;       // filler past the chunk's end: NaN never wins and equals nothing
    uint4 v[kVecPerThread];
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u) {
        const int j = threadIdx.x + u * kArgmaxThreads;
        v[u] = j < nvec ? ld_stream_16B(base + j) : make_uint4(nan2, nan2, nan2, nan2);
    }
    // pass 1: maximum (NaN never wins: max returns the other operand)
    __nv_bfloat162 m2 = *reinterpret_cast<const __nv_bfloat162 *>(&neg_inf2);
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u) {
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162 *>(&v[u].x));
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162 *>(&v[u].y));
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162 *>(&v[u].z));
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162 *>(&v[u].w));
    }
    float m = fmaxf(__low2float(m2), __high2float(m2));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    __shared__ float s_m[kArgmaxThreads / 32];
    __shared__ int s_i[kArgmaxThreads / 32];
    if ((threadIdx.x & 31) == 0) s_m[threadIdx.x >> 5] = m;
    __syncthreads();
    m = s_m[0];
#pragma unroll
    for (int w = 1; w < kArgmaxThreads / 32; ++w) m = fmaxf(m, s_m[w]);
    // pass 2: first position whose value equals the maximum (+0 == -0; NaN equals nothing)
    const __nv_bfloat162 bm2 = __float2bfloat162_rn(m);
    int idx = 0x7fffffff;
#pragma unroll
    for (int u = kVecPerThread - 1; u >= 0; --u) {
        const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
        uint32_t e[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) e[i] = __heq2_mask(*reinterpret_cast<const __nv_bfloat162 *>(&w[i]), bm2);
        if (e[0] | e[1] | e[2] | e[3]) {
            int pos = 0;
            if (e[0]) pos = (e[0] & 0xffffu) ? 0 : 1;
            else if (e[1]) pos = (e[1] & 0xffffu) ? 2 : 3;
            else if (e[2]) pos = (e[2] & 0xffffu) ? 4 : 5;
            else pos = (e[3] & 0xffffu) ? 6 : 7;
            idx = begin + (threadIdx.x + u * kArgmaxThreads) * 8 + pos;      // descending u: the lowest survives
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) idx = min(idx, __shfl_xor_sync(0xffffffffu, idx, o));
    if ((threadIdx.x & 31) == 0) s_i[threadIdx.x >> 5] = idx;
    __syncthreads();
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 1; w < kArgmaxThreads / 32; ++w) idx = min(idx, s_i[w]);
        idx = min(idx, s_i[0]);
        unsigned long long key;
        if (idx == 0x7fffffff) {         // empty chunk, or nothing but NaN: lowest key, first index of the chunk
            key = (unsigned long long)(0xffffffffu - (uint32_t)(begin < vocab ? begin : 0));
        } else {
            const uint32_t bits = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(m));
            key = ((unsigned long long)bf16_key(bits) << 32) | (unsigned long long)(0xffffffffu - (uint32_t)idx);
        }
        keys[(long long)row * chunks + chunk] = key;
    }
}

// One CTA: reduce chunk keys per row, then accept the longest matching draft prefix per sequence.
__global__ void __launch_bounds__(256)
ts_accept_finish_kernel(const unsigned long long *__restrict__ keys, int chunks, const int32_t *__restrict__ draft,
                        int B, int gamma, int32_t *target_argmax, int32_t *accept_len, int32_t *out_tokens)
{
    const int R = gamma + 1;
    // lane groups of the acceptance step below; a thread's first draft token does not come from the kernel
    // before, so it is fetched ahead of the wait for it
    const int lane = threadIdx.x & 31;
    int g = 1;
    while (g < R && g < 32) g <<= 1;
    const int per_warp = 32 / g, sub = lane / g, li = lane % g;
    const int b_first = (threadIdx.x >> 5) * per_warp + sub;
    int32_t d_first = -1;
    if (b_first < B && li < gamma) d_first = draft[(long long)b_first * gamma + li];
    grid_dependency_wait();       // the chunk keys of the kernel before
    for (int r = threadIdx.x; r < B * R; r += blockDim.x) {
        unsigned long long key = 0ull;
        for (int c = 0; c < chunks; ++c) key = key_max(key, keys[(long long)r * chunks + c]);
        target_argmax[r] = (int32_t)(0xffffffffu - (uint32_t)(key & 0xffffffffull));
    }
    __syncthreads();
    // A group of g lanes per sequence (g = the power of two that covers the gamma + 1 positions, at most
    // 32), one lane per position: the draft and target tokens arrive with one round of loads and the first
    // mismatch falls out of a ballot (a thread walking the block position by position paid one memory
    // round trip per accepted token).
    const int nslots = (blockDim.x >> 5) * per_warp;
    const unsigned gmask = g == 32 ? 0xffffffffu : ((1u << g) - 1u);
    for (int b0 = (threadIdx.x >> 5) * per_warp; b0 < B; b0 += nslots) {      // warp-uniform trip count
        const int b = b0 + sub;
        const bool live = b < B;
        const int32_t *d = draft + (long long)(live ? b : 0) * gamma;
        const int32_t *t = target_argmax + (long long)(live ? b : 0) * R;
        int a = gamma;
        bool found = false;
        for (int i0 = 0; i0 < gamma; i0 += g) {                                // g < 32 only when gamma < g: one pass
            const int i = i0 + li;
            const bool have = i0 == 0 && b == b_first;                          // fetched before the wait
            const bool miss = live && !found && i < gamma && (have ? d_first : d[i]) != t[i];
            const unsigned m = (__ballot_sync(0xffffffffu, miss) >> (sub * g)) & gmask;
            if (m && !found) { a = i0 + __ffs(m) - 1; found = true; }
        }
        if (live && li == 0) accept_len[b] = a;
        for (int i0 = 0; i0 < R; i0 += g) {
            const int i = i0 + li;
            if (!live || i >= R) continue;
            int32_t tok = -1;
            if (i < a) tok = d[i];
            else if (i == a) tok = t[i];
            out_tokens[(long long)b * R + i] = tok;
        }
    }
}

static int pick_chunks(long long rows, int vocab)
{
    if (rows <= 0) return 1;
    // about two CTAs per SM on a 148-SM part: every CTA pays a fixed reduction and launch cost, and more,
    // smaller chunks measured slower (80 rows: 13.3 us with 5 chunks per row, 17.4 us with 15)
    long long c = (296 + rows - 1) / rows;
    const long long by_len = (vocab + 4095) / 4096;   // keep at least ~4096 elements per chunk
    if (c > by_len) c = by_len;
    if (c > kMaxChunks) c = kMaxChunks;
    if (c < 1) c = 1;
    return (int)c;
}

// Launch the chunk kernel (fast register path when the layout allows it) and the finishing kernel.
static int launch_accept(const void *logits, long long row_stride, const int32_t *draft, int num_seqs, int gamma,
                         int vocab, int32_t *target_argmax, int32_t *accept_len, int32_t *out_tokens,
                         unsigned long long *keys, cudaStream_t s)
{
    const long long rows = (long long)num_seqs * (gamma + 1);
    int chunks, chunk_len;
    const char *pdl = getenv("TS_PDL");
    const bool overlap = !(pdl && pdl[0] == '0');     // programmatic dependent launches (every kernel waits first)
    const int fast_chunks = (vocab + kFastChunk - 1) / kFastChunk;
    const bool fast = (row_stride % 8 == 0) && (vocab % 8 == 0) && fast_chunks <= kMaxChunks;
    if (fast) {
        // at least enough chunks to hold a chunk in registers; more when there are few rows
        chunks = pick_chunks(rows, vocab);
        if (chunks < fast_chunks) chunks = fast_chunks;
        chunk_len = (vocab + chunks - 1) / chunks;
        chunk_len = (chunk_len + 7) / 8 * 8;
        if (launch_overlapped(ts_argmax_reg_kernel, dim3((unsigned)chunks, (unsigned)rows), dim3(kArgmaxThreads), 0, s,
                              overlap, static_cast<const uint16_t *>(logits), row_stride, vocab, chunk_len, keys) != cudaSuccess)
            return TS_ERR_CUDA;
    } else {
        chunks = pick_chunks(rows, vocab);
        chunk_len = (vocab + chunks - 1) / chunks;
        chunk_len = (chunk_len + 7) / 8 * 8;
        if (launch_overlapped(ts_argmax_chunk_kernel, dim3((unsigned)chunks, (unsigned)rows), dim3(kArgmaxThreads), 0, s,
                              overlap, static_cast<const uint16_t *>(logits), row_stride, vocab, chunk_len, keys) != cudaSuccess)
            return TS_ERR_CUDA;
    }
    const cudaError_t e = launch_overlapped(ts_accept_finish_kernel, dim3(1), dim3(256), 0, s, overlap,
                                            (const unsigned long long *)keys, chunks, draft, num_seqs, gamma,
                                            target_argmax, accept_len, out_tokens);
    return e == cudaSuccess ? TS_OK : TS_ERR_CUDA;
}

}  // namespace ts

extern "C" {

size_t ts_accept_workspace_bytes(int32_t num_seqs, int32_t gamma, int32_t vocab)
{
    if (num_seqs < 0 || gamma < 0 || vocab < 1) return 0;
    const long long rows = (long long)num_seqs * (gamma + 1);
    const size_t bytes = (size_t)rows * ts::kMaxChunks * sizeof(unsigned long long);
    return bytes < 256 ? 256 : bytes;
}

int ts_accept_greedy(const void *logits, int64_t row_stride, const int32_t *draft, int32_t num_seqs, int32_t gamma,
                     int32_t vocab, int32_t *target_argmax, int32_t *accept_len, int32_t *out_tokens, void *workspace,
                     size_t workspace_bytes, void *stream)
{
    if (num_seqs < 0 || gamma < 0 || vocab < 1) return TS_ERR_INVALID_ARG;
    if (!logits || !target_argmax || !accept_len || !out_tokens || !workspace) return TS_ERR_INVALID_ARG;
    if (gamma > 0 && !draft) return TS_ERR_INVALID_ARG;
    if (row_stride < vocab) return TS_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(logits) & 15u) || (reinterpret_cast<uintptr_t>(workspace) & 15u))
        return TS_ERR_INVALID_ARG;
    if (workspace_bytes < ts_accept_workspace_bytes(num_seqs, gamma, vocab)) return TS_ERR_WORKSPACE;
    const long long rows = (long long)num_seqs * (gamma + 1);
    if (rows == 0) return TS_OK;
    if (rows > 65535) return TS_ERR_UNSUPPORTED;
    return ts::launch_accept(logits, row_stride, draft, num_seqs, gamma, vocab, target_argmax, accept_len, out_tokens,
                             static_cast<unsigned long long *>(workspace), static_cast<cudaStream_t>(stream));
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------
// Acceptance without any caller-supplied or allocated scratch
// ------------------------------------------------------------------------------------------------
namespace ts {

constexpr int kNoAllocMaxRows = 1024;   // num_seqs * (gamma + 1) accepted by ts_accept_greedy_noalloc

// Chunk keys of ts_accept_greedy_noalloc: 1024 rows x 64 chunks x 8 B = 512 KB, resident on every
// GPU that loads this library until the process exits.  Every call on a device shares it.
static __device__ __align__(256) unsigned long long g_noalloc_keys[kNoAllocMaxRows * kMaxChunks];

// Device address of g_noalloc_keys on the current device.  In host code the array's name is only a
// handle for the runtime, not a device pointer, so the address is asked for once per device (with
// that device current) and remembered.
static int noalloc_keys_ptr(unsigned long long **out)
{
    static std::mutex mu;
    static unsigned long long *cached[64] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return TS_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (dev >= 0 && dev < 64 && cached[dev]) {
        *out = cached[dev];
        return TS_OK;
    }
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_keys) != cudaSuccess || !p) return TS_ERR_CUDA;
    if (dev >= 0 && dev < 64) cached[dev] = static_cast<unsigned long long *>(p);
    *out = static_cast<unsigned long long *>(p);
    return TS_OK;
}

}  // namespace ts

extern "C" int ts_accept_greedy_noalloc(const void *logits, int64_t row_stride, const int32_t *draft,
                                        int32_t num_seqs, int32_t gamma, int32_t vocab, int32_t *target_argmax,
                                        int32_t *accept_len, int32_t *out_tokens, void *stream)
{
    if (num_seqs < 0 || gamma < 0 || vocab < 1) return TS_ERR_INVALID_ARG;
    if (!logits || !target_argmax || !accept_len || !out_tokens) return TS_ERR_INVALID_ARG;
    if (gamma > 0 && !draft) return TS_ERR_INVALID_ARG;
    if (row_stride < vocab) return TS_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(logits) & 15u) return TS_ERR_INVALID_ARG;
    const long long rows = (long long)num_seqs * (gamma + 1);
    if (rows > ts::kNoAllocMaxRows) return TS_ERR_UNSUPPORTED;     // beyond the built-in scratch
    if (rows == 0) return TS_OK;
    unsigned long long *keys = nullptr;
    const int rc = ts::noalloc_keys_ptr(&keys);
    if (rc != TS_OK) return rc;
    // every key this call reads in the second kernel is written by the first one, so nothing in the
    // shared array has to start at zero
    return ts::launch_accept(logits, row_stride, draft, num_seqs, gamma, vocab, target_argmax, accept_len, out_tokens,
                             keys, static_cast<cudaStream_t>(stream));
}
