// Lossless draft acceptance under temperature / top-k / top-p sampling for sm_100a.
//
// Kernel 1 streams the logits once (HBM-bound, same register-resident chunks as the greedy argmax)
// and leaves the top_k best (value, index) pairs of every chunk; kernel 2 (one CTA per sequence)
// merges the chunks of each row, builds the filtered distribution and walks the draft block.
// Selection is exact and integer-only (ordered bf16 keys, ties to the lower index); probabilities
// are fp32.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

#include "../../include/tailsieve.h"
#include "ts_common.cuh"

namespace ts {
namespace smp {

constexpr int kThreads = 256;
constexpr int kVecPerThread = 16;
constexpr int kChunkMax = kThreads * kVecPerThread * 8;      // 32768 logits per chunk
constexpr int kMaxTopK = 32;
constexpr int kMaxChunks = 16;
constexpr int kCap = 2048;                                   // candidate slots per chunk

// 16-bit ordered key of a bf16 value (thresholds only): NaN -> 0, -0 = +0, larger value -> larger key.
__device__ __forceinline__ uint32_t bf16_key(uint32_t u)
{
    u &= 0xffffu;
    if ((u & 0x7fffu) > 0x7f80u) return 0u;          // NaN: below everything
    if (u == 0x8000u) u = 0u;                          // -0 -> +0
    const uint32_t ord = (u & 0x8000u) ? (~u & 0xffffu) : (u | 0x8000u);
    return ord + 1u;
}
// Inverse of bf16_key for keys >= 1 (returns +0 for the zero key).
__device__ __forceinline__ uint32_t key_to_bf16(uint32_t key)
{
    const uint32_t ord = key - 1u;
    return (ord & 0x8000u) ? (ord & 0x7fffu) : (~ord & 0xffffu);
}
// 32-bit ordered key of an fp32 value (candidates: a penalised logit is no bf16 number any more).
__device__ __forceinline__ uint32_t f32_key(uint32_t f)
{
    if ((f & 0x7fffffffu) > 0x7f800000u) return 0u;  // NaN
    if (f == 0x80000000u) f = 0u;                      // -0 -> +0
    const uint32_t ord = (f & 0x80000000u) ? ~f : (f | 0x80000000u);
    return ord + 1u;
}
__device__ __forceinline__ float key_to_f32(uint32_t key)
{
    const uint32_t ord = key - 1u;
    return __uint_as_float((ord & 0x80000000u) ? (ord & 0x7fffffffu) : ~ord);
}
// Key of element idx of a row: its bf16 bits as they are, or -- if the token is present -- of the original
// logit (re-read from memory: the register copy was rounded) minus the penalty, in fp32.
__device__ __forceinline__ uint32_t element_key(uint32_t bits16, bool present, const uint16_t *rowp, int idx, float pen)
{
    if (!present) return f32_key((bits16 & 0xffffu) << 16);
    const float y = __uint_as_float((uint32_t)rowp[idx] << 16) - pen;
    return f32_key(__float_as_uint(y));
}
// Register copies of penalised logits: (logit - penalty), computed in fp32 as for the exact keys, rounded
// to bf16.  Thresholds and the candidate test work on these copies; that is sound because the rounding is
// monotone (if r(y) > r(x) then y > x: k copies above a threshold mean k true values above whatever lies
// below it), and the rare candidates get their exact fp32 value back from the original logit.
__device__ __forceinline__ void patch_vector(uint4 &x, uint32_t m, float pen)
{
    uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float lo = __uint_as_float(w[i] << 16) - ((m >> (2 * i)) & 1u ? pen : 0.f);
        const float hi = __uint_as_float(w[i] & 0xffff0000u) - ((m >> (2 * i + 1)) & 1u ? pen : 0.f);
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w[i]) : "f"(hi), "f"(lo));
    }
    x = make_uint4(w[0], w[1], w[2], w[3]);
}
__device__ __forceinline__ uint4 ld_stream_16B(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ unsigned long long pack_key(uint32_t key16, int idx)
{
    return ((unsigned long long)key16 << 32) | (unsigned long long)(0xffffffffu - (uint32_t)idx);
}

__device__ __forceinline__ void push_candidates(uint4 v, uint32_t e0, uint32_t e1, uint32_t e2, uint32_t e3, int idx0,
                                             int *cnt, unsigned long long *cand, uint32_t present, const uint16_t *rowp,
                                             float pen)
{
    // one bit per element that passed the threshold test (almost always a single one): the loop runs once per
    // candidate instead of visiting all eight slots
    uint32_t b8 = (e0 & 1u) | ((e0 >> 15) & 2u) | ((e1 & 1u) << 2) | ((e1 >> 13) & 8u) |
                  ((e2 & 1u) << 4) | ((e2 >> 11) & 0x20u) | ((e3 & 1u) << 6) | ((e3 >> 9) & 0x80u);
    while (b8) {
        const int i = __ffs(b8) - 1;
        b8 &= b8 - 1u;
        const int wi = i >> 1;
        const uint32_t word = wi == 0 ? v.x : (wi == 1 ? v.y : (wi == 2 ? v.z : v.w));
        const uint32_t bits = (i & 1) ? word >> 16 : word;
        const int s = atomicAdd(cnt, 1);
        if (s < kCap) cand[s] = pack_key(element_key(bits, (present >> i) & 1u, rowp, idx0 + i, pen), idx0 + i);
    }
}

// Degenerate chunk (thousands of ties at the threshold): extract the best key below the previous
// one, top_k times, re-reading the chunk from memory each time.  Slow, exact, and only reached by
// pathological inputs such as a constant row.
// The tokens of a chunk that are present for its row, beyond the caller's bitmap: the block's earlier
// drafts that fall into the chunk, as (vector index, bit of the element inside the vector) pairs.
struct DraftHits {
    int n;
    int vec[256];
    uint8_t bit[256];
};
__device__ __forceinline__ uint32_t present_mask(int j, const uint8_t *srow, const DraftHits *dh)
{
    uint32_t m = srow ? srow[j] : 0u;
    for (int e = 0; e < dh->n; ++e)
        if (dh->vec[e] == j) m |= dh->bit[e];
    return m;
}

__device__ __noinline__ void slow_topk(const uint4 *base, int nvec, int begin, int top_k, unsigned long long *dst,
                                       unsigned long long *s_red, const uint8_t *srow, const DraftHits *dh,
                                       const uint16_t *rowp, float pen)
{
    const int tid = threadIdx.x;
    unsigned long long prev = ~0ull;
    for (int r = 0; r < top_k; ++r) {
        unsigned long long best = 0ull;
        for (int j = tid; j < nvec; j += kThreads) {
            const uint4 x = base[j];
            const uint32_t w[4] = {x.x, x.y, x.z, x.w};
            const int idx0 = begin + j * 8;
            const uint32_t pm = pen != 0.f ? present_mask(j, srow, dh) : 0u;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t ka = element_key(w[i], (pm >> (2 * i)) & 1u, rowp, idx0 + 2 * i, pen);
                const uint32_t kb = element_key(w[i] >> 16, (pm >> (2 * i + 1)) & 1u, rowp, idx0 + 2 * i + 1, pen);
                const unsigned long long a = pack_key(ka, idx0 + 2 * i), b = pack_key(kb, idx0 + 2 * i + 1);
                if (ka && a < prev && a > best) best = a;
                if (kb && b < prev && b > best) best = b;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { const unsigned long long x = __shfl_xor_sync(0xffffffffu, best, o); best = x > best ? x : best; }
        if ((tid & 31) == 0) s_red[tid >> 5] = best;
        __syncthreads();
        best = s_red[0];
#pragma unroll
        for (int w = 1; w < kThreads / 32; ++w) best = s_red[w] > best ? s_red[w] : best;
        __syncthreads();
        if (tid == 0) dst[r] = best;
        if (best == 0ull) break;
        prev = best;
    }
}

// grid = (chunks, rows).  out[(row * chunks + chunk) * top_k + j] = j-th best key of the chunk (0 = none).
// PEN: a presence penalty applies (seen-token bitmap and / or earlier drafts of the block).
template <bool PEN>
__global__ void __launch_bounds__(kThreads, 3)
ts_topk_chunk_kernel(const uint16_t *__restrict__ logits, long long row_stride, int vocab, int chunk_len, int top_k,
                     unsigned long long *__restrict__ out, const uint8_t *__restrict__ seen, long long seen_stride,
                     float pen, const int32_t *__restrict__ draft, int gamma)
{
    __shared__ DraftHits s_dh;
    __shared__ unsigned long long s_cand[kCap];
    __shared__ unsigned long long s_red[kThreads / 32];
    __shared__ int s_cnt;
    __shared__ uint32_t s_tkey[kThreads];
    __shared__ uint32_t s_t1;
    const int chunk = blockIdx.x, row = blockIdx.y, chunks = gridDim.x;
    const int tid = threadIdx.x;
    const int begin = chunk * chunk_len;
    int end = begin + chunk_len;
    if (end > vocab) end = vocab;
    const int nvec = end > begin ? (end - begin) >> 3 : 0;
    const uint16_t *rowp = logits + (long long)row * row_stride;
    const uint4 *base = reinterpret_cast<const uint4 *>(rowp + begin);
    unsigned long long *dst = out + ((long long)row * chunks + chunk) * top_k;
    const uint32_t nan2 = 0x7fc07fc0u;
    uint4 v[kVecPerThread];
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u) {
        const int j = tid + u * kThreads;
        v[u] = j < nvec ? ld_stream_16B(base + j) : make_uint4(nan2, nan2, nan2, nan2);
    }
    if (tid == 0) { s_cnt = 0; s_dh.n = 0; }
    // ---- presence penalty: lower the register copies of the present tokens (rounded down to bf16)
    uint32_t pmask[kVecPerThread / 4];                  // one byte per vector: which of its 8 elements are present
    const uint8_t *srow = nullptr;
    if (PEN) {
        const int R = gamma + 1, b = row / R, irow = row % R;
        srow = seen ? seen + (long long)b * seen_stride + (begin >> 3) : nullptr;
        __syncthreads();
        for (int jj = tid; jj < irow; jj += kThreads) {
            const int d = draft[(long long)b * gamma + jj];
            if (d >= begin && d < end) {
                const int slot = atomicAdd(&s_dh.n, 1);
                s_dh.vec[slot] = (d - begin) >> 3;
                s_dh.bit[slot] = (uint8_t)(1u << (d & 7));
            }
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < kVecPerThread / 4; ++q) pmask[q] = 0u;
#pragma unroll
        for (int u = 0; u < kVecPerThread; ++u) {
            const int j = tid + u * kThreads;
            if (srow && j < nvec) pmask[u >> 2] |= (uint32_t)srow[j] << (8 * (u & 3));
        }
        for (int e = 0; e < s_dh.n; ++e) {
            const int j = s_dh.vec[e];
            if ((j & (kThreads - 1)) == tid) {
                const int u = j >> 8;
#pragma unroll
                for (int q = 0; q < kVecPerThread / 4; ++q)
                    if (q == (u >> 2)) pmask[q] |= (uint32_t)s_dh.bit[e] << (8 * (u & 3));
            }
        }
#pragma unroll
        for (int u = 0; u < kVecPerThread; ++u) {
            const uint32_t m = (pmask[u >> 2] >> (8 * (u & 3))) & 0xffu;
            if (m) patch_vector(v[u], m, pen);
        }
    }
    // ---- the largest element of every thread (NaN never wins)
    __nv_bfloat162 m2 = *reinterpret_cast<const __nv_bfloat162 *>(&nan2);
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u) {
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162 *>(&v[u].x));
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162 *>(&v[u].y));
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162 *>(&v[u].z));
        m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162 *>(&v[u].w));
    }
    const uint32_t mbits = *reinterpret_cast<const uint32_t *>(&m2);
    const uint32_t k0 = bf16_key(mbits), k1 = bf16_key(mbits >> 16);
    const uint32_t tkey = k0 > k1 ? k0 : k1;
    // ---- threshold T1 = the top_k-th largest of the 256 thread maxima (0 if fewer than top_k threads
    //      hold a number): the top_k-th largest element of the chunk is >= T1, so the chunk's top_k are
    //      all >= T1, and on random data only a few dozen elements are.  Warp 0 finds it by binary search
    //      on the 17-bit key, each lane counting over the 8 maxima it holds.
    s_tkey[tid] = tkey;
    __syncthreads();
    if (tid < 32) {
        uint32_t k8[kThreads / 32];
#pragma unroll
        for (int i = 0; i < kThreads / 32; ++i) k8[i] = s_tkey[tid + 32 * i];
        const int want = top_k < kThreads ? top_k : kThreads;
        // count(>= lo) >= want holds for lo = the smallest maximum (all 256 lie at or above it) and fails
        // for hi = the largest + 1: the search runs over the spread of the maxima, not over all keys
        uint32_t kmin = k8[0], kmax = k8[0];
#pragma unroll
        for (int i = 1; i < kThreads / 32; ++i) { kmin = k8[i] < kmin ? k8[i] : kmin; kmax = k8[i] > kmax ? k8[i] : kmax; }
        uint32_t lo = __reduce_min_sync(0xffffffffu, kmin), hi = __reduce_max_sync(0xffffffffu, kmax) + 1u;
        while (hi - lo > 1u) {
            const uint32_t mid = (lo + hi) >> 1;
            int c = 0;
#pragma unroll
            for (int i = 0; i < kThreads / 32; ++i) c += k8[i] >= mid;
            c = __reduce_add_sync(0xffffffffu, c);           // one warp-wide add instead of a ballot per key
            if (c >= want) lo = mid; else hi = mid;
        }
        if (tid == 0) s_t1 = lo;
    }
    __syncthreads();
    const uint32_t t1 = s_t1;
    const uint32_t t1bits = t1 ? key_to_bf16(t1) : 0xff80u;          // no k-th maximum: everything that is not NaN
    const uint32_t t1x2 = t1bits | (t1bits << 16);
    const __nv_bfloat162 tt = *reinterpret_cast<const __nv_bfloat162 *>(&t1x2);
    // ---- candidates (rare: a few hundred of the chunk's 32768 elements; the push is kept out of line
    //      so that the unrolled scan stays small)
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u) {
        const uint32_t e0 = __hge2_mask(*reinterpret_cast<const __nv_bfloat162 *>(&v[u].x), tt);
        const uint32_t e1 = __hge2_mask(*reinterpret_cast<const __nv_bfloat162 *>(&v[u].y), tt);
        const uint32_t e2 = __hge2_mask(*reinterpret_cast<const __nv_bfloat162 *>(&v[u].z), tt);
        const uint32_t e3 = __hge2_mask(*reinterpret_cast<const __nv_bfloat162 *>(&v[u].w), tt);
        if (e0 | e1 | e2 | e3)
            push_candidates(v[u], e0, e1, e2, e3, begin + (tid + u * kThreads) * 8, &s_cnt, s_cand,
                            PEN ? (pmask[u >> 2] >> (8 * (u & 3))) & 0xffu : 0u, rowp, pen);
    }
    for (int j = tid; j < top_k; j += kThreads) dst[j] = 0ull;
    __syncthreads();
    const int cnt = s_cnt;
    if (cnt <= kCap) {
        // ---- rank the candidates; the best top_k go out in order
        //      (by counting, `per` lanes to a candidate, each over a strided share of the list)
        int per = 1;
        while (per < 32 && cnt * per * 2 <= kThreads) per <<= 1;
        const int sub = tid & (per - 1);
        for (int c0 = 0; c0 < cnt; c0 += kThreads / per) {
            const int c = c0 + tid / per;
            const unsigned long long mine = c < cnt ? s_cand[c] : ~0ull;
            int rank = 0;
            int j = sub;
            for (; j + 3 * per < cnt; j += 4 * per) {
                const unsigned long long a0 = s_cand[j], a1 = s_cand[j + per], a2 = s_cand[j + 2 * per], a3 = s_cand[j + 3 * per];
                rank += (int)(a0 > mine) + (int)(a1 > mine) + (int)(a2 > mine) + (int)(a3 > mine);
            }
            for (; j < cnt; j += per) rank += s_cand[j] > mine;
            for (int o = per >> 1; o > 0; o >>= 1) rank += __shfl_xor_sync(0xffffffffu, rank, o);
            if (c < cnt && sub == 0 && rank < top_k) dst[rank] = mine;
        }
    } else {
        slow_topk(base, nvec, begin, top_k, dst, s_red, srow, &s_dh, rowp, PEN ? pen : 0.f);
    }
}

// One CTA per sequence, one warp per row (rows beyond the number of warps are taken in turn); warp 0
// then walks the draft block with one kept token per lane.
__global__ void __launch_bounds__(1024)
ts_sample_finish_kernel(const unsigned long long *__restrict__ keys, int chunks, int top_k,
                        const int32_t *__restrict__ draft,
                        const float *__restrict__ uniforms, int gamma, float inv_temperature, float top_p,
                        const float *__restrict__ draft_probs, long long q_stride, int vocab,
                        int32_t *accept_len, int32_t *out_tokens)
{
    extern __shared__ unsigned char smem[];
    constexpr uint32_t FULL = 0xffffffffu;
    const int R = gamma + 1;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    const int total = chunks * top_k;
    int32_t *s_ids = reinterpret_cast<int32_t *>(smem);                       // [R][32]
    float *s_p = reinterpret_cast<float *>(smem + (size_t)R * 32 * 4);         // [R][32]
    float *s_q = reinterpret_cast<float *>(smem + (size_t)R * 32 * 8);         // [R][32]: proposal at the kept tokens
    unsigned long long *s_best = reinterpret_cast<unsigned long long *>(smem + (size_t)R * 32 * 12);  // [warps][32]
    unsigned long long *s_cand = s_best + nwarps * 32;                         // [warps][chunks * top_k]
    const int b = blockIdx.x;
    // warp 0 walks the draft block at the end; the inputs of its first 32 steps do not come from the kernel
    // before, so they are fetched ahead of the wait for it (lane l holds step l's uniforms, draft token and
    // that token's proposal probability)
    float ua_l = 0.f, us_l = 0.f, qx_l = 1.f;
    int32_t x_l = -1;
    if (warp == 0 && lane <= gamma) {
        const float2 u2 = *reinterpret_cast<const float2 *>(uniforms + ((long long)b * R + lane) * 2);
        ua_l = u2.x;
        us_l = u2.y;
        x_l = lane < gamma ? draft[(long long)b * gamma + lane] : -1;
        if (draft_probs && lane < gamma)
            qx_l = (x_l >= 0 && x_l < vocab) ? draft_probs[((long long)b * gamma + lane) * q_stride + x_l] : 0.f;
    }
    grid_dependency_wait();       // the chunk keys of the kernel before
    for (int i = warp; i < R; i += nwarps) {
        const long long row = (long long)b * R + i;
        const unsigned long long *src = keys + row * total;
        unsigned long long *best = s_best + warp * 32;
        unsigned long long *cand = s_cand + (size_t)warp * total;
        best[lane] = 0ull;
        for (int c = lane; c < total; c += 32) cand[c] = src[c];
        __syncwarp();
        // Merge of the chunks' lists (each sorted in descending order, empty slots = key 0 last).  Only entries
        // at or above T = the smallest of the lists' m-th entries, m = ceil(top_k / chunks), can be among the
        // top_k overall (chunks * m >= top_k entries lie at or above T); on random data that is a quarter of
        // the chunks * top_k candidates.  They are compacted to the front of the list in place and ranked
        // by counting among themselves (the sweep over all candidates was the longest phase of this kernel:
        // seventeen warps of one SM issuing it at once).
        const int mth = (top_k + chunks - 1) / chunks;
        unsigned long long thr = ~0ull;
        for (int cc = lane; cc < chunks; cc += 32) {
            const unsigned long long x = cand[cc * top_k + mth - 1];
            thr = x < thr ? x : thr;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { const unsigned long long y = __shfl_xor_sync(FULL, thr, o); thr = y < thr ? y : thr; }
        int cnt = 0;                                     // a short list (thr == 0) keeps every entry that exists
        for (int c0 = 0; c0 < total; c0 += 32) {
            const int c = c0 + lane;
            const unsigned long long x = c < total ? cand[c] : 0ull;
            const bool keep = x != 0ull && x >= thr;
            const unsigned mask = __ballot_sync(FULL, keep);
            __syncwarp();
            if (keep) cand[cnt + __popc(mask & ((1u << lane) - 1u))] = x;      // at or before the place it was read from
            cnt += __popc(mask);
            __syncwarp();
        }
        for (int c = lane; c < cnt; c += 32) {
            const unsigned long long mine = cand[c];
            int rank = 0;
            int j = 0;
            for (; j + 3 < cnt; j += 4) {
                const unsigned long long x0 = cand[j], x1 = cand[j + 1], x2 = cand[j + 2], x3 = cand[j + 3];
                rank += (int)(x0 > mine) + (int)(x1 > mine) + (int)(x2 > mine) + (int)(x3 > mine);
            }
            for (; j < cnt; ++j) rank += cand[j] > mine;
            if (rank < top_k) best[rank] = mine;
        }
        __syncwarp();
        const unsigned long long key = best[lane];
        const bool valid = lane < top_k && key != 0ull;
        const int idx = valid ? (int)(0xffffffffu - (uint32_t)(key & 0xffffffffull)) : -1;
        // the (penalised) logit itself, carried exactly by the key
        float x = -INFINITY;
        if (valid) x = key_to_f32((uint32_t)(key >> 32));
        const float z = x * inv_temperature;
        const float z0 = __shfl_sync(FULL, z, 0);
        float e = valid ? expf(z - z0) : 0.f;
        if (valid && z == z0) e = 1.f;                                           // also covers z0 = -inf
        float sum = e;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(FULL, sum, o);
        const float p = sum > 0.f ? e / sum : 0.f;
        float cum = p;                                                            // inclusive prefix sum in rank order
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const float y = __shfl_up_sync(FULL, cum, o); if (lane >= o) cum += y; }
        const bool keep = valid && (lane == 0 || (cum - p) < top_p);
        // nucleus membership must be a prefix: a lane is kept only if every earlier one is
        const unsigned kept_mask = __ballot_sync(FULL, keep);
        const int nkept = kept_mask == FULL ? 32 : __ffs(~kept_mask) - 1;          // length of the leading run of ones
        const bool kept = lane < nkept;
        float ks = kept ? p : 0.f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ks += __shfl_xor_sync(FULL, ks, o);
        s_ids[i * 32 + lane] = kept ? idx : -1;
        s_p[i * 32 + lane] = kept ? p / ks : 0.f;
        // sampled drafts: the proposal is needed at the kept tokens only (the target is zero elsewhere)
        if (draft_probs && i < gamma)
            s_q[i * 32 + lane] = kept ? draft_probs[((long long)b * gamma + i) * q_stride + idx] : 0.f;
    }
    __syncthreads();
    if (warp == 0) {
        int32_t *out = out_tokens + (long long)b * R;
        for (int i = lane; i < R; i += 32) out[i] = -1;
        __syncwarp();
        int a = 0;
        for (int i = 0; i <= gamma; ++i) {
            if ((i & 31) == 0 && i > 0) {
                // the next 32 steps' inputs in one round of loads (read inside the walk, each step paid a
                // memory round trip before it could decide)
                const int il = i + lane;
                if (il <= gamma) {
                    const float2 u2 = *reinterpret_cast<const float2 *>(uniforms + ((long long)b * R + il) * 2);
                    ua_l = u2.x;
                    us_l = u2.y;
                    x_l = il < gamma ? draft[(long long)b * gamma + il] : -1;
                    if (draft_probs && il < gamma)
                        qx_l = (x_l >= 0 && x_l < vocab) ? draft_probs[((long long)b * gamma + il) * q_stride + x_l] : 0.f;
                }
            }
            const int32_t id = s_ids[i * 32 + lane];
            const float pj = s_p[i * 32 + lane];
            const float ua = __shfl_sync(FULL, ua_l, i & 31), us = __shfl_sync(FULL, us_l, i & 31);
            bool is_draft = false;
            if (i < gamma) {
                const int32_t xtok = __shfl_sync(FULL, x_l, i & 31);
                is_draft = (id == xtok) && id >= 0;
                const unsigned hit = __ballot_sync(FULL, is_draft);
                const float px = hit ? __shfl_sync(FULL, pj, __ffs(hit) - 1) : 0.f;
                const float qx = __shfl_sync(FULL, qx_l, i & 31);
                if (ua * qx < px) {                 // accepted (probability min(1, p / q)): next position
                    if (lane == 0) out[i] = xtok;
                    ++a;
                    continue;
                }
                if (draft_probs) {
                    // rejected: one token from norm(max(0, p - q)); from p itself if nothing is left of it
                    float r = id >= 0 ? fmaxf(pj - s_q[i * 32 + lane], 0.f) : 0.f;
                    if (!__ballot_sync(FULL, r > 0.f)) r = id >= 0 ? pj : 0.f;
                    float cum = r, tot = r;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) { const float y = __shfl_up_sync(FULL, cum, o); if (lane >= o) cum += y; }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(FULL, tot, o);
                    const unsigned over = __ballot_sync(FULL, r > 0.f && cum > us * tot);
                    const unsigned lives = __ballot_sync(FULL, r > 0.f);
                    int pick = -1;
                    if (over) pick = __ffs(over) - 1;
                    else if (lives) pick = 31 - __clz(lives);
                    const int32_t y = pick >= 0 ? __shfl_sync(FULL, id, pick) : -1;
                    if (lane == 0) out[i] = y;
                    break;
                }
            }
            // one token from the (residual) distribution, then stop
            const float w = (id >= 0 && !is_draft) ? pj : 0.f;
            float cum = w, tot = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const float y = __shfl_up_sync(FULL, cum, o); if (lane >= o) cum += y; }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(FULL, tot, o);
            const bool live = id >= 0 && !is_draft;
            const unsigned over = __ballot_sync(FULL, live && cum > us * tot);
            const unsigned lives = __ballot_sync(FULL, live);
            int pick = -1;
            if (over) pick = __ffs(over) - 1;
            else if (lives) pick = 31 - __clz(lives);          // rounding left the last one
            const int32_t y = pick >= 0 ? __shfl_sync(FULL, id, pick) : -1;
            if (lane == 0) out[i] = y;
            break;
        }
        if (lane == 0) accept_len[b] = a;
    }
}

static int pick_chunks(long long rows, int vocab)
{
    // a chunk must fit in registers; beyond that, only as many chunks as it takes to have about two
    // CTAs per SM (every CTA pays a fixed selection overhead)
    const int need = (vocab + kChunkMax - 1) / kChunkMax;
    long long c = (296 + rows - 1) / rows;
    const long long by_len = (vocab + 4095) / 4096;
    if (c > by_len) c = by_len;
    if (c > kMaxChunks) c = kMaxChunks;
    if (c < need) c = need;
    if (const char *e = getenv("TS_SAMPLE_CHUNKS")) {
        const long long v = atoll(e);
        if (v >= need && v <= kMaxChunks) c = v;
    }
    return (int)c;
}

}  // namespace smp
}  // namespace ts

extern "C" {

size_t ts_sample_workspace_bytes(int32_t num_seqs, int32_t gamma, int32_t vocab, int32_t top_k)
{
    if (num_seqs < 0 || gamma < 0 || vocab < 1 || top_k < 1 || top_k > ts::smp::kMaxTopK) return 0;
    if ((vocab + ts::smp::kChunkMax - 1) / ts::smp::kChunkMax > ts::smp::kMaxChunks) return 0;
    const size_t bytes = (size_t)num_seqs * (gamma + 1) * ts::smp::kMaxChunks * top_k * sizeof(unsigned long long);
    return bytes < 256 ? 256 : bytes;
}

int ts_accept_sample(const void *logits, int64_t row_stride, const int32_t *draft, const float *uniforms,
                     int32_t num_seqs, int32_t gamma, int32_t vocab, float temperature, int32_t top_k, float top_p,
                     int32_t *accept_len, int32_t *out_tokens, void *workspace, size_t workspace_bytes, void *stream)
{
    return ts_accept_sample_penalized(logits, row_stride, draft, uniforms, num_seqs, gamma, vocab, temperature, top_k,
                                      top_p, 0.f, nullptr, 0, accept_len, out_tokens, workspace, workspace_bytes, stream);
}

int ts_accept_sample_penalized(const void *logits, int64_t row_stride, const int32_t *draft, const float *uniforms,
                               int32_t num_seqs, int32_t gamma, int32_t vocab, float temperature, int32_t top_k,
                               float top_p, float presence_penalty, const uint8_t *seen, int64_t seen_stride,
                               int32_t *accept_len, int32_t *out_tokens, void *workspace, size_t workspace_bytes,
                               void *stream)
{
    return ts_accept_sample_proposal(logits, row_stride, draft, nullptr, 0, uniforms, num_seqs, gamma, vocab, temperature,
                                     top_k, top_p, presence_penalty, seen, seen_stride, accept_len, out_tokens, workspace,
                                     workspace_bytes, stream);
}

int ts_accept_sample_proposal(const void *logits, int64_t row_stride, const int32_t *draft, const float *draft_probs,
                              int64_t draft_probs_row_stride, const float *uniforms, int32_t num_seqs, int32_t gamma,
                              int32_t vocab, float temperature, int32_t top_k, float top_p, float presence_penalty,
                              const uint8_t *seen, int64_t seen_stride, int32_t *accept_len, int32_t *out_tokens,
                              void *workspace, size_t workspace_bytes, void *stream)
{
    using namespace ts::smp;
    if (draft_probs && draft_probs_row_stride < vocab) return TS_ERR_INVALID_ARG;
    if (isnan(presence_penalty) || isinf(presence_penalty)) return TS_ERR_INVALID_ARG;
    if (seen && seen_stride * 8 < vocab) return TS_ERR_INVALID_ARG;
    if (num_seqs < 0 || gamma < 0 || vocab < 1) return TS_ERR_INVALID_ARG;
    if (!logits || !uniforms || !accept_len || !out_tokens || !workspace) return TS_ERR_INVALID_ARG;
    if (gamma > 0 && !draft) return TS_ERR_INVALID_ARG;
    if (!(temperature > 0.f) || isinf(temperature) || !(top_p > 0.f) || top_p > 1.f) return TS_ERR_INVALID_ARG;
    if (top_k < 1) return TS_ERR_INVALID_ARG;
    if (top_k > kMaxTopK || gamma > 255) return TS_ERR_UNSUPPORTED;
    if (row_stride < vocab) return TS_ERR_INVALID_ARG;
    if (row_stride % 8 != 0 || vocab % 8 != 0) return TS_ERR_UNSUPPORTED;      // rows must be 16-byte aligned
    if ((vocab + kChunkMax - 1) / kChunkMax > kMaxChunks) return TS_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(logits) & 15u) || (reinterpret_cast<uintptr_t>(workspace) & 15u)) return TS_ERR_INVALID_ARG;
    const size_t need = ts_sample_workspace_bytes(num_seqs, gamma, vocab, top_k);
    if (need == 0) return TS_ERR_UNSUPPORTED;
    if (workspace_bytes < need) return TS_ERR_WORKSPACE;
    const long long rows = (long long)num_seqs * (gamma + 1);
    if (rows == 0) return TS_OK;
    if (rows > 65535) return TS_ERR_UNSUPPORTED;
    const int chunks = pick_chunks(rows, vocab);
    int chunk_len = (vocab + chunks - 1) / chunks;
    chunk_len = (chunk_len + 7) / 8 * 8;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned long long *keys = static_cast<unsigned long long *>(workspace);
    // a penalty of zero, or nothing present (no bitmap and no earlier drafts), is the plain kernel
    if (presence_penalty != 0.f && (seen || gamma > 0))
        ts_topk_chunk_kernel<true><<<dim3((unsigned)chunks, (unsigned)rows), kThreads, 0, s>>>(
            static_cast<const uint16_t *>(logits), row_stride, vocab, chunk_len, top_k, keys, seen, seen_stride,
            presence_penalty, draft, gamma);
    else
        ts_topk_chunk_kernel<false><<<dim3((unsigned)chunks, (unsigned)rows), kThreads, 0, s>>>(
            static_cast<const uint16_t *>(logits), row_stride, vocab, chunk_len, top_k, keys, nullptr, 0, 0.f, draft,
            gamma);
    if (cudaGetLastError() != cudaSuccess) return TS_ERR_CUDA;
    const int R = gamma + 1;
    int warps = R < 32 ? R : 32;
    size_t smem;
    for (;;) {
        smem = (size_t)R * 32 * 12 + (size_t)warps * 32 * 8 + (size_t)warps * chunks * top_k * 8;
        if (smem <= 48 * 1024 || warps == 1) break;
        warps = (warps + 1) / 2;
    }
    if (smem > 48 * 1024) return TS_ERR_UNSUPPORTED;
    const char *pdl = getenv("TS_PDL");
    const bool overlap = !(pdl && pdl[0] == '0');
    const cudaError_t e = ts::launch_overlapped(ts_sample_finish_kernel, dim3((unsigned)num_seqs), dim3(warps * 32), smem, s,
                                                overlap, (const unsigned long long *)keys, chunks, (int)top_k, draft,
                                                uniforms, (int)gamma, 1.0f / temperature, top_p, draft_probs,
                                                (long long)draft_probs_row_stride, (int)vocab, accept_len, out_tokens);
    return e == cudaSuccess ? TS_OK : TS_ERR_CUDA;
}

}  // extern "C"
