// Paged-KV decode / verify attention for sm_100a.
//
// One persistent kernel serves ts_decode_attn, ts_verify_attn and ts_decode_attn_splitkv.
//
// Work decomposition.  Every (sequence s, kv head g) pair owns ceil(kv_len_s / 64) KV tiles of 64
// tokens.  All pairs' tiles are laid end to end in the order (s, g, tile); that line of W tiles is
// cut into NG equal pieces, one per warp group ("group"; NG = SMs x groups per CTA), so every group
// streams the same number of bytes whatever the length distribution.  A piece that covers a pair
// completely produces that pair's final output; a piece that covers only part of a pair writes an
// fp32 partial (normalised output + log-sum-exp) that a small merge kernel recombines.  In split-KV
// mode the cuts are moved to the caller-visible per-sequence chunk boundaries instead.
//
// Inside a group.  K and V tiles arrive in shared memory through TMA tensor loads (128-byte
// swizzle) into a ring of stages, each with its own pair of mbarriers; lane 0 of the group's first
// warp issues them several tiles ahead.  The math runs on warp-level tensor-core MMAs in the
// "transposed" arrangement: scores S^T[token, row] = K . Q^T with the 64 tokens on the M axis and
// the G*q_len query rows of the pair on the N axis (8 rows per n-tile), then
// O^T[dim, row] += V^T . P^T.  That way every byte of K and V is read from shared memory once per
// warp as an A operand, Q^T lives in registers for the whole segment, and the online-softmax
// statistics are per-column values a lane already owns.  P is fed to the second MMA as a bf16
// hi + lo pair so that its rounding stays below the output's own bf16 rounding.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

#include "../../include/tailsieve.h"
#include "ts_common.cuh"

namespace ts {

// ------------------------------------------------------------------------------------------------
// plan data
// ------------------------------------------------------------------------------------------------
struct GroupStart {
    int32_t s, g, tau, pad;
};

enum : int { kModeFree = 0, kModeChunks = 1 };

struct AttnArgs {
    const uint16_t *q;
    uint16_t *out;
    const int32_t *block_table;
    const int32_t *kv_lens;
    const int32_t *cum_tiles;    // [B+1] exclusive prefix sum of tiles per sequence
    const GroupStart *gstart;    // [NG+1]
    const long long *gpos;       // [NG+1] position of each group's first tile on the tile line
    float *part_o;
    float *part_lse;
    const int32_t *num_splits;   // chunk mode: [B]
    int32_t *status;
    int B, q_len, Hq, Hkv, G, rows, P, max_pages, max_splits, mode;
    int ngrp, ns;                // groups per CTA, pipeline stages per group
    int tok_first;               // 1: token is tensor-map dim 1 and head dim 2; 0: the reverse
    int box_tok;                 // warp-MMA kernel: tokens per 4-D TMA box (16/32/64, <= page size); 0 = one 5-D box per tile
    int lg_page;                 // log2(page size)
    int lg_box;                  // log2(box_tok) when box_tok > 0
    int page_boxes;              // warp-MMA kernel: 1 = 5-D boxes of one 16-token page x both 64-dim halves (page size 16)
    int blk_stride, half_stride; // shared-memory tile layout: bytes between 16-token blocks / between the 64-dim halves
    float scale_log2;            // scale * log2(e)
    long long wait_cycles;       // bound of every mbarrier wait
};

__device__ __forceinline__ int div_up(int a, int b) { return (a + b - 1) / b; }

// Largest s in [0, B] with Hkv * cum[s] <= pos.
__device__ int locate_seq(const int32_t *cum, int B, int Hkv, long long pos)
{
    int lo = 0, hi = B;   // invariant: Hkv*cum[lo] <= pos
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if ((long long)Hkv * cum[mid] <= pos) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// Single-CTA planner: prefix sum of tiles, per-sequence split counts (chunk mode), group starts.
__global__ void __launch_bounds__(1024, 1)
ts_plan_kernel(const int32_t *__restrict__ kv_lens, int B, int Hkv, int NG, int mode, int max_splits,
               int chunks_per_group, int32_t *cum_tiles, GroupStart *gstart, long long *gpos,
               int32_t *num_splits, int32_t *status, float *part_o, float *part_lse,
               int rows_all /* q_len*Hq */, int D)
{
    constexpr int kSmemB = 4096;             // up to this many sequences the prefix sums are also kept in shared
    __shared__ int warp_sums[32];            // memory: the binary searches below are chains of dependent loads
    __shared__ int carry_s;
    __shared__ int32_t s_cum[kSmemB + 1];
    grid_dependency_wait();      // launched ahead of the previous kernel's end: nothing is touched before this
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool in_smem = B <= kSmemB;
    const int32_t *cum = in_smem ? s_cum : cum_tiles;
    if (tid == 0) { carry_s = 0; *status = TS_OK; cum_tiles[0] = 0; s_cum[0] = 0; }
    __syncthreads();
    for (int base = 0; base < B; base += 1024) {
        const int i = base + tid;
        int v = 0;
        if (i < B) { const int n = kv_lens[i]; v = n > 0 ? (n + kTile - 1) / kTile : 0; }
        int x = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, x, o); if (lane >= o) x += y; }
        if (lane == 31) warp_sums[warp] = x;
        __syncthreads();
        if (warp == 0) {
            int w = warp_sums[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, w, o); if (lane >= o) w += y; }
            warp_sums[lane] = w;
        }
        __syncthreads();
        const int incl = carry_s + x + (warp > 0 ? warp_sums[warp - 1] : 0);
        if (i < B) { cum_tiles[i + 1] = incl; if (in_smem) s_cum[i + 1] = incl; }
        __syncthreads();
        if (tid == 1023) carry_s = incl;
        __syncthreads();
    }
    __threadfence_block();
    __syncthreads();
    const long long W = (long long)Hkv * cum[B];

    if (mode == kModeChunks) {
        long long want = (long long)NG * chunks_per_group;
        int chunk = (int)((W + want - 1) / want);
        if (chunk < 1) chunk = 1;
        for (int s = tid; s < B; s += 1024) {
            const int tiles = cum[s + 1] - cum[s];
            int S = div_up(tiles, chunk);
            if (S > max_splits) S = max_splits;
            if (S < 1) S = 1;
            if (tiles > 0) { const int ct = div_up(tiles, S); S = div_up(tiles, ct); }
            num_splits[s] = S;
        }
        // empty sequences: their single slot is zeros / -inf
        for (int s = 0; s < B; ++s) {
            if (cum[s + 1] != cum[s]) continue;
            float *po = part_o + (size_t)s * max_splits * rows_all * D;
            float *pl = part_lse + (size_t)s * max_splits * rows_all;
            for (int i = tid; i < rows_all * D; i += 1024) po[i] = 0.f;
            for (int i = tid; i < rows_all; i += 1024) pl[i] = -INFINITY;
        }
        __threadfence_block();
        __syncthreads();
    }

    for (int k = tid; k <= NG; k += 1024) {
        long long U = (W * k) / NG;
        int s = locate_seq(cum, B, Hkv, U);
        if (mode == kModeChunks && s < B) {
            const int tiles = cum[s + 1] - cum[s];
            const long long r = U - (long long)Hkv * cum[s];
            const int tau = (int)(r % tiles);
            const int ct = div_up(tiles, num_splits[s]);
            const int rem = tau % ct;
            if (rem) {
                int t2 = tau - rem + ct;
                if (t2 > tiles) t2 = tiles;
                U += (t2 - tau);
                s = locate_seq(cum, B, Hkv, U);
            }
        }
        GroupStart gs;
        gs.s = s; gs.g = 0; gs.tau = 0; gs.pad = 0;
        if (s < B) {
            const int tiles = cum[s + 1] - cum[s];
            const long long r = U - (long long)Hkv * cum[s];
            gs.g = (int)(r / tiles);
            gs.tau = (int)(r % tiles);
            if (gs.tau != 0 && k > 0 && mode == kModeFree) {
                // the pair under this boundary is split between group k - 1 and later ones: say so for the
                // merge kernel -- bit 31: the pair starts inside group k - 1 (which therefore merges it),
                // bit 30: some groups are empty (W < NG), low bits: the last group that holds a part of it
                const long long a0 = U - gs.tau, b0 = a0 + tiles;
                const long long prev = (W * (k - 1)) / NG;
                const int k_last = (int)((b0 * NG - 1) / W);
                gs.pad = (int32_t)((a0 >= prev ? 0x80000000u : 0u) | (W < NG ? 0x40000000u : 0u) | (uint32_t)k_last);
            }
        }
        gstart[k] = gs;
        gpos[k] = U;
    }
}

// ------------------------------------------------------------------------------------------------
// attention kernel
// ------------------------------------------------------------------------------------------------
struct Cursor {
    int s, g, tau, tiles, n;
};

__device__ __forceinline__ void cur_load(Cursor &c, const AttnArgs &a)
{
    if (c.s < a.B) {
        const int n = a.kv_lens[c.s];
        c.n = n > 0 ? n : 0;
        c.tiles = (c.n + kTile - 1) / kTile;
    } else {
        c.n = 0;
        c.tiles = 0;
    }
}
__device__ __forceinline__ void cur_advance(Cursor &c, const AttnArgs &a)
{
    if (++c.tau >= c.tiles) {
        c.tau = 0;
        if (++c.g >= a.Hkv) {
            c.g = 0;
            do { ++c.s; cur_load(c, a); } while (c.s < a.B && c.tiles == 0);
        }
    }
}

template <int D, int NT, int WG>
__global__ void __launch_bounds__(256, 1)
ts_attn_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
               const AttnArgs a)
{
    constexpr int KK = D / 16;            // k-steps of S^T = K Q^T
    constexpr int MD = D / 16;            // m-tiles (16 dims) of O^T = V^T P^T
    constexpr int HALVES = D / 64;        // 128-byte swizzle spans per row
    constexpr int TB = kTile * D * 2;     // bytes of one K (or V) tile
    constexpr uint32_t FULL = 0xffffffffu;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int ngrp = a.ngrp, ns = a.ns;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int grp = warp / WG, wig = warp % WG;
    const int gid = blockIdx.x * ngrp + grp;
    const uint32_t ring = smem_base + (uint32_t)grp * ns * 2 * TB;
    const uint32_t bars = smem_base + (uint32_t)ngrp * ns * 2 * TB + (uint32_t)grp * ns * 16;
    const bool issuer_warp = (wig == 0);

    if (issuer_warp && lane == 0) {
        for (int st = 0; st < ns; ++st) {
            mbar_init(bars + st * 16, 1);
            mbar_init(bars + st * 16 + 8, 1);
        }
        mbar_fence_init();
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
    }
    __syncthreads();
    grid_dependency_wait();       // the planner's output is read from here on

    // ---- this group's piece of the tile line
    const GroupStart gs = a.gstart[gid];
    const long long total_ll = a.gpos[gid + 1] - a.gpos[gid];
    const int total = (int)total_ll;
    if (total <= 0) return;   // whole group (all its warps) leaves together; no CTA-wide sync follows

    Cursor cc;                 // consume cursor
    cc.s = gs.s; cc.g = gs.g; cc.tau = gs.tau;
    cur_load(cc, a);
    Cursor ic = cc;            // issue cursor

    // ---- page-id prefetch state (issuer warp): 2 x 32 block-table entries in registers
    int bt_s = -1, bt_base = 0, bt_cur = 0, bt_nxt = 0;
    bool dead = false;         // set after a wait timed out: later waits are skipped

    const int P = a.P;
    const int tiles_per_page = P > kTile ? P / kTile : 1;

    auto page_id = [&](const Cursor &c, int pg) -> int {
        const int npages = (c.n + P - 1) / P;
        const int32_t *row = a.block_table + (size_t)c.s * a.max_pages;
        if (c.s != bt_s || pg < bt_base || pg >= bt_base + 64) {
            bt_s = c.s;
            bt_base = pg & ~31;
            const int i0 = bt_base + lane, i1 = bt_base + 32 + lane;
            bt_cur = i0 < npages ? __ldg(row + i0) : 0;
            bt_nxt = i1 < npages ? __ldg(row + i1) : 0;
        } else if (pg >= bt_base + 32) {
            bt_cur = bt_nxt;
            bt_base += 32;
            const int i1 = bt_base + 32 + lane;
            bt_nxt = i1 < npages ? __ldg(row + i1) : 0;
        }
        return __shfl_sync(FULL, bt_cur, pg - bt_base);
    };

    // Issue the TMA loads of the tile under the issue cursor into stage `st` (issuer warp only).
    auto issue_tile = [&](int st) {
        const uint32_t kdst = ring + (uint32_t)st * 2 * TB;
        const uint32_t vdst = kdst + TB;
        const uint32_t bk = bars + st * 16, bv = bk + 8;
        int ids[4];
        int nbox = 1, tok_off = 0;
        if (a.box_tok > 0) {
            // general path: boxes of box_tok <= min(P, 64) tokens; boxes that start at or past the end of
            // the sequence are not fetched (their rows are masked, and zero-filled for V, below)
            const int bt = a.box_tok;
            const int t0 = ic.tau * kTile;
            const int left = ic.n - t0;
            nbox = left >= kTile ? (kTile >> a.lg_box) : ((left + bt - 1) >> a.lg_box);
#pragma unroll
            for (int b = 0; b < 4; ++b) ids[b] = (b < nbox) ? page_id(ic, (t0 + b * bt) >> a.lg_page) : 0;
        } else {
            ids[0] = page_id(ic, ic.tau / tiles_per_page);
            tok_off = (ic.tau % tiles_per_page) * kTile;
        }
        if (a.box_tok == 0) {
            if (lane == 0) {
                // one instruction per tile and pool: box = 64 tokens x all halves
                const uint32_t bytes = (uint32_t)TB;
                mbar_expect_tx(bk, bytes);
                tma_load_5d(kdst, &tmK, 0, tok_off, 0, ic.g, ids[0], bk);
                mbar_expect_tx(bv, bytes);
                tma_load_5d(vdst, &tmV, 0, tok_off, 0, ic.g, ids[0], bv);
            }
        } else {
            // lane = (pool, box, half): every box of the tile goes out in one warp instruction
            const int bt = a.box_tok;
            const uint32_t bbytes = (uint32_t)bt * 128u;
            if (lane == 0) {
                const uint32_t bytes = (uint32_t)nbox * bbytes * HALVES;
                mbar_expect_tx(bk, bytes);
                mbar_expect_tx(bv, bytes);
            }
            __syncwarp();
            if (a.page_boxes) {
                // 16-token pages: lanes 0..7 = (pool, page of the tile); one 5-D box carries both halves of a
                // page, landing as [page][half][16 tokens][128 B]
                const int is_v = lane >> 2, b = lane & 3;
                if (lane < 8 && b < nbox) {
                    const int id = b == 0 ? ids[0] : (b == 1 ? ids[1] : (b == 2 ? ids[2] : ids[3]));
                    tma_load_5d((is_v ? vdst : kdst) + b * bbytes * HALVES, is_v ? (const void *)&tmV : (const void *)&tmK,
                                0, 0, 0, ic.g, id, is_v ? bv : bk);
                }
                return;
            }
            // lanes 0..7 = (pool, half, box parity): each issues boxes b and b + 2 of its pool and half,
            // so a tile of 32-token boxes goes out in one warp instruction
            const int is_v = lane >> 2, h = (lane >> 1) & 1, b0 = lane & 1;
            if (lane < 8 && h < HALVES) {
                const void *tm = is_v ? (const void *)&tmV : (const void *)&tmK;
                const uint32_t dst = (is_v ? vdst : kdst) + h * (kTile * 128);
                const uint32_t bar = is_v ? bv : bk;
#pragma unroll
                for (int x = 0; x < 2; ++x) {
                    const int b = b0 + 2 * x;
                    if (b < nbox) {
                        const int id = b0 ? (x ? ids[3] : ids[1]) : (x ? ids[2] : ids[0]);
                        const int off = (ic.tau * kTile + b * bt) & (P - 1);
                        const int c1 = a.tok_first ? off : ic.g;
                        const int c2 = a.tok_first ? ic.g : off;
                        tma_load_4d(dst + b * bbytes, tm, h * 64, c1, c2, id, bar);
                    }
                }
            }
        }
    };

    // ---- prologue: fill the ring
    int issued = 0;
    if (issuer_warp) {
        const int pre = total < ns ? total : ns;
        for (int st = 0; st < pre; ++st) {
            issue_tile(st);
            cur_advance(ic, a);
            ++issued;
        }
    }

    // ---- lane-constant pieces of the shared-memory addressing
    const int l7 = lane & 7;
    // K (non-transposed ldmatrix): matrices (tok 0-7, chunk c), (tok 8-15, c), (tok 0-7, c+1), (tok 8-15, c+1)
    const uint32_t k_row_off = (uint32_t)(l7 + ((lane >> 3) & 1) * 8) * 128u;
    const int k_chunk_l = lane >> 4;
    // V (transposed ldmatrix): matrices (tok 0-7, chunk c), (tok 0-7, c+1), (tok 8-15, c), (tok 8-15, c+1)
    const uint32_t v_row_off = (uint32_t)(l7 + (lane >> 4) * 8) * 128u;
    const int v_chunk_l = (lane >> 3) & 1;

    const int rowbase = wig * 8 * NT;
    const int qcol = 2 * (lane & 3);         // first of this lane's two columns inside an n-tile
    const int trow = lane >> 2;              // token (or dim) row inside an 8-row block

    int consumed = 0;                        // tiles consumed so far by this group
    int remaining = total;

    while (remaining > 0) {
        // ---------------- segment = run of tiles of one (s, g) pair
        const int s = cc.s, g = cc.g, tau0 = cc.tau, n = cc.n, tiles = cc.tiles;
        int seg = tiles - tau0;
        int chunk_idx = 0;
        if (a.mode == kModeChunks) {
            const int ct = div_up(tiles, a.num_splits[s]);
            chunk_idx = tau0 / ct;
            const int to_boundary = ct - tau0 % ct;
            if (to_boundary < seg) seg = to_boundary;
        }
        if (remaining < seg) seg = remaining;

        // Q^T fragments of this warp's rows (B operand: k = dim, n = row)
        uint32_t bq[NT][KK][2];
        int lim[NT][2];
#pragma unroll
        for (int j = 0; j < NT; ++j) {
            const int r = rowbase + 8 * j + trow;
            const bool valid = r < a.rows;
            const int t = valid ? r / a.G : 0, hl = valid ? r % a.G : 0;
            const uint16_t *qp = a.q + (((size_t)s * a.q_len + t) * a.Hq + (size_t)g * a.G + hl) * D + qcol;
#pragma unroll
            for (int kk = 0; kk < KK; ++kk) {
                bq[j][kk][0] = valid ? __ldg(reinterpret_cast<const uint32_t *>(qp + 16 * kk)) : 0u;
                bq[j][kk][1] = valid ? __ldg(reinterpret_cast<const uint32_t *>(qp + 16 * kk + 8)) : 0u;
            }
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int rc = rowbase + 8 * j + qcol + e;
                lim[j][e] = rc < a.rows ? n - a.q_len + rc / a.G : -1;   // last visible token index
            }
        }

        float m_run[NT][2], l_run[NT][2];
        float acc_o[MD][NT][4];
#pragma unroll
        for (int j = 0; j < NT; ++j) { m_run[j][0] = m_run[j][1] = -INFINITY; l_run[j][0] = l_run[j][1] = 0.f; }
#pragma unroll
        for (int md = 0; md < MD; ++md)
#pragma unroll
            for (int j = 0; j < NT; ++j) { acc_o[md][j][0] = acc_o[md][j][1] = acc_o[md][j][2] = acc_o[md][j][3] = 0.f; }

        for (int tau = tau0; tau < tau0 + seg; ++tau) {
            const int st = consumed % ns;
            const uint32_t parity = (uint32_t)(consumed / ns) & 1u;
            const uint32_t kbase = ring + (uint32_t)st * 2 * TB;
            const uint32_t vbase = kbase + TB;
            const uint32_t bk = bars + st * 16, bv = bk + 8;
            const int tok0 = tau * kTile;

            // ---------- S^T = K Q^T
            if (!dead && !mbar_wait_bounded(bk, parity, a.wait_cycles)) { dead = true; atomicExch(a.status, (int)TS_ERR_TIMEOUT); }
            float sacc[4][NT][4];
#pragma unroll
            for (int mi = 0; mi < 4; ++mi)
#pragma unroll
                for (int j = 0; j < NT; ++j) { sacc[mi][j][0] = sacc[mi][j][1] = sacc[mi][j][2] = sacc[mi][j][3] = 0.f; }
#pragma unroll
            for (int kk = 0; kk < KK; ++kk) {
                const int chunk = 2 * kk + k_chunk_l;
                const uint32_t col = (uint32_t)(((chunk & 7) ^ l7) << 4) + (uint32_t)(chunk >> 3) * (uint32_t)a.half_stride;
#pragma unroll
                for (int mi = 0; mi < 4; ++mi) {
                    uint32_t af[4];
                    ldsm_x4(af, kbase + mi * (uint32_t)a.blk_stride + k_row_off + col);
#pragma unroll
                    for (int j = 0; j < NT; ++j) mma_bf16_16816(sacc[mi][j], af, bq[j][kk][0], bq[j][kk][1]);
                }
            }

            // ---------- online softmax (per column = query row)
            const bool need_mask = tok0 + kTile - 1 > n - a.q_len;
            float mx[NT][2];
#pragma unroll
            for (int j = 0; j < NT; ++j) { mx[j][0] = mx[j][1] = -INFINITY; }
#pragma unroll
            for (int mi = 0; mi < 4; ++mi)
#pragma unroll
                for (int j = 0; j < NT; ++j)
#pragma unroll
                    for (int r = 0; r < 4; ++r) {
                        float x = sacc[mi][j][r] * a.scale_log2;
                        if (need_mask) {
                            const int tok = tok0 + 16 * mi + trow + ((r >> 1) << 3);
                            if (tok > lim[j][r & 1]) x = -INFINITY;
                        }
                        sacc[mi][j][r] = x;
                        mx[j][r & 1] = fmaxf(mx[j][r & 1], x);
                    }
            float alpha[NT][2], mref[NT][2];
            bool changed = false;
#pragma unroll
            for (int j = 0; j < NT; ++j)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    float v = mx[j][e];
                    v = fmaxf(v, __shfl_xor_sync(FULL, v, 4));
                    v = fmaxf(v, __shfl_xor_sync(FULL, v, 8));
                    v = fmaxf(v, __shfl_xor_sync(FULL, v, 16));
                    const float m_new = fmaxf(m_run[j][e], v);
                    mref[j][e] = (m_new == -INFINITY) ? 0.f : m_new;
                    alpha[j][e] = ex2(m_run[j][e] - mref[j][e]);     // m_run = -inf -> 0
                    changed |= (m_new != m_run[j][e]);
                    m_run[j][e] = m_new;
                    l_run[j][e] *= alpha[j][e];
                }
            if (__any_sync(FULL, changed)) {
#pragma unroll
                for (int md = 0; md < MD; ++md)
#pragma unroll
                    for (int j = 0; j < NT; ++j) {
                        acc_o[md][j][0] *= alpha[j][0]; acc_o[md][j][1] *= alpha[j][1];
                        acc_o[md][j][2] *= alpha[j][0]; acc_o[md][j][3] *= alpha[j][1];
                    }
            }
            // P^T fragments (B operand of the second MMA: k = token, n = row), bf16 hi + lo
            uint32_t bph[4][NT][2], bpl[4][NT][2];
#pragma unroll
            for (int mi = 0; mi < 4; ++mi)
#pragma unroll
                for (int j = 0; j < NT; ++j) {
                    float p[4];
#pragma unroll
                    for (int r = 0; r < 4; ++r) {
                        p[r] = ex2(sacc[mi][j][r] - mref[j][r & 1]);
                        l_run[j][r & 1] += p[r];
                    }
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        const uint32_t hi = pack_bf16x2(p[2 * hh], p[2 * hh + 1]);
                        const uint32_t lo = pack_bf16x2(p[2 * hh] - bf16lo_to_f32(hi), p[2 * hh + 1] - bf16hi_to_f32(hi));
                        bph[mi][j][hh] = movmatrix_trans(hi);
                        bpl[mi][j][hh] = movmatrix_trans(lo);
                    }
                }

            // ---------- O^T += V^T P^T
            if (!dead && !mbar_wait_bounded(bv, parity, a.wait_cycles)) { dead = true; atomicExch(a.status, (int)TS_ERR_TIMEOUT); }
            const int valid_tok = n - tok0;          // tokens of this tile that exist
            if (valid_tok < kTile) {
                // rows past the sequence end may hold anything (also NaN): zero them so that 0 * v = 0
                for (int r = valid_tok + (lane >> 3); r < kTile; r += 4)
#pragma unroll
                    for (int h = 0; h < HALVES; ++h) {
                        const uint32_t addr = vbase + h * (uint32_t)a.half_stride + (r >> 4) * (uint32_t)a.blk_stride + (r & 15) * 128 + l7 * 16;
                        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0u) : "memory");
                    }
                __syncwarp();
            }
#pragma unroll
            for (int md = 0; md < MD; ++md) {
                const int chunk = 2 * md + v_chunk_l;
                const uint32_t col = (uint32_t)(((chunk & 7) ^ l7) << 4) + (uint32_t)(chunk >> 3) * (uint32_t)a.half_stride;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    uint32_t af[4];
                    ldsm_x4_trans(af, vbase + ks * (uint32_t)a.blk_stride + v_row_off + col);
#pragma unroll
                    for (int j = 0; j < NT; ++j) {
                        mma_bf16_16816(acc_o[md][j], af, bph[ks][j][0], bph[ks][j][1]);
                        mma_bf16_16816(acc_o[md][j], af, bpl[ks][j][0], bpl[ks][j][1]);
                    }
                }
            }

            // ---------- release the stage and refill it
            if (valid_tok < kTile) fence_proxy_async_smem();
            if (WG == 1) __syncwarp(); else named_bar_sync(1 + grp, WG * 32);
            ++consumed;
            if (issuer_warp && issued < total) {
                issue_tile(st);
                cur_advance(ic, a);
                ++issued;
            }
        }

        // ---------------- epilogue of the segment
        const bool full_pair = (tau0 == 0 && seg == tiles);
        const bool write_final = (a.mode == kModeFree) && full_pair;
        size_t slot = 0;
        if (a.mode == kModeFree) slot = (size_t)2 * gid + (tau0 > 0 ? 0 : 1);
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                float l = l_run[j][e];
                l += __shfl_xor_sync(FULL, l, 4);
                l += __shfl_xor_sync(FULL, l, 8);
                l += __shfl_xor_sync(FULL, l, 16);
                const float inv = l > 0.f ? 1.f / l : 0.f;
                const int rc = rowbase + 8 * j + qcol + e;
                if (rc >= a.rows) continue;
                const int t = rc / a.G, hl = rc % a.G;
                const size_t row_th = ((size_t)s * a.q_len + t) * a.Hq + (size_t)g * a.G + hl;   // (s, t, h) flat
                if (write_final) {
                    uint16_t *op = a.out + row_th * D;
#pragma unroll
                    for (int md = 0; md < MD; ++md) {
                        const float v0 = acc_o[md][j][e] * inv, v1 = acc_o[md][j][2 + e] * inv;
                        const uint32_t pk = pack_bf16x2(v0, v1);
                        op[16 * md + trow] = (uint16_t)(pk & 0xffffu);
                        op[16 * md + trow + 8] = (uint16_t)(pk >> 16);
                    }
                } else {
                    float *po, *pl;
                    if (a.mode == kModeFree) {
                        po = a.part_o + (slot * a.rows + rc) * D;
                        pl = a.part_lse + slot * a.rows + rc;
                    } else {
                        const size_t rows_all = (size_t)a.q_len * a.Hq;
                        const size_t base = ((size_t)s * a.max_splits + chunk_idx) * rows_all + ((size_t)t * a.Hq + (size_t)g * a.G + hl);
                        po = a.part_o + base * D;
                        pl = a.part_lse + base;
                    }
#pragma unroll
                    for (int md = 0; md < MD; ++md) {
                        po[16 * md + trow] = acc_o[md][j][e] * inv;
                        po[16 * md + trow + 8] = acc_o[md][j][2 + e] * inv;
                    }
                    if (trow == 0) *pl = l > 0.f ? (m_run[j][e] + log2f(l)) * 0.6931471805599453f : -INFINITY;
                }
            }

        remaining -= seg;
        cc.tau += seg - 1;
        cur_advance(cc, a);
    }
    // After a timed-out wait the loop above ran on without waiting, so copies of the last tiles may still
    // be on their way into this CTA's shared memory: give each of them one more bounded wait before leaving.
    if (dead) {
        for (int t = total > ns ? total - ns : 0; t < total; ++t) {
            const uint32_t b = bars + (t % ns) * 16;
            const uint32_t par = (uint32_t)(t / ns) & 1u;
            mbar_wait_bounded(b, par, a.wait_cycles);
            mbar_wait_bounded(b + 8, par, a.wait_cycles);
        }
    }
}

}  // namespace ts

#include "ts_attn_tc.cuh"

namespace ts {

// ------------------------------------------------------------------------------------------------
// merge kernels
// ------------------------------------------------------------------------------------------------
// One warp merges one output row: `count` parts, part i at po + i*o_stride / pl + i*l_stride.
template <int D>
__device__ __forceinline__ void merge_row(const float *po, size_t o_stride, const float *pl, size_t l_stride,
                                          int count, uint16_t *out_row, int lane)
{
    constexpr int V = D / 32;     // floats per lane
    float M = -INFINITY;
    for (int i = 0; i < count; ++i) M = fmaxf(M, pl[(size_t)i * l_stride]);
    float acc[V];
#pragma unroll
    for (int v = 0; v < V; ++v) acc[v] = 0.f;
    float Wsum = 0.f;
    if (M != -INFINITY) {
        for (int i = 0; i < count; ++i) {
            const float lse = pl[(size_t)i * l_stride];
            if (lse == -INFINITY) continue;
            const float w = expf(lse - M);
            Wsum += w;
            const float *p = po + (size_t)i * o_stride + lane * V;
#pragma unroll
            for (int v = 0; v < V; ++v) acc[v] += w * p[v];
        }
    }
    const float inv = Wsum > 0.f ? 1.f / Wsum : 0.f;
    uint16_t *o = out_row + lane * V;
#pragma unroll
    for (int v = 0; v < V; v += 2) {
        const uint32_t pk = pack_bf16x2(acc[v] * inv, acc[v + 1] * inv);
        *reinterpret_cast<uint32_t *>(o + v) = pk;
    }
}

// Free mode: one CTA per group of the tile line.  CTA k merges the pair that straddles the end of
// group k's piece if that pair starts inside the piece (so every split pair is merged exactly once,
// by the group that holds its first part), and zero-fills the outputs of empty sequences k, k+NG, ...
// Pairs covered by a single group were written directly by the attention kernel.
template <int D>
__global__ void __launch_bounds__(1024)
ts_merge_free_kernel(const int32_t *__restrict__ cum_tiles, const GroupStart *__restrict__ gstart,
                     const long long *__restrict__ gpos, const float *__restrict__ part_o,
                     const float *__restrict__ part_lse, uint16_t *out, int B, int q_len, int Hq, int Hkv,
                     int NG, int per_row)
{
    grid_dependency_wait();       // partials and direct outputs of the attention kernel
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k_first = blockIdx.x;
    const int G = Hq / Hkv, rows = G * q_len;
    // ---- empty sequences: zeros
    for (int s0 = k_first; s0 < B; s0 += NG) {
        if (cum_tiles[s0 + 1] != cum_tiles[s0]) continue;
        uint32_t *o = reinterpret_cast<uint32_t *>(out + (size_t)s0 * q_len * Hq * D);
        for (int i = threadIdx.x; i < q_len * Hq * D / 2; i += blockDim.x) o[i] = 0u;
    }
    // ---- the pair cut by the end of this group's piece
    // (the planner left in nx.pad whether this group merges the pair, how far its parts reach, and whether
    //  any group is empty)
    const GroupStart nx = gstart[k_first + 1];
    if (nx.s >= B || nx.tau == 0) return;                  // the piece ends on a pair boundary
    const uint32_t info = (uint32_t)nx.pad;
    if (!(info & 0x80000000u)) return;                     // the pair started in an earlier group: merged there
    const int s = nx.s, g = nx.g;
    const int k_last = (int)(info & 0xffffu);
    const bool some_empty = (info & 0x40000000u) != 0;
    const int cnt = k_last - k_first + 1;
    // `per_row` warps share an output row of the pair: warp `sub` of them takes the parts sub, sub + per_row, ...
    // and the partial sums meet in shared memory.  (With one long sequence in the batch a pair is cut into
    // dozens of parts: one warp walking them in rounds of dependent loads took 35 us for 55 parts.)
    __shared__ float s_acc[32][D];
    __shared__ float s_w[32], s_m[32];
    const int nwarps = blockDim.x >> 5;
    const int slots = nwarps / per_row;                    // rows in flight at a time
    const int slot = warp / per_row, sub = warp % per_row;
    constexpr int V = D / 32;
    for (int r0 = 0; r0 < rows; r0 += slots) {
        const int r = r0 + slot;
        const bool active = r < rows && slot < slots;
        float acc[V];
#pragma unroll
        for (int v = 0; v < V; ++v) acc[v] = 0.f;
        float Wsum = 0.f;
        float M = -INFINITY;                               // largest log-sum-exp among this warp's parts
        if (active) {
            // parts: group k_first wrote slot 2k+1 (pair starts inside it); later groups wrote slot 2k
            // (pair started before them).  Groups whose piece of the tile line is empty (only when W < NG)
            // wrote nothing: a piece is empty exactly when its start equals the next group's.
            // This warp's parts are k_first + sub, + per_row, ...; lane i looks at the i-th of them (+ 32, ...),
            // so that their log-sum-exps come in with one round of loads, and the warp weighs its parts
            // against its own maximum: the warps of a row are put on a common scale when they meet.
            const int mine = (cnt - sub + per_row - 1) / per_row;            // parts of this warp
            for (int b0 = 0; b0 < mine; b0 += 32) {
                const int k = k_first + sub + (b0 + lane) * per_row;
                float lse = -INFINITY;
                if (b0 + lane < mine && (!some_empty || gpos[k] != gpos[k + 1]))
                    lse = part_lse[((size_t)2 * k + (k == k_first ? 1 : 0)) * rows + r];
                M = fmaxf(M, lse);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
            if (M != -INFINITY) {
                for (int b0 = 0; b0 < mine; b0 += 32) {
                    const int kl = k_first + sub + (b0 + lane) * per_row;
                    float wl = 0.f;
                    if (b0 + lane < mine && (!some_empty || gpos[kl] != gpos[kl + 1])) {
                        const float lse = part_lse[((size_t)2 * kl + (kl == k_first ? 1 : 0)) * rows + r];
                        wl = lse == -INFINITY ? 0.f : expf(lse - M);
                    }
                    const int nj = mine - b0 < 32 ? mine - b0 : 32;
#pragma unroll 4
                    for (int jj = 0; jj < nj; ++jj) {
                        const float w = __shfl_sync(0xffffffffu, wl, jj);
                        if (w == 0.f) continue;                       // empty group or empty part: not read
                        const int k = k_first + sub + (b0 + jj) * per_row;
                        const float *p = part_o + (((size_t)2 * k + (k == k_first ? 1 : 0)) * rows + r) * D + lane * V;
                        Wsum += w;
#pragma unroll
                        for (int v = 0; v < V; ++v) acc[v] += w * p[v];
                    }
                }
            }
        }
        if (per_row > 1) {                                 // CTA-uniform
            if (active && sub != 0) {
#pragma unroll
                for (int v = 0; v < V; ++v) s_acc[warp][lane * V + v] = acc[v];
                if (lane == 0) { s_w[warp] = Wsum; s_m[warp] = M; }
            }
            __syncthreads();
            if (active && sub == 0) {
                float Mall = M;
                for (int o = 1; o < per_row; ++o) Mall = fmaxf(Mall, s_m[warp + o]);
                if (Mall != -INFINITY) {
                    const float f0 = M == -INFINITY ? 0.f : expf(M - Mall);
                    Wsum *= f0;
#pragma unroll
                    for (int v = 0; v < V; ++v) acc[v] *= f0;
                    for (int o = 1; o < per_row; ++o) {
                        const float mo = s_m[warp + o];
                        if (mo == -INFINITY) continue;
                        const float f = expf(mo - Mall);
                        Wsum += f * s_w[warp + o];
#pragma unroll
                        for (int v = 0; v < V; ++v) acc[v] += f * s_acc[warp + o][lane * V + v];
                    }
                }
            }
        }
        if (active && sub == 0) {
            const int t = r / G, hl = r % G;
            uint16_t *orow = out + (((size_t)s * q_len + t) * Hq + (size_t)g * G + hl) * D;
            const float inv = Wsum > 0.f ? 1.f / Wsum : 0.f;
            uint16_t *o = orow + lane * V;
#pragma unroll
            for (int v = 0; v < V; v += 2) *reinterpret_cast<uint32_t *>(o + v) = pack_bf16x2(acc[v] * inv, acc[v + 1] * inv);
        }
        if (per_row > 1) __syncthreads();                  // the shared sums are free for the next rows
    }
}

// Caller-visible dense layout: one CTA (NW warps) per output row (s, t, h).  The splits of the row
// are dealt round robin to the warps (lanes across head_dim), four loads in flight per warp; the
// warps' partial sums are combined through shared memory.  NW = 16 when a row can have many parts
// (a hundred parts over 4 warps is a chain of seven dependent rounds of loads; over 16 warps two).
template <int D, int NW>
__global__ void __launch_bounds__(NW * 32)
ts_merge_dense_kernel(const float *__restrict__ part_o, const float *__restrict__ part_lse,
                      const int32_t *__restrict__ num_splits, uint16_t *out, int B, int rows_all, int max_splits)
{
    constexpr int V = D / 32;     // floats per lane
    __shared__ float s_max[NW];
    __shared__ float s_w[NW];
    __shared__ float s_acc[NW][D];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long row = blockIdx.x;
    const int s = (int)(row / rows_all), r = (int)(row % rows_all);
    int S = num_splits[s];
    if (S > max_splits) S = max_splits;
    if (S < 0) S = 0;
    const size_t o_stride = (size_t)rows_all * D, l_stride = (size_t)rows_all;
    const float *po = part_o + ((size_t)s * max_splits * rows_all + r) * D;
    const float *pl = part_lse + (size_t)s * max_splits * rows_all + r;
    // maximum of the log-sum-exps
    float M = -INFINITY;
    for (int i = threadIdx.x; i < S; i += NW * 32) M = fmaxf(M, pl[(size_t)i * l_stride]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    if (lane == 0) s_max[warp] = M;
    __syncthreads();
    M = s_max[0];
#pragma unroll
    for (int w = 1; w < NW; ++w) M = fmaxf(M, s_max[w]);
    float acc[V];
#pragma unroll
    for (int v = 0; v < V; ++v) acc[v] = 0.f;
    float Wsum = 0.f;
    if (M != -INFINITY) {
        for (int i0 = warp; i0 < S; i0 += 4 * NW) {
            float w[4];
            float x[4][V];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + NW * u;
                const float lse = i < S ? pl[(size_t)i * l_stride] : -INFINITY;
                w[u] = lse == -INFINITY ? 0.f : expf(lse - M);
                const float *p = po + (size_t)(i < S ? i : 0) * o_stride + lane * V;
#pragma unroll
                for (int v = 0; v < V; ++v) x[u][v] = w[u] != 0.f ? p[v] : 0.f;    // empty parts are not read into the sum
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                Wsum += w[u];
#pragma unroll
                for (int v = 0; v < V; ++v) acc[v] += w[u] * x[u][v];
            }
        }
    }
    if (lane == 0) s_w[warp] = Wsum;
#pragma unroll
    for (int v = 0; v < V; ++v) s_acc[warp][lane * V + v] = acc[v];
    __syncthreads();
    if (warp == 0) {
        float Wt = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) Wt += s_w[w];
        const float inv = Wt > 0.f ? 1.f / Wt : 0.f;
        uint16_t *o = out + (size_t)row * D + lane * V;
#pragma unroll
        for (int v = 0; v < V; v += 2) {
            const int d = lane * V + v;
            float a0 = 0.f, a1 = 0.f;
#pragma unroll
            for (int w = 0; w < NW; ++w) { a0 += s_acc[w][d]; a1 += s_acc[w][d + 1]; }
            *reinterpret_cast<uint32_t *>(o + v) = pack_bf16x2(a0 * inv, a1 * inv);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct WorkspaceLayout {
    size_t status, cum_tiles, gstart, gpos, part_lse, part_o, total;
};

static WorkspaceLayout layout_workspace(const ts_attn_params *p, bool with_partials)
{
    WorkspaceLayout w;
    const size_t rows = (size_t)(p->num_q_heads / p->num_kv_heads) * p->q_len;
    size_t off = 0;
    w.status = off; off += 256;
    w.cum_tiles = off; off = align_up(off + ((size_t)p->num_seqs + 1) * 4, 256);
    w.gstart = off; off = align_up(off + ((size_t)kMaxGroups + 1) * sizeof(GroupStart), 256);
    w.gpos = off; off = align_up(off + ((size_t)kMaxGroups + 1) * 8, 256);
    w.part_lse = off;
    if (with_partials) off = align_up(off + (size_t)2 * kMaxGroups * rows * 4, 256);
    w.part_o = off;
    if (with_partials) off = align_up(off + (size_t)2 * kMaxGroups * rows * p->head_dim * 4, 256);
    w.total = off;
    return w;
}

static int check_params(const ts_attn_params *p)
{
    if (!p) return TS_ERR_INVALID_ARG;
    if (p->num_seqs < 0 || p->q_len < 1 || p->num_q_heads < 1 || p->num_kv_heads < 1 || p->num_pages < 1 ||
        p->max_pages_per_seq < 1)
        return TS_ERR_INVALID_ARG;
    if (p->num_q_heads % p->num_kv_heads != 0) return TS_ERR_INVALID_ARG;
    if (p->kv_page_stride <= 0 || p->kv_token_stride <= 0 || p->kv_head_stride <= 0) return TS_ERR_INVALID_ARG;
    if (p->kv_page_stride % 8 || p->kv_token_stride % 8 || p->kv_head_stride % 8) return TS_ERR_INVALID_ARG;
    if (p->head_dim != 64 && p->head_dim != 128) return TS_ERR_UNSUPPORTED;
    if (p->page_size != 16 && p->page_size != 32 && p->page_size != 64 && p->page_size != 128) return TS_ERR_UNSUPPORTED;
    const long long rows = (long long)(p->num_q_heads / p->num_kv_heads) * p->q_len;
    if (rows > (p->head_dim == 128 ? kMaxRowsD128 : kMaxRows)) return TS_ERR_UNSUPPORTED;
    if (!(p->scale == p->scale) || isinf(p->scale)) return TS_ERR_INVALID_ARG;
    return TS_OK;
}

static bool misaligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

// box_tok = 0: one 5-D box per 64-token tile when the page holds a whole tile, else one 4-D box per page;
// box_tok > 0: 4-D boxes of that many tokens (must divide 64 and not exceed the page size).
static int make_tensor_map(CUtensorMap *tm, const void *pool, const ts_attn_params *p, int *tok_first, int box_tok_req,
                           bool page_boxes = false)
{
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return TS_ERR_CUDA;
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    CUresult r;
    if (page_boxes) {
        // 5-D with a box of one whole short page: (64 dims, page_size tokens, all halves) of one head, landing
        // in shared memory as [half][token][128 B]
        *tok_first = 1;
        const cuuint64_t halves = (cuuint64_t)p->head_dim / 64;
        cuuint64_t dims[5] = {64, (cuuint64_t)p->page_size, halves, (cuuint64_t)p->num_kv_heads, (cuuint64_t)p->num_pages};
        cuuint64_t strides[4] = {(cuuint64_t)p->kv_token_stride * 2, 128, (cuuint64_t)p->kv_head_stride * 2,
                                 (cuuint64_t)p->kv_page_stride * 2};
        cuuint32_t box[5] = {64, (cuuint32_t)p->page_size, (cuuint32_t)halves, 1, 1};
        r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(pool), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        return r == CUDA_SUCCESS ? TS_OK : TS_ERR_UNSUPPORTED;
    }
    if (p->page_size >= kTile && box_tok_req == 0) {
        // 5-D: (64 dims, token, 64-dim half, head, page).  One box = 64 tokens x all halves, laid out in
        // shared memory as [half][token][128 B]: a whole K or V tile per TMA instruction.
        *tok_first = 1;
        const cuuint64_t halves = (cuuint64_t)p->head_dim / 64;
        cuuint64_t dims[5] = {64, (cuuint64_t)p->page_size, halves, (cuuint64_t)p->num_kv_heads, (cuuint64_t)p->num_pages};
        cuuint64_t strides[4] = {(cuuint64_t)p->kv_token_stride * 2, 128, (cuuint64_t)p->kv_head_stride * 2,
                                 (cuuint64_t)p->kv_page_stride * 2};
        cuuint32_t box[5] = {64, (cuuint32_t)kTile, (cuuint32_t)halves, 1, 1};
        r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(pool), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        return r == CUDA_SUCCESS ? TS_OK : TS_ERR_UNSUPPORTED;
    }
    // 4-D (64 dims, then {token, head} by ascending stride, page), one box per (box_tok tokens, half)
    const bool tf = p->kv_token_stride <= p->kv_head_stride;
    *tok_first = tf ? 1 : 0;
    cuuint64_t dims[4], strides[3];
    cuuint32_t box[4];
    const cuuint32_t box_tok = box_tok_req > 0 ? (cuuint32_t)box_tok_req : (cuuint32_t)p->page_size;
    dims[0] = (cuuint64_t)p->head_dim;
    box[0] = 64;
    if (tf) {
        dims[1] = (cuuint64_t)p->page_size; strides[0] = (cuuint64_t)p->kv_token_stride * 2; box[1] = box_tok;
        dims[2] = (cuuint64_t)p->num_kv_heads; strides[1] = (cuuint64_t)p->kv_head_stride * 2; box[2] = 1;
    } else {
        dims[1] = (cuuint64_t)p->num_kv_heads; strides[0] = (cuuint64_t)p->kv_head_stride * 2; box[1] = 1;
        dims[2] = (cuuint64_t)p->page_size; strides[1] = (cuuint64_t)p->kv_token_stride * 2; box[2] = box_tok;
    }
    dims[3] = (cuuint64_t)p->num_pages; strides[2] = (cuuint64_t)p->kv_page_stride * 2; box[3] = 1;
    r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(pool), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? TS_OK : TS_ERR_UNSUPPORTED;
}

struct DeviceInfo {
    int sms = 0;
    int smem_optin = 0;
    int clock_khz = 0;
    bool ok = false;
};

static const DeviceInfo &device_info()
{
    static DeviceInfo info[64];
    static DeviceInfo bad;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return bad;
    DeviceInfo &d = info[dev];
    if (!d.ok) {
        if (cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return bad;
        if (cudaDeviceGetAttribute(&d.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return bad;
        if (cudaDeviceGetAttribute(&d.clock_khz, cudaDevAttrClockRate, dev) != cudaSuccess) d.clock_khz = 2000000;
        d.ok = d.sms > 0;
    }
    return d;
}

static int env_int(const char *name, int dflt)
{
    const char *v = getenv(name);
    if (!v || !*v) return dflt;
    return atoi(v);
}

template <int D, int NT, int WG>
static int launch_attn(const CUtensorMap &tk, const CUtensorMap &tv, AttnArgs &a, int sms, int smem_optin,
                       cudaStream_t stream, bool dry, int *ng_out)
{
    constexpr int TB = kTile * D * 2;
    // groups per CTA and stages per group: as much shared memory in flight as fits, at most 256 threads
    int ngrp = env_int("TS_ATTN_NGRP", WG == 1 ? 3 : (WG == 2 ? 3 : 2));
    if (ngrp * WG * 32 > 256) ngrp = 256 / (WG * 32);
    if (ngrp < 1) ngrp = 1;
    int ns = env_int("TS_ATTN_STAGES", 0);
    const int budget = smem_optin - 2048;
    if (ns <= 0) ns = budget / (ngrp * 2 * TB);
    if (ns > 8) ns = 8;
    while (ns > 1 && (size_t)ngrp * ns * 2 * TB + 1024 + (size_t)ngrp * ns * 16 > (size_t)budget) --ns;
    if (ns < 2) { ngrp = 1; ns = 2; }
    const size_t smem = (size_t)ngrp * ns * 2 * TB + (size_t)ngrp * ns * 16 + 1024;
    if (smem > (size_t)smem_optin) return TS_ERR_UNSUPPORTED;
    int grid = sms;
    const int grid_cap = env_int("TS_ATTN_GRID", 0);      // testing knob: fewer CTAs, longer pieces
    if (grid_cap > 0 && grid_cap < grid) grid = grid_cap;
    if ((long long)grid * ngrp > kMaxGroups) grid = kMaxGroups / ngrp;
    *ng_out = grid * ngrp;
    a.ngrp = ngrp;
    a.ns = ns;
    if (dry) return TS_OK;
    static bool attr_set[64] = {};      // per device: the attribute belongs to the device's copy of the kernel
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return TS_ERR_CUDA;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        if (cudaFuncSetAttribute(ts_attn_kernel<D, NT, WG>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) != cudaSuccess)
            return TS_ERR_CUDA;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    const cudaError_t e = launch_overlapped(ts_attn_kernel<D, NT, WG>, dim3(grid), dim3(ngrp * WG * 32), smem, stream,
                                            env_int("TS_PDL", 1) != 0, tk, tv, a);
    return e == cudaSuccess ? TS_OK : TS_ERR_CUDA;
}

// tcgen05 kernel: one CTA per SM, each CTA is one group of the tile line.
static int launch_attn_tc(const CUtensorMap &tk, const CUtensorMap &tv, AttnArgs &a, int sms, int smem_optin,
                          cudaStream_t stream, bool dry, int *ng_out)
{
    if ((size_t)smem_optin < tc::kSmemBytes) return TS_ERR_UNSUPPORTED;
    int grid = sms;
    const int grid_cap = env_int("TS_ATTN_GRID", 0);
    if (grid_cap > 0 && grid_cap < grid) grid = grid_cap;
    if (grid > kMaxGroups) grid = kMaxGroups;
    *ng_out = grid;
    a.ngrp = 1;
    a.ns = tc::kStages;
    if (dry) return TS_OK;
    static bool attr_set[64] = {};      // per device
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return TS_ERR_CUDA;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        if (cudaFuncSetAttribute(tc::ts_attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::kSmemBytes) != cudaSuccess)
            return TS_ERR_CUDA;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    const cudaError_t e = launch_overlapped(tc::ts_attn_tc_kernel, dim3(grid), dim3(tc::kThreads), tc::kSmemBytes, stream,
                                            env_int("TS_PDL", 1) != 0, tk, tv, a);
    return e == cudaSuccess ? TS_OK : TS_ERR_CUDA;
}

static bool use_tc_kernel(int D, int rows, float scale_log2)
{
    return D == 128 && rows >= env_int("TS_ATTN_TC_MIN_ROWS", 17) && rows <= 128 && scale_log2 > 0.f &&
           env_int("TS_ATTN_TC", 1) != 0;
}

template <int D>
static int dispatch_attn(int rows, const CUtensorMap &tk, const CUtensorMap &tv, AttnArgs &a, int sms, int smem_optin,
                         cudaStream_t stream, bool dry, int *ng)
{
    // more than two n-tiles of rows at head_dim 128 and a positive scale: tcgen05 path (up to 16 rows
    // the warp-MMA kernel measures faster: 88 vs 73 % of the HBM peak on the bulk lengths at 16 rows);
    // TS_ATTN_TC=0 keeps the warp-MMA path for any row count
    if (use_tc_kernel(D, rows, a.scale_log2))
        return launch_attn_tc(tk, tv, a, sms, smem_optin, stream, dry, ng);
    if (rows <= 8) return launch_attn<D, 1, 1>(tk, tv, a, sms, smem_optin, stream, dry, ng);
    if (rows <= 16) return launch_attn<D, 2, 1>(tk, tv, a, sms, smem_optin, stream, dry, ng);
    // 17..32 rows: two warps of two n-tiles each share a stage (70 % of the HBM peak on the bulk lengths at
    // 20 rows against 58 % for one warp of three n-tiles)
    if (rows <= 32) return launch_attn<D, 2, 2>(tk, tv, a, sms, smem_optin, stream, dry, ng);
    if (rows <= 48) return launch_attn<D, 3, 2>(tk, tv, a, sms, smem_optin, stream, dry, ng);
    if (rows <= 72) return launch_attn<D, 3, 3>(tk, tv, a, sms, smem_optin, stream, dry, ng);
    if (rows <= 96) return launch_attn<D, 3, 4>(tk, tv, a, sms, smem_optin, stream, dry, ng);
    return TS_ERR_UNSUPPORTED;
}

static void *g_ev_start = nullptr, *g_ev_stop = nullptr;   // optional timing events (benchmarks)

// Shared driver of the three attention entry points.
static int run_attention(const ts_attn_params *p, const void *q, const void *k_pool, const void *v_pool,
                         const int32_t *block_table, const int32_t *kv_lens, int mode, int max_splits, void *out,
                         float *part_o, float *part_lse, int32_t *num_splits, void *workspace, size_t workspace_bytes,
                         void *stream_v)
{
    int rc = check_params(p);
    if (rc != TS_OK) return rc;
    if (!q || !k_pool || !v_pool || !block_table || !kv_lens || !workspace) return TS_ERR_INVALID_ARG;
    if (misaligned(q) || misaligned(k_pool) || misaligned(v_pool) || misaligned(block_table) || misaligned(kv_lens) ||
        misaligned(workspace))
        return TS_ERR_INVALID_ARG;
    const bool free_mode = (mode == kModeFree);
    if (free_mode) {
        if (!out || misaligned(out)) return TS_ERR_INVALID_ARG;
    } else {
        if (!part_o || !part_lse || !num_splits || misaligned(part_o) || misaligned(part_lse) || misaligned(num_splits))
            return TS_ERR_INVALID_ARG;
        if (max_splits < 1 || max_splits > 4096) return TS_ERR_INVALID_ARG;
    }
    const WorkspaceLayout w = layout_workspace(p, free_mode);
    if (workspace_bytes < w.total) return TS_ERR_WORKSPACE;
    if (p->num_seqs == 0) return TS_OK;

    const DeviceInfo &dev = device_info();
    if (!dev.ok) return TS_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    uint8_t *ws = static_cast<uint8_t *>(workspace);

    // TMA box: the tcgen05 kernel takes a whole tile per instruction where the page allows it; the
    // warp-MMA kernel takes boxes of TS_ATTN_BOX_TOK tokens (0 = a whole tile per instruction too)
    const int rows_all = (p->num_q_heads / p->num_kv_heads) * p->q_len;
    const float scale_log2 = p->scale * 1.4426950408889634f;
    int box_tok = 0;
    if (!use_tc_kernel(p->head_dim, rows_all, scale_log2)) {
        // measured on the decode batches (one n-tile of rows): 32-token boxes, all issued by one warp
        // instruction, stream 3-5 % faster than one box per tile; with more rows the issuing warp's
        // extra instructions cost more than they gain
        box_tok = env_int("TS_ATTN_BOX_TOK", (rows_all <= 8 && p->head_dim == 128) ? 32 : 0);
        if (box_tok != 0 && box_tok != 16 && box_tok != 32 && box_tok != 64) box_tok = 0;
        if (box_tok > p->page_size || (box_tok == 0 && p->page_size < kTile)) box_tok = p->page_size;
    }
    // 16-token pages at head_dim 128 (warp-MMA kernel): one box per page carrying both halves -- 8 boxes of
    // 4 KB per tile instead of 16 of 2 KB (TS_ATTN_PAGE_BOXES=0 keeps the latter)
    const bool page_boxes = !use_tc_kernel(p->head_dim, rows_all, scale_log2) && p->page_size == 16 &&
                            p->head_dim == 128 && box_tok == 16 && env_int("TS_ATTN_PAGE_BOXES", 1) != 0;
    CUtensorMap tk, tv;
    int tok_first = 1, tf2 = 1;
    rc = make_tensor_map(&tk, k_pool, p, &tok_first, box_tok, page_boxes);
    if (rc != TS_OK) return rc;
    rc = make_tensor_map(&tv, v_pool, p, &tf2, box_tok, page_boxes);
    if (rc != TS_OK) return rc;

    AttnArgs a;
    a.q = static_cast<const uint16_t *>(q);
    a.out = static_cast<uint16_t *>(out);
    a.block_table = block_table;
    a.kv_lens = kv_lens;
    a.cum_tiles = reinterpret_cast<const int32_t *>(ws + w.cum_tiles);
    a.gstart = reinterpret_cast<const GroupStart *>(ws + w.gstart);
    a.gpos = reinterpret_cast<const long long *>(ws + w.gpos);
    a.part_o = free_mode ? reinterpret_cast<float *>(ws + w.part_o) : part_o;
    a.part_lse = free_mode ? reinterpret_cast<float *>(ws + w.part_lse) : part_lse;
    a.num_splits = num_splits;
    a.status = reinterpret_cast<int32_t *>(ws + w.status);
    a.B = p->num_seqs; a.q_len = p->q_len; a.Hq = p->num_q_heads; a.Hkv = p->num_kv_heads;
    a.G = p->num_q_heads / p->num_kv_heads; a.rows = a.G * p->q_len; a.P = p->page_size;
    a.max_pages = p->max_pages_per_seq; a.max_splits = max_splits; a.mode = mode;
    a.ngrp = 1; a.ns = 2; a.tok_first = tok_first;
    a.box_tok = box_tok;
    a.lg_page = 0;
    while ((1 << a.lg_page) < p->page_size) ++a.lg_page;
    a.lg_box = 0;
    while ((1 << a.lg_box) < box_tok) ++a.lg_box;
    a.page_boxes = page_boxes ? 1 : 0;
    a.blk_stride = page_boxes ? 16 * 128 * (p->head_dim / 64) : 16 * 128;
    a.half_stride = page_boxes ? 16 * 128 : kTile * 128;
    a.scale_log2 = scale_log2;
    a.wait_cycles = (long long)dev.clock_khz * 2000LL;   // about two seconds of SM clocks

    // first pass fixes the launch geometry (NG) without launching
    int NG = 0;
    rc = (p->head_dim == 128) ? dispatch_attn<128>(a.rows, tk, tv, a, dev.sms, dev.smem_optin, stream, true, &NG)
                              : dispatch_attn<64>(a.rows, tk, tv, a, dev.sms, dev.smem_optin, stream, true, &NG);
    if (rc != TS_OK) return rc;

    const int chunks_per_group = env_int("TS_SPLIT_CHUNKS_PER_GROUP", 16);
    {
        const bool overlap = env_int("TS_PDL", 1) != 0;
        const cudaError_t e = launch_overlapped(
            ts_plan_kernel, dim3(1), dim3(1024), 0, stream, overlap, kv_lens, a.B, a.Hkv, NG, mode, max_splits,
            chunks_per_group, reinterpret_cast<int32_t *>(ws + w.cum_tiles), reinterpret_cast<GroupStart *>(ws + w.gstart),
            reinterpret_cast<long long *>(ws + w.gpos), num_splits, reinterpret_cast<int32_t *>(ws + w.status), a.part_o,
            a.part_lse, p->q_len * p->num_q_heads, p->head_dim);
        if (e != cudaSuccess) return TS_ERR_CUDA;
    }
    if (cudaGetLastError() != cudaSuccess) return TS_ERR_CUDA;

    if (g_ev_start && g_ev_stop) cudaEventRecord(static_cast<cudaEvent_t>(g_ev_start), stream);
    rc = (p->head_dim == 128) ? dispatch_attn<128>(a.rows, tk, tv, a, dev.sms, dev.smem_optin, stream, false, &NG)
                              : dispatch_attn<64>(a.rows, tk, tv, a, dev.sms, dev.smem_optin, stream, false, &NG);
    if (rc != TS_OK) return rc;
    if (g_ev_start && g_ev_stop) cudaEventRecord(static_cast<cudaEvent_t>(g_ev_stop), stream);

    if (free_mode) {
        const bool overlap = env_int("TS_PDL", 1) != 0;
        const dim3 mgrid((unsigned)NG);
        // one warp per output row of a pair, as many as the pair has rows; when the tile line gives every
        // (sequence, kv-head) pair many pieces -- few, long sequences -- up to eight warps share a row
        int mwarps = a.rows < 4 ? 4 : (a.rows > 32 ? 32 : a.rows);
        const long long pairs = (long long)a.B * a.Hkv;
        int per_row = 1;
        if (env_int("TS_MERGE_PER_ROW", 0) > 0) per_row = env_int("TS_MERGE_PER_ROW", 0);
        else if ((long long)NG >= 4 * pairs) per_row = 8;
        while (per_row > 1 && (mwarps * per_row > 32 || a.rows > mwarps)) per_row >>= 1;
        mwarps *= per_row;
        const dim3 mblock((unsigned)mwarps * 32);
        cudaError_t e;
        if (p->head_dim == 128)
            e = launch_overlapped(ts_merge_free_kernel<128>, mgrid, mblock, 0, stream, overlap, a.cum_tiles, a.gstart,
                                  a.gpos, (const float *)a.part_o, (const float *)a.part_lse, a.out, a.B, a.q_len, a.Hq,
                                  a.Hkv, NG, per_row);
        else
            e = launch_overlapped(ts_merge_free_kernel<64>, mgrid, mblock, 0, stream, overlap, a.cum_tiles, a.gstart,
                                  a.gpos, (const float *)a.part_o, (const float *)a.part_lse, a.out, a.B, a.q_len, a.Hq,
                                  a.Hkv, NG, per_row);
        if (e != cudaSuccess) return TS_ERR_CUDA;
        if (cudaGetLastError() != cudaSuccess) return TS_ERR_CUDA;
    }
    return TS_OK;
}

}  // namespace ts

// ------------------------------------------------------------------------------------------------
// C ABI
// ------------------------------------------------------------------------------------------------
extern "C" {

size_t ts_attn_workspace_bytes(const ts_attn_params *p)
{
    if (ts::check_params(p) != TS_OK) return 0;
    return ts::layout_workspace(p, true).total;
}

size_t ts_splitkv_workspace_bytes(const ts_attn_params *p)
{
    if (ts::check_params(p) != TS_OK) return 0;
    return ts::layout_workspace(p, false).total;
}

int ts_decode_attn(const ts_attn_params *p, const void *q, const void *k_pool, const void *v_pool,
                   const int32_t *block_table, const int32_t *kv_lens, void *out, void *workspace,
                   size_t workspace_bytes, void *stream)
{
    if (p && p->q_len != 1) return TS_ERR_INVALID_ARG;
    return ts::run_attention(p, q, k_pool, v_pool, block_table, kv_lens, ts::kModeFree, 0, out, nullptr, nullptr,
                             nullptr, workspace, workspace_bytes, stream);
}

int ts_verify_attn(const ts_attn_params *p, const void *q, const void *k_pool, const void *v_pool,
                   const int32_t *block_table, const int32_t *kv_lens, void *out, void *workspace,
                   size_t workspace_bytes, void *stream)
{
    return ts::run_attention(p, q, k_pool, v_pool, block_table, kv_lens, ts::kModeFree, 0, out, nullptr, nullptr,
                             nullptr, workspace, workspace_bytes, stream);
}

int ts_decode_attn_splitkv(const ts_attn_params *p, const void *q, const void *k_pool, const void *v_pool,
                           const int32_t *block_table, const int32_t *kv_lens, int32_t max_splits, float *partial_o,
                           float *partial_lse, int32_t *num_splits, void *workspace, size_t workspace_bytes,
                           void *stream)
{
    return ts::run_attention(p, q, k_pool, v_pool, block_table, kv_lens, ts::kModeChunks, max_splits, nullptr,
                             partial_o, partial_lse, num_splits, workspace, workspace_bytes, stream);
}

int ts_lse_merge(const ts_attn_params *p, int32_t max_splits, const float *partial_o, const float *partial_lse,
                 const int32_t *num_splits, void *out, void *stream)
{
    if (!p || !partial_o || !partial_lse || !num_splits || !out) return TS_ERR_INVALID_ARG;
    if (p->num_seqs < 0 || p->q_len < 1 || p->num_q_heads < 1 || max_splits < 1) return TS_ERR_INVALID_ARG;
    if (p->head_dim != 64 && p->head_dim != 128) return TS_ERR_UNSUPPORTED;
    if (ts::misaligned(partial_o) || ts::misaligned(partial_lse) || ts::misaligned(num_splits) || ts::misaligned(out))
        return TS_ERR_INVALID_ARG;
    if (p->num_seqs == 0) return TS_OK;
    const int rows_all = p->q_len * p->num_q_heads;
    const long long rows = (long long)p->num_seqs * rows_all;
    if (rows > 0x7fffffffLL) return TS_ERR_UNSUPPORTED;
    const unsigned grid = (unsigned)rows;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint16_t *o = static_cast<uint16_t *>(out);
    const bool wide = max_splits > 32;          // many parts per row: 16 warps share them
    if (p->head_dim == 128) {
        if (wide) ts::ts_merge_dense_kernel<128, 16><<<grid, 512, 0, s>>>(partial_o, partial_lse, num_splits, o, p->num_seqs, rows_all, max_splits);
        else ts::ts_merge_dense_kernel<128, 4><<<grid, 128, 0, s>>>(partial_o, partial_lse, num_splits, o, p->num_seqs, rows_all, max_splits);
    } else {
        if (wide) ts::ts_merge_dense_kernel<64, 16><<<grid, 512, 0, s>>>(partial_o, partial_lse, num_splits, o, p->num_seqs, rows_all, max_splits);
        else ts::ts_merge_dense_kernel<64, 4><<<grid, 128, 0, s>>>(partial_o, partial_lse, num_splits, o, p->num_seqs, rows_all, max_splits);
    }
    return cudaGetLastError() == cudaSuccess ? TS_OK : TS_ERR_CUDA;
}

int ts_set_attn_timing_events(void *start_event, void *stop_event)
{
    ts::g_ev_start = start_event;
    ts::g_ev_stop = stop_event;
    return TS_OK;
}

const char *ts_status_string(int status)
{
    switch (status) {
    case TS_OK: return "TS_OK";
    case TS_ERR_INVALID_ARG: return "TS_ERR_INVALID_ARG";
    case TS_ERR_UNSUPPORTED: return "TS_ERR_UNSUPPORTED";
    case TS_ERR_WORKSPACE: return "TS_ERR_WORKSPACE";
    case TS_ERR_CUDA: return "TS_ERR_CUDA";
    case TS_ERR_TIMEOUT: return "TS_ERR_TIMEOUT";
    default: return "TS_ERR_UNKNOWN";
    }
}

}  // extern "C"
