// Verify-attention kernel on the 5th-generation tensor cores (tcgen05 + TMEM), head_dim 128.
//
// Used when the (GQA group x q_len) tile of a (sequence, kv head) pair has more than 16 rows (and at
// most 128), i.e. for speculative verification.  The warp-level MMA path tops out at ~550 TFLOP/s on this GPU, which
// is less than a 68-row tile needs to keep up with HBM; tcgen05.mma has about three times that.
//
// One CTA per SM = one "group" of the planner's tile line.  Roles:
//   warp 0      TMA producer: K/V tiles (64 tokens) into a 6-stage shared-memory ring
//   warp 1      first MMA issuer (one lane):   S[M x 64]  = Q[M x 128] . K^T   (8 x N64 K16)
//   warp 2      second MMA issuer (one lane):  O[M x 128] += P[M x 64] . V      (8 x N128 K16,
//               P as bf16 hi and lo).  Issuing one tcgen05.mma costs a thread 60-100 cycles here, more
//               than these small MMAs take to execute, so the two kinds are issued by different threads.
//               M = 64 when the pair has at most 64 rows (half of the tensor datapath then idles: the
//               kernel is power-bound when it runs for long), else 128.
//   warps 3..6, 7..10  two softmax warpgroups, one thread per query row (TMEM lane) each; group w
//               takes the tiles of parity w: S is read from TMEM, masked, exponentiated; each group
//               has its own O accumulator in TMEM, kept there for the whole segment and rescaled
//               only when a row's running maximum grows by more than 2^8 (lazy rescale), so the
//               common tile costs no TMEM round trip for O.  The two accumulators are merged by
//               their (max, sum) statistics at the end of the segment by group 0, while group 1 fetches
//               the next pair's Q tile.  A warp without a valid row only keeps step with the barriers.
// There are four S/P buffers (two per softmax group): the first MMA runs up to four tiles ahead of the
// second, so each softmax group finds its next scores ready when it finishes a tile.  P overwrites
// S in TMEM and is the A operand of the second MMA from there.  Every mbarrier wait is bounded.
#pragma once

namespace ts {
namespace tc {

#ifndef TS_TC_STAGES
#define TS_TC_STAGES 6
#endif
constexpr int kStages = TS_TC_STAGES;
constexpr int kThreads = 352;          // TMA warp, two MMA-issuing warps, two softmax warpgroups of 4 warps
constexpr uint32_t kQBytes = 32768;          // 2 halves x 128 rows x 128 B
constexpr uint32_t kStageBytes = 32768;      // K 16 KB + V 16 KB
constexpr uint32_t kOffQ = 0;
constexpr uint32_t kOffStage = kOffQ + kQBytes;
constexpr uint32_t kOffBar = kOffStage + kStages * kStageBytes;
constexpr uint32_t kOffStats = kOffBar + 384;            // 128 x (m, l) of the second softmax warpgroup
constexpr uint32_t kSmemBytes = kOffStats + 1024 + 1024;  // + alignment slack
constexpr uint32_t kTmemCols = 512;          // four S/P buffers (64 each) + O0, O1 (128 each)
constexpr uint32_t kTmemO = 256;             // first column of O0
constexpr float kLazyTau = 8.0f;             // log2 units

// ------------------------------------------------------------------ tcgen05 wrappers
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Same with the A operand read from TMEM (rows = lanes, two bf16 along K per 32-bit column).
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]),
          "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(taddr)
        : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle.  K-major operands: `sbo` = bytes between 8-row
// groups, `lbo` unused.  MN-major operands: `lbo` = bytes between 64-element groups along M/N,
// `sbo` = bytes between 8-row groups along K.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr, uint32_t lbo, uint32_t sbo)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffffu) >> 4);
    d |= (uint64_t)((lbo >> 4) & 0x3fffu) << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3fffu) << 32;
    d |= (uint64_t)1 << 46;     // descriptor version of this architecture
    d |= (uint64_t)2 << 61;     // 128-byte swizzle
    return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, M x N tile, A K-major, B K- or MN-major.
__host__ __device__ constexpr uint32_t idesc_bf16(int M, int N, int b_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}

// Optional phase timing of one softmax thread (CTA 0, first warp of each group): build with
// -DTS_TC_TRACE; sums of SM clock cycles land in the 16 x 8-byte words after the status word.
#ifdef TS_TC_TRACE
// absolute timestamps of pipeline events of tiles 200..207 of CTA 0 (event e of tile t at ev[(t-200)*8 + e])
#define TS_EVENT(t, e) { if (blockIdx.x == 0 && (t) >= 200 && (t) < 208) reinterpret_cast<long long *>(a.part_o)[((t) - 200) * 16 + (e)] = clock64(); }
#define TS_TRACE_DECL long long tr_t = clock64(), tr_acc[6] = {0, 0, 0, 0, 0, 0};
#define TS_TRACE(i) { const long long tr_n = clock64(); tr_acc[i] += tr_n - tr_t; tr_t = tr_n; }
#else
#define TS_EVENT(t, e) {}
#define TS_TRACE_DECL
#define TS_TRACE(i) {}
#endif

struct Segment {
    int s, g, tau0, n, tiles, len, chunk_idx;
};

// The run of tiles of one (s, g) pair that starts at the cursor (same rule in every role).
__device__ __forceinline__ Segment segment_at(const Cursor &cc, int remaining, const AttnArgs &a)
{
    Segment sg;
    sg.s = cc.s; sg.g = cc.g; sg.tau0 = cc.tau; sg.n = cc.n; sg.tiles = cc.tiles; sg.chunk_idx = 0;
    int len = cc.tiles - cc.tau;
    if (a.mode == kModeChunks) {
        const int ct = div_up(cc.tiles, a.num_splits[cc.s]);
        sg.chunk_idx = cc.tau / ct;
        const int to_boundary = ct - cc.tau % ct;
        if (to_boundary < len) len = to_boundary;
    }
    if (remaining < len) len = remaining;
    sg.len = len;
    return sg;
}

__global__ void __launch_bounds__(kThreads, 1)
ts_attn_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const AttnArgs a)
{
    constexpr uint32_t FULL = 0xffffffffu;
    constexpr int D = 128;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gid = blockIdx.x;
    // Up to 64 rows per pair the MMAs are issued with M = 64: half of the tensor datapath stays idle, which
    // is what the sustained speed of this power-bound kernel turns on.  An M = 64 tile keeps row 16 j + i
    // (i < 16) in TMEM lane 32 j + i, accumulators and the P operand alike.
    const bool m64 = a.rows <= 64;

    // barrier addresses
    const uint32_t bar0 = base + kOffBar;
    auto kfull = [&](int st) { return bar0 + 8u * st; };
    auto vfull = [&](int st) { return bar0 + 8u * (kStages + st); };
    auto kvfree = [&](int st) { return bar0 + 8u * (2 * kStages + st); };
    const uint32_t bsf = bar0 + 8u * (3 * kStages);
    auto sfull = [&](int b) { return bsf + 8u * b; };            // per S/P buffer (4)
    auto pfull = [&](int b) { return bsf + 8u * (4 + b); };      // per S/P buffer (4)
    const uint32_t qfull = bsf + 8u * 10;
    auto pdone = [&](int b) { return bsf + 8u * (11 + b); };     // per S/P buffer (4): its PV has finished
    const uint32_t tmem_slot = bsf + 8u * 15;

    grid_dependency_wait();      // the planner's output is read from here on
    const GroupStart gs = a.gstart[gid];
    const int total = (int)(a.gpos[gid + 1] - a.gpos[gid]);
    if (total <= 0) return;      // whole CTA leaves together, before anything is allocated

    if (warp == 0 && lane == 0) {
        for (int st = 0; st < kStages; ++st) { mbar_init(kfull(st), 1); mbar_init(vfull(st), 1); mbar_init(kvfree(st), 1); }
        for (int b = 0; b < 4; ++b) { mbar_init(sfull(b), 1); mbar_init(pfull(b), 4); mbar_init(pdone(b), 1); }
        mbar_init(qfull, 4);
        mbar_fence_init();
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
        fence_before_sync();
    }
    __syncthreads();
    fence_after_sync();
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

    bool dead = false;
    auto wait = [&](uint32_t bar, uint32_t parity) {
        if (!dead && !mbar_wait_bounded(bar, parity, a.wait_cycles)) { dead = true; atomicExch(a.status, (int)TS_ERR_TIMEOUT); }
    };

    Cursor cc;
    cc.s = gs.s; cc.g = gs.g; cc.tau = gs.tau;
    cur_load(cc, a);

    if (warp == 0) {
        // ============================================================ TMA producer
        // Kept free of integer divisions and long dependent chains: this warp has to issue one tile
        // (4 tensor loads) every ~1000 cycles to stay ahead of the tensor pipe.
        Cursor ic = cc;
        int bt_s = -1, bt_base = 0, bt_cur = 0, bt_nxt = 0;
        const int P = a.P;
        const int lgP = 31 - __clz(P);                    // page sizes are powers of two
        const int box_tok = P < kTile ? P : kTile;
        const uint32_t box_bytes = (uint32_t)box_tok * 128u;
        auto page_id = [&](const Cursor &c, int npages, int pg) -> int {
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
        int st = 0;
        TS_TRACE_DECL
        uint32_t free_par = 0;                            // parity of the kvfree phase to wait for (from the 2nd lap on)
        for (int it = 0; it < total; ++it) {
            TS_TRACE(0)
            if (it >= kStages) wait(kvfree(st), free_par);
            TS_TRACE(1)
            const uint32_t kdst = base + kOffStage + (uint32_t)st * kStageBytes;
            const int npages = (ic.n + P - 1) >> lgP;
            int ids[4];
            int nbox = 1, tok_off = 0;
            if (P < kTile) {
                const int sh = 6 - lgP;                   // pages per tile = 1 << sh
                const int first = ic.tau << sh;
                nbox = npages - first < (1 << sh) ? npages - first : (1 << sh);
#pragma unroll
                for (int b = 0; b < 4; ++b) ids[b] = (b < nbox) ? page_id(ic, npages, first + b) : 0;
            } else {
                const int sh = lgP - 6;                   // tiles per page = 1 << sh
                ids[0] = page_id(ic, npages, ic.tau >> sh);
                tok_off = (ic.tau & ((1 << sh) - 1)) << 6;
            }
            TS_TRACE(2)
            const uint32_t bytes = (P >= kTile) ? 16384u : (uint32_t)nbox * box_bytes * 2;
            if (lane == 0) {
                TS_EVENT(it, 7)
                mbar_expect_tx(kfull(st), bytes);
                mbar_expect_tx(vfull(st), bytes);
            }
            __syncwarp();
            TS_TRACE(3)
            if (P >= kTile) {
                // lanes 0 and 1: one instruction per pool, a whole 64-token tile (both halves) each
                if (lane < 2) {
                    const void *tm = lane ? (const void *)&tmV : (const void *)&tmK;
                    tma_load_5d(kdst + (lane ? 16384u : 0u), tm, 0, tok_off, 0, ic.g, ids[0], lane ? vfull(st) : kfull(st));
                }
            } else if (lane < 4) {
                // short pages: lanes 0..3 = (K, dims 0-63), (K, 64-127), (V, 0-63), (V, 64-127), one box per page
                const int c1 = a.tok_first ? 0 : ic.g;
                const int c2 = a.tok_first ? ic.g : 0;
                const bool is_v = lane >= 2;
                const int h = lane & 1;
                const void *tm = is_v ? (const void *)&tmV : (const void *)&tmK;
                const uint32_t bar = is_v ? vfull(st) : kfull(st);
                const uint32_t dst = kdst + (is_v ? 16384u : 0u) + (uint32_t)h * 8192u;
#pragma unroll
                for (int b = 0; b < 4; ++b)
                    if (b < nbox) tma_load_4d(dst + b * box_bytes, tm, h * 64, c1, c2, ids[b], bar);
            }
            TS_TRACE(4)
            cur_advance(ic, a);
            if (++st == kStages) { st = 0; if (it >= kStages) free_par ^= 1u; }
            TS_TRACE(5)
        }
        // After a timed-out wait this warp went on issuing without waiting: give the copies of the last
        // tiles one more bounded wait each, so that none is still writing shared memory when the CTA leaves.
        if (dead) {
            for (int t = total > kStages ? total - kStages : 0; t < total; ++t) {
                mbar_wait_bounded(kfull(t % kStages), (uint32_t)(t / kStages) & 1u, a.wait_cycles);
                mbar_wait_bounded(vfull(t % kStages), (uint32_t)(t / kStages) & 1u, a.wait_cycles);
            }
        }
#ifdef TS_TC_TRACE
        if (blockIdx.x == 0 && lane == 0) {
            long long *dbg = reinterpret_cast<long long *>(a.part_o) + 128;
            for (int i = 0; i < 6; ++i) dbg[i] = tr_acc[i];
            dbg[6] = total;
        }
#endif
    } else if (warp == 1) {
        // ============================================================ first MMA issuer: S = Q . K^T
        if (lane == 0) {
            const uint32_t idesc_qk = m64 ? idesc_bf16(64, 64, 0) : idesc_bf16(128, 64, 0);
            const uint64_t dk = smem_desc_sw128(0, 16, 1024);          // K-major operands (Q, K tile)
            const uint32_t q_lo = ((base + kOffQ) & 0x3ffffu) >> 4;
            int t = 0, remaining = total, seg_no = 0, st = 0;
            uint32_t st_par = 0;
            TS_TRACE_DECL
            while (remaining > 0) {
                const Segment sg = segment_at(cc, remaining, a);
                wait(qfull, (uint32_t)seg_no & 1u);
                for (int j = 0; j < sg.len; ++j, ++t) {
                    // tile t uses S/P buffer 2*(t&1) + ((t>>1)&1); each buffer turns over every 4 tiles
                    const int buf = ((t & 1) << 1) | ((t >> 1) & 1);
                    TS_TRACE(0)
                    if (t >= 4) wait(pdone(buf), (uint32_t)((t >> 2) - 1) & 1u);   // P of tile t-4 has been consumed
                    TS_EVENT(t, 2)
                    wait(kfull(st), st_par);
                    fence_after_sync();
                    TS_TRACE(1)
                    TS_EVENT(t, 0)
                    const uint32_t k_lo = ((base + kOffStage + (uint32_t)st * kStageBytes) & 0x3ffffu) >> 4;
                    const uint32_t s_tmem = tmem_base + (uint32_t)buf * 64;
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        const uint64_t ad = dk | (uint64_t)(q_lo + (kk >> 2) * (16384 >> 4) + (kk & 3) * 2);
                        const uint64_t bd = dk | (uint64_t)(k_lo + (kk >> 2) * (8192 >> 4) + (kk & 3) * 2);
                        umma_bf16(s_tmem, ad, bd, idesc_qk, kk == 0 ? 0u : 1u);
                    }
                    umma_commit(sfull(buf));
                    TS_TRACE(2)
                    TS_EVENT(t, 1)
                    if (++st == kStages) { st = 0; st_par ^= 1u; }
                }
                remaining -= sg.len;
                cc.tau += sg.len - 1;
                cur_advance(cc, a);
                ++seg_no;
            }
#ifdef TS_TC_TRACE
            if (blockIdx.x == 0) {
                long long *dbg = reinterpret_cast<long long *>(a.status) + 25;
                for (int i = 0; i < 6; ++i) dbg[i] = tr_acc[i];
                dbg[6] = total;
            }
#endif
        }
        __syncwarp();
    } else if (warp == 2) {
        // ============================================================ second MMA issuer: O += P . V
        if (lane == 0) {
            const uint32_t idesc_pv = m64 ? idesc_bf16(64, 128, 1) : idesc_bf16(128, 128, 1);
            const uint64_t dv = smem_desc_sw128(0, 8192, 1024);        // MN-major operand (V tile)
            int t = 0, remaining = total, st = 0;
            uint32_t st_par = 0;
            TS_TRACE_DECL
            while (remaining > 0) {
                const Segment sg = segment_at(cc, remaining, a);
                for (int j = 0; j < sg.len; ++j, ++t) {
                    const int w = t & 1, buf = (w << 1) | ((t >> 1) & 1);
                    TS_TRACE(0)
                    wait(pfull(buf), (uint32_t)(t >> 2) & 1u);
                    TS_TRACE(3)
                    TS_EVENT(t, 5)
                    wait(vfull(st), st_par);
                    fence_after_sync();
                    TS_TRACE(4)
                    const uint32_t p_tmem = tmem_base + (uint32_t)buf * 64;       // P overwrote S in place
                    const uint32_t v_lo = ((base + kOffStage + (uint32_t)st * kStageBytes + 16384) & 0x3ffffu) >> 4;
                    const uint32_t o_tmem = tmem_base + kTmemO + (uint32_t)w * 128;
                    const bool first = j < 2;                 // tiles 0 and 1 of a segment start O0 / O1 afresh
#pragma unroll
                    for (int part = 0; part < 2; ++part)      // hi (columns 0..31), then lo (32..63)
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {
                            const uint64_t bd = dv | (uint64_t)(v_lo + ks * (2048 >> 4));
                            umma_bf16_ts(o_tmem, p_tmem + part * 32 + ks * 8, bd, idesc_pv, (first && part == 0 && ks == 0) ? 0u : 1u);
                        }
                    umma_commit(pdone(buf));
                    umma_commit(kvfree(st));
                    TS_TRACE(5)
                    TS_EVENT(t, 6)
                    if (++st == kStages) { st = 0; st_par ^= 1u; }
                }
                remaining -= sg.len;
                cc.tau += sg.len - 1;
                cur_advance(cc, a);
            }
#ifdef TS_TC_TRACE
            if (blockIdx.x == 0) {
                long long *dbg = reinterpret_cast<long long *>(a.status) + 2 + 16;
                for (int i = 0; i < 6; ++i) dbg[i] = tr_acc[i];
                dbg[6] = total;
            }
#endif
        }
        __syncwarp();
    } else {
        // ============================================================ softmax warpgroups (one thread per row)
        const int wg = (warp - 3) >> 2;                   // 0 or 1: parity of the tiles this group takes
        // A warp reaches the 32 TMEM lanes of its quarter q4 = warp % 4 only, and warp % 4 is also the SM
        // sub-partition (scheduler) it issues from.  Sub-partition 3 hosts no single-thread role, 0 the TMA
        // producer, 2 the PV issuer, 1 the QK issuer, so the 32-row blocks of a pair are handed to the
        // quarters in that order: with few rows the busy softmax warps stay off the MMA issuers' schedulers.
        const int q4 = warp & 3;
        const int blk = (0x0231 >> (4 * q4)) & 3;         // quarter 3 -> first block of rows, then 0, 2, 1
        const int per_q = m64 ? 16 : 32;                  // rows of the MMA tile per quarter
        const bool lane_used = lane < per_q;
        // row of the MMA tile (= row of the Q tile in shared memory) behind this thread's TMEM lane; the
        // unused upper lanes of an M = 64 quarter get indices past the tile (scratch slots, never a tile row)
        const int mrow = lane_used ? q4 * per_q + lane : 64 + q4 * 16 + (lane - 16);
        const int row = blk * per_q + lane;               // query row of the pair that lives there
        const uint32_t tlane = (uint32_t)(q4 * 32) << 16;
        const bool row_valid = lane_used && row < a.rows;
        const int t_row = row_valid ? row / a.G : 0, hl = row_valid ? row % a.G : 0;
        const int tid_wg = (threadIdx.x - 96) & 127;      // 0..127 inside the group
        // A warp none of whose 32 rows exists has nothing to compute: its rows of Q are zeros, so its rows of
        // S are zeros (or NaN under a poisoned key), which is all the P those rows need -- nobody reads their
        // O.  It only keeps step with the barriers.  At 20 rows (gamma 4) that is 3 of a group's 4 warps.
        const bool idle_warp = blk * per_q >= a.rows;
        const uint32_t o_col = kTmemO + (uint32_t)wg * 128u;
        const uint32_t stats = base + kOffStats + (uint32_t)mrow * 8u;
        // This group's PVs are numbered u = it >> 1; PV u signals pdone of buffer 2*wg + (u & 1), phase u >> 1.
        // A parity wait only tells the current phase from the previous one, so the phases of each of the two
        // barriers are observed in order, and PV u - 2 (the previous phase of the barrier PV u will signal) is
        // observed before P of tile u is released: PV u cannot complete earlier.  That is all the common tile
        // waits for: its P is released while PV u - 1 may still be running (the tensor core accumulates in
        // issue order).  Only a rescale of O, and the end of a segment, wait for every PV issued so far.
        int seen = 0;                                     // PVs of this group observed so far
        auto observe_upto = [&](int u_target) {
            while (seen <= u_target) {
                wait(pdone((wg << 1) | (seen & 1)), (uint32_t)(seen >> 1) & 1u);
                ++seen;
            }
        };
        // Q tile of pair (s_, g_) -> shared memory (K-major, 128-byte swizzle; rows past the tile are
        // zero-filled): this thread's row, as asynchronous 16-byte copies.
        auto issue_q = [&](int s_, int g_) {
            const uint16_t *src = a.q + (((size_t)s_ * a.q_len + t_row) * a.Hq + (size_t)g_ * a.G + hl) * D;
            const uint32_t qrow = base + kOffQ + (uint32_t)mrow * 128u;
            if (!lane_used) return;                          // M = 64: the upper lanes of a quarter own no tile row
            const uint32_t nbytes = row_valid ? 16u : 0u;
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                const uint32_t addr = qrow + (uint32_t)(c >> 3) * 16384u + (uint32_t)(((c & 7) ^ (mrow & 7)) << 4);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(addr), "l"(src + 8 * c), "r"(nbytes) : "memory");
            }
        };
        // The copies of this thread have landed; make them visible to the tensor core and count the warp in.
        auto publish_q = [&]() {
            asm volatile("cp.async.wait_all;" ::: "memory");
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(qfull);
        };
        int it0 = 0, remaining = total, seg_no = 0;
        if (wg == 1 && remaining > 0) {
            const Segment s0 = segment_at(cc, remaining, a);
            issue_q(s0.s, s0.g);
            publish_q();
        }
        TS_TRACE_DECL
        while (remaining > 0) {
            const Segment sg = segment_at(cc, remaining, a);
            const bool has_next = remaining > sg.len;
            // Group 1 owns the Q tile: it fetches the next pair's while group 0 writes this pair's result.
            Cursor nc = cc;
            if (wg == 1 && has_next) {
                nc.tau += sg.len - 1;
                cur_advance(nc, a);
            }
            // Group 1 may not hand the first P of a new segment to the PV issuer (which overwrites O1)
            // before group 0 has read O1 of the previous segment: named barrier 3.
            bool need_o_sync = (wg == 1 && seg_no > 0);
            float m_used = -INFINITY, l_sum = 0.f;
            const int lim = row_valid ? sg.n - a.q_len + t_row : -1;
            int last_t = -1;                              // last tile of this group in the segment
            for (int j = ((it0 & 1) == wg) ? 0 : 1; j < sg.len; j += 2) {
                const int it = it0 + j;
                const int st = it % kStages;
                const int tok0 = (sg.tau0 + j) * kTile;
                last_t = it;
                const int buf = (wg << 1) | ((it >> 1) & 1);
                const uint32_t sp_tmem = tmem_base + tlane + (uint32_t)buf * 64;
                TS_TRACE(0)
                if (wg == 1 && has_next && j + 2 >= sg.len && row_valid) {
                    // last tile of this group in the segment: pull the next pair's Q rows into L2, so that the
                    // copy at the end of the segment does not wait for HBM
                    const uint16_t *src = a.q + (((size_t)nc.s * a.q_len + t_row) * a.Hq + (size_t)nc.g * a.G + hl) * D;
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(src));
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(src + 64));
                }
                wait(sfull(buf), (uint32_t)(it >> 2) & 1u);
                fence_after_sync();
                TS_TRACE(1)
                float alpha = 1.f, rowsum = 0.f;
                bool rescale = false;
                const bool need_mask = tok0 + kTile - 1 > sg.n - a.q_len;
                if (!idle_warp) {
                uint32_t xr[2][32];
                tmem_ld32(sp_tmem, xr[0]);
                tmem_ld32(sp_tmem + 32, xr[1]);
                tmem_wait_ld();
                TS_TRACE(2)
                if (q4 == 3 && lane == 0) TS_EVENT(it, 3)
                // mask (only near the sequence end) and row maximum of the raw scores (scale > 0 here)
                if (need_mask) {
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (tok0 + 32 * h + c > lim) xr[h][c] = 0xff800000u;      // -inf
                }
                float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int c = 0; c < 32; ++c) mx4[c & 3] = fmaxf(mx4[c & 3], __uint_as_float(xr[h][c]));
                const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * a.scale_log2;
                const float m_new = fmaxf(m_used, mx);
                if (j < 2 || m_new > m_used + kLazyTau) {
                    alpha = ex2(m_used - ((m_new == -INFINITY) ? 0.f : m_new));
                    rescale = row_valid && (j >= 2) && (m_new != m_used);
                    m_used = m_new;
                }
                const float mref = (m_used == -INFINITY) ? 0.f : m_used;
                // P = exp2(x - m) as bf16 hi + lo, written over S in TMEM: the A operand of the second MMA.
                TS_TRACE(3)
                float rs4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t hi[16], lo[16];
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        const float p0 = ex2(fmaf(__uint_as_float(xr[h][2 * k]), a.scale_log2, -mref));
                        const float p1 = ex2(fmaf(__uint_as_float(xr[h][2 * k + 1]), a.scale_log2, -mref));
                        rs4[k & 3] += p0 + p1;
                        hi[k] = pack_bf16x2(p0, p1);
                        lo[k] = pack_bf16x2(p0 - bf16lo_to_f32(hi[k]), p1 - bf16hi_to_f32(hi[k]));
                    }
                    tmem_st16(sp_tmem + 16 * h, hi);
                    tmem_st16(sp_tmem + 32 + 16 * h, lo);
                }
                rowsum = (rs4[0] + rs4[1]) + (rs4[2] + rs4[3]);
                }
                TS_TRACE(4)
                // V rows past the sequence end may hold anything: zero them (0 * NaN)
                const int valid_tok = sg.n - tok0;
                if (valid_tok < kTile) {
                    wait(vfull(st), (uint32_t)(it / kStages) & 1u);
                    const uint32_t vb = base + kOffStage + (uint32_t)st * kStageBytes + 16384;
                    for (int i = tid_wg; i < (kTile - valid_tok) * 16; i += 128) {
                        const int r = valid_tok + (i >> 4), c = i & 15;
                        const uint32_t addr = vb + (uint32_t)(c >> 3) * 8192u + (uint32_t)r * 128u + (uint32_t)((c & 7) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0u) : "memory");
                    }
                }
                const int u = it >> 1;
                if (u >= 2 && !idle_warp) observe_upto(u - 2);
                // lazy rescale of this group's O in TMEM (warp-collective): every PV into it must have finished
                if (__any_sync(FULL, rescale)) {
                    observe_upto(u - 1);
                    fence_after_sync();
                    const float f = rescale ? alpha : 1.f;
#pragma unroll 1
                    for (int ch = 0; ch < 4; ++ch) {
                        uint32_t o[32];
                        tmem_ld32(tmem_base + tlane + o_col + 32 * ch, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * f);
                        tmem_st32(tmem_base + tlane + o_col + 32 * ch, o);
                    }
                }
                tmem_wait_st();
                fence_before_sync();
                if (valid_tok < kTile) fence_proxy_async_smem();
                __syncwarp();
                if (need_o_sync) { named_bar_sync(3, 256); need_o_sync = false; }
                if (lane == 0) mbar_arrive(pfull(buf));
                if (q4 == 3 && lane == 0) TS_EVENT(it, 4)
                l_sum = l_sum * alpha + rowsum;
                TS_TRACE(5)
            }
            // ---- end of the segment: merge the two groups' accumulators, write the result
            if (last_t >= 0 && !idle_warp) observe_upto(last_t >> 1);
            if (q4 == 3 && lane == 0) TS_EVENT(it0 + sg.len - 1, 8 + wg)
            if (need_o_sync) named_bar_sync(3, 256);      // no tile of this segment was ours: still pair up
            if (wg == 1) {
                asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(stats), "f"(m_used), "f"(l_sum) : "memory");
                fence_before_sync();
                named_bar_sync(1, 256);       // every S = Q K^T and P V of the segment has completed
                named_bar_sync(2, 256);       // group 0 has read the statistics: the slot may be rewritten
                if (has_next) {
                    issue_q(nc.s, nc.g);       // the tile is free: every Q K^T of the segment is done
                    publish_q();
                    if (q4 == 0 && lane == 0) TS_EVENT(it0 + sg.len - 1, 10)
                }
            } else {
                named_bar_sync(1, 256);
                fence_after_sync();
                float m1, l1;
                asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(m1), "=f"(l1) : "r"(stats));
                named_bar_sync(2, 256);
                const float M = fmaxf(m_used, m1);
                const float Mref = (M == -INFINITY) ? 0.f : M;
                const float w0 = l_sum > 0.f ? ex2(m_used - Mref) : 0.f;
                const float w1 = l1 > 0.f ? ex2(m1 - Mref) : 0.f;
                const float L = w0 * l_sum + w1 * l1;
                const float inv = L > 0.f ? 1.f / L : 0.f;
                const float f0 = w0 * inv, f1 = w1 * inv;
                const bool use0 = l_sum > 0.f, use1 = l1 > 0.f;     // an unused accumulator may hold anything
                const bool full_pair = (sg.tau0 == 0 && sg.len == sg.tiles);
                const bool write_final = (a.mode == kModeFree) && full_pair;
                const size_t row_th = ((size_t)sg.s * a.q_len + t_row) * a.Hq + (size_t)sg.g * a.G + hl;
                float *po = nullptr, *pl = nullptr;
                if (!write_final) {
                    if (a.mode == kModeFree) {
                        const size_t slot = (size_t)2 * gid + (sg.tau0 > 0 ? 0 : 1);
                        po = a.part_o + (slot * a.rows + row) * D;
                        pl = a.part_lse + slot * a.rows + row;
                    } else {
                        const size_t rows_all = (size_t)a.q_len * a.Hq;
                        const size_t b0 = ((size_t)sg.s * a.max_splits + sg.chunk_idx) * rows_all + ((size_t)t_row * a.Hq + (size_t)sg.g * a.G + hl);
                        po = a.part_o + b0 * D;
                        pl = a.part_lse + b0;
                    }
                }
                const bool any0 = __any_sync(FULL, use0), any1 = __any_sync(FULL, use1);
#pragma unroll 1
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t o[32], o1[32];
#pragma unroll
                    for (int c = 0; c < 32; ++c) { o[c] = 0u; o1[c] = 0u; }
                    if (any0) tmem_ld32(tmem_base + tlane + kTmemO + 32 * ch, o);
                    if (any1) tmem_ld32(tmem_base + tlane + kTmemO + 128 + 32 * ch, o1);
                    tmem_wait_ld();
                    float r[32];
#pragma unroll
                    for (int c = 0; c < 32; ++c)
                        r[c] = (use0 ? __uint_as_float(o[c]) * f0 : 0.f) + (use1 ? __uint_as_float(o1[c]) * f1 : 0.f);
                    if (row_valid) {
                        if (write_final) {
                            uint4 *dst = reinterpret_cast<uint4 *>(a.out + row_th * D + 32 * ch);
#pragma unroll
                            for (int v = 0; v < 4; ++v) {
                                uint4 w;
                                w.x = pack_bf16x2(r[8 * v + 0], r[8 * v + 1]);
                                w.y = pack_bf16x2(r[8 * v + 2], r[8 * v + 3]);
                                w.z = pack_bf16x2(r[8 * v + 4], r[8 * v + 5]);
                                w.w = pack_bf16x2(r[8 * v + 6], r[8 * v + 7]);
                                dst[v] = w;
                            }
                        } else {
                            float4 *dst = reinterpret_cast<float4 *>(po + 32 * ch);
#pragma unroll
                            for (int v = 0; v < 8; ++v) dst[v] = make_float4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                        }
                    }
                }
                fence_before_sync();
                if (has_next) asm volatile("bar.arrive 3, 256;" ::: "memory");   // O0 and O1 have been read
                if (q4 == 3 && lane == 0) TS_EVENT(it0 + sg.len - 1, 11)
                if (row_valid && !write_final) *pl = L > 0.f ? (Mref + log2f(L)) * 0.6931471805599453f : -INFINITY;
            }
            ++seg_no;
            it0 += sg.len;
            remaining -= sg.len;
            cc.tau += sg.len - 1;
            cur_advance(cc, a);
        }
#ifdef TS_TC_TRACE
        if (blockIdx.x == 0 && q4 == 3 && lane == 0) {
            long long *dbg = reinterpret_cast<long long *>(a.status) + 2 + 8 * wg;
            for (int i = 0; i < 6; ++i) dbg[i] = tr_acc[i];
            dbg[6] = total;
        }
#endif
    }

#ifdef TS_TC_TRACE
    // (written by the traced threads inside their branch; nothing to do here)
#endif
    // ---- teardown
    fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace tc
}  // namespace ts
