// Tensor-core corpus scan for sm_100a: coarse scores s = bf16(q).bf16(x) - |bf16(x)|^2 / 2 for
// every corpus row and up to 256 miss queries per pass, with the per-query best-k' selection
// fused into the accumulator read-out (Algorithm 1: the database call of the misses).
//
// One persistent block per SM, 4 + 8 warps:
//   warp 0   one lane issues TMA loads (cp.async.bulk.tensor, no multicast) of 128-row x 64-col
//            bf16 corpus tiles, and of the matching query tile unless the whole query block
//            fits in shared memory and is loaded once, into a ring of mbarrier-guarded stages;
//   warp 1   allocates tensor memory; one lane issues tcgen05.mma (M = 128 corpus rows,
//            N = padded query count, K = 16 per instruction, fp32 accumulators in tensor memory,
//            two accumulator buffers so that the read-out of tile t overlaps the products of t+1);
//   warp 2   keeps the score bounds that the blocks share fresh (see the bound warp below);
//   warps 4-11 read the accumulators (tcgen05.ld, one corpus row per thread, the two warps of a
//            tensor-memory lane quarter splitting the columns) into registers, hand the
//            accumulator buffer back at once, then compare every score with the query's
//            threshold and append survivors to warp-private candidate lists; a warp sorts and
//            cuts a list of its own when it could overflow.
// Row tiles are dealt to the pairs of blocks in contiguous runs whose lengths follow the speed
// each pair showed in the previous launch.
// Every wait on an mbarrier is bounded in time; on expiry the block latches PROX_ERR_TIMEOUT,
// stops issuing work, lets copies in flight land, frees its tensor memory and returns.
#include <cuda.h>

#include <new>

#include "prox_internal.h"
#include "scan_readout.cuh"
#include "sm100_ptx.cuh"
#include "topk_device.cuh"

namespace prox {

using namespace sm100;

namespace {

#ifndef PROX_READ_WARPS
#define PROX_READ_WARPS 8
#endif
constexpr int kReadWarps = PROX_READ_WARPS;          // 4, 8, 12 or 16
constexpr int kReadPerQuarter = kReadWarps / 4;      // warps that share a tensor-memory lane quarter
constexpr int kReadGroups = (kScanQ / 32 + kReadPerQuarter - 1) / kReadPerQuarter;   // most 32-column groups of one warp
constexpr int kReadCols = 32 * kReadGroups;          // most query columns one read-out warp takes
constexpr int kThreads = 128 + 32 * kReadWarps;      // producer, MMA, bound, (idle), read-out warps
constexpr int kMaxStages = 8;
constexpr int kChunkK = 64;                          // bf16 elements per 128-byte swizzle row
constexpr int kATileBytes = kTileRows * 128;         // 16 KB
constexpr int kTileRegion = 216 * 1024;              // shared memory for operand tiles
constexpr int kQResidentMax = 128 * 1024;            // query block kept resident up to this size
constexpr int kTmemCols = 512;

struct ScanArgs {
    DevState *st;
    const int *n_active;    // device: how many queries the whole call serves (misses, or the batch for the probe)
    const float *xh;
    uint32_t *thr_g;
    uint32_t *top1;
    u64 *buf;
    int32_t *buf_cnt;
    size_t buf_pass_stride, cnt_pass_stride;   // entries of buf / buf_cnt that belong to one pass
    long long N;
    int d, kp;
    int ks;                 // 64-column groups per pipeline stage (1 or 2; the tensor maps' boxes match)
    const float *w_in;      // speed of every pair (or block) as the previous launch measured it, tiles per ns
    float *w_out;           // ... as this launch measures it
};

struct Control {
    unsigned long long full[kMaxStages], empty[kMaxStages], tmem_full[2], tmem_empty[2], q_full;
    alignas(16) float thr[kScanQ];   // per query: scores at or below it cannot be among the best k'
    uint32_t best[4][kScanQ];        // best score appended per query by each lane quarter (ordered-uint form)
    int wcnt[kReadWarps][kReadCols];   // entries in each read-out warp's private candidate lists
    uint32_t tmem_base;
    int abort_flag;                  // set by any thread whose wait ran out
    int done;                        // read-out warps that have finished (the bound warp stops at kReadWarps)
    int first_pub;                   // read-out warps that have published the bests of their first tile
    uint32_t issued;                 // tiles whose products have all been issued (the MMA issuers take turns)
    long long t_begin, t_end;        // row tiles of this pair (or block)
};

// One read-out warp owns, for every query column it reads, a private candidate list in global
// memory (CAP entries): it appends the scores that beat the query's threshold and, when a list
// could overflow during the next tile, sorts it and keeps the best k'.  No other warp touches the
// list, so the read-out needs no block-wide barrier.
//
// PAIR = true runs two blocks per MMA (a cluster of two, tcgen05 cta_group::2): a pair takes 256
// corpus rows per tile, each block loading its own 128 rows and half of the query rows, so a
// block ingests a third less per corpus row than alone.  Block 0 of the pair issues the MMAs.
template <int CAP, bool PAIR, bool DUAL>
__global__ void __launch_bounds__(kThreads, 1)
scan_tc_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_q16,
               const __grid_constant__ CUtensorMap tm_q32, const __grid_constant__ CUtensorMap tm_q64,
               const __grid_constant__ CUtensorMap tm_q128, const __grid_constant__ CUtensorMap tm_q256,
               const ScanArgs a) {
    extern __shared__ unsigned char smem_dyn[];
    __shared__ Control ctl;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = PAIR ? cluster_rank() : 0u;        // 0: the block of the pair that issues MMAs
    const int unit = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;      // pair (or block) index
    const int n_units = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    constexpr int kUnitRows = PAIR ? 2 * kTileRows : kTileRows;            // corpus rows per tile of a unit

    // The queries are taken in passes of up to kScanQ; the pairs (or blocks) are dealt to the passes
    // round robin and each pass's pairs split the row tiles among themselves, so that one launch
    // serves the whole batch and a small matrix is not walked four times by idle-starting blocks.
    const int n_act = *a.n_active;
    const int n_pass = (n_act + kScanQ - 1) / kScanQ;
    if (n_pass <= 0) {                                    // nothing to scan for
        if (blockIdx.x == 0)
            for (int u = tid; u < n_units; u += kThreads) a.w_out[u] = a.w_in[u];
        return;
    }
    const int pass = unit % n_pass;
    const int sub = unit / n_pass, n_sub = (n_units - pass + n_pass - 1) / n_pass;    // place among the pass's pairs
    const int q0 = pass * kScanQ;
    const int nq = n_act - q0 < kScanQ ? n_act - q0 : kScanQ;
    // lists of the other passes that this block will not write must read as empty
    for (int p2 = 0; p2 < n_pass; ++p2)
        if (p2 != pass)
            for (int idx = tid; idx < 4 * kScanQ; idx += kThreads)
                a.buf_cnt[(size_t)p2 * a.cnt_pass_stride + (size_t)blockIdx.x * 4 * kScanQ + idx] = 0;
    const int n_pad = nq <= 32 ? 32 : (nq <= 64 ? 64 : (nq <= 128 ? 128 : 256));
    const int q_rows = PAIR ? n_pad / 2 : n_pad;             // query rows this block stages (half of B in a pair)
    const CUtensorMap *tm_q = q_rows == 16 ? &tm_q16 : (q_rows == 32 ? &tm_q32 : (q_rows == 64 ? &tm_q64 : (q_rows == 128 ? &tm_q128 : &tm_q256)));
    const int q_row0 = q0 + (int)rank * q_rows;
    const int nk = a.d / kChunkK;                            // 64-column groups of a row
    const int ks = a.ks;                                     // column groups per stage (one barrier round trip)
    const int nst = nk / ks;                                 // stages per tile
    const int b_tile_bytes = q_rows * 128;
    const int q_block_bytes = b_tile_bytes * nk;
    const bool resident = q_block_bytes <= kQResidentMax;
    const int stage_bytes = ks * (resident ? kATileBytes : kATileBytes + b_tile_bytes);
    int stages = (kTileRegion - (resident ? q_block_bytes : 0)) / stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    // Two MMA issuers take the tiles in turn (see there).  An issuer waits for the first stage of its
    // tile before its turn, i.e. while the other issuer may still be consuming the tile before; an
    // mbarrier wait tells only the parity of a phase, so the fill waited for must be the very next
    // one of its stage: the fill before it (stages earlier) has to belong to a tile that was issued
    // before this issuer's previous tile.  That holds when the ring has at least two tiles' worth of stages.
    // (DUAL: the launch allows it, for few dimensions; with many, a tile's products outlast the issuer's chain anyway)
    const bool dual = DUAL && nst <= 2 && stages >= 2 * nst;

    const uint32_t tiles0 = (smem_u32(smem_dyn) + 1023u) & ~1023u;       // 1024-byte aligned
    const uint32_t q_res0 = tiles0;
    const uint32_t stage0 = tiles0 + (resident ? (uint32_t)q_block_bytes : 0u);
    volatile int *abort_flag = &ctl.abort_flag;
    uint32_t *thr_g = a.thr_g + q0;
    uint32_t *top1 = a.top1 + (size_t)q0 * 4 * gridDim.x;      // [query][block][lane quarter]
    const long long ntiles = (a.N + kUnitRows - 1) / kUnitRows;
    // barriers the MMA-issuing block waits on: in a pair, both blocks signal block 0's copy
    const uint32_t tx_mult = PAIR ? 2u : 1u;

    if (tid == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(smem_u32(&ctl.full[s]), 1);
            mbar_init(smem_u32(&ctl.empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl.tmem_full[b]), 1);
            mbar_init(smem_u32(&ctl.tmem_empty[b]), PAIR ? 2 * kReadWarps : kReadWarps);
        }
        mbar_init(smem_u32(&ctl.q_full), 1);
        ctl.abort_flag = 0;
        ctl.done = 0;
        ctl.first_pub = 0;
        ctl.issued = 0u;
        // Row tiles are dealt out in contiguous runs whose lengths follow the speeds that the
        // previous launch measured (SMs differ by their place on the die: up to a quarter in
        // tiles per second), so that all pairs end together.  Every block adds the same numbers
        // in the same order and so arrives at the same split.
        {
            const long long nt = (a.N + kUnitRows - 1) / kUnitRows;
            double mean = 0.0;
            for (int j = 0; j < n_sub; ++j) mean += (double)a.w_in[pass + j * n_pass];
            mean /= n_sub;
            double total = 0.0, before = 0.0, upto = 0.0;
            for (int j = 0; j < n_sub; ++j) {
                double w = (double)a.w_in[pass + j * n_pass];
                if (!(w > 0.7 * mean)) w = 0.7 * mean;     // one odd measurement must not starve a pair
                if (w > 1.4 * mean) w = 1.4 * mean;
                if (j < sub) before += w;
                if (j <= sub) upto += w;
                total += w;
            }
            long long b0 = (long long)((double)nt * (before / total));
            long long b1 = sub == n_sub - 1 ? nt : (long long)((double)nt * (upto / total));
            if (b0 > nt) b0 = nt;
            if (b1 > nt) b1 = nt;
            if (b1 < b0) b1 = b0;
            ctl.t_begin = b0;
            ctl.t_end = b1;
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    for (int q = tid; q < kScanQ; q += kThreads) {
        ctl.thr[q] = q < nq ? -INFINITY : INFINITY;
        ctl.best[0][q] = 0u; ctl.best[1][q] = 0u; ctl.best[2][q] = 0u; ctl.best[3][q] = 0u;
    }
    for (int i = tid; i < kReadWarps * kReadCols; i += kThreads) (&ctl.wcnt[0][0])[i] = 0;
    if (warp == 1) tmem_alloc<PAIR>(smem_u32(&ctl.tmem_base), kTmemCols);
    tc_fence_before();
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();               // both blocks' barriers exist before any remote signal
    tc_fence_after();
    const uint32_t tmem_base = ctl.tmem_base;
    const long long t_begin = ctl.t_begin, t_end = ctl.t_end;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint32_t q_full_bar = PAIR ? map_to_rank(smem_u32(&ctl.q_full), 0) : smem_u32(&ctl.q_full);
            if (resident) {
                if (rank == 0) mbar_expect_tx(smem_u32(&ctl.q_full), tx_mult * (uint32_t)q_block_bytes);
                for (int st = 0; st < nst; ++st) {
                    if constexpr (PAIR) tma_load_3d_pair(q_res0 + st * ks * b_tile_bytes, tm_q, 0, q_row0, st * ks, q_full_bar);
                    else tma_load_3d(q_res0 + st * ks * b_tile_bytes, tm_q, 0, q_row0, st * ks, q_full_bar);
                }
            }
            uint32_t g = 0;
            bool ok = true;
            for (long long tile = t_begin; ok && tile < t_end; ++tile) {
                const int row0 = (int)(tile * kUnitRows) + (int)rank * kTileRows;
                // (no L2 prefetch of the next tile: measured, it makes a quarter of the rows come from DRAM
                // twice and every shape slower, by 11 % at 256 queries over 24 M rows)
                for (int st = 0; st < nst; ++st, ++g) {
                    const int s = g % stages;
                    const uint32_t ph = (g / stages) & 1u;
                    if (!mbar_wait(smem_u32(&ctl.empty[s]), ph ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t dst = stage0 + s * stage_bytes;        // [ks corpus groups][ks query groups]
                    if constexpr (PAIR) {
                        const uint32_t fb = map_to_rank(smem_u32(&ctl.full[s]), 0);
                        if (rank == 0) mbar_expect_tx(smem_u32(&ctl.full[s]), 2u * (uint32_t)stage_bytes);
                        tma_load_3d_pair(dst, &tm_x, 0, row0, st * ks, fb);
                        if (!resident) tma_load_3d_pair(dst + ks * kATileBytes, tm_q, 0, q_row0, st * ks, fb);
                    } else {
                        const uint32_t fb = smem_u32(&ctl.full[s]);
                        mbar_expect_tx(fb, (uint32_t)stage_bytes);
                        tma_load_3d(dst, &tm_x, 0, row0, st * ks, fb);
                        if (!resident) tma_load_3d(dst + ks * kATileBytes, tm_q, 0, q_row0, st * ks, fb);
                    }
                }
            }
        }
    } else if (warp == 1 || warp == 3) {
        // ------------------------------------------------------------ MMA issuers
        // One thread issues a tile's products: every tcgen05.mma costs it about a hundred cycles,
        // and with the waits and commits of a tile the chain of one thread is longer than the
        // products of a tile of 128 dimensions take.  So two threads (warps 1 and 3) take the
        // tiles in turn: while one issues, the other has already waited for its row tile and its
        // accumulator buffer and only waits for its turn, which keeps the products in tile order.
        const uint32_t me = warp == 1 ? 0u : 1u;
        const uint32_t n_issuers = dual ? 2u : 1u;
        if (lane == 0 && rank == 0 && me < n_issuers) {
            const uint32_t idesc = instr_desc_bf16(kUnitRows, n_pad);
            bool ok = true;
            if (resident) ok = mbar_wait(smem_u32(&ctl.q_full), 0, abort_flag);
            volatile uint32_t *issued = &ctl.issued;
            for (uint32_t it = me; ok && t_begin + (long long)it < t_end; it += n_issuers) {
                const uint32_t b = it & 1u, bph = (it >> 1) & 1u;
                uint32_t g = it * (uint32_t)nst;
                // what the tile needs first; its turn last
                if (!mbar_wait(smem_u32(&ctl.full[g % stages]), (g / stages) & 1u, abort_flag)) { ok = false; break; }
                if (!mbar_wait(smem_u32(&ctl.tmem_empty[b]), bph ^ 1u, abort_flag)) { ok = false; break; }
                if (dual) {
                    const unsigned long long t0 = global_ns();
                    uint32_t spins = 0;
                    while (*issued != it) {
                        if ((++spins & 1023u) == 0u && (*abort_flag || global_ns() - t0 > kWaitLimitNs)) { *abort_flag = 1; ok = false; break; }
                    }
                    if (!ok) break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + b * (uint32_t)kScanQ;
                for (int st = 0; st < nst; ++st, ++g) {
                    const int s = g % stages;
                    const uint32_t ph = (g / stages) & 1u;
                    if (st > 0 && !mbar_wait(smem_u32(&ctl.full[s]), ph, abort_flag)) { ok = false; break; }
                    const uint32_t a_addr = stage0 + s * stage_bytes;
                    const uint32_t b_addr = resident ? q_res0 + st * ks * b_tile_bytes : a_addr + ks * kATileBytes;
                    for (int ka = 0; ka < ks; ++ka) {
                        const uint64_t a_desc = smem_desc_sw128(a_addr + ka * kATileBytes);
                        const uint64_t b_desc = smem_desc_sw128(b_addr + ka * b_tile_bytes);
#pragma unroll
                        for (int k4 = 0; k4 < kChunkK / 16; ++k4) {   // 16 bf16 = 32 bytes = 2 descriptor units
                            const uint32_t acc = (st | ka | k4) ? 1u : 0u;
                            if constexpr (PAIR) tc_mma_bf16_pair(d_tmem, a_desc + 2 * k4, b_desc + 2 * k4, idesc, acc);
                            else tc_mma_bf16(d_tmem, a_desc + 2 * k4, b_desc + 2 * k4, idesc, acc);
                        }
                    }
                    if (st == nst - 1 && dual) {                  // the other thread's turn
                        __threadfence_block();
                        *issued = it + 1u;
                    }
                    // the stage is free (in both blocks of a pair) once these are done
                    if constexpr (PAIR) tc_commit_pair(smem_u32(&ctl.empty[s]));
                    else tc_commit(smem_u32(&ctl.empty[s]));
                }
                if (!ok) { if (dual) *abort_flag = 1; break; }
                // accumulator complete
                if constexpr (PAIR) tc_commit_pair(smem_u32(&ctl.tmem_full[b]));
                else tc_commit(smem_u32(&ctl.tmem_full[b]));
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------ bound warp
        // Blocks scan disjoint rows, so the k'-th largest of the blocks' best scores for a query
        // is matched or exceeded by at least k' distinct rows: a lower bound of the query's global
        // k'-th best that tightens as every block publishes better rows.  Each block keeps the
        // bounds of the queries q = block (mod blocks) fresh while its read-out runs.
        // The rows of a block split further into its four lane quarters, so there are four times
        // as many disjoint row sets as blocks: a tighter bound, and one that exists for k' up to that.
        const int P = 4 * gridDim.x;
        const int my = PAIR ? 2 * sub + (int)rank : sub;        // this block among the blocks of its pass
        const int nb = PAIR ? 2 * n_sub : n_sub;
        if (a.kp <= 4 * nb && P <= 1024) {
            volatile int *done = &ctl.done;
            int jq = my, jobs = 0;
            // The first bounds are worth the most (until they arrive every row passes), and there is
            // nothing to select from before the first tile has been read out: the blocks start in
            // step, so this block's own first publication tells when the others' are due.
            {
                volatile int *first_pub = &ctl.first_pub;
                while (*first_pub < kReadWarps && *done < kReadWarps && !*abort_flag) __nanosleep(200);
            }
            while (*done < kReadWarps && !*abort_flag) {
                if (jq >= nq) jq = my;
                if (jq < nq) {
                    uint32_t t[32];
#pragma unroll
                    for (int i8 = 0; i8 < 32; ++i8) {
                        const int eidx = i8 * 32 + lane;
                        t[i8] = (eidx < P) ? __ldcg(&top1[(size_t)jq * P + eidx]) : 0u;
                    }
                    // the k'-th largest of them, bit by bit: the largest value that at least k' reach
                    // (the first rounds stop at 16 bits: a bound 2^-7 below the exact one, in half the time)
                    uint32_t rth = 0u;
                    const int low_bit = jobs < 6 ? 16 : 0;
#pragma unroll 1
                    for (int bit = 31; bit >= low_bit; --bit) {
                        const uint32_t cand = rth | (1u << bit);
                        int n_ge = 0;
#pragma unroll
                        for (int i8 = 0; i8 < 32; ++i8) n_ge += t[i8] >= cand ? 1 : 0;
                        n_ge = __reduce_add_sync(0xffffffffu, n_ge);
                        if (n_ge >= a.kp) rth = cand;
                    }
                    if (lane == 0 && rth != 0u) atomicMax(&thr_g[jq], rth);
                }
                jq += nb;
                // bounds move fast while the first tiles come in and slowly afterwards; this warp
                // shares an issue port with read-out warps, so it backs off once they have settled
                // (in short naps, so that the block does not outlive its read-out by a long one)
                const int naps = ++jobs < 48 ? 1 : 10;
                if (jobs < 6) __nanosleep(300);                 // the first rounds follow one another closely
                else
                    for (int n = 0; n < naps && *done < kReadWarps; ++n) __nanosleep(2000);
            }
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------ accumulator read-out
        // Warp w may read tensor-memory lanes 32 (w mod 4) .. +31 (one corpus row per thread); the
        // warps that share a lane quarter split the query columns.  A warp copies
        // its columns into registers and frees the accumulator buffer before it looks at them, so
        // a slow tile (appends, a list to cut) does not hold back the products two tiles on.
        const int e = warp - 4;                                   // 0..15
        const int quarter = warp & 3;
        const int part = e >> 2;
        // the 32-column groups of the query block are dealt to the warps of the quarter as evenly as they go
        const int n_grp = n_pad / 32, g_base = n_grp / kReadPerQuarter, g_rem = n_grp % kReadPerQuarter;
        const int cw = 32 * (g_base + (part < g_rem ? 1 : 0));    // columns of this warp
        const int col_begin = 32 * (part * g_base + (part < g_rem ? part : g_rem));
        const bool active = cw > 0;
        const int ncol = active ? (nq - col_begin < cw ? (nq - col_begin > 0 ? nq - col_begin : 0) : cw) : 0;
        int *wcnt = ctl.wcnt[e];
        // lists of this warp: [(block * 4 + quarter) * kScanQ + query] * CAP
        u64 *lists = a.buf + (size_t)pass * a.buf_pass_stride + ((size_t)(blockIdx.x * 4 + quarter) * kScanQ) * CAP;
        int32_t *lists_cnt = a.buf_cnt + (size_t)pass * a.cnt_pass_stride + (size_t)(blockIdx.x * 4 + quarter) * kScanQ;
        uint32_t it = 0;
        uint32_t published[kReadGroups];
        float tmin[kReadGroups];                                  // lower bound of the thresholds of each 32-column group
#pragma unroll
        for (int i = 0; i < kReadGroups; ++i) { published[i] = 0u; tmin[i] = -INFINITY; }
        long long row = t_begin * kUnitRows + (long long)rank * kTileRows + quarter * 32 + lane;
        float hn = (t_begin < t_end && row < a.N) ? a.xh[row] : INFINITY;
        const unsigned long long ns0 = global_ns();
        bool alive = true;
        const uint32_t empty_bar0 = PAIR ? map_to_rank(smem_u32(&ctl.tmem_empty[0]), 0) : smem_u32(&ctl.tmem_empty[0]);
        const uint32_t empty_bar1 = PAIR ? map_to_rank(smem_u32(&ctl.tmem_empty[1]), 0) : smem_u32(&ctl.tmem_empty[1]);
        for (long long tile = t_begin; alive && tile < t_end; ++tile, ++it) {
            const uint32_t b = it & 1u, bph = (it >> 1) & 1u;
            // loads whose latency hides behind the wait and the read-out
            const long long row_next = row + kUnitRows;
            const float hn_next = (tile + 1 < t_end && row_next < a.N) ? a.xh[row_next] : INFINITY;
            // (the shared bounds are looked at on every tile at first and on every eighth tile once they
            // move slowly: at 128 dimensions the read-out of a tile, not its products, sets the pace)
            uint32_t g_thr[kReadGroups];
            const bool thr_tile = it < 16 || (it & 7u) == 1u;
#pragma unroll
            for (int i = 0; i < kReadGroups; ++i) {
                const int c = col_begin + lane + 32 * i;
                g_thr[i] = (thr_tile && lane + 32 * i < ncol) ? __ldcg(&thr_g[c]) : 0u;
            }
            bool ok = mbar_wait(smem_u32(&ctl.tmem_full[b]), bph, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) { alive = false; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + b * (uint32_t)kScanQ;
            // The shared bounds read above go into the block's thresholds (a stale, lower threshold
            // only lets more rows through, so plain stores that the warps of a column share are
            // enough).  While the first tiles come in every tile that is still tested against an
            // open threshold floods the lists, so the bounds are applied before the test; later
            // they are applied after it, where the latency of their load is hidden.
            const bool early = it < 8;
            if (early) {
#pragma unroll
                for (int i = 0; i < kReadGroups; ++i) {
                    const int lc = lane + 32 * i;
                    if (lc < ncol) {
                        const float g = o2f(g_thr[i]);
                        if (g > ctl.thr[col_begin + lc]) ctl.thr[col_begin + lc] = g;
                    }
                }
                __syncwarp();
            }
            // 64 columns at a time; the accumulator buffer goes back to the MMA issuer as soon as
            // the last of them are in registers, before they are looked at.  Rows past the end carry
            // an infinite half norm, columns past nq an infinite threshold: neither can pass, so
            // the compare loop needs no bounds tests.
            bool need = false;
#pragma unroll 1
            for (int c0 = 0; c0 < kReadCols; c0 += 64) {
                const bool last = c0 + 64 >= cw;
                uint32_t v0[32], v1[32];
                if (active && c0 < cw) {
                    tc_ld32(taddr + col_begin + c0, v0);
                    if (c0 + 32 < cw) tc_ld32(taddr + col_begin + c0 + 32, v1);
                    tc_wait_ld();
                }
                if (last) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        if constexpr (PAIR) mbar_arrive_cluster(b ? empty_bar1 : empty_bar0);
                        else mbar_arrive(b ? empty_bar1 : empty_bar0);
                    }
                }
                if (active && c0 < cw)
                {
                    // (selected, not indexed: the array stays in registers)
                    constexpr int G = kReadGroups;
                    const int rd = c0 >> 6;                                   // 64-column round
                    const float ta = rd == 0 ? tmin[0] : (rd == 1 ? tmin[G > 2 ? 2 : 0] : (rd == 2 ? tmin[G > 4 ? 4 : 0] : tmin[G > 6 ? 6 : 0]));
                    const float tb = rd == 0 ? tmin[G > 1 ? 1 : 0] : (rd == 1 ? tmin[G > 3 ? 3 : 0] : (rd == 2 ? tmin[G > 5 ? 5 : 0] : tmin[G > 7 ? 7 : 0]));
                    readout64<CAP>(v0, v1, c0 + 32 < cw, col_begin + c0, c0, hn, ta, tb, (int32_t)row, ctl.thr, wcnt,
                                   ctl.best[quarter], lists, need);
                }
                if (last) break;
            }
            if (!early && thr_tile) {
#pragma unroll
                for (int i = 0; i < kReadGroups; ++i) {
                    const int lc = lane + 32 * i;
                    if (lc < ncol) {
                        const float g = o2f(g_thr[i]);
                        if (g > ctl.thr[col_begin + lc]) ctl.thr[col_begin + lc] = g;
                    }
                }
            }
            // the warp publishes the best score of its lane quarter for each of its columns, and takes
            // the smallest threshold of each of its column groups for the first level of the test
            // (every tile at first, every sixteenth once the bounds move slowly; thresholds only rise,
            // so an older minimum is still a lower bound)
            if (it < 16 || (it & 15u) == 0u) {
#pragma unroll
                for (int i = 0; i < kReadGroups; ++i) {
                    float t = ctl.thr[col_begin + ((lane + 32 * i) < cw ? lane + 32 * i : 0)];
#pragma unroll
                    for (int m = 16; m > 0; m >>= 1) t = fminf(t, __shfl_xor_sync(0xffffffffu, t, m));
                    tmin[i] = t;
                }
#pragma unroll
                for (int i = 0; i < kReadGroups; ++i) {
                    const int lc = lane + 32 * i;
                    if (lc < ncol) {
                        const int c = col_begin + lc;
                        const uint32_t bq = ctl.best[quarter][c];
                        if (bq > published[i]) {
                            top1[((size_t)c * gridDim.x + blockIdx.x) * 4 + quarter] = bq;
                            published[i] = bq;
                        }
                    }
                }
                if (it == 0) {
                    __syncwarp();
                    if (lane == 0) atomicAdd(&ctl.first_pub, 1);
                }
            }
            if (need) {                                           // warp-uniform
                __syncwarp();
                for (int i = 0; i < kReadGroups; ++i) {
                    const int lc = lane + 32 * i;
                    unsigned mm = __ballot_sync(0xffffffffu, lc < ncol && wcnt[lc] > CAP - 33);
                    while (mm) {
                        const int l = __ffs(mm) - 1;
                        mm &= mm - 1;
                        const int lcc = l + 32 * i, c = col_begin + lcc;
                        warp_compact<CAP>(lists + (size_t)c * CAP, &wcnt[lcc], &ctl.thr[c], &thr_g[c], a.kp, nullptr,
                                          blockIdx.x, gridDim.x, false);
                    }
                }
                __syncwarp();
            }
            row = row_next;
            hn = hn_next;
        }
        // the speed of this pair (or block) for the next launch's split; kept when the launch was
        // too short to tell (the same test in every block, so all keep or all renew)
        if (rank == 0 && e == 0 && lane == 0) {
            const unsigned long long ns = global_ns() - ns0;
            const bool long_enough = ntiles >= 32LL * n_sub;
            a.w_out[unit] = (long_enough && alive && it > 0 && ns > 0) ? (float)((double)it / (double)ns) : a.w_in[unit];
        }
        // the lists go to the merge as they are: it drops what the shared bound has ruled out
        __syncwarp();
        for (int lc = lane; lc < ncol; lc += 32) {
            const int n = wcnt[lc] < CAP ? wcnt[lc] : CAP;
            lists_cnt[col_begin + lc] = alive ? n : 0;
        }
        if (lane == 0) atomicAdd(&ctl.done, 1);
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();               // no signal to the other block is still under way
    if (ctl.abort_flag) {
        if (tid == 0) atomicCAS(&a.st->error, 0, PROX_ERR_TIMEOUT);
        // let copies and products that were already issued finish before memory is handed back
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc<PAIR>(tmem_base, kTmemCols);
    }
}

#include "scan_tc_multi.cuh"

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

// A row-major bf16 matrix seen as (64-column group, row, column within the group): one box is
// box_rows rows of ks neighbouring groups, landing in shared memory group after group.
bool make_map(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t ks) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {kChunkK, rows, cols / kChunkK};
    const cuuint64_t strides[2] = {cols * 2, kChunkK * 2};
    const cuuint32_t box[3] = {kChunkK, box_rows, ks};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct Maps {
    CUtensorMap x, q16, q32, q64, q128, q256;
    int ks = 1;
    bool ok = false;
    float *speed = nullptr;        // device, 2 x kMaxUnits: the pairs' speeds, written by one launch, read by the next
    int units = 0;                 // pairs (or blocks) the speeds were measured for
    unsigned launch_no = 0;
};
constexpr int kMaxUnits = 256;

// Equal speeds for every pair: the state before the first measurement.
__global__ void speed_init_kernel(float *speed) {
    for (int i = threadIdx.x; i < 2 * kMaxUnits; i += blockDim.x) speed[i] = 1.f;
}

}  // namespace

template <int CAP, bool PAIR, bool DUAL>
static void set_scan_smem() {
    cudaFuncSetAttribute(scan_tc_kernel<CAP, PAIR, DUAL>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTileRegion + 1024);
}
template <int CAP, bool PAIR, bool DUAL>
static cudaError_t launch_scan_kernel(const cudaLaunchConfig_t &cfg, const Maps &maps, const ScanArgs &a) {
    return cudaLaunchKernelEx(&cfg, scan_tc_kernel<CAP, PAIR, DUAL>, maps.x, maps.q16, maps.q32, maps.q64, maps.q128, maps.q256, a);
}
template <int CAP>
static cudaError_t launch_scan_kernel(bool pair, bool dual, const cudaLaunchConfig_t &cfg, const Maps &maps, const ScanArgs &a) {
    if (pair) return dual ? launch_scan_kernel<CAP, true, true>(cfg, maps, a) : launch_scan_kernel<CAP, true, false>(cfg, maps, a);
    return dual ? launch_scan_kernel<CAP, false, true>(cfg, maps, a) : launch_scan_kernel<CAP, false, false>(cfg, maps, a);
}

// Tensor maps and the speed table of one scanned matrix: made once, at prox_create, so that the
// batch calls neither allocate nor copy.
static void ensure_maps(prox_handle *h, void **state, const __nv_bfloat16 *xb, long long rows,
                        const __nv_bfloat16 *qb) {
    if (*state) return;
    Maps *m = new (std::nothrow) Maps();
    if (!m) return;
    *state = m;
    const uint32_t ks = ((h->d / kChunkK) % 2 == 0) ? 2 : 1;
    m->ks = (int)ks;
    if (cudaMalloc(&m->speed, sizeof(float) * 2 * kMaxUnits) != cudaSuccess) { m->speed = nullptr; cudaGetLastError(); }
    m->ok = m->speed != nullptr && make_map(&m->x, xb, (uint64_t)rows, (uint64_t)h->d, kTileRows, ks) &&
            make_map(&m->q16, qb, kMaxBatch, (uint64_t)h->d, 16, ks) &&
            make_map(&m->q32, qb, kMaxBatch, (uint64_t)h->d, 32, ks) &&
            make_map(&m->q64, qb, kMaxBatch, (uint64_t)h->d, 64, ks) &&
            make_map(&m->q128, qb, kMaxBatch, (uint64_t)h->d, 128, ks) &&
            make_map(&m->q256, qb, kMaxBatch, (uint64_t)h->d, 256, ks);
    if (m->speed) {
        // equal speeds from the start, for the launch shape the handle takes by default: the first scan of a
        // handle may be recorded (prox_record_batch), and a recording must not carry the table's reset
        speed_init_kernel<<<1, 256>>>(m->speed);
        const bool pair = h->scan_ctas >= 2 && rows >= 2 * kTileRows;
        m->units = pair ? (h->scan_ctas & ~1) / 2 : h->scan_ctas;
    }
    set_scan_smem<256, false, false>(); set_scan_smem<512, false, false>(); set_scan_smem<256, true, false>(); set_scan_smem<512, true, false>();
    set_scan_smem<256, false, true>(); set_scan_smem<512, false, true>(); set_scan_smem<256, true, true>(); set_scan_smem<512, true, true>();
    cudaFuncSetAttribute(scan_tc_multi_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTileRegionM + 1024);
    cudaFuncSetAttribute(scan_tc_multi_kernel<512>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTileRegionM + 1024);
}

void init_scan_tc(prox_handle *h) {
    if (h->d % kChunkK) return;
    if (h->N >= kTileRows) ensure_maps(h, &h->tc_state, h->xb, (long long)h->N, h->qb);
    if (h->probe_tc) ensure_maps(h, &h->tc_state_keys, h->keys_b, (long long)h->C, h->pqb);
}

// One pass of the tensor-core scan of `rows` bf16 rows (xb, half norms xh) against the bf16 query
// block qb.  Returns nonzero when the tensor-core path cannot run (no tensor-map encoder in the
// driver, out of memory for the maps); the caller then falls back.
static int launch_scan_generic(prox_handle *h, void **state, const __nv_bfloat16 *xb, const float *xh, long long rows,
                               const __nv_bfloat16 *qb, const int *n_active, int n_max, int kp, cudaStream_t s) {
    if (!*state) return 1;
    Maps &maps = *static_cast<Maps *>(*state);
    if (!maps.ok) return 1;
    ScanArgs a;
    a.st = h->st; a.n_active = n_active; a.xh = xh; a.thr_g = h->thr_g; a.top1 = h->top1; a.buf = h->buf;
    a.buf_cnt = h->buf_cnt; a.buf_pass_stride = h->buf_pass_stride; a.cnt_pass_stride = h->cnt_pass_stride;
    a.N = rows; a.d = h->d; a.kp = kp; a.ks = maps.ks;
    const bool pair = h->scan_mode != PROX_SCAN_TC_SINGLE && h->scan_ctas >= 2 && rows >= 2 * kTileRows;
    const int grid = pair ? (h->scan_ctas & ~1) : h->scan_ctas;
    const int units = pair ? grid / 2 : grid;
    if (units > kMaxUnits) return 1;
    if (maps.units != units) {                            // first launch, or the launch shape changed: equal speeds
        speed_init_kernel<<<1, 256, 0, s>>>(maps.speed);
        maps.units = units;
    }
    a.w_in = maps.speed + (maps.launch_no & 1u) * kMaxUnits;
    a.w_out = maps.speed + ((maps.launch_no + 1u) & 1u) * kMaxUnits;
    h->scan_lists = 4 * grid;                             // one candidate list per read-out lane quarter
    h->scan_list_stride = h->tc_cap;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kTileRegion + 1024;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = pair ? 2 : 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // two MMA issuers when a row tile is one or two ring stages (up to 256 dimensions)
    const bool dual = (h->d / kChunkK) / maps.ks <= 2;
    // up to 128 dimensions and more queries than one pass takes: every pair serves all passes (the row tiles
    // are read once instead of once per pass)
    const bool multi = pair && (h->d / kChunkK) / maps.ks == 1 && n_max > kScanQ && h->scan_mode == PROX_SCAN_AUTO;
    cudaError_t e;
    if (multi) {
        cfg.dynamicSmemBytes = kTileRegionM + 1024;
        e = h->tc_cap == 256 ? cudaLaunchKernelEx(&cfg, scan_tc_multi_kernel<256>, maps.x, maps.q128, a)
                             : cudaLaunchKernelEx(&cfg, scan_tc_multi_kernel<512>, maps.x, maps.q128, a);
    } else {
        e = h->tc_cap == 256 ? launch_scan_kernel<256>(pair, dual, cfg, maps, a) : launch_scan_kernel<512>(pair, dual, cfg, maps, a);
    }
    if (e != cudaSuccess) {                               // the caller falls back: leave no error behind, keep the speeds' turn
        cudaGetLastError();
        return 1;
    }
    maps.launch_no++;
    h->launches++;
    return 0;
}

// The corpus scan of the misses, all passes of the batch in one launch.  Nonzero: the handle cannot
// take the tensor-core path (d not a multiple of 64, fewer corpus rows than one tile); the caller
// then runs the CUDA-core scan.
int launch_scan_tc(prox_handle *h, int B, cudaStream_t s) {
    if (h->d % kChunkK || h->N < kTileRows) return 1;
    return launch_scan_generic(h, &h->tc_state, h->xb, h->xh, (long long)h->N, h->qb, &h->st->n_miss, B, h->kp, s);
}

// The coarse probe: the same scan over the bf16 copies of the cached keys, all batch queries,
// keeping the kProbeKp best slots per query.
int launch_probe_scan_tc(prox_handle *h, int B, cudaStream_t s) {
    return launch_scan_generic(h, &h->tc_state_keys, h->keys_b, h->kh, (long long)h->C, h->pqb, &h->st->n_probe, B,
                               kProbeKp, s);
}

void free_scan_tc(prox_handle *h) {
    for (void **st : {&h->tc_state, &h->tc_state_keys}) {
        Maps *m = static_cast<Maps *>(*st);
        if (m && m->speed) cudaFree(m->speed);
        delete m;
        *st = nullptr;
    }
}

}  // namespace prox
