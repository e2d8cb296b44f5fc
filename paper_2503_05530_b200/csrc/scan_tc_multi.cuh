// The tensor-core scan for few dimensions (d <= 128) and batches of more than 256 queries: every pair of
// blocks serves ALL passes of 256 queries.  Included by scan_tcgen05.cu inside its unnamed namespace
// (ScanArgs, the constants and the PTX wrappers are those of that file).
//
// With the passes side by side on their own pairs (scan_tc_kernel), every pass brings the corpus
// rows from DRAM and from L2 into shared memory itself: four times the bytes for 1024 queries, and at
// 128 dimensions that traffic is a sizeable part of the energy of a launch that runs at the power
// cap.  Here a row tile is loaded once and multiplied with the query blocks of all passes, which
// all stay resident in shared memory (4 x 32 KB per block at d = 128): the unit of work is (row tile,
// pass), the accumulator buffers alternate from unit to unit, the two MMA issuers take the units in
// turn, and the read-out warps keep one set of thresholds and list counts per pass.  The blocks'
// best scores per query go straight to the shared table in global memory (no per-block copy: the
// shared memory is full).
#pragma once

constexpr int kMultiPass = kMaxBatch / kScanQ;           // 4 passes at most
constexpr int kTileRegionM = 204 * 1024;                 // shared memory for the query blocks and the ring

struct ControlM {
    unsigned long long full[kMaxStages], empty[kMaxStages], tmem_full[2], tmem_empty[2], q_full;
    alignas(16) float thr[kMultiPass][kScanQ];           // per pass and query: scores at or below it cannot be among the best k'
    int wcnt[kMultiPass][kReadWarps][kReadCols];         // entries in each read-out warp's private lists, per pass
    float tmin[kMultiPass][kReadWarps][kReadGroups];     // smallest threshold of each 32-column group of a warp, per pass
    uint32_t tmem_base;
    int abort_flag, done, first_pub;
    uint32_t issued;                                     // units whose products have all been issued
    long long t_begin, t_end;
};

template <int CAP>
__global__ void __launch_bounds__(kThreads, 1)
scan_tc_multi_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_q,
                     const ScanArgs a) {
    extern __shared__ unsigned char smem_dyn[];
    __shared__ ControlM ctl;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_rank();                    // 0: the block of the pair that issues MMAs
    const int unit = (int)(blockIdx.x >> 1), n_units = (int)(gridDim.x >> 1);
    constexpr int kUnitRows = 2 * kTileRows;                 // corpus rows per tile of a pair
    constexpr int kQRows = kScanQ / 2;                       // query rows of a pass that one block stages

    const int n_act = *a.n_active;
    const int n_pass = (n_act + kScanQ - 1) / kScanQ;
    if (n_pass <= 0) {
        if (blockIdx.x == 0)
            for (int u = tid; u < n_units; u += kThreads) a.w_out[u] = a.w_in[u];
        return;
    }
    const int nk = a.d / kChunkK;                            // 1 or 2 column groups: one ring stage per tile
    const int ks = a.ks;
    const int b_tile_bytes = kQRows * 128;
    const int q_block_bytes = b_tile_bytes * nk;             // one pass's query rows of this block
    const int stage_bytes = ks * kATileBytes;
    int stages = (kTileRegionM - n_pass * q_block_bytes) / stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;

    const uint32_t tiles0 = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    const uint32_t q_res0 = tiles0;
    const uint32_t stage0 = tiles0 + (uint32_t)(n_pass * q_block_bytes);
    volatile int *abort_flag = &ctl.abort_flag;
    const long long ntiles = (a.N + kUnitRows - 1) / kUnitRows;

    if (tid == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(smem_u32(&ctl.full[s]), 1);
            // a stage is free when the products of every pass over it are done; with two passes or more both
            // issuers have units in every tile, and each commits its own products
            mbar_init(smem_u32(&ctl.empty[s]), n_pass >= 2 ? 2 : 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl.tmem_full[b]), 1);
            mbar_init(smem_u32(&ctl.tmem_empty[b]), 2 * kReadWarps);
        }
        mbar_init(smem_u32(&ctl.q_full), 1);
        ctl.abort_flag = 0;
        ctl.done = 0;
        ctl.first_pub = 0;
        ctl.issued = 0u;
        {
            // contiguous runs of row tiles, as long as the pairs' measured speeds say (see scan_tc_kernel)
            double mean = 0.0;
            for (int j = 0; j < n_units; ++j) mean += (double)a.w_in[j];
            mean /= n_units;
            double total = 0.0, before = 0.0, upto = 0.0;
            for (int j = 0; j < n_units; ++j) {
                double w = (double)a.w_in[j];
                if (!(w > 0.7 * mean)) w = 0.7 * mean;
                if (w > 1.4 * mean) w = 1.4 * mean;
                if (j < unit) before += w;
                if (j <= unit) upto += w;
                total += w;
            }
            long long b0 = (long long)((double)ntiles * (before / total));
            long long b1 = unit == n_units - 1 ? ntiles : (long long)((double)ntiles * (upto / total));
            if (b0 > ntiles) b0 = ntiles;
            if (b1 > ntiles) b1 = ntiles;
            if (b1 < b0) b1 = b0;
            ctl.t_begin = b0;
            ctl.t_end = b1;
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    for (int i = tid; i < kMultiPass * kScanQ; i += kThreads)
        (&ctl.thr[0][0])[i] = i < n_act ? -INFINITY : INFINITY;          // (pass * 256 + column is the query's index)
    for (int i = tid; i < kMultiPass * kReadWarps * kReadCols; i += kThreads) (&ctl.wcnt[0][0][0])[i] = 0;
    for (int i = tid; i < kMultiPass * kReadWarps * kReadGroups; i += kThreads) (&ctl.tmin[0][0][0])[i] = -INFINITY;
    if (warp == 1) tmem_alloc<true>(smem_u32(&ctl.tmem_base), kTmemCols);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = ctl.tmem_base;
    const long long t_begin = ctl.t_begin, t_end = ctl.t_end;
    const uint32_t n_my_units = (uint32_t)((t_end - t_begin) * n_pass);      // (row tile, pass) pairs of this pair of blocks

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint32_t q_full_bar = map_to_rank(smem_u32(&ctl.q_full), 0);
            if (rank == 0) mbar_expect_tx(smem_u32(&ctl.q_full), 2u * (uint32_t)(n_pass * q_block_bytes));
            for (int p = 0; p < n_pass; ++p)                 // the query rows of every pass stay resident
                tma_load_3d_pair(q_res0 + p * q_block_bytes, &tm_q, 0, p * kScanQ + (int)rank * kQRows, 0, q_full_bar);
            bool ok = true;
            uint32_t g = 0;
            for (long long tile = t_begin; ok && tile < t_end; ++tile, ++g) {
                const int row0 = (int)(tile * kUnitRows) + (int)rank * kTileRows;
                const int s = g % stages;
                const uint32_t ph = (g / stages) & 1u;
                if (!mbar_wait(smem_u32(&ctl.empty[s]), ph ^ 1u, abort_flag)) { ok = false; break; }
                const uint32_t fb = map_to_rank(smem_u32(&ctl.full[s]), 0);
                if (rank == 0) mbar_expect_tx(smem_u32(&ctl.full[s]), 2u * (uint32_t)stage_bytes);
                tma_load_3d_pair(stage0 + s * stage_bytes, &tm_x, 0, row0, 0, fb);
            }
        }
    } else if (warp == 1 || warp == 3) {
        // ------------------------------------------------------------ MMA issuers
        // The two threads take the units in turn (see scan_tc_kernel): a thread waits for its unit's row
        // tile and accumulator buffer ahead of its turn.  The ring holds at least two tiles and a tile is one
        // stage, so the fill waited for is the next one of its stage: the tile two before was issued whole
        // before this thread's previous unit.
        const uint32_t me = warp == 1 ? 0u : 1u;
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = instr_desc_bf16(kUnitRows, kScanQ);
            bool ok = mbar_wait(smem_u32(&ctl.q_full), 0, abort_flag);
            volatile uint32_t *issued = &ctl.issued;
            for (uint32_t u = me; ok && u < n_my_units; u += 2u) {
                const uint32_t tile_i = u / (uint32_t)n_pass, pass = u - tile_i * (uint32_t)n_pass;
                const uint32_t b = u & 1u, bph = (u >> 1) & 1u;
                const int s = (int)(tile_i % (uint32_t)stages);
                const uint32_t ph = (tile_i / (uint32_t)stages) & 1u;
                if (!mbar_wait(smem_u32(&ctl.full[s]), ph, abort_flag)) { ok = false; break; }
                if (!mbar_wait(smem_u32(&ctl.tmem_empty[b]), bph ^ 1u, abort_flag)) { ok = false; break; }
                {
                    const unsigned long long t0 = global_ns();
                    uint32_t spins = 0;
                    while (*issued != u) {
                        if ((++spins & 1023u) == 0u && (*abort_flag || global_ns() - t0 > kWaitLimitNs)) { *abort_flag = 1; ok = false; break; }
                    }
                    if (!ok) break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + b * (uint32_t)kScanQ;
                const uint32_t a_addr = stage0 + s * stage_bytes;
                const uint32_t b_addr = q_res0 + pass * (uint32_t)q_block_bytes;
                for (int ka = 0; ka < ks; ++ka) {
                    const uint64_t a_desc = smem_desc_sw128(a_addr + ka * kATileBytes);
                    const uint64_t b_desc = smem_desc_sw128(b_addr + ka * b_tile_bytes);
#pragma unroll
                    for (int k4 = 0; k4 < kChunkK / 16; ++k4)
                        tc_mma_bf16_pair(d_tmem, a_desc + 2 * k4, b_desc + 2 * k4, idesc, (ka | k4) ? 1u : 0u);
                }
                __threadfence_block();
                *issued = u + 1u;                               // the other thread's turn
                // this thread's last unit of the tile: its products over the stage are all issued
                if ((u + 2u) / (uint32_t)n_pass != tile_i) tc_commit_pair(smem_u32(&ctl.empty[s]));
                tc_commit_pair(smem_u32(&ctl.tmem_full[b]));    // accumulator complete
            }
            if (!ok) *abort_flag = 1;
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------ bound warp
        // The k'-th largest of all blocks' (and lane quarters') best scores for a query is a lower bound
        // of its global k'-th best (see scan_tc_kernel); here every block holds rows for every query.
        const int P = 4 * gridDim.x;
        const int my = (int)blockIdx.x, nb = (int)gridDim.x;
        if (a.kp <= 4 * nb && P <= 1024) {
            volatile int *done = &ctl.done;
            int jq = my, jobs = 0;
            {
                volatile int *first_pub = &ctl.first_pub;
                while (*first_pub < kReadWarps && *done < kReadWarps && !*abort_flag) __nanosleep(200);
            }
            while (*done < kReadWarps && !*abort_flag) {
                if (jq >= n_act) jq = my;
                if (jq < n_act) {
                    uint32_t t[32];
#pragma unroll
                    for (int i8 = 0; i8 < 32; ++i8) {
                        const int eidx = i8 * 32 + lane;
                        t[i8] = (eidx < P) ? __ldcg(&a.top1[(size_t)jq * P + eidx]) : 0u;
                    }
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
                    if (lane == 0 && rth != 0u) atomicMax(&a.thr_g[jq], rth);
                }
                jq += nb;
                const int naps = ++jobs < 48 ? 1 : 10;
                if (jobs < 6) __nanosleep(300);
                else
                    for (int n = 0; n < naps && *done < kReadWarps; ++n) __nanosleep(2000);
            }
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------ accumulator read-out
        // As in scan_tc_kernel (a warp reads its lane quarter's rows of its 128 query columns), unit by
        // unit; what belongs to a pass (thresholds, list counts, group minima, lists, shared bounds)
        // is picked by the unit's pass.
        const int e = warp - 4;
        const int quarter = warp & 3;
        const int part = e >> 2;
        constexpr int cw = kReadCols;                             // 128 columns of every pass
        const int col_begin = part * cw;
        const int best_stride = 4 * (int)gridDim.x;               // the shared table is [query][block][lane quarter]
        uint32_t u = 0, it = 0;                                   // unit and row tile counters
        long long row = t_begin * kUnitRows + (long long)rank * kTileRows + quarter * 32 + lane;
        float hn = (t_begin < t_end && row < a.N) ? a.xh[row] : INFINITY;
        float hn_next = INFINITY;
        const unsigned long long ns0 = global_ns();
        bool alive = true;
        const uint32_t empty_bar0 = map_to_rank(smem_u32(&ctl.tmem_empty[0]), 0);
        const uint32_t empty_bar1 = map_to_rank(smem_u32(&ctl.tmem_empty[1]), 0);
        for (; alive && u < n_my_units; ++u) {
            const uint32_t b = u & 1u, bph = (u >> 1) & 1u;
            const int pass = (int)(u - it * (uint32_t)n_pass);
            const int nq_p = n_act - pass * kScanQ < kScanQ ? n_act - pass * kScanQ : kScanQ;
            const int ncol = nq_p - col_begin < cw ? (nq_p - col_begin > 0 ? nq_p - col_begin : 0) : cw;
            float *thr_p = ctl.thr[pass];
            int *wcnt = ctl.wcnt[pass][e];
            float *tmin_p = ctl.tmin[pass][e];
            uint32_t *thr_g = a.thr_g + pass * kScanQ;
            uint32_t *best_p = a.top1 + ((size_t)pass * kScanQ * gridDim.x + blockIdx.x) * 4 + quarter;
            u64 *lists = a.buf + (size_t)pass * a.buf_pass_stride + ((size_t)(blockIdx.x * 4 + quarter) * kScanQ) * CAP;
            // loads whose latency hides behind the wait and the read-out (the next tile's half norm once per tile)
            if (pass == 0) {
                const long long row_next = row + kUnitRows;
                hn_next = (t_begin + it + 1 < t_end && row_next < a.N) ? a.xh[row_next] : INFINITY;
            }
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
            const bool early = it < 8;
            if (early) {
#pragma unroll
                for (int i = 0; i < kReadGroups; ++i) {
                    const int lc = lane + 32 * i;
                    if (lc < ncol) {
                        const float g = o2f(g_thr[i]);
                        if (g > thr_p[col_begin + lc]) thr_p[col_begin + lc] = g;
                    }
                }
                __syncwarp();
            }
            // 64 columns at a time; the buffer goes back to the issuers once the last are in registers
            bool need = false;
#pragma unroll 1
            for (int c0 = 0; c0 < cw; c0 += 64) {
                const bool last = c0 + 64 >= cw;
                uint32_t v0[32], v1[32];
                tc_ld32(taddr + col_begin + c0, v0);
                tc_ld32(taddr + col_begin + c0 + 32, v1);
                tc_wait_ld();
                if (last) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(b ? empty_bar1 : empty_bar0);
                }
                const int g0 = c0 >> 5;
                readout64<CAP>(v0, v1, true, col_begin + c0, c0, hn, tmin_p[g0], tmin_p[g0 + 1], (int32_t)row, thr_p, wcnt,
                               best_p, lists, need, best_stride);
            }
            if (!early && thr_tile) {
#pragma unroll
                for (int i = 0; i < kReadGroups; ++i) {
                    const int lc = lane + 32 * i;
                    if (lc < ncol) {
                        const float g = o2f(g_thr[i]);
                        if (g > thr_p[col_begin + lc]) thr_p[col_begin + lc] = g;
                    }
                }
            }
            // the smallest threshold of each column group, for the first level of the test (every tile at
            // first, every sixteenth later; thresholds only rise, so an older minimum is still a lower bound)
            if (it < 16 || (it & 15u) == 0u) {
                __syncwarp();
#pragma unroll
                for (int i = 0; i < kReadGroups; ++i) {
                    float t = thr_p[col_begin + lane + 32 * i];
#pragma unroll
                    for (int m = 16; m > 0; m >>= 1) t = fminf(t, __shfl_xor_sync(0xffffffffu, t, m));
                    if (lane == 0) tmin_p[i] = t;
                }
                __syncwarp();
            }
            if (u + 1u == (uint32_t)n_pass) {                     // the first tile is read out for every pass
                __syncwarp();
                if (lane == 0) atomicAdd(&ctl.first_pub, 1);
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
                        warp_compact<CAP>(lists + (size_t)c * CAP, &wcnt[lcc], &thr_p[c], &thr_g[c], a.kp, nullptr,
                                          blockIdx.x, gridDim.x, false);
                    }
                }
                __syncwarp();
            }
            if (pass == n_pass - 1) {                             // next row tile
                ++it;
                row += kUnitRows;
                hn = hn_next;
            }
        }
        // the speed of this pair for the next launch's split (kept when the launch was too short to tell)
        if (rank == 0 && e == 0 && lane == 0) {
            const unsigned long long ns = global_ns() - ns0;
            const bool long_enough = ntiles >= 32LL * n_units;
            a.w_out[unit] = (long_enough && alive && it > 0 && ns > 0) ? (float)((double)it / (double)ns) : a.w_in[unit];
        }
        // the lists of every pass go to the merge as they are
        __syncwarp();
        for (int p = 0; p < kMultiPass; ++p) {
            int32_t *lists_cnt = a.buf_cnt + (size_t)p * a.cnt_pass_stride + (size_t)(blockIdx.x * 4 + quarter) * kScanQ;
            const int nq_p = n_act - p * kScanQ < kScanQ ? n_act - p * kScanQ : kScanQ;
            for (int lc = lane; lc < cw; lc += 32) {
                const int c = col_begin + lc;
                const int n = ctl.wcnt[p][e][lc] < CAP ? ctl.wcnt[p][e][lc] : CAP;
                lists_cnt[c] = (alive && p < n_pass && c < nq_p) ? n : 0;
            }
        }
        if (lane == 0) atomicAdd(&ctl.done, 1);
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (ctl.abort_flag) {
        if (tid == 0) atomicCAS(&a.st->error, 0, PROX_ERR_TIMEOUT);
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc<true>(tmem_base, kTmemCols);
    }
}
