// Tensor-core corpus scan for sm_100a: coarse scores s = bf16(q).bf16(x) - |bf16(x)|^2 / 2 for
// every corpus row and up to 256 miss queries per pass, with the per-query best-k' selection
// fused into the accumulator read-out (Algorithm 1, line 6: the database call of the misses).
//
// One persistent block per SM, 12 warps:
//   warp 0   one lane issues TMA loads (cp.async.bulk.tensor, no multicast) of 128-row x 64-col
//            bf16 corpus tiles, and of the matching query tile unless the whole query block
//            fits in shared memory and is loaded once, into a ring of mbarrier-guarded stages;
//   warp 1   allocates tensor memory; one lane issues tcgen05.mma (M = 128 corpus rows,
//            N = padded query count, K = 16 per instruction, fp32 accumulators in tensor memory,
//            two accumulator buffers so that the read-out of tile t overlaps the products of t+1);
//   warp 2   keeps the score bounds that the blocks share fresh (see the bound warp below);
//   warps 4-11 read the accumulators (tcgen05.ld, one corpus row per thread, two warps per
//            tensor-memory lane quarter splitting the columns), subtract the row's half norm,
//            compare with the query's threshold and append survivors to warp-private candidate
//            lists; a warp sorts and cuts a list of its own when it could overflow.
// Every wait on an mbarrier is bounded in time; on expiry the block latches PROX_ERR_TIMEOUT,
// stops issuing work, lets copies in flight land, frees its tensor memory and returns.
#include <cuda.h>

#include <new>

#include "prox_internal.h"
#include "topk_device.cuh"

namespace prox {

namespace {

constexpr int kThreads = 384;                        // producer, MMA, bound, (idle), 8 read-out warps
constexpr int kReadWarps = 8;
constexpr int kMaxStages = 8;
constexpr int kChunkK = 64;                          // bf16 elements per 128-byte swizzle row
constexpr int kATileBytes = kTileRows * 128;         // 16 KB
constexpr int kTileRegion = 216 * 1024;              // shared memory for operand tiles
constexpr int kQResidentMax = 128 * 1024;            // query block kept resident up to this size
constexpr int kTmemCols = 512;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: false if the limit ran out or another thread of the block gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
#pragma unroll 1
    for (int i = 0; i < 128; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
#pragma unroll 1
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_ns() - t0 > kWaitLimitNs) {
            *abort_flag = 1;
            return false;
        }
        __nanosleep(32);
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
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
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major operand tile whose rows are 128 bytes
// (64 bf16) written by TMA with the 128-byte swizzle: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t desc = 0;
    desc |= (uint64_t)((addr & 0x3ffffu) >> 4);          // start address, 16-byte units
    desc |= (uint64_t)(1024u >> 4) << 32;                // stride between 8-row groups
    desc |= 1ull << 46;                                  // descriptor version of sm_100
    desc |= 2ull << 61;                                  // 128-byte swizzle
    return desc;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t instr_desc_bf16(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTileRows >> 4) << 24);
}

struct ScanArgs {
    DevState *st;
    const float *xh;
    uint32_t *thr_g;
    uint32_t *top1;
    u64 *buf;
    int32_t *buf_cnt;
    long long N;
    int d, pass, kp;
};

struct Control {
    unsigned long long full[kMaxStages], empty[kMaxStages], tmem_full[2], tmem_empty[2], q_full;
    alignas(16) float thr[kScanQ];   // per query: scores at or below it cannot be among the best k'
    uint32_t best[kScanQ];           // best score this block has appended per query (ordered-uint form)
    int wcnt[kReadWarps][kScanQ / 2];  // entries in each read-out warp's private candidate lists
    uint32_t tmem_base;
    int abort_flag;                  // set by any thread whose wait ran out
    int done;                        // read-out warps that have finished (the bound warp stops at kReadWarps)
};

// One read-out warp owns, for every query column it reads, a private candidate list in global
// memory (CAP entries): it appends the scores that beat the query's threshold and, when a list
// could overflow during the next tile, sorts it and keeps the best k'.  No other warp touches the
// list, so the read-out needs no block-wide barrier.
// Slow path of the read-out, entered by the whole warp when some lane has a passing column:
// per column, the passing lanes take consecutive slots of the warp's list (the counter is
// private to the warp, so a ballot replaces atomics) and the warp's best score is folded in.
template <int CAP>
__device__ __forceinline__ void append32(const uint32_t (&v)[32], int c0, int lc0, float hn, int32_t row,
                                         const float *thr, int *wcnt, uint32_t *best, u64 *lists, bool &need) {
    const int lane = threadIdx.x & 31;
    const unsigned lt = (1u << lane) - 1u;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        const bool p = __uint_as_float(v[j]) - thr[c0 + j] > hn;    // the same arithmetic as the shortcut
        const unsigned mask = __ballot_sync(0xffffffffu, p);
        if (mask) {
            const int base = wcnt[lc0 + j];
            const u64 ent = pack_entry(__uint_as_float(v[j]) - hn, row);
            const int pos = base + __popc(mask & lt);
            if (p && pos < CAP) lists[(size_t)(c0 + j) * CAP + pos] = ent;
            const uint32_t mx = __reduce_max_sync(0xffffffffu, p ? (uint32_t)(ent >> 32) : 0u);
            const int n_new = base + __popc(mask);
            if (lane == 0) {
                wcnt[lc0 + j] = n_new;
                atomicMax(&best[c0 + j], mx);
            }
            if (n_new > CAP - 33) need = true;                    // this list must be cut before the next tile
        }
    }
    __syncwarp();
}

// 32 accumulator columns (queries c0 .. c0+31) of one corpus row.  A column passes when
// acc - thr > half norm, i.e. score = acc - half norm beats the threshold up to one rounding
// (the certificate's slack covers it); the common case, no column passes, is decided by one
// maximum over the 32 differences.
template <int CAP>
__device__ __forceinline__ void readout32(const uint32_t (&v)[32], int c0, int lc0, float hn,
                                          int32_t row, const float *thr, int *wcnt, uint32_t *best, u64 *lists,
                                          bool &need) {
    float m = -INFINITY;
#pragma unroll
    for (int j4 = 0; j4 < 8; ++j4) {
        const float4 t4 = *reinterpret_cast<const float4 *>(&thr[c0 + 4 * j4]);
        const float a0 = __uint_as_float(v[4 * j4]) - t4.x, a1 = __uint_as_float(v[4 * j4 + 1]) - t4.y;
        const float a2 = __uint_as_float(v[4 * j4 + 2]) - t4.z, a3 = __uint_as_float(v[4 * j4 + 3]) - t4.w;
        m = fmaxf(m, fmaxf(fmaxf(a0, a1), fmaxf(a2, a3)));
    }
    if (__any_sync(0xffffffffu, m > hn)) append32<CAP>(v, c0, lc0, hn, row, thr, wcnt, best, lists, need);
}

template <int CAP>
__global__ void __launch_bounds__(kThreads, 1)
scan_tc_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_q32,
               const __grid_constant__ CUtensorMap tm_q64, const __grid_constant__ CUtensorMap tm_q128,
               const __grid_constant__ CUtensorMap tm_q256, const ScanArgs a) {
    extern __shared__ unsigned char smem_dyn[];
    __shared__ Control ctl;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    const int q0 = a.pass * kScanQ;
    int nq = a.st->n_miss - q0;
    if (nq > kScanQ) nq = kScanQ;
    if (nq <= 0) return;                                  // nothing missed in this pass
    const int n_pad = nq <= 32 ? 32 : (nq <= 64 ? 64 : (nq <= 128 ? 128 : 256));
    const CUtensorMap *tm_q = n_pad == 32 ? &tm_q32 : (n_pad == 64 ? &tm_q64 : (n_pad == 128 ? &tm_q128 : &tm_q256));
    const int nk = a.d / kChunkK;
    const int b_tile_bytes = n_pad * 128;
    const int q_block_bytes = b_tile_bytes * nk;
    const bool resident = q_block_bytes <= kQResidentMax;
    const int stage_bytes = resident ? kATileBytes : kATileBytes + b_tile_bytes;
    int stages = (kTileRegion - (resident ? q_block_bytes : 0)) / stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;

    const uint32_t tiles0 = (smem_u32(smem_dyn) + 1023u) & ~1023u;       // 1024-byte aligned
    const uint32_t q_res0 = tiles0;
    const uint32_t stage0 = tiles0 + (resident ? (uint32_t)q_block_bytes : 0u);
    volatile int *abort_flag = &ctl.abort_flag;
    uint32_t *thr_g = a.thr_g + q0;
    uint32_t *top1 = a.top1 + (size_t)q0 * gridDim.x;
    const long long ntiles = (a.N + kTileRows - 1) / kTileRows;

    if (tid == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(smem_u32(&ctl.full[s]), 1);
            mbar_init(smem_u32(&ctl.empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl.tmem_full[b]), 1);
            mbar_init(smem_u32(&ctl.tmem_empty[b]), kReadWarps);
        }
        mbar_init(smem_u32(&ctl.q_full), 1);
        ctl.abort_flag = 0;
        ctl.done = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    for (int q = tid; q < kScanQ; q += kThreads) { ctl.thr[q] = q < nq ? -INFINITY : INFINITY; ctl.best[q] = 0u; }
    for (int i = tid; i < kReadWarps * (kScanQ / 2); i += kThreads) (&ctl.wcnt[0][0])[i] = 0;
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&ctl.tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl.tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            if (resident) {
                mbar_expect_tx(smem_u32(&ctl.q_full), (uint32_t)q_block_bytes);
                for (int kc = 0; kc < nk; ++kc)
                    tma_load_2d(q_res0 + kc * b_tile_bytes, tm_q, kc * kChunkK, q0, smem_u32(&ctl.q_full));
            }
            uint32_t g = 0;
            bool ok = true;
            for (long long tile = blockIdx.x; ok && tile < ntiles; tile += gridDim.x) {
                const int row0 = (int)(tile * kTileRows);
                for (int kc = 0; kc < nk; ++kc, ++g) {
                    const int s = g % stages;
                    const uint32_t ph = (g / stages) & 1u;
                    if (!mbar_wait(smem_u32(&ctl.empty[s]), ph ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t fb = smem_u32(&ctl.full[s]);
                    const uint32_t dst = stage0 + s * stage_bytes;
                    mbar_expect_tx(fb, (uint32_t)stage_bytes);
                    tma_load_2d(dst, &tm_x, kc * kChunkK, row0, fb);
                    if (!resident) tma_load_2d(dst + kATileBytes, tm_q, kc * kChunkK, q0, fb);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = instr_desc_bf16(n_pad);
            bool ok = true;
            if (resident) ok = mbar_wait(smem_u32(&ctl.q_full), 0, abort_flag);
            uint32_t g = 0, it = 0;
            for (long long tile = blockIdx.x; ok && tile < ntiles; tile += gridDim.x, ++it) {
                const uint32_t b = it & 1u, bph = (it >> 1) & 1u;
                if (!mbar_wait(smem_u32(&ctl.tmem_empty[b]), bph ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + b * (uint32_t)kScanQ;
                for (int kc = 0; kc < nk; ++kc, ++g) {
                    const int s = g % stages;
                    const uint32_t ph = (g / stages) & 1u;
                    if (!mbar_wait(smem_u32(&ctl.full[s]), ph, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = stage0 + s * stage_bytes;
                    const uint32_t b_addr = resident ? q_res0 + kc * b_tile_bytes : a_addr + kATileBytes;
                    const uint64_t a_desc = smem_desc_sw128(a_addr), b_desc = smem_desc_sw128(b_addr);
#pragma unroll
                    for (int k4 = 0; k4 < kChunkK / 16; ++k4)     // 16 bf16 = 32 bytes = 2 descriptor units
                        tc_mma_bf16(d_tmem, a_desc + 2 * k4, b_desc + 2 * k4, idesc, (kc | k4) ? 1u : 0u);
                    tc_commit(smem_u32(&ctl.empty[s]));           // the stage is free once these are done
                }
                if (ok) tc_commit(smem_u32(&ctl.tmem_full[b]));   // accumulator complete
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------ bound warp
        // Blocks scan disjoint rows, so the k'-th largest of the blocks' best scores for a query
        // is matched or exceeded by at least k' distinct rows: a lower bound of the query's global
        // k'-th best that tightens as every block publishes better rows.  Each block keeps the
        // bounds of the queries q = block (mod blocks) fresh while its read-out runs.
        const int P = gridDim.x;
        if (a.kp <= P && P <= 256) {
            volatile int *done = &ctl.done;
            int jq = blockIdx.x;
            while (*done < kReadWarps && !*abort_flag) {
                if (jq >= nq) jq = blockIdx.x;
                if (jq < nq) {
                    u64 t[8];
#pragma unroll
                    for (int i8 = 0; i8 < 8; ++i8) {
                        const int eidx = i8 * 32 + lane;
                        t[i8] = (eidx < P) ? (u64)__ldcg(&top1[(size_t)jq * P + eidx]) : 0ull;
                    }
                    warp_sort_desc<8>(t);
                    u64 rth = 0ull;
#pragma unroll
                    for (int i8 = 0; i8 < 8; ++i8) rth |= (i8 * 32 + lane == a.kp - 1) ? t[i8] : 0ull;
                    rth = __shfl_sync(0xffffffffu, rth, (a.kp - 1) & 31);
                    if (lane == 0 && (uint32_t)rth != 0u) atomicMax(&thr_g[jq], (uint32_t)rth);
                }
                jq += P;
                __nanosleep(2000);
            }
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------ accumulator read-out
        // Eight warps: warp w may read tensor-memory lanes 32 (w mod 4) .. +31 (one corpus row per
        // thread); the two warps that share a lane quarter split the query columns.
        const int e = warp - 4;                                   // 0..7
        const int quarter = warp & 3;
        const int half = e >> 2;
        const int cw = n_pad >= 64 ? n_pad / 2 : 32;              // columns per warp
        const int col_begin = half * cw;
        const bool active = col_begin < n_pad;
        const int ncol = active ? (nq - col_begin < cw ? (nq - col_begin > 0 ? nq - col_begin : 0) : cw) : 0;
        int *wcnt = ctl.wcnt[e];
        // lists of this warp: [(block * 4 + quarter) * kScanQ + query] * CAP
        u64 *lists = a.buf + ((size_t)(blockIdx.x * 4 + quarter) * kScanQ) * CAP;
        int32_t *lists_cnt = a.buf_cnt + (size_t)(blockIdx.x * 4 + quarter) * kScanQ;
        uint32_t it = 0;
        uint32_t published[4] = {0u, 0u, 0u, 0u};
        long long row = (long long)blockIdx.x * kTileRows + quarter * 32 + lane;
        float hn = (blockIdx.x < ntiles && row < a.N) ? a.xh[row] : INFINITY;
        bool alive = true;
        for (long long tile = blockIdx.x; alive && tile < ntiles; tile += gridDim.x, ++it) {
            const uint32_t b = it & 1u, bph = (it >> 1) & 1u;
            // loads whose latency hides behind the wait and the read-out
            const long long row_next = row + (long long)gridDim.x * kTileRows;
            const float hn_next = (tile + gridDim.x < ntiles && row_next < a.N) ? a.xh[row_next] : INFINITY;
            uint32_t g_thr[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int c = col_begin + lane + 32 * i;
                g_thr[i] = (lane + 32 * i < ncol) ? __ldcg(&thr_g[c]) : 0u;
            }
            bool ok = mbar_wait(smem_u32(&ctl.tmem_full[b]), bph, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) { alive = false; break; }
            tc_fence_after();
            // rows past the end carry an infinite half norm, columns past nq an infinite threshold:
            // neither can pass, so the compare loop needs no bounds tests
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + b * (uint32_t)kScanQ;
            bool need = false;
            if (active) {
                for (int c0 = col_begin; c0 < col_begin + cw; c0 += 64) {
                    const bool two = c0 + 32 < col_begin + cw;
                    uint32_t v0[32], v1[32];
                    tc_ld32(taddr + c0, v0);
                    if (two) tc_ld32(taddr + c0 + 32, v1);
                    tc_wait_ld();
                    readout32<CAP>(v0, c0, c0 - col_begin, hn, (int32_t)row, ctl.thr, wcnt, ctl.best, lists, need);
                    if (two)
                        readout32<CAP>(v1, c0 + 32, c0 + 32 - col_begin, hn, (int32_t)row, ctl.thr, wcnt,
                                       ctl.best, lists, need);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl.tmem_empty[b]));
            // threshold upkeep for this warp's columns: a stale (lower) threshold only lets more
            // rows through, so plain stores shared with the other warps are enough
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int lc = lane + 32 * i;
                if (lc < ncol) {
                    const int c = col_begin + lc;
                    const float g = o2f(g_thr[i]);
                    if (g > ctl.thr[c]) ctl.thr[c] = g;
                    if (quarter == 0) {                           // one warp per column publishes the block's best
                        const uint32_t bq = ctl.best[c];
                        if (bq > published[i]) {
                            top1[(size_t)c * gridDim.x + blockIdx.x] = bq;
                            published[i] = bq;
                        }
                    }
                }
            }
            if (need) {                                           // warp-uniform
                __syncwarp();
                for (int i = 0; i < 4; ++i) {
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
        // final cut of every list, dropping what the shared bound has already ruled out
        __syncwarp();
        for (int lc = 0; lc < ncol; ++lc) {
            const int c = col_begin + lc;
            if (alive)
                warp_compact<CAP>(lists + (size_t)c * CAP, &wcnt[lc], &ctl.thr[c], &thr_g[c], a.kp, nullptr, blockIdx.x,
                                  gridDim.x, true);
            if (lane == 0) lists_cnt[c] = alive ? wcnt[lc] : 0;
        }
        if (lane == 0) atomicAdd(&ctl.done, 1);
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (ctl.abort_flag) {
        if (tid == 0) atomicCAS(&a.st->error, 0, PROX_ERR_TIMEOUT);
        // let copies and products that were already issued finish before memory is handed back
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

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

bool make_map(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {kChunkK, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct Maps {
    CUtensorMap x, q32, q64, q128, q256;
    bool ok = false;
};

}  // namespace

// Returns nonzero when the tensor-core path cannot take this handle (d not a multiple of 64,
// fewer corpus rows than one tile, or no tensor-map encoder in the driver); the caller then
// runs the CUDA-core scan.
int launch_scan_pass_tc(prox_handle *h, int pass, cudaStream_t s) {
    if (h->d % kChunkK || h->N < kTileRows) return 1;
    if (!h->tc_state) {
        Maps *m = new (std::nothrow) Maps();
        if (!m) return 1;
        h->tc_state = m;
        m->ok = make_map(&m->x, h->xb, (uint64_t)h->N, (uint64_t)h->d, kTileRows) &&
                make_map(&m->q32, h->qb, kMaxBatch, (uint64_t)h->d, 32) &&
                make_map(&m->q64, h->qb, kMaxBatch, (uint64_t)h->d, 64) &&
                make_map(&m->q128, h->qb, kMaxBatch, (uint64_t)h->d, 128) &&
                make_map(&m->q256, h->qb, kMaxBatch, (uint64_t)h->d, 256);
        cudaFuncSetAttribute(scan_tc_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTileRegion + 1024);
        cudaFuncSetAttribute(scan_tc_kernel<512>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTileRegion + 1024);
    }
    Maps &maps = *static_cast<Maps *>(h->tc_state);
    if (!maps.ok) return 1;
    ScanArgs a;
    a.st = h->st; a.xh = h->xh; a.thr_g = h->thr_g; a.top1 = h->top1; a.buf = h->buf; a.buf_cnt = h->buf_cnt;
    a.N = (long long)h->N; a.d = h->d; a.pass = pass; a.kp = h->kp;
    h->scan_lists = 4 * h->scan_ctas;                     // one candidate list per read-out lane quarter
    h->scan_list_stride = h->tc_cap;
    if (h->tc_cap == 256)
        scan_tc_kernel<256><<<h->scan_ctas, kThreads, kTileRegion + 1024, s>>>(maps.x, maps.q32, maps.q64, maps.q128,
                                                                              maps.q256, a);
    else
        scan_tc_kernel<512><<<h->scan_ctas, kThreads, kTileRegion + 1024, s>>>(maps.x, maps.q32, maps.q64, maps.q128,
                                                                              maps.q256, a);
    h->launches++;
    return 0;
}

void free_scan_tc(prox_handle *h) {
    delete static_cast<Maps *>(h->tc_state);
    h->tc_state = nullptr;
}

}  // namespace prox
