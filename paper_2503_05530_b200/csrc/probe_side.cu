// The part of the probe that the in-order replay needs pair by pair (the key distances of
// Algorithm 1 for the keys whose residence can change inside the batch): every query against the
// at-risk slots and against the earlier queries of its own batch.  For large batches this is a
// dense B x 2B x d contraction, taken here on the tensor cores over the bf16 copies (mma.sync
// m16n8k16, fp32 accumulation: a small product next to the key scan, so the warp-level form is
// enough); every pair whose coarse distance could hide a true distance within tau goes to a pair
// list, and only those pairs are measured in fp64.  The bound that decides "could hide" covers the
// bf16 rounding of both vectors and the fp32 sum, so the pairs within tau are all in the list: the
// result is the exact set, with exact fp64 distances, as the fp64 rows would have given it.
#include <cuda_bf16.h>

#include "prox_internal.h"

namespace prox {

namespace {

constexpr int kSideTile = 128;            // queries x columns of one block
constexpr int kSideK = 64;                // dimensions per pipeline step
constexpr int kSideLd = kSideK + 8;       // row pitch in shared memory (bf16): fragment loads without bank conflicts
constexpr int kSideStages = 3;            // steps in flight: the operands come from L2, a microsecond away
constexpr int kSideSmem = kSideStages * 2 * kSideTile * kSideLd * 2;   // bytes of dynamic shared memory

__device__ __forceinline__ void cp_async16(void *dst, const void *src, bool pred) {
    const unsigned d = (unsigned)__cvta_generic_to_shared(dst);
    const int n = pred ? 16 : 0;                             // 0: the 16 bytes are filled with zeros
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

}  // namespace

// Largest coarse squared distance that a pair whose true squared distance is at most tau can show:
// rounding to bf16 moves either vector by at most a resp. e, the fp32 sum and norms by the slack.
__device__ __forceinline__ double side_coarse_bound(double root_tau, double a, double e, double qn, double kn, int d) {
    const double slack = 4.0 * (double)(d + 16) * 5.9604644775390625e-08 * (2.0 * qn * kn + kn * kn + qn * qn);
    const double r = root_tau + a + e;
    return r * r * (1.0 + 1e-6) + slack * (1.0 + 1e-6) + 4e-7 * (qn * qn + kn * kn) + 1e-30;
}

// Column space: code < kMaxBatch = position in the at-risk list, code >= kMaxBatch = kMaxBatch + j
// for query j of the batch (only j < i counts for query i).  grid = (query tiles, 2 * kMaxBatch / 128).
__global__ void __launch_bounds__(256)
probe_side_kernel(DevState *st, const __nv_bfloat16 *__restrict__ pqb, const float *__restrict__ pqbn,
                  const float *__restrict__ pqerr, const __nv_bfloat16 *__restrict__ keys_b,
                  const float *__restrict__ kh, const int32_t *__restrict__ risk_slot, int B, int d, double tau,
                  uint32_t *pairs) {
    extern __shared__ __align__(16) unsigned char side_smem[];
    typedef __nv_bfloat16 (*Tile)[kSideTile][kSideLd];
    Tile As = reinterpret_cast<Tile>(side_smem);                                   // [kSideStages][kSideTile][kSideLd]
    Tile Bs = reinterpret_cast<Tile>(side_smem + (size_t)kSideStages * kSideTile * kSideLd * 2);
    __shared__ float col_n2[kSideTile], col_err[kSideTile];
    __shared__ double col_n[kSideTile];                       // |bf16 column|, one square root per column instead of one per pair
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int R = st->n_risk;
    const int i0 = blockIdx.x * kSideTile;
    const bool batch_cols = (int)blockIdx.y >= kMaxBatch / kSideTile;
    const int c0 = (batch_cols ? (int)blockIdx.y - kMaxBatch / kSideTile : (int)blockIdx.y) * kSideTile;   // first at-risk position or batch index
    const int n_cols = batch_cols ? B : R;
    if (c0 >= n_cols) return;
    if (batch_cols && c0 >= i0 + kSideTile - 1) return;       // no column of the tile precedes a query of the tile

    // rows this thread copies: four of A (queries) and four of B (columns), 16 bytes of each per step
    const int lr = tid >> 3, part = tid & 7;
    const __nv_bfloat16 *a_src[4], *b_src[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int r = lr + 32 * u;
        a_src[u] = (i0 + r < B) ? pqb + (size_t)(i0 + r) * d + part * 8 : nullptr;
        const int c = c0 + r;
        b_src[u] = nullptr;
        if (c < n_cols) b_src[u] = (batch_cols ? pqb + (size_t)c * d : keys_b + (size_t)risk_slot[c] * d) + part * 8;
    }
    if (tid < kSideTile) {
        const int c = c0 + tid;
        float n2 = 0.f, er = 0.f;
        if (c < n_cols) {
            if (batch_cols) { n2 = pqbn[c]; er = pqerr[c]; }
            else { n2 = 2.f * kh[risk_slot[c]]; er = st->ke_max; }
        }
        col_n2[tid] = n2;
        col_err[tid] = er;
        col_n[tid] = sqrt((double)n2);
    }
    auto load_stage = [&](int stage, int k0) {
        const bool in_row = k0 + part * 8 < d;                // d is a multiple of 16: the last step may be half empty
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int r = lr + 32 * u;
            const bool pa = in_row && a_src[u] != nullptr, pb = in_row && b_src[u] != nullptr;
            cp_async16(&As[stage][r][part * 8], pa ? a_src[u] + k0 : pqb, pa);
            cp_async16(&Bs[stage][r][part * 8], pb ? b_src[u] + k0 : pqb, pb);
        }
        cp_async_commit();
    };

    float acc[2][8][4];
#pragma unroll
    for (int mi = 0; mi < 2; ++mi)
#pragma unroll
        for (int ni = 0; ni < 8; ++ni)
#pragma unroll
            for (int r = 0; r < 4; ++r) acc[mi][ni][r] = 0.f;
    const int wm = warp & 3, wn = warp >> 2;                  // the warp's 32 queries x 64 columns
    const int g = lane >> 2, t = lane & 3;
    const int steps = (d + kSideK - 1) / kSideK;

    // (one commit group per step, empty past the last step, so that "all but the newest two" is always step s)
    load_stage(0, 0);
    if (steps > 1) load_stage(1, kSideK); else cp_async_commit();
    for (int s = 0; s < steps; ++s) {
        if (s + 2 < steps) load_stage((s + 2) % kSideStages, (s + 2) * kSideK); else cp_async_commit();
        cp_async_wait<2>();
        __syncthreads();
        const int st_ = s % kSideStages;
#pragma unroll
        for (int kk = 0; kk < kSideK / 16; ++kk) {
            uint32_t af[2][4];
#pragma unroll
            for (int mi = 0; mi < 2; ++mi) {
                const int r = wm * 32 + mi * 16 + g;
                af[mi][0] = *reinterpret_cast<const uint32_t *>(&As[st_][r][kk * 16 + 2 * t]);
                af[mi][1] = *reinterpret_cast<const uint32_t *>(&As[st_][r + 8][kk * 16 + 2 * t]);
                af[mi][2] = *reinterpret_cast<const uint32_t *>(&As[st_][r][kk * 16 + 2 * t + 8]);
                af[mi][3] = *reinterpret_cast<const uint32_t *>(&As[st_][r + 8][kk * 16 + 2 * t + 8]);
            }
#pragma unroll
            for (int ni = 0; ni < 8; ++ni) {
                const int c = wn * 64 + ni * 8 + g;
                uint32_t bf[2];
                bf[0] = *reinterpret_cast<const uint32_t *>(&Bs[st_][c][kk * 16 + 2 * t]);
                bf[1] = *reinterpret_cast<const uint32_t *>(&Bs[st_][c][kk * 16 + 2 * t + 8]);
                mma_bf16_16816(acc[0][ni], af[0], bf);
                mma_bf16_16816(acc[1][ni], af[1], bf);
            }
        }
        __syncthreads();
    }

    // coarse distance |bf16 q|^2 + |bf16 key|^2 - 2 q.key against the bound of the pair
    const double root_tau = sqrt(tau);
#pragma unroll
    for (int mi = 0; mi < 2; ++mi) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int i = i0 + wm * 32 + mi * 16 + g + 8 * half;
            if (i >= B) continue;
            const double qn2 = (double)pqbn[i], qn = sqrt(qn2), qa = (double)pqerr[i];
#pragma unroll
            for (int ni = 0; ni < 8; ++ni) {
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
                    const int lc = wn * 64 + ni * 8 + 2 * t + cc;
                    const int c = c0 + lc;
                    if (c >= n_cols || (batch_cols && c >= i)) continue;
                    const double n2 = (double)col_n2[lc];
                    const double coarse = qn2 + n2 - 2.0 * (double)acc[mi][ni][2 * half + cc];
                    if (coarse <= side_coarse_bound(root_tau, qa, (double)col_err[lc], qn, col_n[lc], d)) {
                        const int pos = atomicAdd(&st->n_pairs, 1);
                        if (pos < kPairCap) pairs[pos] = ((uint32_t)i << 16) | (uint32_t)(batch_cols ? kMaxBatch + c : c);
                        else st->side_overflow = 1;
                    }
                }
            }
        }
    }
}

// Exact fp64 distance of every listed pair; the pairs within tau become the candidates of their
// query (unsorted here: the candidate kernel sorts them).
__global__ void __launch_bounds__(256)
probe_pairs_exact_kernel(const DevState *__restrict__ st, const float *__restrict__ keys,
                         const float *__restrict__ queries, const int32_t *__restrict__ risk_slot, int d, double tau,
                         const uint32_t *__restrict__ pairs, double *cand_d, int32_t *cand_code, int32_t *n_cand) {
    if (st->side_overflow) return;                            // the fp64 rows take over
    const int n = st->n_pairs < kPairCap ? st->n_pairs : kPairCap;
    const int lane = threadIdx.x & 31;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    for (int p = warp; p < n; p += nwarps) {
        const uint32_t pr = pairs[p];
        const int i = (int)(pr >> 16), code = (int)(pr & 0xffffu);
        const float *q = queries + (size_t)i * d;
        const float *x = code < kMaxBatch ? keys + (size_t)risk_slot[code] * d : queries + (size_t)(code - kMaxBatch) * d;
        double acc = 0.0;
        for (int j = lane; j < d; j += 32) {
            const double df = (double)q[j] - (double)x[j];
            acc = fma(df, df, acc);
        }
#pragma unroll
        for (int m = 16; m > 0; m >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, m);
        if (lane == 0 && acc <= tau) {
            const int pos = atomicAdd(&n_cand[i], 1);
            cand_d[(size_t)i * (2 * kMaxBatch) + pos] = acc;
            cand_code[(size_t)i * (2 * kMaxBatch) + pos] = code;
        }
    }
}

// Kernel attributes belong to a device: set when a handle is created there.
void set_probe_side_attributes() {
    cudaFuncSetAttribute(probe_side_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSideSmem);
}

void launch_probe_side(prox_handle *h, const float *q, int B, cudaStream_t s) {
    dim3 grid((B + kSideTile - 1) / kSideTile, 2 * kMaxBatch / kSideTile);
    probe_side_kernel<<<grid, 256, kSideSmem, s>>>(h->st, h->pqb, h->pqbn, h->pqerr, h->keys_b, h->kh, h->risk_slot, B, h->d,
                                           (double)h->tau, h->side_pairs);
    probe_pairs_exact_kernel<<<h->num_sms * 4, 256, 0, s>>>(h->st, h->keys, q, h->risk_slot, h->d, (double)h->tau,
                                                           h->side_pairs, h->cand_d, h->cand_code, h->n_cand);
    h->launches += 2;
}

}  // namespace prox
