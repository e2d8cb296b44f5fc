// Nearest cached key per query with no allocation anywhere on the call path.
//
// Who needs this: code that is not allowed to call cudaMalloc when it wants a lookup -- a plugin
// running inside a host application that owns the memory pool and forbids outside allocations,
// a service with a frozen memory budget.
// Such a caller passes the keys, the queries and the outputs (all memory it already owns); the
// partial results that the blocks exchange live in an array that is part of the library image.
//
// The array is one per GPU and is shared by every call on that GPU: it keeps whatever the last
// call left there, and two calls that run at the same time on one GPU would overwrite each
// other's partial results.  Order such calls on one stream (or otherwise keep them from
// overlapping).
#include <cstdarg>
#include <mutex>

#include "prox_internal.h"

namespace prox {
void set_last_error(const char *fmt, ...);      // prox_api.cu: text for prox_last_error()
}

namespace {

constexpr int kNaMaxB = PROX_STATIC_MAX_BATCH;       // queries per call
constexpr int kNaMaxSplits = 64;                     // blocks that share one tile of queries
constexpr int kNaQ = 32, kNaC = 64, kNaD = 32;       // tile: queries x keys x dimensions
constexpr int kNaQTiles = kNaMaxB / kNaQ;

struct NaScratch {
    double part_min[kNaMaxB * kNaMaxSplits];         // nearest distance each block found, per query
    int32_t part_arg[kNaMaxB * kNaMaxSplits];        // and its slot
    unsigned ticket[kNaQTiles];                      // blocks of a query tile that have finished; must start at 0
};

// Lives in the library image on every GPU that loads it (about 192 KB) until the process exits.
static __device__ __align__(256) unsigned char g_na_scratch[sizeof(NaScratch)];

// Squared distances in fp64 over the fp32 values, difference form (the distances and argmin of Algorithm 1, for
// a batch): each block scans a range of keys for 32 queries; the block that finishes last for
// a query tile reduces the partial minima (ties go to the lowest slot) and writes the outputs.
__global__ void __launch_bounds__(256)
nearest_static_kernel(const float *__restrict__ keys, long long n_keys, int d, const float *__restrict__ queries,
                      int B, NaScratch *sc, int32_t *out_slot, float *out_dist) {
    __shared__ double qs[kNaQ][kNaD + 1];
    __shared__ double ks[kNaC][kNaD + 1];
    __shared__ int s_last;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const long long ntiles = (n_keys + kNaC - 1) / kNaC;
    const int S = gridDim.y, sp = blockIdx.y;
    const long long per = (ntiles + S - 1) / S;
    const long long t_begin = sp * per;
    const long long t_end = (t_begin + per < ntiles) ? t_begin + per : ntiles;
    const int q0 = blockIdx.x * kNaQ;

    double best_d[2] = {INFINITY, INFINITY};
    int best_s[2] = {0x7fffffff, 0x7fffffff};
    for (long long t = t_begin; t < t_end; ++t) {
        const long long c0 = t * kNaC;
        double acc[2][4] = {{0.0, 0.0, 0.0, 0.0}, {0.0, 0.0, 0.0, 0.0}};
        for (int kc = 0; kc < d; kc += kNaD) {
            __syncthreads();
            for (int it = 0; it < (kNaQ * kNaD) / 256; ++it) {
                const int idx = it * 256 + tid, r = idx / kNaD, c = idx % kNaD;
                qs[r][c] = (q0 + r < B && kc + c < d) ? (double)queries[(size_t)(q0 + r) * d + kc + c] : 0.0;
            }
            for (int it = 0; it < (kNaC * kNaD) / 256; ++it) {
                const int idx = it * 256 + tid, r = idx / kNaD, c = idx % kNaD;
                ks[r][c] = (c0 + r < n_keys && kc + c < d) ? (double)keys[(size_t)(c0 + r) * d + kc + c] : 0.0;
            }
            __syncthreads();
#pragma unroll 8
            for (int j = 0; j < kNaD; ++j) {
                const double qa = qs[ty * 2][j], qb = qs[ty * 2 + 1][j];
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const double kv = ks[tx + 16 * b][j];
                    const double d0 = qa - kv, d1 = qb - kv;
                    acc[0][b] = fma(d0, d0, acc[0][b]);
                    acc[1][b] = fma(d1, d1, acc[1][b]);
                }
            }
        }
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const long long col = c0 + tx + 16 * b;
                if (col < n_keys && (acc[a][b] < best_d[a] || (acc[a][b] == best_d[a] && (int)col < best_s[a]))) {
                    best_d[a] = acc[a][b];
                    best_s[a] = (int)col;
                }
            }
    }
#pragma unroll
    for (int a = 0; a < 2; ++a) {
#pragma unroll
        for (int m = 1; m < 16; m <<= 1) {
            const double od = __shfl_xor_sync(0xffffffffu, best_d[a], m);
            const int os = __shfl_xor_sync(0xffffffffu, best_s[a], m);
            if (od < best_d[a] || (od == best_d[a] && os < best_s[a])) { best_d[a] = od; best_s[a] = os; }
        }
        const int i = q0 + ty * 2 + a;
        if (tx == 0 && i < B) {
            sc->part_min[(size_t)i * kNaMaxSplits + sp] = best_d[a];
            sc->part_arg[(size_t)i * kNaMaxSplits + sp] = best_s[a];
        }
    }
    // the block that arrives last for this query tile reduces the partial minima
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(&sc->ticket[blockIdx.x], 1u) == (unsigned)(S - 1));
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const int lane = tid & 31, warp = tid >> 5;
    for (int r = warp; r < kNaQ; r += 8) {
        const int i = q0 + r;
        if (i >= B) continue;
        double bd = INFINITY;
        int bs = 0x7fffffff;
        for (int s = lane; s < S; s += 32) {
            const double v = __ldcg(&sc->part_min[(size_t)i * kNaMaxSplits + s]);
            const int a = __ldcg(&sc->part_arg[(size_t)i * kNaMaxSplits + s]);
            if (v < bd || (v == bd && a < bs)) { bd = v; bs = a; }
        }
#pragma unroll
        for (int m = 1; m < 32; m <<= 1) {
            const double od = __shfl_xor_sync(0xffffffffu, bd, m);
            const int os = __shfl_xor_sync(0xffffffffu, bs, m);
            if (od < bd || (od == bd && os < bs)) { bd = od; bs = os; }
        }
        if (lane == 0) {
            out_slot[i] = bs;
            out_dist[i] = (float)bd;
        }
    }
    if (tid == 0) sc->ticket[blockIdx.x] = 0;           // leave the counter clean for the next call
}

struct PerDevice {
    NaScratch *scratch = nullptr;     // device address of g_na_scratch on this GPU
    int sms = 0;
};
PerDevice g_dev[64];
std::mutex g_dev_mutex;

}  // namespace

extern "C" int32_t prox_nearest_key_static(const float *keys, int64_t n_keys, int32_t d, const float *queries,
                                           int32_t B, int32_t *out_slot, float *out_dist, void *stream) {
    if (!keys || !queries || !out_slot || !out_dist) {
        prox::set_last_error("prox_nearest_key_static: NULL pointer");
        return PROX_ERR_INVALID_ARG;
    }
    if (B < 1 || B > PROX_STATIC_MAX_BATCH) {
        prox::set_last_error("prox_nearest_key_static: B = %d is outside [1, %d], the size the built-in scratch holds",
                             (int)B, (int)PROX_STATIC_MAX_BATCH);
        return PROX_ERR_INVALID_ARG;
    }
    if (n_keys < 1 || n_keys > PROX_STATIC_MAX_KEYS || d < 1 || d > 4096) {
        prox::set_last_error("prox_nearest_key_static: need 1 <= n_keys <= %lld and 1 <= d <= 4096",
                             (long long)PROX_STATIC_MAX_KEYS);
        return PROX_ERR_INVALID_ARG;
    }
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        prox::set_last_error("prox_nearest_key_static: no usable current CUDA device");
        return PROX_ERR_CUDA;
    }
    PerDevice pd;
    {
        // once per GPU, with that GPU current: the name g_na_scratch is only a host-side stand-in,
        // the kernel needs the address the runtime reports for it
        std::lock_guard<std::mutex> lock(g_dev_mutex);
        if (!g_dev[dev].scratch) {
            NaScratch *p = nullptr;
            cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void **>(&p), g_na_scratch);
            int sms = 0;
            if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
            if (e != cudaSuccess || !p) {
                cudaGetLastError();
                prox::set_last_error("prox_nearest_key_static: set-up failed: %s", cudaGetErrorString(e));
                return PROX_ERR_CUDA;
            }
            g_dev[dev].scratch = p;
            g_dev[dev].sms = sms;
        }
        pd = g_dev[dev];
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the arrival counters must start at zero even if an earlier call was cut short
    if (cudaMemsetAsync(pd.scratch->ticket, 0, sizeof(unsigned) * kNaQTiles, s) != cudaSuccess) {
        prox::set_last_error("prox_nearest_key_static: %s", cudaGetErrorString(cudaGetLastError()));
        return PROX_ERR_CUDA;
    }
    const int qtiles = (B + kNaQ - 1) / kNaQ;
    const long long ntiles = (n_keys + kNaC - 1) / kNaC;
    long long S = (4LL * pd.sms + qtiles - 1) / qtiles;
    if (S > ntiles) S = ntiles;
    if (S > kNaMaxSplits) S = kNaMaxSplits;
    if (S < 1) S = 1;
    nearest_static_kernel<<<dim3(qtiles, (unsigned)S), 256, 0, s>>>(keys, (long long)n_keys, d, queries, B, pd.scratch,
                                                                    out_slot, out_dist);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        prox::set_last_error("prox_nearest_key_static: %s", cudaGetErrorString(e));
        return PROX_ERR_CUDA;
    }
    return PROX_OK;
}
