// A corpus split by rows over several GPUs: the exchange record of one shard's miss results and
// the merge of all shards' records into the k nearest rows of the whole corpus (the database
// call of Algorithm 1, answered by G shards).
#include "prox_internal.h"

namespace prox {

// One shard's record: kMax = B * k fp64 distances, then B * k int64 ids of the whole corpus.
// Miss j of the batch owns entries j*k .. j*k+k-1; places beyond the number of misses are
// filled with (+inf, -1) so that every byte of the record is defined.
__global__ void __launch_bounds__(256)
shard_pack_kernel(const DevState *__restrict__ st, int B, int k, long long row_offset,
                  const int32_t *__restrict__ res_ids, const double *__restrict__ res_dists, double *x_dist,
                  long long *x_id) {
    const int n = B * k;
    const int live = st->n_miss * k;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < n; e += gridDim.x * blockDim.x) {
        const bool on = e < live && res_ids[e] >= 0;
        x_dist[e] = on ? res_dists[e] : __longlong_as_double(0x7ff0000000000000LL);
        x_id[e] = on ? (long long)res_ids[e] + row_offset : -1LL;
    }
}

// (distance, id) order of the result lists: nearer first, ties by lower id; an empty place
// (id -1) comes after everything.
__device__ __forceinline__ bool entry_before(double da, long long ia, double db, long long ib) {
    if (ia < 0) return false;
    if (ib < 0) return true;
    return da < db || (da == db && ia < ib);
}

// One warp per miss: lane g walks the (sorted) list of shard g; k rounds, each taking the
// smallest head of the G lists.  G <= 32.
__global__ void __launch_bounds__(128)
shard_merge_kernel(const DevState *__restrict__ st, int B, int k, int G, const unsigned char *__restrict__ gathered,
                   int32_t *res_ids, double *res_dists) {
    const int lane = threadIdx.x & 31;
    const int m = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (m >= st->n_miss) return;
    const size_t n = (size_t)B * k;
    const size_t rec = n * 16;
    const double *dl = nullptr;
    const long long *il = nullptr;
    if (lane < G) {
        dl = reinterpret_cast<const double *>(gathered + (size_t)lane * rec) + (size_t)m * k;
        il = reinterpret_cast<const long long *>(gathered + (size_t)lane * rec + n * 8) + (size_t)m * k;
    }
    int pos = 0;
    double hd = 0.0;
    long long hi = -1;
    if (lane < G) { hd = dl[0]; hi = il[0]; }
    for (int r = 0; r < k; ++r) {
        double bd = hd;
        long long bi = hi;
        int bl = lane;
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) {
            const double od = __shfl_xor_sync(0xffffffffu, bd, s);
            const long long oi = __shfl_xor_sync(0xffffffffu, bi, s);
            const int ol = __shfl_xor_sync(0xffffffffu, bl, s);
            // equal (distance, id) pairs cannot come from two shards (ids are disjoint); the lane
            // number settles the order among empty heads so that all lanes agree
            if (entry_before(od, oi, bd, bi) || (oi < 0 && bi < 0 && ol < bl)) { bd = od; bi = oi; bl = ol; }
        }
        if (lane == 0) {
            res_ids[(size_t)m * k + r] = (int32_t)bi;
            res_dists[(size_t)m * k + r] = bi >= 0 ? bd : 0.0;
        }
        if (lane == bl && bi >= 0) {
            ++pos;
            if (pos < k) { hd = dl[pos]; hi = il[pos]; } else { hi = -1; }
        }
    }
}

void launch_shard_pack(prox_handle *h, int B, void *xchg, cudaStream_t s) {
    const int n = B * h->k;
    double *x_dist = static_cast<double *>(xchg);
    long long *x_id = reinterpret_cast<long long *>(x_dist + n);
    shard_pack_kernel<<<(n + 255) / 256, 256, 0, s>>>(h->st, B, h->k, (long long)h->row_offset, h->res_ids,
                                                      h->res_dists, x_dist, x_id);
    h->launches++;
}

void launch_shard_merge(prox_handle *h, int B, const void *gathered, int G, cudaStream_t s) {
    shard_merge_kernel<<<(B * 32 + 127) / 128, 128, 0, s>>>(h->st, B, h->k, G,
                                                           static_cast<const unsigned char *>(gathered), h->res_ids,
                                                           h->res_dists);
    h->launches++;
}

}  // namespace prox
