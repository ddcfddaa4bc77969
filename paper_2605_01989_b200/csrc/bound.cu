// dblp_check_bound: per (worker, bucket) popcount of the received bitmap and the tolerance test
// (Section III-B: retransmission stops once missing / total <= p; Algorithm 2: stop signal, else bitmap reply).
#include "common.cuh"

namespace dblp {

constexpr int kBoundThreads = 512;

__global__ void __launch_bounds__(kBoundThreads)
k_bound(const uint32_t* __restrict__ bitmap, uint64_t row_words, const uint32_t* __restrict__ bucket_bounds, uint32_t B,
        uint32_t bound_scalar, const uint32_t* __restrict__ bound_per_bucket, uint32_t* __restrict__ recv_cnt,
        uint32_t* __restrict__ missing_cnt, uint8_t* ok, uint32_t* __restrict__ all_ok, uint32_t* ticket)
{
    __shared__ uint32_t s_warp[kBoundThreads / 32];
    __shared__ bool s_last;
    const uint32_t b = blockIdx.x, w = blockIdx.y;
    const uint32_t lo = bucket_bounds[b], hi = bucket_bounds[b + 1];
    const uint32_t* row = bitmap + (uint64_t)w * row_words;
    uint32_t n = 0;
    if (hi > lo) {
        const uint32_t first = lo >> 5, last = (hi - 1) >> 5;          // words that hold bits of [lo, hi)
        for (uint32_t k = first + threadIdx.x; k <= last; k += kBoundThreads) {
            uint32_t x = __ldg(&row[k]);
            if (k == first) x &= 0xFFFFFFFFu << (lo & 31);
            if (k == last && (hi & 31)) x &= (1u << (hi & 31)) - 1u;
            n += __popc(x);
        }
    }
    n = __reduce_add_sync(0xFFFFFFFFu, n);
    if ((threadIdx.x & 31) == 0) s_warp[threadIdx.x >> 5] = n;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t got = 0;
        for (int k = 0; k < kBoundThreads / 32; ++k) got += s_warp[k];
        const uint64_t total = hi - lo, miss = total - got;
        const uint64_t p = bound_per_bucket ? bound_per_bucket[b] : bound_scalar;
        const uint64_t cell = (uint64_t)w * B + b;
        recv_cnt[cell] = got;
        missing_cnt[cell] = (uint32_t)miss;
        ok[cell] = miss * 1000000ull <= p * total;
        // the block that finishes last (a counter, nobody waits) folds the flags into all_ok and rearms the counter
        __threadfence();
        s_last = atomicAdd(ticket, 1u) == gridDim.x * gridDim.y - 1;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    int bad = 0;
    const uint32_t cells = gridDim.x * gridDim.y;
    for (uint32_t i = threadIdx.x; i < cells; i += kBoundThreads) bad |= !__ldcg(&ok[i]);
    const int any_bad = __syncthreads_or(bad);
    if (threadIdx.x == 0) {
        *all_ok = any_bad ? 0u : 1u;
        *ticket = 0;
    }
}

}  // namespace dblp

using namespace dblp;

extern "C" int dblp_check_bound(const dblp_plan_t* plan, const uint32_t* recv_bitmap, const uint32_t* bound_ppm,
                                uint32_t n_bounds, uint32_t* recv_cnt, uint32_t* missing_cnt, uint8_t* ok,
                                uint32_t* all_ok, void* stream)
{
    DBLP_REQUIRE(plan && recv_bitmap && bound_ppm && recv_cnt && missing_cnt && ok && all_ok, DBLP_EINVAL,
                 "check_bound: null argument");
    DBLP_REQUIRE(n_bounds == 1 || n_bounds == plan->B, DBLP_EINVAL, "check_bound: n_bounds must be 1 or B = %u", plan->B);
    DBLP_REQUIRE(plan->W <= 65535, DBLP_ECAPACITY, "check_bound: more than 65535 workers");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const uint32_t* per_bucket = nullptr;
    if (n_bounds > 1) {
        DBLP_CUDA(cudaMemcpyAsync(plan->d_bound_ppm, bound_ppm, sizeof(uint32_t) * n_bounds, cudaMemcpyHostToDevice, s));
        per_bucket = plan->d_bound_ppm;
    }
    dim3 grid(plan->B, plan->W);
    k_bound<<<grid, kBoundThreads, 0, s>>>(recv_bitmap, plan->row_words, plan->d_bucket_bounds, plan->B, bound_ppm[0],
                                           per_bucket, recv_cnt, missing_cnt, ok, all_ok, plan->d_ticket);
    DBLP_LAUNCHED();
    return DBLP_OK;
}

// The same rule as k_bound's, on the host, for counts that were summed over several GPUs.
extern "C" int dblp_bound_ok(uint64_t missing, uint64_t total, uint32_t bound_ppm)
{
    return missing * 1000000ull <= (uint64_t)bound_ppm * total ? 1 : 0;
}
