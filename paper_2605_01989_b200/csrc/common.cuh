// Shared declarations of libdblp's translation units: the plan object, error plumbing, the launch counter and the
// counter-based generator used by the loss and arrival kernels.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <vector>

#include "dblp.h"

namespace dblp {

constexpr uint32_t kEmpty32 = 0xFFFFFFFFu;
constexpr unsigned long long kEmpty64 = ~0ull;
constexpr uint32_t kMaxWorkersPerLaunch = 64;  // gradient pointers travel in the kernel parameter block

// Purposes of a Philox draw: kept apart by the low byte of counter word 2.
enum : uint32_t { kStreamPacket = 1, kStreamGeInit = 2, kStreamWindow = 3, kStreamPerm = 4 };

void set_error(const char* fmt, ...);
extern std::atomic<uint64_t> g_launches;

#define DBLP_CUDA(call)                                                                         \
    do {                                                                                        \
        cudaError_t e_ = (call);                                                                \
        if (e_ != cudaSuccess) {                                                                \
            dblp::set_error("%s failed: %s (%s:%d)", #call, cudaGetErrorString(e_), __FILE__, __LINE__); \
            return DBLP_ECUDA;                                                                  \
        }                                                                                       \
    } while (0)

#define DBLP_LAUNCHED()                                                                         \
    do {                                                                                        \
        dblp::g_launches.fetch_add(1, std::memory_order_relaxed);                               \
        cudaError_t e_ = cudaGetLastError();                                                    \
        if (e_ != cudaSuccess) {                                                                \
            dblp::set_error("kernel launch failed: %s (%s:%d)", cudaGetErrorString(e_), __FILE__, __LINE__); \
            return DBLP_ECUDA;                                                                  \
        }                                                                                       \
    } while (0)

#define DBLP_REQUIRE(cond, status, ...)                                                         \
    do {                                                                                        \
        if (!(cond)) {                                                                          \
            dblp::set_error(__VA_ARGS__);                                                       \
            return (status);                                                                    \
        }                                                                                       \
    } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies, an xor mix with the key, and a Weyl
// step on the key.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), hi1 = __umulhi(0xCD9E8D57u, c.z);
        const uint32_t lo0 = 0xD2511F53u * c.x, lo1 = 0xCD9E8D57u * c.z;
        c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
        k.x += 0x9E3779B9u;
        k.y += 0xBB67AE85u;
    }
    return c;
}

struct DrawKey {
    uint2 key;         // seed low, high
    uint32_t attempt8; // attempt << 8
    uint32_t round;
};

__device__ __forceinline__ uint4 draw(const DrawKey& k, uint64_t a, uint32_t stream)
{
    return philox4x32_10(make_uint4((uint32_t)a, (uint32_t)(a >> 32), stream | k.attempt8, k.round), k.key);
}

}  // namespace dblp

// The plan: immutable after creation.  Device tables:
//   chunk_desc[c]   = (first element of chunk c in the flat gradient) << 16 | elements in the chunk
//   chunk_tensor[c] = tensor the chunk belongs to
//   numel[t], base[t] (first flat element of tensor t), chunkbase[t] (sequence number of its first chunk; [T] = C)
//   bucket_bounds[0..B], bound_ppm[B] (staging for per-bucket tolerances), ticket (see k_bound)
// The staging buffer and the ticket make a plan serve one dblp_check_bound at a time.
struct dblp_plan {
    uint32_t T, W, B, P, es, E, VE, VPC;
    // where packets live: header of slot i at hdr_ring + i * hdr_stride, payload at payload_ring + pay_off + i * pay_stride
    // (separate rings: 32, P, 0; datagrams with the header in front: 32 + P, 32 + P, 32)
    uint32_t hdr_stride, pay_stride, pay_off;
    int dtype, device;
    uint64_t C, N, M, row_words;
    std::vector<uint64_t> h_numel, h_base;
    std::vector<uint32_t> h_chunkbase;
    uint64_t* d_numel;
    uint64_t* d_base;
    uint32_t* d_chunkbase;
    uint64_t* d_chunk_desc;
    uint32_t* d_chunk_tensor;
    uint32_t* d_bucket_bounds;
    uint32_t* d_bound_ppm;
    uint32_t* d_ticket;     // "blocks finished" counter of k_bound; zero between launches
    // launch shape of the masked reduce (configure_reduce): red_variant = items per thread of the tiled kernel,
    // 0 = the simple one-vector-per-thread kernel
    uint32_t red_variant, red_CH, red_tiles, red_grid, red_rows;
    size_t red_smem;
};

namespace dblp {
int configure_reduce(dblp_plan* p, uint32_t ch_override, uint32_t grid_override);
}
