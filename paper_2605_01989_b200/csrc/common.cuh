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
//   tensor_tab[t]   = (numel low, numel high, sequence number of the tensor's first chunk, 0): what the integrity
//                     check needs, in one 16-byte load;  base[t] = first flat element of tensor t
//   bucket_bounds[0..B], bound_ppm[B] (staging for per-bucket tolerances), ticket (see k_bound)
// The staging buffer and the ticket make a plan serve one dblp_check_bound at a time.
struct dblp_plan {
    uint32_t T, W, B, P, es, E, VE, VPC;
    // where packets live: header of slot i at hdr_ring + i * hdr_stride, payload at payload_ring + pay_off + i * pay_stride
    // (separate rings: 32, P, 0; datagrams with the header in front: 32 + P, 32 + P, 32)
    uint32_t hdr_stride, pay_stride, pay_off;
    int dtype, device;
    uint64_t C, N, M, row_words;
    // A shard of a split server (dblp_plan_set_shard) covers sequence numbers seq_off .. seq_off + C - 1 of a worker
    // stream of C_stream chunks; otherwise C_stream = C and seq_off = 0.  Only the loss process looks at these.
    uint64_t C_stream, seq_off;
    std::vector<uint64_t> h_numel, h_base;
    std::vector<uint32_t> h_chunkbase;
    uint4* d_tensor_tab;
    uint64_t* d_base;
    uint64_t* d_chunk_desc;
    uint32_t* d_chunk_tensor;
    uint32_t* d_bucket_bounds;
    uint32_t* d_bound_ppm;
    uint32_t* d_ticket;     // "blocks finished" counter of k_bound; zero between launches
    // Host-side resources of the whole-round calls (round.cu): a high-priority stream for the work that runs beside
    // the two bandwidth-bound kernels, a stream for host-to-device copies, and the events that order them.  They make
    // a plan serve one whole-round call at a time.
    cudaStream_t side, copy, back;
    cudaEvent_t ev_fork, ev_join, ev_claimed, ev_done, ev_copy[2], ev_part[2], ev_back;
    // launch shape of the masked reduce (configure_reduce): red_variant = items per thread of the tiled kernel,
    // 0 = the simple one-vector-per-thread kernel
    uint32_t red_variant, red_CH, red_tiles, red_grid, red_rows;
    size_t red_smem;
    // block order of packetize: 1 = tile by tile with all workers of a tile together, 0 = worker by worker.
    // Tile-major leaves the end of every worker's ring in L2, which is where the masked reduce starts reading (it
    // walks the tiles from the last one down); it pays while the ring is only a few times the L2 and costs about 2 %
    // of the copy rate on rings of many GB, so the plan picks it for rings up to 16 times the L2.
    uint32_t pack_tile_major;
    // dblp_round_reset as one kernel that leaves the claim table in L2 (tables up to a quarter of the L2), instead of
    // three memsets
    uint32_t reset_in_l2;
    // dblp_round_receive groups the arrivals by slot range before claiming (dblp_aggregate_claim_grouped): chosen when
    // headers and claim table together exceed the L2
    uint32_t claim_grouped;
    void* d_claim_ws;       // scratch of the grouped claims (dblp_claim_workspace_bytes(M, M) bytes); null unless claim_grouped
    size_t claim_ws_bytes;
};

namespace dblp {
int configure_reduce(dblp_plan* p, uint32_t ch_override, uint32_t grid_override);
// dblp_packetize for workers w0 .. w0 + nw - 1 and chunks chunk_lo .. chunk_hi - 1 only; grads[k] is worker (w0 + k)'s
// whole gradient.
int packetize_workers(const dblp_plan* plan, const void* const* grads, uint32_t w0, uint32_t nw, uint32_t round,
                      dblp_hdr_t* hdr_ring, void* payload_ring, uint64_t chunk_lo, uint64_t chunk_hi, cudaStream_t s);
// dblp_aggregate_claim, optionally as one of several passes over the arrival list: with part_hi != 0 only the entries
// whose slot number modulo C lies in [part_lo, part_hi) are examined (and counted); part_hi = 0 takes all.
int claim_arrivals(const dblp_plan* plan, const dblp_hdr_t* hdr_ring, uint64_t n_slots, const uint32_t* arrival,
                   const uint64_t* n_arrived_dev, uint64_t arrival_cap, uint32_t round, uint64_t* slot_key,
                   dblp_counters_t* counters, uint32_t part_lo, uint32_t part_hi, cudaStream_t s);
// dblp_aggregate_reduce for chunks chunk_lo .. chunk_hi - 1 (whole tiles of the tiled reduce: chunk_lo a multiple of
// red_CH, chunk_hi a multiple of it or C); needs red_variant != 0.
int reduce_chunks(const dblp_plan* plan, const void* payload_ring, const uint64_t* slot_key, float* agg_out, uint32_t flags,
                  uint64_t chunk_lo, uint64_t chunk_hi, cudaStream_t s);
}
