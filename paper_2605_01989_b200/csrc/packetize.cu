// dblp_packetize: gradients -> header ring + payload ring (Algorithm 1 "split data into chunks"; Sections IV-A, IV-B).
//
// A pure copy, bound by HBM.  A block owns a tile of CH consecutive chunks (about 32 KB) of one worker: it first brings the tile's
// chunk descriptors into shared memory (so that no payload load waits on a table lookup), writes the tile's headers,
// then streams the tile's 16-byte vectors, kPackUnroll per thread per pass with all loads issued before the first
// store.  The source follows the descriptors, so tensors of any size are handled: a vector that is ragged (end of a
// short chunk) or whose source is not 16-byte aligned is assembled from element loads, and the slot's tail is written
// as zero.  Blocks run either worker by worker (grid.y = worker) or tile by tile with a tile's workers side by side
// (one-dimensional grid, nw_fast = workers of the launch); the plan chooses, see dblp_plan::pack_tile_major.
#include "common.cuh"

namespace dblp {

struct GradPtrs {
    const void* p[kMaxWorkersPerLaunch];
};

constexpr int kPackThreads = 256;
constexpr int kPackUnroll = 4;       // 2 and 8 vectors per thread per pass measured slower

__device__ __forceinline__ uint4 ld_stream16(const void* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ void st_stream16(void* p, uint4 v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

constexpr uint32_t kPackMaxTile = 256;     // chunks per tile at most (descriptors live in static shared memory)

// Headers are re-read in arrival (that is, random) order by the bookkeeping a moment later: ask L2 to keep them
// while the payloads stream through.
__device__ __forceinline__ void st_keep16(void* p, uint4 v)
{
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(policy));
    asm volatile("st.global.L2::cache_hint.v4.u32 [%0], {%1,%2,%3,%4}, %5;" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w),
                 "l"(policy)
                 : "memory");
}

template <int ES>
__global__ void __launch_bounds__(kPackThreads)
k_packetize(GradPtrs grads, uint32_t w0, uint32_t nw_fast, uint32_t c_lo, uint32_t c_hi, uint32_t C, uint32_t VPC,
            uint32_t pay_stride, uint32_t hdr_stride, uint32_t CH, uint32_t round,
            const uint64_t* __restrict__ chunk_desc, const uint32_t* __restrict__ chunk_tensor,
            const uint64_t* __restrict__ tensor_base, dblp_hdr_t* __restrict__ hdr_ring, uint8_t* __restrict__ ring)
{
    constexpr uint32_t VE = 16 / ES;
    __shared__ uint64_t s_desc[kPackMaxTile];
    uint32_t tile = blockIdx.x, wl = blockIdx.y;
    if (nw_fast) {                                      // tile-major: consecutive blocks are the workers of one tile
        tile = blockIdx.x / nw_fast;
        wl = blockIdx.x - tile * nw_fast;
    }
    const uint32_t w = w0 + wl, tid = threadIdx.x;
    const uint8_t* __restrict__ g = static_cast<const uint8_t*>(grads.p[wl]);
    const uint32_t c0 = c_lo + tile * CH, nch = min(CH, c_hi - c0);     // the launch covers chunks c_lo .. c_hi - 1
    const uint64_t slot0 = (uint64_t)w * C + c0;

    for (uint32_t k = tid; k < nch; k += kPackThreads) {
        const uint64_t d = __ldg(&chunk_desc[c0 + k]);
        s_desc[k] = d;
        const uint32_t t = __ldg(&chunk_tensor[c0 + k]);
        const uint64_t off = (d >> 16) - __ldg(&tensor_base[t]);
        uint4* h = reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(hdr_ring) + (slot0 + k) * hdr_stride);
        st_keep16(h, make_uint4(c0 + k, round, (uint32_t)(d & 0xFFFFu) * ES, t));
        st_keep16(h + 1, make_uint4((uint32_t)off, (uint32_t)(off >> 32), w, 0u));
    }
    __syncthreads();

    const uint32_t nvec = nch * VPC;
    uint8_t* __restrict__ out = ring + slot0 * pay_stride;        // first slot of the tile
    for (uint32_t i0 = tid; i0 < nvec; i0 += kPackThreads * kPackUnroll) {
        uint4 val[kPackUnroll];
#pragma unroll
        for (int u = 0; u < kPackUnroll; ++u) {
            const uint32_t i = i0 + u * kPackThreads;
            val[u] = make_uint4(0, 0, 0, 0);
            if (i >= nvec) continue;
            const uint32_t cl = i / VPC, v = i - cl * VPC;
            const uint64_t d = s_desc[cl];
            const uint32_t len = (uint32_t)(d & 0xFFFFu), e0 = v * VE;
            if (e0 >= len) continue;                       // wholly past the data of a short chunk: zero fill
            const uint32_t nv = min(VE, len - e0);
            const uint8_t* src = g + ((d >> 16) + e0) * ES;
            if (nv == VE && (reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
                val[u] = ld_stream16(src);
            } else {
                uint32_t wd[4] = {0, 0, 0, 0};
#pragma unroll
                for (uint32_t e = 0; e < VE; ++e) {
                    if (e < nv) {
                        if (ES == 4) wd[e] = __ldg(reinterpret_cast<const uint32_t*>(src) + e);
                        else wd[e >> 1] |= (uint32_t)__ldg(reinterpret_cast<const uint16_t*>(src) + e) << (16 * (e & 1));
                    }
                }
                val[u] = make_uint4(wd[0], wd[1], wd[2], wd[3]);
            }
        }
#pragma unroll
        for (int u = 0; u < kPackUnroll; ++u) {
            const uint32_t i = i0 + u * kPackThreads;
            if (i >= nvec) continue;
            const uint32_t cl = i / VPC, v = i - cl * VPC;
            st_stream16(out + (uint64_t)cl * pay_stride + (uint64_t)v * 16, val[u]);
        }
    }
}

int packetize_workers(const dblp_plan* plan, const void* const* grads, uint32_t w_first, uint32_t n_workers, uint32_t round,
                      dblp_hdr_t* hdr_ring, void* payload_ring, uint64_t chunk_lo, uint64_t chunk_hi, cudaStream_t s)
{
    DBLP_REQUIRE(chunk_lo < chunk_hi && chunk_hi <= plan->C, DBLP_EINVAL, "packetize: empty or out-of-range chunk range");
    // about 32 KB of payload per block: measured against 8, 16 and 64 KB (64 KB: 4 % slower on 10-50 GB rings; 16 KB:
    // faster on 10 GB, slower on 50 GB; 8 KB: slower everywhere)
    uint32_t CH = (2048u + plan->VPC - 1) / plan->VPC;
    if (CH > kPackMaxTile) CH = kPackMaxTile;
    const uint64_t gx = (chunk_hi - chunk_lo + CH - 1) / CH;
    DBLP_REQUIRE(gx * kMaxWorkersPerLaunch < (1ull << 31), DBLP_ECAPACITY, "packetize: grid too large");
    for (uint32_t w0 = w_first; w0 < w_first + n_workers; w0 += kMaxWorkersPerLaunch) {
        const uint32_t nw = min(kMaxWorkersPerLaunch, w_first + n_workers - w0);
        GradPtrs gp{};
        for (uint32_t k = 0; k < nw; ++k) gp.p[k] = grads[w0 - w_first + k];
        const uint32_t nw_fast = plan->pack_tile_major ? nw : 0u;
        const dim3 grid = nw_fast ? dim3((unsigned)(gx * nw), 1) : dim3((unsigned)gx, nw);
        if (plan->es == 4)
            k_packetize<4><<<grid, kPackThreads, 0, s>>>(gp, w0, nw_fast, (uint32_t)chunk_lo, (uint32_t)chunk_hi, (uint32_t)plan->C, plan->VPC, plan->pay_stride, plan->hdr_stride, CH, round,
                plan->d_chunk_desc, plan->d_chunk_tensor, plan->d_base, hdr_ring, static_cast<uint8_t*>(payload_ring) + plan->pay_off);
        else
            k_packetize<2><<<grid, kPackThreads, 0, s>>>(gp, w0, nw_fast, (uint32_t)chunk_lo, (uint32_t)chunk_hi, (uint32_t)plan->C, plan->VPC, plan->pay_stride, plan->hdr_stride, CH, round,
                plan->d_chunk_desc, plan->d_chunk_tensor, plan->d_base, hdr_ring, static_cast<uint8_t*>(payload_ring) + plan->pay_off);
        DBLP_LAUNCHED();
    }
    return DBLP_OK;
}

}  // namespace dblp

using namespace dblp;

extern "C" int dblp_packetize(const dblp_plan_t* plan, const void* const* grads, uint32_t round, dblp_hdr_t* hdr_ring,
                              void* payload_ring, void* stream)
{
    DBLP_REQUIRE(plan && grads && hdr_ring && payload_ring, DBLP_EINVAL, "packetize: null argument");
    DBLP_REQUIRE(aligned16(hdr_ring) && aligned16(payload_ring), DBLP_EALIGN, "packetize: rings must be 16-byte aligned");
    for (uint32_t w = 0; w < plan->W; ++w) {
        DBLP_REQUIRE(grads[w], DBLP_EINVAL, "packetize: gradient pointer of worker %u is null", w);
        DBLP_REQUIRE((reinterpret_cast<uintptr_t>(grads[w]) % plan->es) == 0, DBLP_EALIGN,
                     "packetize: gradient of worker %u is not element-aligned", w);
    }
    return packetize_workers(plan, grads, 0, plan->W, round, hdr_ring, payload_ring, 0, plan->C, static_cast<cudaStream_t>(stream));
}
