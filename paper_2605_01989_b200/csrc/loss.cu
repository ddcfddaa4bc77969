// dblp_apply_loss: the seeded loss process (delivered bitmap) and the permuted arrival list.
// The paper injects loss without naming a generator (Section II-C "randomly zeroing out a fraction"; Section V-B
// "manually injecting bursty packet loss"); the processes are defined in dblp.h, in integers, on Philox4x32-10 draws.
//
// Memoryless kinds (none / iid / microburst): one thread per packet, warp ballot -> one bitmap word per warp.
// Gilbert-Elliott: the two-state chain is sequential by definition.  Each packet's transition is a function
// {Good, Bad} -> {Good, Bad} (four possibilities, two bits); composition is associative, so the state at every packet
// follows from a prefix "sum" of functions: a warp draws the 32 packets of a bitmap word in parallel and scans their
// functions with shuffles, a block combines its warps, a second small pass over the block totals gives every block
// its entry state, and a third pass judges every packet in its now known state (ballot -> bitmap word).
// The start of a worker's row contributes a constant function (its drawn initial state), which resets the chain with
// no special casing.  None of the passes waits on another block.
// Arrival: pi(a) for a = 0 .. M-1 by a 4-round Feistel network with cycle walking (each thread walks four
// consecutive a one after the other, which evens out the walk lengths across a warp); survivors are compacted in
// order of a with ballot / popcount prefix sums over three passes.
#include "common.cuh"

namespace dblp {

constexpr int kLossThreads = 256;
constexpr int kGeThreads = 256;
constexpr int kGeWordsPerWarp = 4;
constexpr int kGeWordsPerBlock = kGeThreads / 32 * kGeWordsPerWarp;   // bitmap words one block of the chain passes covers
constexpr int kScanThreads = 1024;   // single-block scans over block totals
constexpr int kPermThreads = 1024;   // arrival positions per block of the compaction passes
constexpr int kPermWalkers = 256;    // threads of k_perm_flags; each walks kPermThreads / kPermWalkers positions

struct LossParams {
    uint32_t kind;
    uint64_t t_drop, t_gb, t_bg, t_init_bad, t_drop_good, t_drop_bad, window_len, t_drop_in, t_drop_out;
};

// ------------------------------------------------------------------------------------------------ memoryless kinds
__global__ void __launch_bounds__(kLossThreads)
k_loss_pointwise(LossParams m, DrawKey dk, uint32_t W, uint64_t C, uint64_t row_words, uint64_t C_stream, uint64_t seq_off,
                 const uint32_t* __restrict__ sent, uint32_t* __restrict__ delivered)
{
    // C_stream, seq_off: the plan covers sequence numbers seq_off .. seq_off + C - 1 of a worker stream of C_stream
    // chunks (a shard of a split server; C_stream = C and seq_off = 0 otherwise).  Draws and the burst window live in
    // the stream's numbering, so every shard sees the packet fates of the unsplit round.
    __shared__ uint64_t s_window_start;
    if (m.kind == DBLP_LOSS_MICROBURST) {
        if (threadIdx.x == 0) s_window_start = (uint64_t)draw(dk, 0, kStreamWindow).x % (C_stream - m.window_len + 1);
        __syncthreads();
    }
    const uint64_t i = (uint64_t)blockIdx.x * kLossThreads + threadIdx.x;   // (row, word, lane)
    const uint64_t row_bits = row_words * 32;
    if (i >= row_bits * W) return;
    const uint32_t w = (uint32_t)(i / row_bits);
    const uint64_t seq = i - (uint64_t)w * row_bits;
    bool alive = false;
    if (seq < C && (!sent || ((__ldg(&sent[(uint64_t)w * row_words + (seq >> 5)]) >> (seq & 31)) & 1u))) {
        uint64_t t = 0;
        const uint64_t gseq = seq_off + seq;
        if (m.kind == DBLP_LOSS_IID) t = m.t_drop;
        else if (m.kind == DBLP_LOSS_MICROBURST)
            t = (gseq >= s_window_start && gseq < s_window_start + m.window_len) ? m.t_drop_in : m.t_drop_out;
        const uint32_t u = draw(dk, (uint64_t)w * C_stream + gseq, kStreamPacket).x;
        alive = !((uint64_t)u < t);
    }
    const uint32_t word = __ballot_sync(0xFFFFFFFFu, alive);
    if ((threadIdx.x & 31) == 0) delivered[(uint64_t)w * row_words + (seq >> 5)] = word;
}

// ------------------------------------------------------------------------------------------------ Gilbert-Elliott
// A function f on one bit is stored as f(0) | f(1) << 1.  State 0 = Good, 1 = Bad.
__device__ __forceinline__ uint32_t fn_apply(uint32_t f, uint32_t x) { return (f >> x) & 1u; }
__device__ __forceinline__ uint32_t fn_after(uint32_t later, uint32_t earlier)   // later o earlier
{
    return fn_apply(later, earlier & 1u) | (fn_apply(later, earlier >> 1) << 1);
}
constexpr uint32_t kFnIdentity = 2u;

// One bitmap word (row w, word k) handled by a whole warp: lane b owns packet k*32+b.
struct GeLane {
    uint32_t before;     // composition of the word's packets that precede this lane's (identity for lane 0)
    uint32_t word_fn;    // composition of all the word's packets (uniform across the warp)
    uint32_t reset;      // kFnIdentity, or the constant function of the row's initial state (first word of a row)
    bool valid, drop_if_good, drop_if_bad;
};

__device__ __forceinline__ GeLane ge_word(const LossParams& m, const DrawKey& dk, const uint32_t* sent, uint64_t j, uint64_t C,
                                          uint64_t row_words)
{
    GeLane g;
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t w = (uint32_t)(j / row_words);
    const uint64_t k = j - (uint64_t)w * row_words;
    const uint64_t seq = k * 32 + lane;
    g.valid = seq < C && (!sent || ((__ldg(&sent[j]) >> lane) & 1u));   // packets that are not sent leave the chain alone
    uint32_t fn = kFnIdentity;          // so do the padding bits past the end of the row
    g.drop_if_good = g.drop_if_bad = false;
    if (g.valid) {
        const uint4 u = draw(dk, (uint64_t)w * C + seq, kStreamPacket);
        const uint32_t to_bad = (uint64_t)u.y < m.t_gb, stay_bad = !((uint64_t)u.y < m.t_bg);
        fn = to_bad | (stay_bad << 1);
        g.drop_if_good = (uint64_t)u.x < m.t_drop_good;
        g.drop_if_bad = (uint64_t)u.x < m.t_drop_bad;
    }
    uint32_t inc = fn;                  // inclusive scan over the lanes: lower lanes are applied first
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= (uint32_t)d) inc = fn_after(inc, o);
    }
    g.before = __shfl_up_sync(0xFFFFFFFFu, inc, 1);
    if (lane == 0) g.before = kFnIdentity;
    g.word_fn = __shfl_sync(0xFFFFFFFFu, inc, 31);
    g.reset = kFnIdentity;
    if (k == 0) {
        const uint32_t bad = (uint64_t)draw(dk, w, kStreamGeInit).x < m.t_init_bad;
        g.reset = bad | (bad << 1);
    }
    return g;
}

// Composition of the functions of the block's warps that come before this warp; *block_total receives all of them.
// warp_fn is uniform within each warp.
__device__ __forceinline__ uint32_t ge_block_prefix(uint32_t warp_fn, uint32_t* block_total)
{
    __shared__ uint32_t s_warp[kGeThreads / 32];
    const uint32_t warp = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0) s_warp[warp] = warp_fn;
    __syncthreads();
    uint32_t before = kFnIdentity, all = kFnIdentity;
    for (uint32_t k = 0; k < kGeThreads / 32; ++k) {
        if (k == warp) before = all;
        all = fn_after(s_warp[k], all);
    }
    *block_total = all;
    return before;
}

__global__ void __launch_bounds__(kGeThreads)
k_ge_partial(LossParams m, DrawKey dk, uint32_t W, uint64_t C, uint64_t row_words, const uint32_t* __restrict__ sent,
             uint8_t* __restrict__ block_fn)
{
    const uint64_t n_words = row_words * W;
    const uint64_t j0 = (uint64_t)blockIdx.x * kGeWordsPerBlock + (threadIdx.x >> 5) * kGeWordsPerWarp;
    uint32_t f = kFnIdentity;
    for (int q = 0; q < kGeWordsPerWarp; ++q) {
        if (j0 + q < n_words) {
            const GeLane g = ge_word(m, dk, sent, j0 + q, C, row_words);
            f = fn_after(g.word_fn, fn_after(g.reset, f));
        }
    }
    uint32_t total;
    ge_block_prefix(f, &total);
    if (threadIdx.x == 0) block_fn[blockIdx.x] = (uint8_t)total;
}

// One block: turns the per-block functions into the state with which each block is entered.
__global__ void __launch_bounds__(kScanThreads)
k_ge_block_states(const uint8_t* __restrict__ block_fn, uint8_t* __restrict__ block_state, uint32_t n_blocks)
{
    __shared__ uint32_t s_warp[kScanThreads / 32];
    const uint32_t per = (n_blocks + kScanThreads - 1) / kScanThreads;
    const uint32_t lo = min(n_blocks, threadIdx.x * per), hi = min(n_blocks, lo + per);
    uint32_t f = kFnIdentity;
    for (uint32_t b = lo; b < hi; ++b) f = fn_after(block_fn[b], f);
    // exclusive scan of f over the block's threads (thread order = application order)
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = f;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= (uint32_t)d) inc = fn_after(inc, o);
    }
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    uint32_t before = kFnIdentity;
    for (uint32_t k = 0; k < warp; ++k) before = fn_after(s_warp[k], before);
    uint32_t exc = __shfl_up_sync(0xFFFFFFFFu, inc, 1);
    if (lane == 0) exc = kFnIdentity;
    before = fn_after(exc, before);
    for (uint32_t b = lo; b < hi; ++b) {
        block_state[b] = (uint8_t)fn_apply(before, 0);   // the value fed in is irrelevant: word 0 starts with a reset
        before = fn_after(block_fn[b], before);
    }
}

__global__ void __launch_bounds__(kGeThreads)
k_ge_apply(LossParams m, DrawKey dk, uint32_t W, uint64_t C, uint64_t row_words, const uint32_t* __restrict__ sent,
           const uint8_t* __restrict__ block_state, uint32_t* __restrict__ delivered)
{
    const uint64_t n_words = row_words * W;
    const uint64_t j0 = (uint64_t)blockIdx.x * kGeWordsPerBlock + (threadIdx.x >> 5) * kGeWordsPerWarp;
    GeLane g[kGeWordsPerWarp];
    uint32_t f = kFnIdentity;
#pragma unroll
    for (int q = 0; q < kGeWordsPerWarp; ++q) {
        if (j0 + q < n_words) {
            g[q] = ge_word(m, dk, sent, j0 + q, C, row_words);
            f = fn_after(g[q].word_fn, fn_after(g[q].reset, f));
        }
    }
    uint32_t total;
    const uint32_t before = ge_block_prefix(f, &total);
    uint32_t state = fn_apply(before, block_state[blockIdx.x]);       // state in which the warp's first word is entered
#pragma unroll
    for (int q = 0; q < kGeWordsPerWarp; ++q) {
        if (j0 + q < n_words) {
            state = fn_apply(g[q].reset, state);
            const uint32_t mine = fn_apply(g[q].before, state);      // the packet is judged in the state it is sent in
            const bool alive = g[q].valid && !(mine ? g[q].drop_if_bad : g[q].drop_if_good);
            const uint32_t word = __ballot_sync(0xFFFFFFFFu, alive);
            if ((threadIdx.x & 31) == 0) delivered[j0 + q] = word;
            state = fn_apply(g[q].word_fn, state);
        }
    }
}

// ------------------------------------------------------------------------------------------------ arrival order
struct PermParams {
    uint32_t half;   // bits per Feistel half
    uint32_t mask;   // (1 << half) - 1
    uint32_t M;
};

__device__ __forceinline__ uint32_t feistel(const PermParams& pp, const DrawKey& dk, uint32_t x)
{
    uint32_t L = x >> pp.half, R = x & pp.mask;
#pragma unroll
    for (uint32_t r = 0; r < 4; ++r) {
        const uint32_t F = philox4x32_10(make_uint4(R, r, kStreamPerm | dk.attempt8, dk.round), dk.key).x & pp.mask;
        const uint32_t nl = R;
        R = L ^ F;
        L = nl;
    }
    return (L << pp.half) | R;
}

__global__ void __launch_bounds__(kPermWalkers)
k_perm_flags(PermParams pp, DrawKey dk, uint64_t C, uint64_t row_words, const uint32_t* __restrict__ delivered,
             uint32_t* __restrict__ perm_flag, uint32_t* __restrict__ block_count)
{
    constexpr uint32_t K = kPermThreads / kPermWalkers;
    __shared__ uint32_t s_warp[kPermWalkers / 32];
    const uint32_t a0 = blockIdx.x * kPermThreads + threadIdx.x * K;
    const uint32_t n = a0 < pp.M ? min(K, pp.M - a0) : 0;
    uint32_t out[K];
#pragma unroll
    for (uint32_t q = 0; q < K; ++q) out[q] = 0;
    uint32_t k = 0, x = a0, flags = 0;
    while (k < n) {       // every walk ends: a cycle of the permutation of [0, 2^b) that starts below M returns below M
        x = feistel(pp, dk, x);
        if (x < pp.M) {
            const uint32_t w = (uint32_t)(x / C);
            const uint64_t seq = x - (uint64_t)w * C;
            const uint32_t flag = (__ldg(&delivered[(uint64_t)w * row_words + (seq >> 5)]) >> (seq & 31)) & 1u;
#pragma unroll
            for (uint32_t q = 0; q < K; ++q)
                if (q == k) out[q] = x | (flag << 31);
            flags += flag;
            ++k;
            x = a0 + k;
        }
    }
#pragma unroll
    for (uint32_t q = 0; q < K; ++q)
        if (q < n) perm_flag[a0 + q] = out[q];
    flags = __reduce_add_sync(0xFFFFFFFFu, flags);
    if ((threadIdx.x & 31) == 0) s_warp[threadIdx.x >> 5] = flags;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t total = 0;
        for (int q = 0; q < kPermWalkers / 32; ++q) total += s_warp[q];
        block_count[blockIdx.x] = total;
    }
}

// One block: exclusive prefix sum of the per-block survivor counts (in place) and the total.
__global__ void __launch_bounds__(kScanThreads)
k_count_scan(uint32_t* __restrict__ block_count, uint32_t n_blocks, uint64_t* __restrict__ n_arrived)
{
    __shared__ uint32_t s_warp[kScanThreads / 32];
    const uint32_t per = (n_blocks + kScanThreads - 1) / kScanThreads;
    const uint32_t lo = min(n_blocks, threadIdx.x * per), hi = min(n_blocks, lo + per);
    uint32_t sum = 0;
    for (uint32_t b = lo; b < hi; ++b) sum += block_count[b];
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= (uint32_t)d) inc += o;
    }
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    uint32_t before = 0;
    for (uint32_t k = 0; k < warp; ++k) before += s_warp[k];
    uint32_t run = before + inc - sum;
    for (uint32_t b = lo; b < hi; ++b) {
        const uint32_t n = block_count[b];
        block_count[b] = run;
        run += n;
    }
    if (threadIdx.x == kScanThreads - 1) *n_arrived = run;
}

__global__ void __launch_bounds__(kPermThreads)
k_arrival_scatter(uint32_t M, const uint32_t* __restrict__ perm_flag, const uint32_t* __restrict__ block_offset,
                  uint32_t* __restrict__ arrival)
{
    __shared__ uint32_t s_warp[kPermThreads / 32];
    const uint32_t a = blockIdx.x * kPermThreads + threadIdx.x;
    const uint32_t pf = a < M ? perm_flag[a] : 0u;
    const bool flag = pf >> 31;
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t ballot = __ballot_sync(0xFFFFFFFFu, flag);
    if (lane == 0) s_warp[warp] = __popc(ballot);
    __syncthreads();
    if (!flag) return;
    uint32_t pos = block_offset[blockIdx.x] + __popc(ballot & ((1u << lane) - 1u));
    for (uint32_t k = 0; k < warp; ++k) pos += s_warp[k];
    arrival[pos] = pf & 0x7FFFFFFFu;
}

// dst row w = bits seq_off .. seq_off + C - 1 of src row w (rows of src_words / dst_words words; padding bits zero).
__global__ void __launch_bounds__(256)
k_bitmap_columns(const uint32_t* __restrict__ src, uint64_t src_words, uint32_t W, uint64_t seq_off, uint64_t C,
                 uint32_t* __restrict__ dst, uint64_t dst_words)
{
    const uint64_t j = (uint64_t)blockIdx.x * 256 + threadIdx.x;
    if (j >= dst_words * W) return;
    const uint32_t w = (uint32_t)(j / dst_words);
    const uint64_t k = j - (uint64_t)w * dst_words;
    const uint64_t first = seq_off + k * 32;                      // stream number of this word's bit 0
    const uint32_t* row = src + (uint64_t)w * src_words;
    const uint64_t sw = first >> 5;
    const uint32_t sh = (uint32_t)(first & 31);
    uint32_t x = row[sw] >> sh;
    if (sh && sw + 1 < src_words) x |= row[sw + 1] << (32 - sh);
    const uint64_t left = C - k * 32;                              // bits of the row that remain from this word on
    if (left < 32) x &= (1u << left) - 1u;
    dst[j] = x;
}

struct WorkspaceLayout {
    size_t perm_flag, block_count, ge_fn, ge_state, ge_mask, total;
    uint32_t n_perm_blocks, n_ge_blocks;
    uint64_t stream_words;      // bitmap words per row of the whole worker stream
    bool shard;
};

static WorkspaceLayout layout(const dblp_plan* p)
{
    WorkspaceLayout l{};
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    l.shard = p->C_stream != p->C;
    l.stream_words = (p->C_stream + 31) / 32;
    l.n_perm_blocks = (uint32_t)((p->M + kPermThreads - 1) / kPermThreads);
    l.n_ge_blocks = (uint32_t)((l.stream_words * p->W + kGeWordsPerBlock - 1) / kGeWordsPerBlock);
    l.perm_flag = 0;
    l.block_count = up(l.perm_flag + p->M * sizeof(uint32_t));
    l.ge_fn = up(l.block_count + (size_t)l.n_perm_blocks * sizeof(uint32_t));
    l.ge_state = up(l.ge_fn + l.n_ge_blocks);
    l.ge_mask = up(l.ge_state + l.n_ge_blocks);       // a shard's burst chain is run over the whole stream, then cut
    l.total = l.shard ? up(l.ge_mask + l.stream_words * p->W * sizeof(uint32_t)) : l.ge_mask;
    return l;
}

}  // namespace dblp

using namespace dblp;

extern "C" int dblp_workspace_bytes(const dblp_plan_t* plan, size_t* bytes)
{
    DBLP_REQUIRE(plan && bytes, DBLP_EINVAL, "workspace_bytes: null argument");
    *bytes = layout(plan).total;
    return DBLP_OK;
}

extern "C" int dblp_apply_loss_resend(const dblp_plan_t* plan, const dblp_loss_model_t* model, uint64_t seed,
                                      uint32_t round, uint32_t attempt, const uint32_t* sent_bits,
                                      uint32_t* delivered_bits, uint32_t* arrival, uint64_t* n_arrived_dev, void* ws,
                                      size_t ws_bytes, void* stream)
{
    DBLP_REQUIRE(plan && model && delivered_bits && arrival && n_arrived_dev && ws, DBLP_EINVAL, "apply_loss: null argument");
    DBLP_REQUIRE(model->kind <= DBLP_LOSS_MICROBURST, DBLP_EINVAL, "apply_loss: unknown loss kind %u", model->kind);
    DBLP_REQUIRE(attempt < (1u << 24), DBLP_ECAPACITY, "apply_loss: attempt must be below 2^24");
    const WorkspaceLayout l = layout(plan);
    DBLP_REQUIRE(ws_bytes >= l.total, DBLP_ECAPACITY, "apply_loss: workspace of %zu bytes, %zu needed", ws_bytes, l.total);
    DBLP_REQUIRE((reinterpret_cast<uintptr_t>(ws) & 255u) == 0, DBLP_EALIGN, "apply_loss: workspace must be 256-byte aligned");
    const uint64_t limit = 1ull << 32;
    DBLP_REQUIRE(model->t_drop <= limit && model->t_gb <= limit && model->t_bg <= limit && model->t_init_bad <= limit &&
                 model->t_drop_good <= limit && model->t_drop_bad <= limit && model->t_drop_in <= limit &&
                 model->t_drop_out <= limit, DBLP_EINVAL, "apply_loss: thresholds must lie in [0, 2^32]");
    if (model->kind == DBLP_LOSS_MICROBURST)
        DBLP_REQUIRE(model->window_len <= plan->C_stream, DBLP_EINVAL, "apply_loss: window longer than a worker's stream");
    DBLP_REQUIRE(!(l.shard && sent_bits && model->kind == DBLP_LOSS_GE), DBLP_EINVAL,
                 "apply_loss: a burst chain over a subset of sent packets needs the whole stream's send set, which a "
                 "shard plan does not have");

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t* base = static_cast<uint8_t*>(ws);
    uint32_t* perm_flag = reinterpret_cast<uint32_t*>(base + l.perm_flag);
    uint32_t* block_count = reinterpret_cast<uint32_t*>(base + l.block_count);
    uint8_t* ge_fn = base + l.ge_fn;
    uint8_t* ge_state = base + l.ge_state;

    LossParams m{model->kind, model->t_drop, model->t_gb, model->t_bg, model->t_init_bad, model->t_drop_good,
                 model->t_drop_bad, model->window_len, model->t_drop_in, model->t_drop_out};
    DrawKey dk{make_uint2((uint32_t)seed, (uint32_t)(seed >> 32)), attempt << 8, round};

    if (model->kind == DBLP_LOSS_GE) {
        // the chain is sequential along the whole worker stream: a shard runs it over the stream and keeps its columns
        uint32_t* chain_out = l.shard ? reinterpret_cast<uint32_t*>(base + l.ge_mask) : delivered_bits;
        k_ge_partial<<<l.n_ge_blocks, kGeThreads, 0, s>>>(m, dk, plan->W, plan->C_stream, l.stream_words, sent_bits, ge_fn);
        DBLP_LAUNCHED();
        k_ge_block_states<<<1, kScanThreads, 0, s>>>(ge_fn, ge_state, l.n_ge_blocks);
        DBLP_LAUNCHED();
        k_ge_apply<<<l.n_ge_blocks, kGeThreads, 0, s>>>(m, dk, plan->W, plan->C_stream, l.stream_words, sent_bits, ge_state,
                                                       chain_out);
        DBLP_LAUNCHED();
        if (l.shard) {
            const uint64_t words = plan->row_words * plan->W;
            k_bitmap_columns<<<(unsigned)((words + 255) / 256), 256, 0, s>>>(chain_out, l.stream_words, plan->W, plan->seq_off,
                                                                            plan->C, delivered_bits, plan->row_words);
            DBLP_LAUNCHED();
        }
    } else {
        const uint64_t threads = plan->row_words * 32 * plan->W;
        k_loss_pointwise<<<(unsigned)((threads + kLossThreads - 1) / kLossThreads), kLossThreads, 0, s>>>(
            m, dk, plan->W, plan->C, plan->row_words, plan->C_stream, plan->seq_off, sent_bits, delivered_bits);
        DBLP_LAUNCHED();
    }

    PermParams pp{};
    uint32_t bits = 2;
    while (bits < 32 && (1ull << bits) < plan->M) bits += 2;
    pp.half = bits / 2;
    pp.mask = (1u << pp.half) - 1u;
    pp.M = (uint32_t)plan->M;
    k_perm_flags<<<l.n_perm_blocks, kPermWalkers, 0, s>>>(pp, dk, plan->C, plan->row_words, delivered_bits, perm_flag, block_count);
    DBLP_LAUNCHED();
    k_count_scan<<<1, kScanThreads, 0, s>>>(block_count, l.n_perm_blocks, n_arrived_dev);
    DBLP_LAUNCHED();
    k_arrival_scatter<<<l.n_perm_blocks, kPermThreads, 0, s>>>(pp.M, perm_flag, block_count, arrival);
    DBLP_LAUNCHED();
    return DBLP_OK;
}

extern "C" int dblp_apply_loss(const dblp_plan_t* plan, const dblp_loss_model_t* model, uint64_t seed, uint32_t round,
                               uint32_t attempt, uint32_t* delivered_bits, uint32_t* arrival, uint64_t* n_arrived_dev,
                               void* ws, size_t ws_bytes, void* stream)
{
    return dblp_apply_loss_resend(plan, model, seed, round, attempt, nullptr, delivered_bits, arrival, n_arrived_dev, ws,
                                  ws_bytes, stream);
}

namespace dblp {
__global__ void __launch_bounds__(256)
k_missing_bits(const uint32_t* __restrict__ bitmap, uint32_t* __restrict__ sent, uint64_t C, uint64_t row_words, uint64_t n_words)
{
    const uint64_t j = (uint64_t)blockIdx.x * 256 + threadIdx.x;
    if (j >= n_words) return;
    const uint64_t k = j % row_words;
    uint32_t x = ~bitmap[j];
    if (k == row_words - 1 && (C & 31)) x &= (1u << (C & 31)) - 1u;       // padding bits are not chunks
    sent[j] = x;
}
}  // namespace dblp

extern "C" int dblp_missing_bits(const dblp_plan_t* plan, const uint32_t* recv_bitmap, uint32_t* sent_bits, void* stream)
{
    DBLP_REQUIRE(plan && recv_bitmap && sent_bits, DBLP_EINVAL, "missing_bits: null argument");
    const uint64_t n = plan->row_words * plan->W;
    k_missing_bits<<<(unsigned)((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(recv_bitmap, sent_bits, plan->C,
                                                                                               plan->row_words, n);
    DBLP_LAUNCHED();
    return DBLP_OK;
}

// ---------------------------------------------------------------------------------------------------- no-allocation variant
// Scratch for callers that cannot obtain device memory at all (see dblp_apply_loss_static in dblp.h).  The array lives
// in this library's device image: every GPU that loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[DBLP_STATIC_SCRATCH_BYTES];

namespace dblp {
constexpr int kMaxDevices = 64;
static std::atomic<void*> g_static_scratch_addr[kMaxDevices];   // device address of the array, per device; null = not looked up yet
}  // namespace dblp

extern "C" int dblp_apply_loss_static(const dblp_plan_t* plan, const dblp_loss_model_t* model, uint64_t seed,
                                      uint32_t round, uint32_t attempt, uint32_t* delivered_bits, uint32_t* arrival,
                                      uint64_t* n_arrived_dev, void* stream)
{
    DBLP_REQUIRE(plan, DBLP_EINVAL, "apply_loss_static: null plan");
    const size_t need = layout(plan).total;
    DBLP_REQUIRE(need <= (size_t)DBLP_STATIC_SCRATCH_BYTES, DBLP_ECAPACITY,
                 "apply_loss_static: this plan needs %zu bytes of scratch, the built-in scratch holds %zu "
                 "(about 2^20 packets per round); use dblp_apply_loss with a caller-provided workspace",
                 need, (size_t)DBLP_STATIC_SCRATCH_BYTES);
    int device = -1;
    DBLP_CUDA(cudaGetDevice(&device));
    DBLP_REQUIRE(device == plan->device, DBLP_EINVAL, "apply_loss_static: device %d is current, the plan lives on device %d",
                 device, plan->device);
    DBLP_REQUIRE(device >= 0 && device < kMaxDevices, DBLP_ECAPACITY, "apply_loss_static: device index %d not supported", device);
    void* addr = g_static_scratch_addr[device].load(std::memory_order_acquire);
    if (!addr) {
        // In host code the array's name is only a handle; the kernels need its address in this device's memory.
        // Threads that get here together all look up the same address and store the same value.
        DBLP_CUDA(cudaGetSymbolAddress(&addr, g_static_scratch));
        DBLP_REQUIRE(addr, DBLP_ECUDA, "apply_loss_static: the scratch symbol has no address on device %d", device);
        g_static_scratch_addr[device].store(addr, std::memory_order_release);
    }
    return dblp_apply_loss(plan, model, seed, round, attempt, delivered_bits, arrival, n_arrived_dev, addr,
                           (size_t)DBLP_STATIC_SCRATCH_BYTES, stream);
}
