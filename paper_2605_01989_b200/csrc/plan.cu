// Plan creation (the constants of Section IV-A turned into device tables), host-side scalar rules (Eq. 1, the
// tolerance schedule of Section IV-D / Algorithm 3) and diagnostics.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>

#include <new>

#include "common.cuh"

namespace dblp {

static thread_local char t_err[512] = "";
std::atomic<uint64_t> g_launches{0};

void set_error(const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(t_err, sizeof(t_err), fmt, ap);
    va_end(ap);
}

static void free_tables(dblp_plan* p)
{
    cudaFree(p->d_tensor_tab);
    cudaFree(p->d_base);
    cudaFree(p->d_chunk_desc);
    cudaFree(p->d_chunk_tensor);
    cudaFree(p->d_bucket_bounds);
    cudaFree(p->d_bound_ppm);
    cudaFree(p->d_ticket);
    cudaFree(p->d_claim_ws);
    if (p->side) cudaStreamDestroy(p->side);
    if (p->copy) cudaStreamDestroy(p->copy);
    if (p->back) cudaStreamDestroy(p->back);
    cudaEvent_t* evs[] = {&p->ev_fork, &p->ev_join,    &p->ev_claimed, &p->ev_done, &p->ev_copy[0],
                          &p->ev_copy[1], &p->ev_part[0], &p->ev_part[1], &p->ev_back};
    for (cudaEvent_t* e : evs)
        if (*e) cudaEventDestroy(*e);
}

// Streams and events of the whole-round calls.  The side stream gets the highest priority the device offers, so that
// its short kernels are scheduled between the blocks of the long bandwidth-bound ones instead of behind them.
static cudaError_t create_round_resources(dblp_plan* p)
{
    int least = 0, greatest = 0;
    cudaError_t e = cudaDeviceGetStreamPriorityRange(&least, &greatest);
    if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&p->side, cudaStreamNonBlocking, greatest);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p->copy, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p->back, cudaStreamNonBlocking);
    cudaEvent_t* evs[] = {&p->ev_fork, &p->ev_join,    &p->ev_claimed, &p->ev_done, &p->ev_copy[0],
                          &p->ev_copy[1], &p->ev_part[0], &p->ev_part[1], &p->ev_back};
    for (cudaEvent_t* ev : evs)
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming);
    return e;
}

template <typename T>
static cudaError_t upload(T** dst, const std::vector<T>& src)
{
    cudaError_t e = cudaMalloc((void**)dst, src.size() * sizeof(T));
    if (e != cudaSuccess) return e;
    return cudaMemcpy(*dst, src.data(), src.size() * sizeof(T), cudaMemcpyHostToDevice);
}

}  // namespace dblp

using namespace dblp;

static int plan_create(const uint64_t* tensor_numel, uint32_t T, int dtype, uint32_t payload_bytes, uint32_t W,
                       const uint64_t* bucket_seq_bounds, uint32_t B, dblp_plan_t** out)
{
    DBLP_REQUIRE(tensor_numel && out && T > 0 && W > 0 && B > 0, DBLP_EINVAL, "plan: null argument or zero count");
    DBLP_REQUIRE(dtype == DBLP_F32 || dtype == DBLP_BF16, DBLP_EINVAL, "plan: unknown dtype %d", dtype);
    DBLP_REQUIRE(payload_bytes >= 16 && payload_bytes <= 65536, DBLP_ECAPACITY, "plan: payload_bytes %u outside [16, 65536]",
                 payload_bytes);
    DBLP_REQUIRE(payload_bytes % 16 == 0, DBLP_EALIGN, "plan: payload_bytes %u is not a multiple of 16", payload_bytes);
    DBLP_REQUIRE(bucket_seq_bounds || B == 1, DBLP_EINVAL, "plan: B = %u needs bucket_seq_bounds", B);

    dblp_plan* p = new (std::nothrow) dblp_plan();
    DBLP_REQUIRE(p, DBLP_EINVAL, "plan: out of host memory");
    struct Guard {              // frees a half-built plan on every early return and on exceptions
        dblp_plan* p;
        ~Guard() { if (p) { free_tables(p); delete p; } }
    } guard{p};
    p->T = T; p->W = W; p->B = B; p->P = payload_bytes; p->dtype = dtype;
    p->es = dtype == DBLP_F32 ? 4 : 2;
    p->E = payload_bytes / p->es;
    p->VE = 16 / p->es;
    p->VPC = payload_bytes / 16;
    p->hdr_stride = 32; p->pay_stride = payload_bytes; p->pay_off = 0;
    p->d_tensor_tab = nullptr; p->d_base = nullptr; p->d_chunk_desc = nullptr;
    p->d_chunk_tensor = p->d_bucket_bounds = p->d_bound_ppm = p->d_ticket = nullptr;
    p->d_claim_ws = nullptr; p->claim_ws_bytes = 0;
    p->side = p->copy = p->back = nullptr;
    p->ev_fork = p->ev_join = p->ev_claimed = p->ev_done = p->ev_copy[0] = p->ev_copy[1] = nullptr;
    p->ev_part[0] = p->ev_part[1] = p->ev_back = nullptr;

    uint64_t base = 0, c = 0;
    p->h_numel.assign(tensor_numel, tensor_numel + T);
    p->h_base.resize(T);
    p->h_chunkbase.resize((size_t)T + 1);
    for (uint32_t t = 0; t < T; ++t) {
        DBLP_REQUIRE(tensor_numel[t] != 0, DBLP_EINVAL, "plan: tensor %u has no elements", t);
        p->h_base[t] = base;
        p->h_chunkbase[t] = (uint32_t)c;
        base += tensor_numel[t];
        c += (tensor_numel[t] + p->E - 1) / p->E;
        DBLP_REQUIRE(base < (1ull << 47) && c * W < (1ull << 31), DBLP_ECAPACITY,
                     "plan: W * C must stay below 2^31 packets and N below 2^47 elements");
    }
    p->h_chunkbase[T] = (uint32_t)c;
    p->C = c; p->N = base; p->M = c * W; p->row_words = (c + 31) / 32;
    p->C_stream = c; p->seq_off = 0;

    std::vector<uint32_t> bounds((size_t)B + 1);
    if (bucket_seq_bounds) {
        bool ok = bucket_seq_bounds[0] == 0 && bucket_seq_bounds[B] == c;
        for (uint32_t b = 0; b < B && ok; ++b) ok = bucket_seq_bounds[b] <= bucket_seq_bounds[b + 1];
        DBLP_REQUIRE(ok, DBLP_EINVAL, "plan: bucket bounds must ascend from 0 to C = %llu", (unsigned long long)c);
        for (uint32_t b = 0; b <= B; ++b) bounds[b] = (uint32_t)bucket_seq_bounds[b];
    } else {
        bounds[0] = 0; bounds[1] = (uint32_t)c;
    }

    std::vector<uint64_t> desc(c);
    std::vector<uint32_t> owner(c);
    for (uint32_t t = 0; t < T; ++t) {
        const uint64_t n = tensor_numel[t], nch = (n + p->E - 1) / p->E;
        for (uint64_t j = 0; j < nch; ++j) {
            const uint64_t off = j * p->E, len = n - off < p->E ? n - off : p->E;
            desc[p->h_chunkbase[t] + j] = ((p->h_base[t] + off) << 16) | len;
            owner[p->h_chunkbase[t] + j] = t;
        }
    }

    std::vector<uint4> tab(T);
    for (uint32_t t = 0; t < T; ++t)
        tab[t] = make_uint4((uint32_t)tensor_numel[t], (uint32_t)(tensor_numel[t] >> 32), p->h_chunkbase[t], 0u);

    cudaError_t e = cudaGetDevice(&p->device);
    if (e == cudaSuccess) e = upload(&p->d_tensor_tab, tab);
    if (e == cudaSuccess) e = upload(&p->d_base, p->h_base);
    if (e == cudaSuccess) e = upload(&p->d_chunk_desc, desc);
    if (e == cudaSuccess) e = upload(&p->d_chunk_tensor, owner);
    if (e == cudaSuccess) e = upload(&p->d_bucket_bounds, bounds);
    if (e == cudaSuccess) e = cudaMalloc((void**)&p->d_bound_ppm, sizeof(uint32_t) * B);
    if (e == cudaSuccess) e = cudaMalloc((void**)&p->d_ticket, sizeof(uint32_t));
    if (e == cudaSuccess) e = cudaMemset(p->d_ticket, 0, sizeof(uint32_t));
    if (e == cudaSuccess) e = create_round_resources(p);
    DBLP_REQUIRE(e == cudaSuccess, DBLP_ECUDA, "plan: device table setup failed: %s", cudaGetErrorString(e));
    const int rc = configure_reduce(p, 0, 0);
    if (rc != DBLP_OK) return rc;
    int l2_bytes = 0;
    e = cudaDeviceGetAttribute(&l2_bytes, cudaDevAttrL2CacheSize, p->device);
    DBLP_REQUIRE(e == cudaSuccess, DBLP_ECUDA, "plan: device query failed: %s", cudaGetErrorString(e));
    p->pack_tile_major = p->M * (uint64_t)payload_bytes <= 16ull * (uint64_t)l2_bytes ? 1u : 0u;
    p->reset_in_l2 = p->M * sizeof(uint64_t) <= (uint64_t)l2_bytes / 4 && p->M >= 8 ? 1u : 0u;
    p->claim_grouped = p->M * (sizeof(dblp_hdr_t) + sizeof(uint64_t)) > (uint64_t)l2_bytes ? 1u : 0u;
    if (p->claim_grouped) {                                         // 8 bytes per packet, e.g. 97 MB for 12 M packets
        const int rcw = dblp_claim_workspace_bytes(p, p->M, p->M, &p->claim_ws_bytes);
        if (rcw != DBLP_OK) return rcw;
        e = cudaMalloc(&p->d_claim_ws, p->claim_ws_bytes);
        DBLP_REQUIRE(e == cudaSuccess, DBLP_ECUDA, "plan: scratch of the grouped claims (%zu bytes): %s", p->claim_ws_bytes,
                     cudaGetErrorString(e));
    }
    guard.p = nullptr;
    *out = p;
    return DBLP_OK;
}

extern "C" int dblp_plan_create(const uint64_t* tensor_numel, uint32_t T, int dtype, uint32_t payload_bytes, uint32_t W,
                                const uint64_t* bucket_seq_bounds, uint32_t B, dblp_plan_t** out)
{
    try {                      // the host tables are std::vectors: running out of host memory must not cross the C ABI
        return plan_create(tensor_numel, T, dtype, payload_bytes, W, bucket_seq_bounds, B, out);
    } catch (...) {
        set_error("plan: out of host memory while building the chunk tables");
        return DBLP_ECAPACITY;
    }
}

extern "C" int dblp_plan_set_wire_format(dblp_plan_t* plan, int format)
{
    DBLP_REQUIRE(plan, DBLP_EINVAL, "plan_set_wire_format: null plan");
    if (format == DBLP_WIRE_RINGS) {
        plan->hdr_stride = 32; plan->pay_stride = plan->P; plan->pay_off = 0;
    } else if (format == DBLP_WIRE_DATAGRAMS) {
        plan->hdr_stride = plan->pay_stride = 32 + plan->P; plan->pay_off = 32;
    } else {
        DBLP_REQUIRE(false, DBLP_EINVAL, "plan_set_wire_format: unknown format %d", format);
    }
    return DBLP_OK;
}

extern "C" int dblp_plan_set_shard(dblp_plan_t* plan, uint64_t stream_chunks, uint64_t seq_offset)
{
    DBLP_REQUIRE(plan, DBLP_EINVAL, "plan_set_shard: null plan");
    DBLP_REQUIRE(seq_offset <= stream_chunks && plan->C <= stream_chunks - seq_offset, DBLP_EINVAL,
                 "plan_set_shard: chunks %llu .. %llu do not lie inside a stream of %llu",
                 (unsigned long long)seq_offset, (unsigned long long)(seq_offset + plan->C), (unsigned long long)stream_chunks);
    DBLP_REQUIRE(stream_chunks * plan->W < (1ull << 31), DBLP_ECAPACITY, "plan_set_shard: W * stream chunks must stay below 2^31");
    plan->C_stream = stream_chunks;
    plan->seq_off = seq_offset;
    return DBLP_OK;
}

extern "C" int dblp_plan_destroy(dblp_plan_t* plan)
{
    if (!plan) return DBLP_OK;
    free_tables(plan);
    delete plan;
    return DBLP_OK;
}

extern "C" int dblp_plan_query(const dblp_plan_t* plan, uint64_t* C, uint64_t* N, uint64_t* M, uint64_t* row_words)
{
    DBLP_REQUIRE(plan, DBLP_EINVAL, "plan_query: null plan");
    if (C) *C = plan->C;
    if (N) *N = plan->N;
    if (M) *M = plan->M;
    if (row_words) *row_words = plan->row_words;
    return DBLP_OK;
}

extern "C" int dblp_loss_model_from_rates(int kind, double mean_loss, double mean_burst_len, double window_frac,
                                          double p_in, double p_out, uint64_t C, dblp_loss_model_t* out)
{
    DBLP_REQUIRE(out, DBLP_EINVAL, "loss_model_from_rates: null output");
    auto thr = [](double p) -> uint64_t {
        if (!(p > 0.0)) return 0;
        if (p >= 1.0) return 1ull << 32;
        return (uint64_t)floor(p * 4294967296.0);
    };
    *out = dblp_loss_model_t{};
    out->kind = (uint32_t)kind;
    switch (kind) {
    case DBLP_LOSS_NONE: break;
    case DBLP_LOSS_IID: out->t_drop = thr(mean_loss); break;
    case DBLP_LOSS_GE: {
        DBLP_REQUIRE(mean_burst_len >= 1.0 && mean_loss >= 0.0 && mean_loss <= 1.0, DBLP_EINVAL,
                     "loss_model_from_rates: burst length must be >= 1 and loss within [0, 1]");
        const double p_bg = 1.0 / mean_burst_len;
        const double p_gb = mean_loss < 1.0 ? p_bg * mean_loss / (1.0 - mean_loss) : 1.0;
        DBLP_REQUIRE(p_gb <= 1.0, DBLP_EINVAL,
                     "loss_model_from_rates: a mean loss of %g cannot be reached with bursts of mean length %g "
                     "(P(Good->Bad) would be %g)", mean_loss, mean_burst_len, p_gb);
        out->t_gb = thr(p_gb); out->t_bg = thr(p_bg); out->t_init_bad = thr(mean_loss);
        out->t_drop_good = 0; out->t_drop_bad = 1ull << 32;
        break;
    }
    case DBLP_LOSS_MICROBURST: {
        uint64_t wl = (uint64_t)ceil(window_frac * (double)C);
        out->window_len = wl > C ? C : wl;
        out->t_drop_in = thr(p_in); out->t_drop_out = thr(p_out);
        break;
    }
    default: DBLP_REQUIRE(false, DBLP_EINVAL, "loss_model_from_rates: unknown kind %d", kind);
    }
    return DBLP_OK;
}

extern "C" int dblp_clr(double norm_prev, double norm_curr, double eta)
{
    if (norm_prev == 0.0) return 1;
    return fabs(norm_prev - norm_curr) / norm_prev >= eta ? 1 : 0;
}

extern "C" uint32_t dblp_select_bound(double norm_prev, double norm_curr, double eta, uint32_t p_low_ppm,
                                      uint32_t p_high_ppm, int at_epoch_start, int first_iteration, uint32_t current_ppm)
{
    if (first_iteration) return p_low_ppm;
    if (!at_epoch_start) return current_ppm;
    return dblp_clr(norm_prev, norm_curr, eta) ? p_low_ppm : p_high_ppm;
}

extern "C" const char* dblp_strerror(int status)
{
    switch (status) {
    case DBLP_OK: return "ok";
    case DBLP_EINVAL: return "invalid argument";
    case DBLP_EALIGN: return "misaligned pointer or size";
    case DBLP_ECAPACITY: return "capacity or limit exceeded";
    case DBLP_ECUDA: return "CUDA runtime error";
    case DBLP_ETIMEOUT: return "timeout";
    default: return "unknown status";
    }
}

extern "C" const char* dblp_last_error(void) { return dblp::t_err; }
extern "C" uint64_t dblp_launch_count(void) { return dblp::g_launches.load(std::memory_order_relaxed); }
