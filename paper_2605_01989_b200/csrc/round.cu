// Whole rounds: the two-stream schedule on device-resident gradients (dblp_round_send, dblp_round_receive,
// dblp_round_device), the same from host buffers with the copies overlapped (dblp_round_host), and the control loop of
// retransmission attempts (dblp_round_until_stop).  Order of steps: Algorithm 3 (server loop) around Algorithms 1 and 2.
//
// Schedule of one round (s = the caller's stream, side = the plan's own high-priority stream):
//
//   s:    fork --- packetize ----------------- join -- claim -- claimed ----- reduce ----------- done' -- (end)
//   side:      \-- round_reset, apply_loss ---/                        \-- bitmap, check_bound --/
//
// The loss process and the arrival order do not depend on the gradients, so the ALU-bound apply_loss runs beside the
// HBM-bound packetize; the masked reduce needs only the claims and the tolerance test only the bitmap, so those run
// beside each other as well.  All ordering is by events; nothing waits on the host.
#include "common.cuh"

using namespace dblp;

namespace {

inline int mark(void* ev, cudaStream_t st)
{
    if (!ev) return DBLP_OK;
    DBLP_CUDA(cudaEventRecord(static_cast<cudaEvent_t>(ev), st));
    return DBLP_OK;
}

#define DBLP_TRY(call)                 \
    do {                               \
        const int rc_ = (call);        \
        if (rc_ != DBLP_OK) return rc_; \
    } while (0)

int check_buffers(const dblp_device_buffers_t* d, const char* who)
{
    DBLP_REQUIRE(d->hdr_ring && d->payload_ring && d->delivered_bits && d->arrival && d->n_arrived && d->recv_bitmap &&
                 d->slot_key && d->counters && d->agg && d->recv_cnt && d->missing_cnt && d->ok && d->all_ok && d->ws,
                 DBLP_EINVAL, "%s: a member of the device buffer set is null", who);
    return DBLP_OK;
}

// side stream: start of the round (Algorithm 2: bitmap <- 0) and the lossy channel; joined by ev_join
int enqueue_channel(const dblp_plan_t* plan, const dblp_loss_model_t* model, uint64_t seed, uint32_t round,
                    const dblp_device_buffers_t* dev, const dblp_round_marks_t* m, cudaStream_t s)
{
    DBLP_CUDA(cudaEventRecord(plan->ev_fork, s));
    DBLP_CUDA(cudaStreamWaitEvent(plan->side, plan->ev_fork, 0));
    DBLP_TRY(mark(m ? m->loss_begin : nullptr, plan->side));
    DBLP_TRY(dblp_round_reset(plan, dev->recv_bitmap, dev->slot_key, dev->counters, plan->side));
    DBLP_TRY(dblp_apply_loss(plan, model, seed, round, 0, dev->delivered_bits, dev->arrival, dev->n_arrived, dev->ws,
                             dev->ws_bytes, plan->side));
    DBLP_TRY(mark(m ? m->loss_end : nullptr, plan->side));
    DBLP_CUDA(cudaEventRecord(plan->ev_join, plan->side));
    return DBLP_OK;
}

}  // namespace

extern "C" int dblp_round_send(const dblp_plan_t* plan, const void* const* grads, const dblp_loss_model_t* model,
                               uint64_t seed, uint32_t round, const dblp_device_buffers_t* dev,
                               const dblp_round_marks_t* marks, void* stream)
{
    DBLP_REQUIRE(plan && grads && model && dev, DBLP_EINVAL, "round_send: null argument");
    DBLP_TRY(check_buffers(dev, "round_send"));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    DBLP_TRY(mark(marks ? marks->begin : nullptr, s));
    DBLP_TRY(enqueue_channel(plan, model, seed, round, dev, marks, s));
    DBLP_TRY(dblp_packetize(plan, grads, round, dev->hdr_ring, dev->payload_ring, s));
    DBLP_TRY(mark(marks ? marks->packetize_end : nullptr, s));
    DBLP_CUDA(cudaStreamWaitEvent(s, plan->ev_join, 0));
    return DBLP_OK;
}

extern "C" int dblp_round_receive(const dblp_plan_t* plan, uint32_t round, uint32_t bound_ppm, uint32_t flags,
                                  const dblp_device_buffers_t* dev, const dblp_round_marks_t* marks, void* stream)
{
    DBLP_REQUIRE(plan && dev, DBLP_EINVAL, "round_receive: null argument");
    DBLP_TRY(check_buffers(dev, "round_receive"));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    DBLP_TRY(mark(marks ? marks->receive_begin : nullptr, s));
    DBLP_TRY(dblp_aggregate_claim(plan, dev->hdr_ring, plan->M, dev->arrival, dev->n_arrived, plan->M, round, dev->slot_key,
                                  dev->counters, s));
    DBLP_TRY(mark(marks ? marks->claim_end : nullptr, s));
    DBLP_CUDA(cudaEventRecord(plan->ev_claimed, s));
    DBLP_CUDA(cudaStreamWaitEvent(plan->side, plan->ev_claimed, 0));
    DBLP_TRY(mark(marks ? marks->bound_begin : nullptr, plan->side));
    DBLP_TRY(dblp_aggregate_bitmap(plan, dev->slot_key, dev->n_arrived, plan->M, dev->recv_bitmap, dev->counters, plan->side));
    DBLP_TRY(dblp_check_bound(plan, dev->recv_bitmap, &bound_ppm, 1, dev->recv_cnt, dev->missing_cnt, dev->ok, dev->all_ok,
                              plan->side));
    DBLP_TRY(mark(marks ? marks->bound_end : nullptr, plan->side));
    DBLP_CUDA(cudaEventRecord(plan->ev_done, plan->side));
    DBLP_TRY(dblp_aggregate_reduce(plan, dev->payload_ring, dev->slot_key, dev->agg, flags, s));
    DBLP_TRY(mark(marks ? marks->reduce_end : nullptr, s));
    DBLP_CUDA(cudaStreamWaitEvent(s, plan->ev_done, 0));
    DBLP_TRY(mark(marks ? marks->end : nullptr, s));
    return DBLP_OK;
}

extern "C" int dblp_round_device(const dblp_plan_t* plan, const void* const* grads, const dblp_loss_model_t* model,
                                 uint64_t seed, uint32_t round, uint32_t bound_ppm, uint32_t flags,
                                 const dblp_device_buffers_t* dev, const dblp_round_marks_t* marks, void* stream)
{
    DBLP_TRY(dblp_round_send(plan, grads, model, seed, round, dev, marks, stream));
    return dblp_round_receive(plan, round, bound_ppm, flags, dev, marks, stream);
}

namespace {

// First flat element of chunk c (c = C gives N), from the plan's per-tensor host tables.
uint64_t first_element_of_chunk(const dblp_plan_t* plan, uint64_t c)
{
    if (c >= plan->C) return plan->N;
    uint32_t lo = 0, hi = plan->T;                       // last tensor whose first chunk is <= c
    while (hi - lo > 1) {
        const uint32_t mid = lo + (hi - lo) / 2;
        if (plan->h_chunkbase[mid] <= c) lo = mid; else hi = mid;
    }
    return plan->h_base[lo] + (c - plan->h_chunkbase[lo]) * plan->E;
}

}  // namespace

// From host buffers.  The round is cut into up to 16 parts, contiguous ranges of chunks (and so of gradient elements)
// of about equal size.  The host-to-device copies run back to back on the plan's copy stream, part by part and worker
// by worker; behind them, on the caller's stream, each slice is packetized as soon as it has landed, and once a part
// is complete for all workers its packets are claimed (a pass over the arrival list that takes only that part's
// slots), its chunks are reduced, and its range of the aggregate starts back to the host on a third stream.  So the
// device-to-host copy of the aggregate overlaps the host-to-device copies of the later parts (the bus carries both
// directions at once), and the call ends one part's worth of work after the last gradient byte has arrived.
// Claims are atomic minima and every chunk is reduced from the finished claim table of its own part, so the results
// are those of the unsplit round.
extern "C" int dblp_round_host(const dblp_plan_t* plan, const void* const* grads_host, const dblp_loss_model_t* model,
                               uint64_t seed, uint32_t round, uint32_t bound_ppm, uint32_t flags,
                               const dblp_device_buffers_t* dev, float* agg_host, dblp_counters_t* counters_host,
                               uint32_t* recv_cnt_host, uint32_t* missing_cnt_host, uint8_t* ok_host,
                               uint32_t* all_ok_host, void* stream)
{
    DBLP_REQUIRE(plan && grads_host && model && dev, DBLP_EINVAL, "round_host: null argument");
    DBLP_REQUIRE(dev->grads, DBLP_EINVAL, "round_host: device buffer for the gradients is null");
    DBLP_TRY(check_buffers(dev, "round_host"));
    DBLP_REQUIRE(aligned16(dev->hdr_ring) && aligned16(dev->payload_ring), DBLP_EALIGN, "round_host: rings must be 16-byte aligned");
    DBLP_REQUIRE(flags == DBLP_SUM || flags == DBLP_MEAN, DBLP_EINVAL, "round_host: unknown flags %u", flags);
    for (uint32_t w = 0; w < plan->W; ++w)
        DBLP_REQUIRE(grads_host[w], DBLP_EINVAL, "round_host: gradient pointer of worker %u is null", w);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t grad_bytes = plan->N * plan->es;

    // parts: whole tiles of the tiled reduce, at least 16 MiB of one worker's gradient each, 16 at most
    uint64_t n_parts = grad_bytes / (16ull << 20);
    if (n_parts > 16) n_parts = 16;
    if (n_parts < 1 || !plan->red_variant) n_parts = 1;
    uint64_t per_part = (plan->C + n_parts - 1) / n_parts;
    if (plan->red_variant) per_part = (per_part + plan->red_CH - 1) / plan->red_CH * plan->red_CH;
    n_parts = (plan->C + per_part - 1) / per_part;

    DBLP_TRY(enqueue_channel(plan, model, seed, round, dev, nullptr, s));     // records ev_fork on s first
    DBLP_CUDA(cudaStreamWaitEvent(plan->copy, plan->ev_fork, 0));            // the copies follow whatever precedes on s
    uint32_t n_copies = 0;
    for (uint64_t k = 0; k < n_parts; ++k) {
        const uint64_t c_lo = k * per_part, c_hi = (k + 1) * per_part < plan->C ? (k + 1) * per_part : plan->C;
        const uint64_t e_lo = first_element_of_chunk(plan, c_lo), e_hi = first_element_of_chunk(plan, c_hi);
        for (uint32_t w = 0; w < plan->W; ++w, ++n_copies) {
            uint8_t* g = static_cast<uint8_t*>(dev->grads) + (size_t)w * grad_bytes;
            DBLP_CUDA(cudaMemcpyAsync(g + e_lo * plan->es, static_cast<const uint8_t*>(grads_host[w]) + e_lo * plan->es,
                                      (e_hi - e_lo) * plan->es, cudaMemcpyHostToDevice, plan->copy));
            DBLP_CUDA(cudaEventRecord(plan->ev_copy[n_copies & 1], plan->copy));
            DBLP_CUDA(cudaStreamWaitEvent(s, plan->ev_copy[n_copies & 1], 0));   // waits for the record just made
            const void* gp = g;
            DBLP_TRY(packetize_workers(plan, &gp, w, 1, round, dev->hdr_ring, dev->payload_ring, c_lo, c_hi, s));
        }
        if (k == 0) DBLP_CUDA(cudaStreamWaitEvent(s, plan->ev_join, 0));     // the arrival list is needed from here on
        DBLP_TRY(claim_arrivals(plan, dev->hdr_ring, plan->M, dev->arrival, dev->n_arrived, plan->M, round, dev->slot_key,
                                dev->counters, (uint32_t)c_lo, n_parts > 1 ? (uint32_t)c_hi : 0u, s));
        if (k + 1 == n_parts) {                                              // all claims made: bitmap and tolerance test
            DBLP_CUDA(cudaEventRecord(plan->ev_claimed, s));
            DBLP_CUDA(cudaStreamWaitEvent(plan->side, plan->ev_claimed, 0));
            DBLP_TRY(dblp_aggregate_bitmap(plan, dev->slot_key, dev->n_arrived, plan->M, dev->recv_bitmap, dev->counters, plan->side));
            DBLP_TRY(dblp_check_bound(plan, dev->recv_bitmap, &bound_ppm, 1, dev->recv_cnt, dev->missing_cnt, dev->ok,
                                      dev->all_ok, plan->side));
            DBLP_CUDA(cudaEventRecord(plan->ev_done, plan->side));
        }
        if (plan->red_variant) DBLP_TRY(reduce_chunks(plan, dev->payload_ring, dev->slot_key, dev->agg, flags, c_lo, c_hi, s));
        else DBLP_TRY(dblp_aggregate_reduce(plan, dev->payload_ring, dev->slot_key, dev->agg, flags, s));
        if (agg_host) {
            DBLP_CUDA(cudaEventRecord(plan->ev_part[k & 1], s));
            DBLP_CUDA(cudaStreamWaitEvent(plan->back, plan->ev_part[k & 1], 0));
            DBLP_CUDA(cudaMemcpyAsync(agg_host + e_lo, dev->agg + e_lo, (e_hi - e_lo) * sizeof(float), cudaMemcpyDeviceToHost,
                                      plan->back));
        }
    }
    DBLP_CUDA(cudaStreamWaitEvent(s, plan->ev_done, 0));

    const size_t cells = (size_t)plan->W * plan->B;
    if (counters_host) DBLP_CUDA(cudaMemcpyAsync(counters_host, dev->counters, sizeof(dblp_counters_t), cudaMemcpyDeviceToHost, s));
    if (recv_cnt_host) DBLP_CUDA(cudaMemcpyAsync(recv_cnt_host, dev->recv_cnt, cells * sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
    if (missing_cnt_host) DBLP_CUDA(cudaMemcpyAsync(missing_cnt_host, dev->missing_cnt, cells * sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
    if (ok_host) DBLP_CUDA(cudaMemcpyAsync(ok_host, dev->ok, cells, cudaMemcpyDeviceToHost, s));
    if (all_ok_host) DBLP_CUDA(cudaMemcpyAsync(all_ok_host, dev->all_ok, sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
    if (agg_host) {
        DBLP_CUDA(cudaEventRecord(plan->ev_back, plan->back));
        DBLP_CUDA(cudaStreamWaitEvent(s, plan->ev_back, 0));
    }
    DBLP_CUDA(cudaStreamSynchronize(s));
    return DBLP_OK;
}

extern "C" int dblp_round_until_stop(const dblp_plan_t* plan, const dblp_loss_model_t* model, uint64_t seed, uint32_t round,
                                     uint32_t bound_ppm, uint32_t max_attempts, int early_stop,
                                     const dblp_device_buffers_t* dev, uint32_t* attempts_used, uint32_t* all_ok_host,
                                     void* stream)
{
    DBLP_REQUIRE(plan && model && dev && attempts_used && all_ok_host, DBLP_EINVAL, "round_until_stop: null argument");
    DBLP_REQUIRE(dev->sent_bits, DBLP_EINVAL, "round_until_stop: sent_bits buffer missing");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    *attempts_used = 0;
    *all_ok_host = 0;
    for (uint32_t k = 0; k < max_attempts; ++k) {
        int rc = dblp_missing_bits(plan, dev->recv_bitmap, dev->sent_bits, s);
        if (rc == DBLP_OK) rc = dblp_apply_loss_resend(plan, model, seed, round, k, dev->sent_bits, dev->delivered_bits,
                                                      dev->arrival, dev->n_arrived, dev->ws, dev->ws_bytes, s);
        if (rc == DBLP_OK) {
            if (early_stop)
                rc = dblp_aggregate_book_stop(plan, dev->hdr_ring, plan->M, dev->arrival, dev->n_arrived, plan->M, round,
                                              bound_ppm, dev->recv_bitmap, dev->slot_key, dev->counters, dev->ws,
                                              dev->ws_bytes, s);
            else
                rc = dblp_aggregate_book(plan, dev->hdr_ring, plan->M, dev->arrival, dev->n_arrived, plan->M, round,
                                         dev->recv_bitmap, dev->slot_key, dev->counters, s);
        }
        if (rc == DBLP_OK) rc = dblp_check_bound(plan, dev->recv_bitmap, &bound_ppm, 1, dev->recv_cnt, dev->missing_cnt,
                                                dev->ok, dev->all_ok, s);
        if (rc != DBLP_OK) return rc;
        // the stop / bitmap reply is a round trip of the protocol: the decision comes back to the host every attempt
        DBLP_CUDA(cudaMemcpyAsync(all_ok_host, dev->all_ok, sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
        DBLP_CUDA(cudaStreamSynchronize(s));
        *attempts_used = k + 1;
        if (*all_ok_host) break;
    }
    return DBLP_OK;
}
