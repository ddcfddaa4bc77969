// dblp_round_host: one whole round driven from host buffers -- copies in, the four steps, copies out, one wait.
#include "common.cuh"

using namespace dblp;

extern "C" int dblp_round_host(const dblp_plan_t* plan, const void* const* grads_host, const dblp_loss_model_t* model,
                               uint64_t seed, uint32_t round, uint32_t bound_ppm, uint32_t flags,
                               const dblp_device_buffers_t* dev, float* agg_host, dblp_counters_t* counters_host,
                               uint32_t* recv_cnt_host, uint32_t* missing_cnt_host, uint8_t* ok_host,
                               uint32_t* all_ok_host, void* stream)
{
    DBLP_REQUIRE(plan && grads_host && model && dev, DBLP_EINVAL, "round_host: null argument");
    DBLP_REQUIRE(plan->W <= 4096, DBLP_ECAPACITY, "round_host: more than 4096 workers");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t grad_bytes = plan->N * plan->es;
    std::vector<const void*> gdev(plan->W);
    for (uint32_t w = 0; w < plan->W; ++w) {
        DBLP_REQUIRE(grads_host[w], DBLP_EINVAL, "round_host: gradient pointer of worker %u is null", w);
        gdev[w] = static_cast<const uint8_t*>(dev->grads) + (size_t)w * grad_bytes;
        DBLP_CUDA(cudaMemcpyAsync(const_cast<void*>(gdev[w]), grads_host[w], grad_bytes, cudaMemcpyHostToDevice, s));
    }
    int rc = dblp_round_reset(plan, dev->recv_bitmap, dev->slot_key, dev->counters, s);
    if (rc == DBLP_OK) rc = dblp_packetize(plan, gdev.data(), round, dev->hdr_ring, dev->payload_ring, s);
    if (rc == DBLP_OK) rc = dblp_apply_loss(plan, model, seed, round, 0, dev->delivered_bits, dev->arrival, dev->n_arrived,
                                           dev->ws, dev->ws_bytes, s);
    if (rc == DBLP_OK) rc = dblp_aggregate(plan, dev->hdr_ring, dev->payload_ring, plan->M, dev->arrival, dev->n_arrived,
                                          plan->M, round, dev->recv_bitmap, dev->slot_key, dev->counters, dev->agg, flags, s);
    if (rc == DBLP_OK) rc = dblp_check_bound(plan, dev->recv_bitmap, &bound_ppm, 1, dev->recv_cnt, dev->missing_cnt,
                                            dev->ok, dev->all_ok, s);
    if (rc != DBLP_OK) return rc;
    const size_t cells = (size_t)plan->W * plan->B;
    if (agg_host) DBLP_CUDA(cudaMemcpyAsync(agg_host, dev->agg, plan->N * sizeof(float), cudaMemcpyDeviceToHost, s));
    if (counters_host) DBLP_CUDA(cudaMemcpyAsync(counters_host, dev->counters, sizeof(dblp_counters_t), cudaMemcpyDeviceToHost, s));
    if (recv_cnt_host) DBLP_CUDA(cudaMemcpyAsync(recv_cnt_host, dev->recv_cnt, cells * sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
    if (missing_cnt_host) DBLP_CUDA(cudaMemcpyAsync(missing_cnt_host, dev->missing_cnt, cells * sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
    if (ok_host) DBLP_CUDA(cudaMemcpyAsync(ok_host, dev->ok, cells, cudaMemcpyDeviceToHost, s));
    if (all_ok_host) DBLP_CUDA(cudaMemcpyAsync(all_ok_host, dev->all_ok, sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
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
