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
