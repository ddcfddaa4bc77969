/*
 * dblp.h -- C ABI of libdblp: the receive-side data path of the Dynamic Bounded-Loss Protocol (DBLP)
 * for W simulated workers whose gradients are resident on one CUDA device (sm_100a).
 *
 * One communication round is four steps:
 *
 *   dblp_packetize   gradients            -> header ring + payload ring      (Algorithm 1, first step)
 *   dblp_apply_loss  seeded loss process  -> delivered bitmap + arrival list (Sections II-C, V-B; property 1)
 *   dblp_aggregate   arrival list + rings -> received bitmap + aggregate     (Algorithm 2; Algorithm 3 "mean")
 *   dblp_check_bound received bitmap      -> per-worker loss counts, stop / continue decision (Section III-B)
 *
 * Each is a call of its own on the caller's stream.  dblp_round_device runs all four as one call and overlaps what is
 * independent: apply_loss (ALU-bound) beside packetize (HBM-bound), and the bitmap + tolerance test beside the masked
 * reduce, on a high-priority stream that the plan owns; dblp_round_host does the same from host buffers with the
 * copies overlapped.  Results are identical either way.
 *
 * Conventions
 *   - Every function returns DBLP_OK (0) or a negative dblp_status_t; nothing throws, aborts or traps.
 *     dblp_last_error() gives the text of the calling thread's most recent failure.
 *   - Unless an argument is marked HOST it is a DEVICE pointer owned by the caller, on the device that was
 *     current when the plan was created.  The library allocates device memory, streams and events only in
 *     dblp_plan_create.
 *   - Per-round calls only enqueue work on the given stream (a cudaStream_t passed as void*; NULL = the
 *     legacy default stream) and do not synchronise.  Counts that a later step needs stay on the device.
 *   - Anomalies found on the device (bad slot index, header that contradicts the plan, wrong round, repeated
 *     packet) are counted in dblp_counters_t and skipped; they never fault.
 *   - Alignment: ring and aggregate base pointers 16-byte aligned; payload_bytes a multiple of 16.
 *     Tensor sizes need no alignment (ragged edges take a scalar path).
 *   - Limits: W * C < 2^31 packets per round, ring slots < 2^32 - 1, payload_bytes <= 65536.
 */
#ifndef DBLP_H
#define DBLP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DBLP_OK = 0,
    DBLP_EINVAL = -1,    /* null pointer, zero size, value out of range */
    DBLP_EALIGN = -2,    /* pointer or payload size not 16-byte aligned */
    DBLP_ECAPACITY = -3, /* a limit above is exceeded, or the workspace is too small */
    DBLP_ECUDA = -4,     /* a CUDA runtime call failed; text in dblp_last_error() */
    DBLP_ETIMEOUT = -5   /* reserved: no call in this library waits on the device */
} dblp_status_t;

typedef enum { DBLP_F32 = 0, DBLP_BF16 = 1 } dblp_dtype_t;
typedef enum { DBLP_LOSS_NONE = 0, DBLP_LOSS_IID = 1, DBLP_LOSS_GE = 2, DBLP_LOSS_MICROBURST = 3 } dblp_loss_kind_t;
enum { DBLP_SUM = 0, DBLP_MEAN = 1, DBLP_OUT_BF16 = 2 }; /* flags of dblp_aggregate; OUT_BF16 only with dblp_aggregate_reduce_ex */

/* Packet header, 32 bytes, stored beside (not inside) the payload.  seq, round and len_bytes are the paper's
 * three fields (Section IV-A); tensor_id and offset_elems are the id/offset tags of the prior work the paper
 * builds on (Section III-A), redundant with seq given the plan and verified against it on receipt; worker stands
 * for the per-worker UDP port (Section IV-D). */
typedef struct {
    uint32_t seq;          /* unique per (worker, round), 0 .. C-1 */
    uint32_t round;        /* communication round the packet was sent in */
    uint32_t len_bytes;    /* valid payload bytes (the last chunk of a tensor is short) */
    uint32_t tensor_id;    /* index into the plan's tensor list */
    uint64_t offset_elems; /* first element of the chunk inside its tensor */
    uint32_t worker;       /* 0 .. W-1 */
    uint32_t reserved;     /* written as 0 */
} dblp_hdr_t;

/* Loss process in integers: a packet's 32-bit draw u drops it iff u < threshold, thresholds in [0, 2^32].
 * The paper injects loss without naming a generator (Sections II-C, V-B); the processes are:
 *   IID         drop iff u0 < t_drop.
 *   MICROBURST  one window of window_len consecutive sequence numbers, the same for every worker;
 *               drop iff u0 < (inside ? t_drop_in : t_drop_out).
 *   GE          two-state chain per worker in seq order: starts Bad iff u_init < t_init_bad; drop iff
 *               u0 < (Bad ? t_drop_bad : t_drop_good); then Bad -> Good iff u1 < t_bg, Good -> Bad iff u1 < t_gb.
 * Draws are Philox4x32-10 with key = seed and counter = (id low, id high, stream | attempt << 8, round),
 * id = worker * C + seq. */
typedef struct {
    uint32_t kind; /* dblp_loss_kind_t */
    uint32_t pad;
    uint64_t t_drop;
    uint64_t t_gb, t_bg, t_init_bad;
    uint64_t t_drop_good, t_drop_bad;
    uint64_t window_len;
    uint64_t t_drop_in, t_drop_out;
} dblp_loss_model_t;

/* Receiver statistics of a round (device memory; all fields accumulate until dblp_round_reset).  n_accepted and n_dup
 * are settled by the bitmap step of the bookkeeping (dblp_aggregate_bitmap): between a dblp_aggregate_claim and its
 * dblp_aggregate_bitmap every valid packet of the call is still counted under n_dup. */
typedef struct {
    uint64_t n_arrived;  /* arrival-list entries examined */
    uint64_t n_accepted; /* packets whose bit was newly set */
    uint64_t n_dup;      /* valid packets of this round whose chunk had already arrived */
    uint64_t n_stale;    /* valid packets of another round (Section III-A: dropped) */
    uint64_t n_invalid;  /* slot outside the ring, or header contradicting the plan (Algorithm 2 integrity check) */
    uint64_t n_late;     /* valid packets of this round that came after their worker's receiver had stopped */
    uint32_t status;     /* bit 0: arrival numbers exceeded 32 bits */
    uint32_t pad;
} dblp_counters_t;

typedef struct dblp_plan dblp_plan_t;

/* ---- plan: the constants exchanged once before training (Section IV-A) -------------------------------------
 * tensor_numel (HOST, T values > 0): elements of each gradient tensor in flat order.  Chunking is per tensor:
 * tensor t yields ceil(n_t / E) chunks, E = payload_bytes / element size; C is their total.
 * bucket_seq_bounds (HOST, B+1 ascending sequence numbers from 0 to C, or NULL with B = 1): the ranges over
 * which dblp_check_bound counts; one bucket is the paper's single bitmap per worker stream.
 * Allocates the plan's device tables on the current device; *out is owned by the caller until dblp_plan_destroy. */
int dblp_plan_create(const uint64_t* tensor_numel, uint32_t T, int dtype, uint32_t payload_bytes, uint32_t W,
                     const uint64_t* bucket_seq_bounds, uint32_t B, dblp_plan_t** out);
int dblp_plan_destroy(dblp_plan_t* plan);
/* C = chunks per worker, N = elements per worker, M = W * C, row_words = ceil(C / 32) words per bitmap row.
 * Any out pointer may be NULL. */
int dblp_plan_query(const dblp_plan_t* plan, uint64_t* C, uint64_t* N, uint64_t* M, uint64_t* row_words);
/* Where packets live.  DBLP_WIRE_RINGS (default): a header ring of 32-byte entries and a payload ring of payload_bytes
 * entries.  DBLP_WIRE_DATAGRAMS: one ring of (32 + payload_bytes)-byte datagrams, header first, as a packet looks on
 * the wire (Section IV-B: chunk and header together fill the UDP payload); pass the ring's base as both hdr_ring and
 * payload_ring to every call.  Set before the first round; results do not depend on it. */
enum { DBLP_WIRE_RINGS = 0, DBLP_WIRE_DATAGRAMS = 1 };
int dblp_plan_set_wire_format(dblp_plan_t* plan, int format);
/* A server split over several devices (Section IV-D's server, sharded by offset range): each device owns a contiguous
 * run of the tensors with a plan of its own, whose packets are the chunks seq_offset .. seq_offset + C - 1 of worker
 * streams that are stream_chunks long in all.  After this call the loss process draws each packet's fate by its number
 * in the whole stream (and runs the burst chain and places the microburst window along the whole stream), so that the
 * shards' delivered bitmaps, side by side, are exactly the delivered bitmap of the unsplit round.  Headers, sequence
 * numbers and the arrival permutation stay local to the shard.  dblp_workspace_bytes grows by one stream-wide bitmap.
 * dblp_apply_loss_resend with a send set and DBLP_LOSS_GE is refused on such a plan (DBLP_EINVAL): the chain would need
 * the send set of the whole stream.  Call before the first round. */
int dblp_plan_set_shard(dblp_plan_t* plan, uint64_t stream_chunks, uint64_t seq_offset);
/* Expert knob: pins the launch shape of the masked reduce (dblp_aggregate_reduce) -- chunks summed per tile and
 * number of persistent blocks; 0 = choose automatically (what dblp_plan_create does).  Results do not depend on it.
 * DBLP_ECAPACITY if the tile's slot entries do not fit in shared memory.  Not to be called while work that uses the
 * plan is being enqueued from another thread. */
int dblp_plan_tune_reduce(dblp_plan_t* plan, uint32_t chunks_per_tile, uint32_t grid_blocks);
/* Bytes of scratch that dblp_apply_loss / dblp_apply_loss_resend need.  dblp_aggregate_book_stop has its own query
 * (dblp_stop_workspace_bytes); the remaining calls need none. */
int dblp_workspace_bytes(const dblp_plan_t* plan, size_t* bytes);

/* HOST helper: rates -> thresholds floor(prob * 2^32).  IID uses mean_loss.  GE is the simple Gilbert chain
 * (every packet sent in Bad is lost): P(Bad->Good) = 1 / mean_burst_len, P(Good->Bad) chosen so the stationary loss
 * is mean_loss, start state drawn from the stationary law; DBLP_EINVAL if that P(Good->Bad) would exceed 1 (the mean
 * loss cannot be reached with bursts that short).  MICROBURST: window_len = ceil(window_frac * C). */
int dblp_loss_model_from_rates(int kind, double mean_loss, double mean_burst_len, double window_frac, double p_in,
                               double p_out, uint64_t C, dblp_loss_model_t* out);

/* ---- packetize (Algorithm 1 "split data into chunks"; Sections IV-A, IV-B) ----------------------------------
 * grads: HOST array of W device pointers, each a flat gradient of N elements of the plan's dtype (element-aligned).
 * Writes M headers to hdr_ring and M payload slots of payload_bytes each to payload_ring; packet (w, seq) goes to
 * slot w * C + seq; bytes of a slot past len_bytes are written as zero.  Rings may hold more than M slots (the
 * rest is untouched). */
int dblp_packetize(const dblp_plan_t* plan, const void* const* grads, uint32_t round, dblp_hdr_t* hdr_ring,
                   void* payload_ring, void* stream);

/* ---- apply_loss: which packets survive, and in which order they arrive ---------------------------------------
 * model: HOST.  delivered_bits: W rows of row_words u32, bit (seq % 32) of word (seq / 32) set iff packet
 * (w, seq) survives; padding bits zero.  arrival: capacity M u32; receives the surviving slot numbers in the order
 * pi(0), pi(1), ... where pi is a seeded permutation of [0, M) (4-round Feistel network on the smallest even
 * number of bits covering M, cycle-walked; round function = one Philox draw).  *n_arrived_dev (u64) = their count.
 * ws: scratch of at least dblp_workspace_bytes(); contents need not be preserved between calls. */
int dblp_apply_loss(const dblp_plan_t* plan, const dblp_loss_model_t* model, uint64_t seed, uint32_t round,
                    uint32_t attempt, uint32_t* delivered_bits, uint32_t* arrival, uint64_t* n_arrived_dev, void* ws,
                    size_t ws_bytes, void* stream);

/* ---- retransmission attempts (Algorithm 1: "for each unsent chunk ... send"; Section III-B: the sender retransmits
 * from the most recent bitmap) -------------------------------------------------------------------------------------
 * dblp_missing_bits: sent_bits <- the chunks whose bit is 0 in recv_bitmap (padding bits stay 0): what a sender
 * transmits after a bitmap reply.  Same layout as the bitmaps.
 * dblp_apply_loss_resend: dblp_apply_loss restricted to the chunks in sent_bits (NULL = all, which is
 * dblp_apply_loss): a chunk that is not sent cannot arrive, and the burst chain, which models the channel while
 * packets cross it, advances only over the packets that are sent.  Draws are keyed by (packet id, attempt), so the
 * fate of a sent packet under a memoryless process does not depend on what else is sent. */
int dblp_missing_bits(const dblp_plan_t* plan, const uint32_t* recv_bitmap, uint32_t* sent_bits, void* stream);
int dblp_apply_loss_resend(const dblp_plan_t* plan, const dblp_loss_model_t* model, uint64_t seed, uint32_t round,
                           uint32_t attempt, const uint32_t* sent_bits, uint32_t* delivered_bits, uint32_t* arrival,
                           uint64_t* n_arrived_dev, void* ws, size_t ws_bytes, void* stream);

/* ---- apply_loss without any allocation (the paper has no counterpart: this entry point exists for the sake of
 * callers, not of the protocol) ---------------------------------------------------------------------------------
 * Same results as dblp_apply_loss, bit for bit, but the scratch is a fixed array inside the library's own device
 * image instead of a caller-provided workspace.  It is meant for callers that hold no allocator for device memory
 * and must not call one: code running inside a memory pool whose owner forbids side allocations, plug-ins loaded
 * into a host process that has already handed all device memory to another runtime, and hard real-time loops where
 * an allocation's latency (or its implicit device synchronisation) is not acceptable.  Inputs and outputs are still
 * the caller's buffers.
 *   - Limit: the plan's dblp_workspace_bytes() must not exceed DBLP_STATIC_SCRATCH_BYTES (4 MiB + 64 KiB, i.e.
 *     roughly W * C <= 2^20 packets per round); larger plans get DBLP_ECAPACITY and a message naming both sizes.
 *   - Cost: every GPU on which the library is loaded keeps those bytes reserved until the process exits.
 *   - The first call on a device looks up the array's device address (one cudaGetSymbolAddress, no allocation) and
 *     caches it; make that first call before starting any stream capture on that device.  The plan's device must be
 *     the current device.
 *   - All calls on a device share the one array.  Nothing in it has to start at zero (each pass overwrites what the
 *     next reads), but two calls whose kernels overlap on the GPU -- different streams, or different host threads
 *     without ordering between them -- race on it.  Order them on one stream or with events.
 *   - Calls no cudaMalloc, cudaFree or other allocating routine. */
#define DBLP_STATIC_SCRATCH_BYTES (4u * 1024u * 1024u + 64u * 1024u)
int dblp_apply_loss_static(const dblp_plan_t* plan, const dblp_loss_model_t* model, uint64_t seed, uint32_t round,
                           uint32_t attempt, uint32_t* delivered_bits, uint32_t* arrival, uint64_t* n_arrived_dev,
                           void* stream);

/* ---- aggregate = bookkeeping + masked reduce ------------------------------------------------------------------
 * dblp_aggregate_book (Algorithm 2, chunk branch; Section III-A round filter): examines arrival[0 .. *n_arrived_dev)
 * (at most arrival_cap entries).  An entry is invalid if its slot >= n_slots or its header contradicts the plan
 * (worker < W, tensor_id < T, offset on a chunk boundary inside the tensor, len_bytes = that chunk's length,
 * seq = that chunk's number); stale if header.round != round; otherwise it claims cell (worker, seq) of slot_key.
 * slot_key: W * C u64, all-ones = nothing arrived yet, else (arrival number << 32) | slot; the claim is an atomic
 * minimum, so the earliest arrival keeps the cell whatever order threads run in, and later ones count as n_dup.
 * Arrival numbers continue from counters->n_arrived, so a further call in the same round (a retransmission
 * attempt) never displaces an earlier packet.  recv_bitmap (W rows of row_words u32) is rewritten from slot_key.
 *
 * dblp_aggregate_reduce (Algorithm 2 "unreceived chunks remain 0-filled / reconstruct"; Algorithm 3 mean): for
 * every element i of chunk c:  agg[i] = (+0.0f + x_0 + x_1 + ...) over the workers w = 0 .. W-1, in that order,
 * whose cell (w, c) is claimed, x_w read from the claimed payload slot (bf16 widened exactly), plain fp32
 * additions; with DBLP_MEAN the sum is divided by (float)W -- all workers, not the number that arrived.
 * The destination is the plan's (tensor base + chunk offset), never the slot's position.  agg_out: N fp32.
 *
 * dblp_aggregate runs both.  slot_key, recv_bitmap and counters are in/out round state (dblp_round_reset). */
/* dblp_aggregate_book = dblp_aggregate_claim (examine the arrivals, claim cells, count stale and invalid ones) followed
 * by dblp_aggregate_bitmap (rewrite recv_bitmap from slot_key; the bits that are new are the packets accepted by this
 * call, the other valid ones were repeats; fold this call's arrival count into counters->n_arrived).  recv_bitmap must
 * be the round's bitmap as the previous bookkeeping call (or dblp_round_reset) left it.
 * The reduce needs only the claims, the tolerance test only the bitmap, so a caller with two streams can run the
 * bitmap and dblp_check_bound beside dblp_aggregate_reduce.  Call dblp_aggregate_bitmap exactly once after each
 * dblp_aggregate_claim, with the same n_arrived_dev and arrival_cap, before the round's next claim. */
int dblp_aggregate_claim(const dblp_plan_t* plan, const dblp_hdr_t* hdr_ring, uint64_t n_slots, const uint32_t* arrival,
                         const uint64_t* n_arrived_dev, uint64_t arrival_cap, uint32_t round, uint64_t* slot_key,
                         dblp_counters_t* counters, void* stream);
/* dblp_aggregate_claim_grouped: the same claims with the same results (claim table and counters are identical), made
 * in a cheaper order for rounds whose headers and claim table do not fit in L2.  The arrival list is first grouped by
 * slot range (a counting sort in three small passes into (position, slot) pairs in ws), then the claims are made range
 * by range, so that the headers and cells they touch stay in L2 instead of costing two random DRAM sectors per packet;
 * a packet's arrival number travels with it, so "first arrival wins" is unchanged.  On 12 M packets the claim stage
 * drops from 0.53 to 0.29 ms; below about 3 M packets the plain order is the faster one.
 * dblp_aggregate_claim chooses by itself: a plan whose headers and claim table exceed the L2 owns a scratch of
 * dblp_claim_workspace_bytes(M, M) bytes (allocated in dblp_plan_create, 8 bytes per packet) and groups every call
 * with n_slots <= M and arrival_cap <= M; such a plan serves one claim at a time.  This entry point is for callers who
 * want the grouping elsewhere or with a scratch of their own.  ws: dblp_claim_workspace_bytes(n_slots, arrival_cap)
 * bytes, 256-byte aligned, contents need not be preserved. */
int dblp_claim_workspace_bytes(const dblp_plan_t* plan, uint64_t n_slots, uint64_t arrival_cap, size_t* bytes);
int dblp_aggregate_claim_grouped(const dblp_plan_t* plan, const dblp_hdr_t* hdr_ring, uint64_t n_slots,
                                 const uint32_t* arrival, const uint64_t* n_arrived_dev, uint64_t arrival_cap,
                                 uint32_t round, uint64_t* slot_key, dblp_counters_t* counters, void* ws, size_t ws_bytes,
                                 void* stream);
int dblp_aggregate_bitmap(const dblp_plan_t* plan, const uint64_t* slot_key, const uint64_t* n_arrived_dev,
                          uint64_t arrival_cap, uint32_t* recv_bitmap, dblp_counters_t* counters, void* stream);
int dblp_aggregate_book(const dblp_plan_t* plan, const dblp_hdr_t* hdr_ring, uint64_t n_slots, const uint32_t* arrival,
                        const uint64_t* n_arrived_dev, uint64_t arrival_cap, uint32_t round, uint32_t* recv_bitmap,
                        uint64_t* slot_key, dblp_counters_t* counters, void* stream);
int dblp_aggregate_reduce(const dblp_plan_t* plan, const void* payload_ring, const uint64_t* slot_key, float* agg_out,
                          uint32_t flags, void* stream);

/* ---- masked reduce with fused extras ---------------------------------------------------------------------------------
 * dblp_aggregate_reduce plus, in the same pass over the data:
 *   norm (Eq. 1 needs the L2 norm of the aggregated gradient): norm_out[0] = sum of agg[i]^2 in fp64, norm_out[1] = its
 *     square root.  Squares of fp32 values are exact in fp64; the additions follow a fixed tree (per thread, warp
 *     shuffle, warps in order, tiles in a fixed order), so the result is reproducible for a given plan and within
 *     about 64 ulp of the exactly rounded sum.  norm_scratch: dblp_norm_scratch_count() doubles (changes when
 *     dblp_plan_tune_reduce changes the tile height).  Both NULL = off.
 *   update (Algorithm 4, worker: w <- w - alpha * g): params[i] = params[i] - lr * agg[i], an fp32 multiply then an
 *     fp32 subtract (no fused multiply-add), for every element; chunks nobody delivered leave params unchanged because
 *     their aggregate is +0.  params: N fp32, in/out.  NULL = off.
 *   bf16 output (flag DBLP_OUT_BF16, may be or-ed with DBLP_MEAN): agg_out is N bf16 values, each the fp32 result
 *     rounded to nearest even (NaN stays a quiet NaN); norm and update still use the fp32 value.
 * For the broadcast half of a round (Algorithm 3 "DBLP_SEND(mean)", Algorithm 4 "DBLP_RECV"), packetize the mean with a
 * W = 1 plan, apply loss, book, and call this with params: the worker's reconstruction and its update in one pass. */
int dblp_norm_scratch_count(const dblp_plan_t* plan, uint64_t* count);
int dblp_aggregate_reduce_ex(const dblp_plan_t* plan, const void* payload_ring, const uint64_t* slot_key, float* agg_out,
                             uint32_t flags, double* norm_scratch, double* norm_out, float* params, float lr,
                             void* stream);

/* ---- order-free reduce (property 1: "gradients should be applied as soon as they arrive") --------------------------
 * Same inputs and the same mathematical result as dblp_aggregate_reduce, but every received payload is added into the
 * aggregate with floating-point atomics in whatever order the hardware runs them, so the fp32 sums are not
 * reproducible bit for bit: each element is within (W - 1) * 2^-24 * sum_w |x_w| of the exact sum.  Provided to measure
 * what the fixed worker order costs; zeroes agg_out first, and scales by 1 / W in a second pass for DBLP_MEAN. */
int dblp_aggregate_reduce_atomic(const dblp_plan_t* plan, const void* payload_ring, const uint64_t* slot_key,
                                 float* agg_out, uint32_t flags, void* stream);

/* ---- bookkeeping with early stop (Algorithm 2, the branch without a probe: "if the loss-tolerance threshold is
 * satisfied, send stop") ------------------------------------------------------------------------------------------
 * As dblp_aggregate_book, but each worker's receiver stops the moment its own missing / C <= bound_ppm / 10^6 holds
 * (one bitmap per worker stream): of a worker's valid packets of this round, taken in arrival order, only those up
 * to and including the one that satisfies the threshold are booked; the rest count as n_late and leave no trace.
 * Integrity and round checks come first, as for a running receiver.  The result equals a sequential walk over the
 * arrival list.  Needs W <= 4096 and a workspace of dblp_stop_workspace_bytes(arrival_cap) bytes, 256-byte aligned. */
int dblp_stop_workspace_bytes(const dblp_plan_t* plan, uint64_t arrival_cap, size_t* bytes);
int dblp_aggregate_book_stop(const dblp_plan_t* plan, const dblp_hdr_t* hdr_ring, uint64_t n_slots,
                             const uint32_t* arrival, const uint64_t* n_arrived_dev, uint64_t arrival_cap,
                             uint32_t round, uint32_t bound_ppm, uint32_t* recv_bitmap, uint64_t* slot_key,
                             dblp_counters_t* counters, void* ws, size_t ws_bytes, void* stream);
int dblp_aggregate(const dblp_plan_t* plan, const dblp_hdr_t* hdr_ring, const void* payload_ring, uint64_t n_slots,
                   const uint32_t* arrival, const uint64_t* n_arrived_dev, uint64_t arrival_cap, uint32_t round,
                   uint32_t* recv_bitmap, uint64_t* slot_key, dblp_counters_t* counters, float* agg_out,
                   uint32_t flags, void* stream);

/* Start of a round (Algorithm 2: bitmap <- 0): recv_bitmap <- 0, slot_key <- all-ones, counters <- 0. */
int dblp_round_reset(const dblp_plan_t* plan, uint32_t* recv_bitmap, uint64_t* slot_key, dblp_counters_t* counters,
                     void* stream);

/* ---- check_bound (Section III-B: stop once missing / total <= p; Algorithm 2: stop signal or bitmap reply) ----
 * For each worker w and bucket b: recv_cnt[w*B+b] = set bits of row w over the bucket's sequence range,
 * missing_cnt = total - recv_cnt, ok = (missing * 10^6 <= bound_ppm * total) in 64-bit integers;
 * *all_ok = 1 iff every ok is 1.  bound_ppm: HOST, n_bounds = 1 (one tolerance for all) or B (per bucket), in parts
 * per million (Table I: 0.8 % = 8000).  Outputs: recv_cnt, missing_cnt u32[W*B], ok u8[W*B], all_ok u32[1].
 * A plan serves one dblp_check_bound at a time (calls on one stream, or ordered by events). */
int dblp_check_bound(const dblp_plan_t* plan, const uint32_t* recv_bitmap, const uint32_t* bound_ppm,
                     uint32_t n_bounds, uint32_t* recv_cnt, uint32_t* missing_cnt, uint8_t* ok, uint32_t* all_ok,
                     void* stream);

/* HOST, pure: the rule above for counts summed over several shards of one worker stream (each GPU of a sharded server
 * counts its own chunk range): 1 iff missing * 10^6 <= bound_ppm * total.  Counts below 2^43 cannot overflow. */
int dblp_bound_ok(uint64_t missing, uint64_t total, uint32_t bound_ppm);

/* ---- phase-aware tolerance (HOST, pure) ----------------------------------------------------------------------
 * dblp_clr: Eq. 1, |norm_prev - norm_curr| / norm_prev >= eta in fp64; norm_prev == 0 counts as critical.
 * dblp_select_bound: Section IV-D / Algorithm 3: the first iteration uses P_low; at the start of an epoch the
 * tolerance becomes P_high unless dblp_clr fires, then P_low; at any other iteration it stays current_ppm. */
int dblp_clr(double norm_prev, double norm_curr, double eta);
uint32_t dblp_select_bound(double norm_prev, double norm_curr, double eta, uint32_t p_low_ppm, uint32_t p_high_ppm,
                           int at_epoch_start, int first_iteration, uint32_t current_ppm);

/* ---- whole rounds ---------------------------------------------------------------------------------------------------
 * The device buffers of a round, all allocated by the caller with the sizes given. */
typedef struct {
    void* grads;               /* W * N elements of the plan's dtype, worker-major; dblp_round_host only */
    dblp_hdr_t* hdr_ring;      /* M headers */
    void* payload_ring;        /* M * payload_bytes */
    uint32_t* delivered_bits;  /* W * row_words */
    uint32_t* arrival;         /* M */
    uint64_t* n_arrived;       /* 1 */
    uint32_t* recv_bitmap;     /* W * row_words */
    uint64_t* slot_key;        /* W * C */
    dblp_counters_t* counters; /* 1 */
    float* agg;                /* N */
    uint32_t* recv_cnt;        /* W * B */
    uint32_t* missing_cnt;     /* W * B */
    uint8_t* ok;               /* W * B */
    uint32_t* all_ok;          /* 1 */
    void* ws;                  /* dblp_workspace_bytes (max with dblp_stop_workspace_bytes(M) for dblp_round_until_stop) */
    size_t ws_bytes;
    uint32_t* sent_bits;       /* W * row_words; used by dblp_round_until_stop only */
} dblp_device_buffers_t;

/* Optional stage marks: CUDA events (cudaEvent_t passed as void*, created by the caller) that a whole-round call
 * records where a stage begins or ends, on the stream that runs the stage, so that a caller can time the stages of the
 * overlapped schedule.  NULL members are skipped; a NULL struct pointer means no marks. */
typedef struct {
    void* begin;          /* caller's stream, before anything */
    void* packetize_end;  /* caller's stream */
    void* loss_begin;     /* side stream: round_reset + apply_loss */
    void* loss_end;
    void* receive_begin;  /* caller's stream, once packetize and apply_loss have both finished */
    void* claim_end;      /* caller's stream: arrivals examined, cells claimed */
    void* reduce_end;     /* caller's stream */
    void* bound_begin;    /* side stream: bitmap + check_bound */
    void* bound_end;
    void* end;            /* caller's stream, after the side stream has been joined */
} dblp_round_marks_t;

/* dblp_round_device = one round of the server on gradients resident in device memory (Algorithm 3: receive from
 * every worker, then the mean; Algorithm 2 inside; Section III-B for the tolerance test):
 *   dblp_round_send     round_reset and apply_loss (attempt 0) on the plan's side stream beside dblp_packetize on the
 *                       caller's stream; returns with the caller's stream waiting for both.
 *   dblp_round_receive  dblp_aggregate_claim, then dblp_aggregate_bitmap + dblp_check_bound (one tolerance for all) on
 *                       the side stream beside dblp_aggregate_reduce; the caller's stream waits for both at the end.
 * grads: HOST array of W device pointers as for dblp_packetize.  flags: DBLP_SUM or DBLP_MEAN.  Packets occupy ring slots
 * 0 .. M-1.  Nothing is allocated and the host is not blocked.  The side stream and its events belong to the plan, so a
 * plan serves one whole-round call at a time (calls on one stream, or ordered by the caller). */
int dblp_round_send(const dblp_plan_t* plan, const void* const* grads, const dblp_loss_model_t* model, uint64_t seed,
                    uint32_t round, const dblp_device_buffers_t* dev, const dblp_round_marks_t* marks, void* stream);
int dblp_round_receive(const dblp_plan_t* plan, uint32_t round, uint32_t bound_ppm, uint32_t flags,
                       const dblp_device_buffers_t* dev, const dblp_round_marks_t* marks, void* stream);
int dblp_round_device(const dblp_plan_t* plan, const void* const* grads, const dblp_loss_model_t* model, uint64_t seed,
                      uint32_t round, uint32_t bound_ppm, uint32_t flags, const dblp_device_buffers_t* dev,
                      const dblp_round_marks_t* marks, void* stream);

/* dblp_round_host = the same round from HOST gradients (grads_host: HOST array of W host pointers, pinned memory
 * recommended).  Gradients of 32 MiB per worker and more are taken in up to 16 parts, contiguous ranges of chunks: the
 * host-to-device copies into dev->grads run back to back on a copy stream of the plan, part by part and worker by
 * worker; each slice is packetized as soon as it has landed; once a part is there for all workers its packets are
 * claimed, its chunks reduced, and its range of the aggregate starts back to agg_host on another stream of the plan,
 * so the copy back overlaps the copies in of the later parts.  The loss process runs beside all of it, the bitmap and
 * the tolerance test after the last claims.  Results are those of dblp_round_device.  The aggregate, the counters and
 * the bound outputs are copied back to the host pointers (NULL to skip) and the call waits for all of it.  Nothing is
 * allocated. */
int dblp_round_host(const dblp_plan_t* plan, const void* const* grads_host, const dblp_loss_model_t* model,
                    uint64_t seed, uint32_t round, uint32_t bound_ppm, uint32_t flags,
                    const dblp_device_buffers_t* dev, float* agg_host, dblp_counters_t* counters_host,
                    uint32_t* recv_cnt_host, uint32_t* missing_cnt_host, uint8_t* ok_host, uint32_t* all_ok_host,
                    void* stream);

/* ---- one round's control loop (Algorithms 1 + 2 together; HOST-blocking) ----------------------------------------------
 * After dblp_round_reset and dblp_packetize: attempt k = 0, 1, ... transmits what the bitmap reports missing
 * (dblp_missing_bits), redraws loss and arrival order with the attempt number (dblp_apply_loss_resend), books the
 * arrivals (dblp_aggregate_book, or dblp_aggregate_book_stop when early_stop != 0) and tests the tolerance
 * (dblp_check_bound, one value for all).  The decision is read back after every attempt -- the protocol's
 * probe / bitmap / stop exchange is a round trip -- and the loop ends when every worker passes or after max_attempts.
 * Packets are read from ring slots 0 .. M-1.  *attempts_used and *all_ok_host are HOST outputs.  The masked reduce is
 * left to the caller (dblp_aggregate_reduce). */
int dblp_round_until_stop(const dblp_plan_t* plan, const dblp_loss_model_t* model, uint64_t seed, uint32_t round,
                          uint32_t bound_ppm, uint32_t max_attempts, int early_stop, const dblp_device_buffers_t* dev,
                          uint32_t* attempts_used, uint32_t* all_ok_host, void* stream);

/* ---- diagnostics -----------------------------------------------------------------------------------------------*/
const char* dblp_strerror(int status);
const char* dblp_last_error(void);  /* HOST string, valid until the calling thread's next failing call */
uint64_t dblp_launch_count(void);   /* kernels launched by this library since it was loaded */

#ifdef __cplusplus
}
#endif
#endif /* DBLP_H */
