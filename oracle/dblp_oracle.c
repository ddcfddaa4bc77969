/*
 * dblp_oracle.c -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, single-pass CPU statement of the receive-side data path of the
 * Dynamic Bounded-Loss Protocol (DBLP): chunking with headers, a seeded loss
 * process, permuted arrival, bitmap bookkeeping, zero-filled reconstruction with
 * the server's reduce, and the tolerance test.  Every function names the passage
 * of the paper it restates.  It shares no code, header, table or constant
 * generator with the CUDA library; only tests, the smoke check and the bench's
 * CPU-baseline leg may call it.
 *
 * Everything is written as the definition reads: no blocking, no fusion, no
 * reordering.  The single concession to the timed multi-core baseline is one
 * OpenMP pragma over chunks in the reduce (each chunk is independent, and the
 * order of the additions inside a chunk is untouched).
 *
 * Pins (see tests/): Philox known answers from the generator's publication;
 * closed forms for the chunk count; identities (reassembly, zero loss = plain
 * left-to-right sum, permutation invariance, popcount = counters); Table I and
 * Eq. 1 boundary cases for the tolerance rules.
 * Parity unpinned: none of the functions below.
 */
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#include <stdlib.h>
#include <math.h>

#define ORC_OK 0
#define ORC_EINVAL (-1)

#define ORC_NONE 0xFFFFFFFFu

/* Header carried beside each payload: the paper's three fields (sequence number,
 * round counter, data length -- Section IV-A) plus the id/offset tagging of the
 * prior work it builds on (Section III-A) and the worker that the paper
 * identifies by UDP port (Section IV-D). */
typedef struct {
    uint32_t seq;
    uint32_t round;
    uint32_t len_bytes;
    uint32_t tensor_id;
    uint64_t offset_elems;
    uint32_t worker;
    uint32_t reserved;
} orc_hdr_t;

typedef struct {
    uint32_t kind;        /* 0 none, 1 iid, 2 Gilbert-Elliott, 3 microburst */
    uint32_t pad;
    uint64_t t_drop;      /* iid: drop iff u < t_drop, u a 32-bit draw, t in [0, 2^32] */
    uint64_t t_gb, t_bg, t_init_bad;
    uint64_t t_drop_good, t_drop_bad;
    uint64_t window_len;
    uint64_t t_drop_in, t_drop_out;
} orc_loss_t;

typedef struct {
    uint64_t n_arrived, n_accepted, n_dup, n_stale, n_invalid, n_late;
    uint32_t status, pad;
} orc_counters_t;

/* ---------------------------------------------------------------------------
 * Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy
 * as 1, 2, 3", SC'11).  Ten rounds; each round multiplies counter words 0 and 2
 * by two fixed multipliers, mixes high halves with the other words and the key,
 * then bumps the key by the Weyl constants.
 * ------------------------------------------------------------------------- */
void dblp_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Stream tags that keep the draws for different purposes apart. */
enum { STREAM_PACKET = 1, STREAM_GE_INIT = 2, STREAM_WINDOW = 3, STREAM_PERM = 4 };

/* One draw: counter = (a low, a high, stream tag | attempt << 8, round), key = seed. */
static void draw(uint64_t seed, uint64_t a, uint32_t stream, uint32_t attempt, uint32_t round, uint32_t out[4])
{
    uint32_t ctr[4] = { (uint32_t)a, (uint32_t)(a >> 32), stream | (attempt << 8), round };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    dblp_oracle_philox4x32_10(ctr, key, out);
}

/* ---------------------------------------------------------------------------
 * Plan = the constants exchanged once before training (Section IV-A): how many
 * chunks a communication cycle has, and which tensor each belongs to.
 * Chunking is per tensor (Section IV-B: "partitions the tensor"): tensor t with
 * n_t elements gives ceil(n_t / E) chunks, E = payload_bytes / elem_size, the
 * last one short.  base[t] = first element of t in the flat gradient;
 * chunkbase[t] = sequence number of t's first chunk; chunkbase[T] = C.
 * ------------------------------------------------------------------------- */
int dblp_oracle_plan(const uint64_t* numel, uint32_t T, uint32_t elem_size, uint32_t payload_bytes,
                     uint64_t* base, uint64_t* chunkbase)
{
    if (!numel || !base || !chunkbase || T == 0) return ORC_EINVAL;
    if (elem_size != 2 && elem_size != 4) return ORC_EINVAL;
    if (payload_bytes == 0 || payload_bytes % elem_size) return ORC_EINVAL;
    uint64_t E = payload_bytes / elem_size;
    uint64_t b = 0, c = 0;
    for (uint32_t t = 0; t < T; ++t) {
        if (numel[t] == 0) return ORC_EINVAL;
        base[t] = b;
        chunkbase[t] = c;
        b += numel[t];
        c += (numel[t] + E - 1) / E;
    }
    chunkbase[T] = c;
    return ORC_OK;
}

/* ---------------------------------------------------------------------------
 * Packetize (Algorithm 1, first step; Sections IV-A, IV-B).  For each worker,
 * tensor and chunk: copy the chunk into its payload slot and fill in the header.
 * Slot of packet (w, seq) is w*C + seq.  Bytes of a short chunk's slot past its
 * data length are written as zero.  With payload_ring == NULL only the headers
 * are produced (they do not depend on the gradient values).
 * ------------------------------------------------------------------------- */
int dblp_oracle_packetize(const uint64_t* numel, uint32_t T, uint32_t elem_size, uint32_t payload_bytes,
                          uint32_t W, const void* const* grads, uint32_t round,
                          orc_hdr_t* hdr_ring, uint8_t* payload_ring)
{
    uint64_t* base = (uint64_t*)malloc(sizeof(uint64_t) * T);
    uint64_t* cb = (uint64_t*)malloc(sizeof(uint64_t) * ((size_t)T + 1));
    if (!base || !cb) { free(base); free(cb); return ORC_EINVAL; }
    int rc = dblp_oracle_plan(numel, T, elem_size, payload_bytes, base, cb);
    if (rc) { free(base); free(cb); return rc; }
    uint64_t E = payload_bytes / elem_size, C = cb[T];
    for (uint32_t w = 0; w < W; ++w) {
        const uint8_t* g = payload_ring ? (const uint8_t*)grads[w] : NULL;
        for (uint32_t t = 0; t < T; ++t) {
            uint64_t nchunks = (numel[t] + E - 1) / E;
            for (uint64_t j = 0; j < nchunks; ++j) {
                uint64_t off = j * E;
                uint64_t len = numel[t] - off < E ? numel[t] - off : E;
                uint64_t seq = cb[t] + j;
                uint64_t slot = (uint64_t)w * C + seq;
                orc_hdr_t* h = &hdr_ring[slot];
                h->seq = (uint32_t)seq;
                h->round = round;
                h->len_bytes = (uint32_t)(len * elem_size);
                h->tensor_id = t;
                h->offset_elems = off;
                h->worker = w;
                h->reserved = 0;
                if (!payload_ring) continue;
                uint8_t* dst = payload_ring + slot * payload_bytes;
                memcpy(dst, g + (base[t] + off) * elem_size, len * elem_size);
                memset(dst + len * elem_size, 0, payload_bytes - len * elem_size);
            }
        }
    }
    free(base); free(cb);
    return ORC_OK;
}

/* Header of one packet alone (for spot checks at sizes where the full ring is
 * too large for the host). */
int dblp_oracle_header_at(const uint64_t* numel, uint32_t T, uint32_t elem_size, uint32_t payload_bytes,
                          uint32_t w, uint64_t seq, uint32_t round, orc_hdr_t* h, uint64_t* base_of_tensor)
{
    uint64_t E = payload_bytes / elem_size, b = 0, c = 0;
    for (uint32_t t = 0; t < T; ++t) {
        uint64_t nchunks = (numel[t] + E - 1) / E;
        if (seq < c + nchunks) {
            uint64_t off = (seq - c) * E;
            uint64_t len = numel[t] - off < E ? numel[t] - off : E;
            h->seq = (uint32_t)seq; h->round = round; h->len_bytes = (uint32_t)(len * elem_size);
            h->tensor_id = t; h->offset_elems = off; h->worker = w; h->reserved = 0;
            *base_of_tensor = b;
            return ORC_OK;
        }
        b += numel[t];
        c += nchunks;
    }
    return ORC_EINVAL;
}

/* ---------------------------------------------------------------------------
 * Bit helpers.  A per-worker bitmap row has ceil(C/32) words; chunk seq is bit
 * (seq mod 32) of word (seq div 32).  Kept as naive as possible.
 * ------------------------------------------------------------------------- */
static uint64_t row_words(uint64_t C) { return (C + 31) / 32; }
static int get_bit(const uint32_t* bm, uint64_t C, uint32_t w, uint64_t seq)
{
    return (bm[(uint64_t)w * row_words(C) + seq / 32] >> (seq % 32)) & 1u;
}
static void set_bit(uint32_t* bm, uint64_t C, uint32_t w, uint64_t seq)
{
    bm[(uint64_t)w * row_words(C) + seq / 32] |= (1u << (seq % 32));
}

/* ---------------------------------------------------------------------------
 * Loss process.  The paper injects loss without giving a generator (Section
 * II-C "randomly zeroing out a fraction"; Section V-B "manually injecting bursty
 * packet loss"), so the three processes are defined here, in integers:
 *   every packet id = w*C + seq owns one Philox draw; word 0 decides the drop,
 *   word 1 drives the burst chain's transition.
 *   iid:         drop iff u0 < t_drop.
 *   microburst:  one window of window_len consecutive seqs, the same for every
 *                worker (the server's ingress is the shared bottleneck,
 *                Section IV-D); drop iff u0 < (inside ? t_drop_in : t_drop_out).
 *   Gilbert-Elliott: per worker a two-state chain walked in seq order;
 *                state0 = Bad iff u_init(w) < t_init_bad;
 *                drop iff u0 < (Bad ? t_drop_bad : t_drop_good);
 *                then Bad stays Bad unless u1 < t_bg, Good turns Bad iff u1 < t_gb.
 * Output: delivered bitmap (1 = survived), rows per worker.
 * A retransmission attempt sends only the chunks the latest bitmap reports
 * missing (Algorithm 1: "for each unsent chunk"; Section III-B).  `sent` (same
 * layout as the output, NULL = everything) is that set: a chunk that is not
 * sent cannot arrive, and the burst chain, which models the channel while
 * packets cross it, advances only over the packets that are sent.
 * ------------------------------------------------------------------------- */
int dblp_oracle_loss_mask_sent(const orc_loss_t* m, uint64_t C, uint32_t W, uint64_t seed, uint32_t round,
                               uint32_t attempt, const uint32_t* sent, uint32_t* delivered,
                               uint64_t* window_start_out)
{
    if (!m || !delivered || C == 0 || W == 0) return ORC_EINVAL;
    memset(delivered, 0, sizeof(uint32_t) * row_words(C) * W);
    uint32_t u[4];
    uint64_t s0 = 0;
    if (m->kind == 3) {
        if (m->window_len > C) return ORC_EINVAL;
        draw(seed, 0, STREAM_WINDOW, attempt, round, u);
        s0 = (uint64_t)u[0] % (C - m->window_len + 1);
    }
    if (window_start_out) *window_start_out = s0;
    for (uint32_t w = 0; w < W; ++w) {
        int bad = 0;
        if (m->kind == 2) {
            draw(seed, w, STREAM_GE_INIT, attempt, round, u);
            bad = (uint64_t)u[0] < m->t_init_bad;
        }
        for (uint64_t seq = 0; seq < C; ++seq) {
            if (sent && !get_bit(sent, C, w, seq)) continue;
            uint64_t id = (uint64_t)w * C + seq;
            draw(seed, id, STREAM_PACKET, attempt, round, u);
            int drop;
            switch (m->kind) {
            case 0: drop = 0; break;
            case 1: drop = (uint64_t)u[0] < m->t_drop; break;
            case 2:
                drop = (uint64_t)u[0] < (bad ? m->t_drop_bad : m->t_drop_good);
                if (bad) bad = !((uint64_t)u[1] < m->t_bg);
                else     bad = ((uint64_t)u[1] < m->t_gb);
                break;
            case 3:
                drop = (uint64_t)u[0] < ((seq >= s0 && seq < s0 + m->window_len) ? m->t_drop_in : m->t_drop_out);
                break;
            default: return ORC_EINVAL;
            }
            if (!drop) set_bit(delivered, C, w, seq);
        }
    }
    return ORC_OK;
}

int dblp_oracle_loss_mask(const orc_loss_t* m, uint64_t C, uint32_t W, uint64_t seed, uint32_t round,
                          uint32_t attempt, uint32_t* delivered, uint64_t* window_start_out)
{
    return dblp_oracle_loss_mask_sent(m, C, W, seed, round, attempt, NULL, delivered, window_start_out);
}

/* What the sender retransmits after a bitmap reply: every chunk whose bit is 0. */
void dblp_oracle_missing_bits(uint64_t C, uint32_t W, const uint32_t* bitmap, uint32_t* sent)
{
    memset(sent, 0, sizeof(uint32_t) * row_words(C) * W);
    for (uint32_t w = 0; w < W; ++w)
        for (uint64_t seq = 0; seq < C; ++seq)
            if (!get_bit(bitmap, C, w, seq)) set_bit(sent, C, w, seq);
}

/* ---------------------------------------------------------------------------
 * Arrival order (property 1, order independence: Sections I and III-A).  A
 * seeded permutation pi of [0, M): a balanced Feistel network of 4 rounds on b
 * bits (b even, b >= 2, 2^b >= M, the smallest such), the round function one
 * Philox draw masked to b/2 bits, walked until the value falls below M.
 * ------------------------------------------------------------------------- */
static uint32_t perm_bits(uint64_t M)
{
    uint32_t b = 2;
    while (b < 64 && ((uint64_t)1 << b) < M) b += 2;
    return b;
}

uint64_t dblp_oracle_perm(uint64_t M, uint64_t seed, uint32_t round, uint32_t attempt, uint64_t a)
{
    uint32_t b = perm_bits(M), half = b / 2;
    uint64_t mask = ((uint64_t)1 << half) - 1;
    uint64_t x = a;
    do {
        uint64_t L = x >> half, R = x & mask;
        for (uint32_t r = 0; r < 4; ++r) {
            uint32_t ctr[4] = { (uint32_t)R, r, STREAM_PERM | (attempt << 8), round };
            uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
            uint32_t u[4];
            dblp_oracle_philox4x32_10(ctr, key, u);
            uint64_t F = (uint64_t)u[0] & mask;
            uint64_t nl = R, nr = L ^ F;
            L = nl; R = nr;
        }
        x = (L << half) | R;
    } while (x >= M);
    return x;
}

/* Survivors in permuted order: arrival = [pi(a) for a = 0..M-1 if delivered(pi(a))].
 * Entries are ring slots (packet ids w*C + seq). */
int dblp_oracle_arrival(uint64_t C, uint32_t W, uint64_t seed, uint32_t round, uint32_t attempt,
                        const uint32_t* delivered, uint32_t* arrival, uint64_t* n_arrived)
{
    uint64_t M = C * W, n = 0;
    if (M >= 0x80000000ull) return ORC_EINVAL;
    for (uint64_t a = 0; a < M; ++a) {
        uint64_t p = dblp_oracle_perm(M, seed, round, attempt, a);
        uint32_t w = (uint32_t)(p / C);
        uint64_t seq = p % C;
        if (get_bit(delivered, C, w, seq)) arrival[n++] = (uint32_t)p;
    }
    *n_arrived = n;
    return ORC_OK;
}

/* ---------------------------------------------------------------------------
 * Bookkeeping (Algorithm 2, the chunk branch of the loop: integrity check,
 * accept, update bitmap; Section III-A: drop what is not of the current round).
 * Walks the arrival list in order.  An entry is
 *   invalid  if its slot is outside the ring or its header contradicts the plan
 *            (worker, tensor, offset on a chunk boundary and inside the tensor,
 *            length = that chunk's length, seq = that chunk's sequence number);
 *   stale    if its round counter is not the current round (older or newer);
 *   a duplicate if the bit of (worker, seq) is already set -- the first arrival
 *            keeps the slot;
 *   accepted otherwise: bit set, slot_of and first_arrival recorded.
 * bitmap, slot_of, first_arrival and counters are in/out so a later attempt can
 * continue the same round (Section III-B: retransmission works from the most
 * recent bitmap).  The arrival number of entry a is counters->n_arrived (as it
 * stood before the call) + a.
 * With early_stop (Algorithm 2, the branch without a probe: "if the
 * loss-tolerance threshold is satisfied, send stop"), each worker's receiver
 * stops the moment its own missing / total <= p holds (total = C, one bitmap
 * per worker stream); whatever that worker delivers afterwards, valid and of
 * this round, is late and ignored.  The integrity and round checks come first,
 * as they do for a running receiver.
 * ------------------------------------------------------------------------- */
int dblp_oracle_book_stop(const uint64_t* numel, uint32_t T, uint32_t elem_size, uint32_t payload_bytes,
                          uint32_t W, const orc_hdr_t* hdr_ring, uint64_t n_slots,
                          const uint32_t* arrival, uint64_t n_arrived, uint32_t round,
                          int early_stop, uint32_t bound_ppm,
                          uint32_t* bitmap, uint32_t* slot_of, uint32_t* first_arrival, orc_counters_t* cnt)
{
    uint64_t* base = (uint64_t*)malloc(sizeof(uint64_t) * T);
    uint64_t* cb = (uint64_t*)malloc(sizeof(uint64_t) * ((size_t)T + 1));
    if (!base || !cb) { free(base); free(cb); return ORC_EINVAL; }
    int rc = dblp_oracle_plan(numel, T, elem_size, payload_bytes, base, cb);
    if (rc) { free(base); free(cb); return rc; }
    uint64_t E = payload_bytes / elem_size, C = cb[T];
    uint64_t first = cnt->n_arrived;
    uint64_t* got = (uint64_t*)calloc(W, sizeof(uint64_t));          /* chunks received so far, per worker */
    if (!got) { free(base); free(cb); return ORC_EINVAL; }
    for (uint32_t w = 0; w < W; ++w)
        for (uint64_t s = 0; s < C; ++s) got[w] += (uint64_t)get_bit(bitmap, C, w, s);
    for (uint64_t a = 0; a < n_arrived; ++a) {
        cnt->n_arrived++;
        uint64_t slot = arrival[a];
        if (slot >= n_slots) { cnt->n_invalid++; continue; }
        const orc_hdr_t* h = &hdr_ring[slot];
        int valid = 0;
        if (h->worker < W && h->tensor_id < T) {
            uint64_t n = numel[h->tensor_id];
            if (h->offset_elems % E == 0 && h->offset_elems < n) {
                uint64_t len = n - h->offset_elems < E ? n - h->offset_elems : E;
                if (h->len_bytes == len * elem_size && h->seq == cb[h->tensor_id] + h->offset_elems / E)
                    valid = 1;
            }
        }
        if (!valid) { cnt->n_invalid++; continue; }
        if (h->round != round) { cnt->n_stale++; continue; }
        if (early_stop && (C - got[h->worker]) * 1000000ull <= (uint64_t)bound_ppm * C) { cnt->n_late++; continue; }
        if (get_bit(bitmap, C, h->worker, h->seq)) { cnt->n_dup++; continue; }
        set_bit(bitmap, C, h->worker, h->seq);
        slot_of[(uint64_t)h->worker * C + h->seq] = (uint32_t)slot;
        first_arrival[(uint64_t)h->worker * C + h->seq] = (uint32_t)(first + a);
        cnt->n_accepted++;
        got[h->worker]++;
    }
    free(base); free(cb); free(got);
    return ORC_OK;
}

int dblp_oracle_book(const uint64_t* numel, uint32_t T, uint32_t elem_size, uint32_t payload_bytes,
                     uint32_t W, const orc_hdr_t* hdr_ring, uint64_t n_slots,
                     const uint32_t* arrival, uint64_t n_arrived, uint32_t round,
                     uint32_t* bitmap, uint32_t* slot_of, uint32_t* first_arrival, orc_counters_t* cnt)
{
    return dblp_oracle_book_stop(numel, T, elem_size, payload_bytes, W, hdr_ring, n_slots, arrival, n_arrived, round,
                                 0, 0, bitmap, slot_of, first_arrival, cnt);
}

/* bf16 -> fp32 is exact: the 16 bits are the top half of the fp32 pattern. */
static float widen_bf16(uint16_t v)
{
    uint32_t bits = (uint32_t)v << 16;
    float f;
    memcpy(&f, &bits, 4);
    return f;
}

/* ---------------------------------------------------------------------------
 * Reduce (Algorithm 2, last three lines: unreceived chunks stay zero, the data
 * is put back in place; Algorithm 3: the server takes the mean over all N
 * workers).  By definition, for element i in chunk c:
 *     agg[i] = sum over w = 0..W-1, in that order, of (received(w,c) ? g_w[i] : nothing)
 * starting from +0.0f, each addition a plain IEEE fp32 add; mean divides that
 * sum by (float)W -- by all workers, not by how many arrived.
 * The value of g_w[i] is read from the payload slot recorded for (w, c), and
 * the destination comes from the plan (tensor base + chunk offset).
 * ------------------------------------------------------------------------- */
int dblp_oracle_reduce(const uint64_t* numel, uint32_t T, uint32_t elem_size, uint32_t payload_bytes,
                       uint32_t W, const uint8_t* payload_ring, const uint32_t* bitmap,
                       const uint32_t* slot_of, int mean, float* agg)
{
    uint64_t* base = (uint64_t*)malloc(sizeof(uint64_t) * T);
    uint64_t* cb = (uint64_t*)malloc(sizeof(uint64_t) * ((size_t)T + 1));
    if (!base || !cb) { free(base); free(cb); return ORC_EINVAL; }
    int rc = dblp_oracle_plan(numel, T, elem_size, payload_bytes, base, cb);
    if (rc) { free(base); free(cb); return rc; }
    uint64_t E = payload_bytes / elem_size, C = cb[T];
    for (uint32_t t = 0; t < T; ++t) {
        int64_t nchunks = (int64_t)((numel[t] + E - 1) / E);
        #pragma omp parallel for schedule(static)
        for (int64_t j = 0; j < nchunks; ++j) {
            uint64_t off = (uint64_t)j * E;
            uint64_t len = numel[t] - off < E ? numel[t] - off : E;
            uint64_t c = cb[t] + (uint64_t)j;
            for (uint64_t e = 0; e < len; ++e) {
                float acc = 0.0f;
                for (uint32_t w = 0; w < W; ++w) {
                    if (!get_bit(bitmap, C, w, c)) continue;
                    const uint8_t* p = payload_ring + (uint64_t)slot_of[(uint64_t)w * C + c] * payload_bytes;
                    float x;
                    if (elem_size == 4) memcpy(&x, p + e * 4, 4);
                    else { uint16_t v; memcpy(&v, p + e * 2, 2); x = widen_bf16(v); }
                    acc = acc + x;
                }
                if (mean) acc = acc / (float)W;
                agg[base[t] + off + e] = acc;
            }
        }
    }
    free(base); free(cb);
    return ORC_OK;
}

/* The same definition evaluated at listed elements only, from the workers' own
 * values at those elements (vals[w*n + k] = g_w[elem[k]]), for sizes at which the
 * rings do not fit on the host. */
int dblp_oracle_reduce_at(const uint64_t* numel, uint32_t T, uint32_t elem_size, uint32_t payload_bytes,
                          uint32_t W, const uint32_t* bitmap, uint64_t n, const uint64_t* elem,
                          const void* vals, int mean, float* out)
{
    uint64_t E = payload_bytes / elem_size, C = 0;
    for (uint32_t t = 0; t < T; ++t) C += (numel[t] + E - 1) / E;
    for (uint64_t k = 0; k < n; ++k) {
        uint64_t b = 0, c0 = 0, c = 0;
        int found = 0;
        for (uint32_t t = 0; t < T; ++t) {
            if (elem[k] < b + numel[t]) { c = c0 + (elem[k] - b) / E; found = 1; break; }
            b += numel[t];
            c0 += (numel[t] + E - 1) / E;
        }
        if (!found) return ORC_EINVAL;
        float acc = 0.0f;
        for (uint32_t w = 0; w < W; ++w) {
            if (!get_bit(bitmap, C, w, c)) continue;
            float x;
            if (elem_size == 4) x = ((const float*)vals)[(uint64_t)w * n + k];
            else x = widen_bf16(((const uint16_t*)vals)[(uint64_t)w * n + k]);
            acc = acc + x;
        }
        if (mean) acc = acc / (float)W;
        out[k] = acc;
    }
    return ORC_OK;
}

/* ---------------------------------------------------------------------------
 * Tolerance test (Section III-B: stop once the ratio of missing packets is equal
 * to or less than p; Algorithm 2: stop signal versus bitmap reply).  Per worker
 * and bucket (a contiguous seq range; one bucket = the paper's single bitmap per
 * worker stream): count received chunks bit by bit, missing = total - received,
 * ok iff missing / total <= p, evaluated exactly with p in parts per million:
 * missing * 10^6 <= p_ppm * total.
 * ------------------------------------------------------------------------- */
int dblp_oracle_check_bound(uint64_t C, uint32_t W, const uint32_t* bitmap,
                            const uint64_t* bucket_bounds, uint32_t B,
                            const uint32_t* bound_ppm, uint32_t n_bounds,
                            uint32_t* recv, uint32_t* missing, uint8_t* ok, uint32_t* all_ok)
{
    if (n_bounds != 1 && n_bounds != B) return ORC_EINVAL;
    uint32_t all = 1;
    for (uint32_t w = 0; w < W; ++w) {
        for (uint32_t b = 0; b < B; ++b) {
            uint64_t lo = bucket_bounds ? bucket_bounds[b] : 0;
            uint64_t hi = bucket_bounds ? bucket_bounds[b + 1] : C;
            uint64_t got = 0;
            for (uint64_t s = lo; s < hi; ++s) got += (uint64_t)get_bit(bitmap, C, w, s);
            uint64_t total = hi - lo, miss = total - got;
            uint64_t p = bound_ppm[n_bounds == 1 ? 0 : b];
            int pass = miss * 1000000ull <= p * total;
            recv[(uint64_t)w * B + b] = (uint32_t)got;
            missing[(uint64_t)w * B + b] = (uint32_t)miss;
            ok[(uint64_t)w * B + b] = (uint8_t)pass;
            if (!pass) all = 0;
        }
    }
    *all_ok = all;
    return ORC_OK;
}

/* ---------------------------------------------------------------------------
 * Critical-learning-regime test (Eq. 1): | ||G_prev|| - ||G_curr|| | / ||G_prev|| >= eta.
 * Evaluated as printed, in fp64.  A zero previous norm (nothing to compare
 * with) counts as critical.  The absolute value makes a rise trigger as well as
 * a drop.
 * ------------------------------------------------------------------------- */
int dblp_oracle_clr(double norm_prev, double norm_curr, double eta)
{
    if (norm_prev == 0.0) return 1;
    double d = norm_prev - norm_curr;
    if (d < 0) d = -d;
    return d / norm_prev >= eta;
}

/* ---------------------------------------------------------------------------
 * Tolerance schedule (Section IV-D; Algorithm 3, the epoch branch).  Training
 * starts at P_low.  At the beginning of an epoch the threshold is reset to
 * P_high and, if the regime test fires, set to P_low.  Otherwise it is kept.
 * ------------------------------------------------------------------------- */
uint32_t dblp_oracle_select_bound(double norm_prev, double norm_curr, double eta,
                                  uint32_t p_low_ppm, uint32_t p_high_ppm,
                                  int at_epoch_start, int first_iteration, uint32_t current_ppm)
{
    if (first_iteration) return p_low_ppm;
    if (!at_epoch_start) return current_ppm;
    uint32_t p = p_high_ppm;
    if (dblp_oracle_clr(norm_prev, norm_curr, eta)) p = p_low_ppm;
    return p;
}

/* ---------------------------------------------------------------------------
 * L2 norm of the aggregated gradient (Eq. 1 compares ||G_prev|| with ||G_curr||;
 * Section III-B: the L2 norm).  By definition ||G||^2 = sum_i g_i^2.  Each square
 * of an fp32 value is exact in fp64; the sum is carried with Neumaier's
 * compensated summation so that the result is the exactly rounded sum to within
 * an ulp or two whatever N is -- the definition's value, not one particular
 * order of additions.
 * ------------------------------------------------------------------------- */
int dblp_oracle_norm(const float* g, uint64_t n, double* sum_sq, double* norm)
{
    double s = 0.0, c = 0.0;
    for (uint64_t i = 0; i < n; ++i) {
        double x = (double)g[i] * (double)g[i];
        double t = s + x;
        if ((s >= 0 ? s : -s) >= x) c += (s - t) + x;
        else c += (x - t) + s;
        s = t;
    }
    *sum_sq = s + c;
    *norm = sqrt(*sum_sq);      /* the C library's sqrt: correctly rounded by IEEE 754 */
    return ORC_OK;
}

/* ---------------------------------------------------------------------------
 * Worker update (Algorithm 4: w <- w - alpha * g_hat): one fp32 multiply, then
 * one fp32 subtract, per element.
 * ------------------------------------------------------------------------- */
void dblp_oracle_sgd_apply(float* params, const float* g, float lr, uint64_t n)
{
    for (uint64_t i = 0; i < n; ++i) {
        float step = lr * g[i];
        params[i] = params[i] - step;
    }
}

/* ---------------------------------------------------------------------------
 * fp32 -> bf16 with round to nearest, ties to even (the optional 16-bit output
 * of the aggregate).  bf16 keeps the upper 16 bits of the fp32 pattern; the
 * discarded 16 bits decide the rounding: above half -> up, below half -> down,
 * exactly half -> to the even neighbour.  A NaN stays a (quiet) NaN.
 * ------------------------------------------------------------------------- */
void dblp_oracle_to_bf16(const float* x, uint16_t* out, uint64_t n)
{
    for (uint64_t i = 0; i < n; ++i) {
        uint32_t b;
        memcpy(&b, &x[i], 4);
        uint32_t upper = b >> 16, rest = b & 0xFFFFu;
        if ((b & 0x7FFFFFFFu) > 0x7F800000u) { out[i] = (uint16_t)(upper | 0x40u); continue; }
        if (rest > 0x8000u || (rest == 0x8000u && (upper & 1u))) upper += 1;   /* a carry into the exponent is the right result */
        out[i] = (uint16_t)upper;
    }
}
