/*
 * qkvshare.h -- C interface of the CacheCard create / inject library (CUDA, sm_100a).
 *
 * A CacheCard is the artifact one agent hands to the next in place of re-prefilling a shared
 * context (Section 4.2 of the QKVShare paper): the sender's FP16 key/value cache, quantised
 * token by token at a bit-width b(t) in {2, 4, 8, 16} (Section 3.3; 16 keeps the token in
 * FP16), packed together with the bit-width vector, the sequence length, model and sender
 * identifiers, a position-offset placeholder and the achieved average bit-width
 * (Section 4.2.1).  The receiver rebuilds FP16 keys and values in the [heads, tokens,
 * head_dim] layout of a HuggingFace cache (Section 4.2.2).
 *
 * The paper fixes no arithmetic or byte layout; this library uses:
 *   groups of 32 consecutive channels of one token row, for K and V alike;
 *   zero = group minimum, scale = (max - min) / (2^b - 1), both fp32;
 *   code = round-to-nearest-even((x - zero) * ((2^b - 1) / (max - min))), clamped to [0, 2^b - 1];
 *   reconstruction = fp16_rne(fl32(code * scale) + zero);  every step one IEEE binary32
 *   operation, never fused; a constant group has scale 0 and all-zero codes.
 * Compact metadata (qkvs_layout_t.meta_bytes = 4).  Section 3.1 counts a 4-bit cache at about
 * 0.5 bytes per element, which eight bytes of scale and zero per 32 elements (two more bits per
 * element) do not leave room for; the paper says nothing on how the metadata is kept.  In this
 * variant a group keeps an FP16 pair: zero, a group minimum, is an FP16 value already and is kept
 * exactly; scale = (max - min) / (2^b - 1) computed as above and then rounded UP to FP16, so that
 * the largest value still maps inside the code range; the codes are taken against the stored
 * scale, code = round-to-nearest-even((x - zero) * fl32(1 / scale)), and reconstruction is the
 * same formula with the two FP16 values widened.  One more bit per element instead of two:
 * 5 / 3 / 9 effective bits at 4 / 2 / 8.  Needs head_dim to be a multiple of 128.
 *
 * Card bytes (little-endian; every section padded with zeros to a multiple of 256):
 *   [0, 256)        qkvs_card_header_t
 *   bits_off        bits[seg][t]  u8           seg = 0 (bits_mode 0) or layer*H + head (mode 1)
 *   offs_off        off[seg][0..T] u32         exclusive prefix sum of record sizes
 *   sbase_off       sbase[0..S] u64            (bits_mode 1 only) start of each stream in the payload
 *   payload_off     streams one after another, stream index s = (layer*2 + kv)*H + head,
 *                   kv 0 = K, 1 = V; token t's record sits at off[seg][t] inside its stream.
 *   record, b < 16: d/32 pairs {scale, zero} (two fp32, or two FP16 in the compact variant), then
 *                   d*b/8 code bytes, which therefore start on a 16-byte boundary; the code of
 *                   channel i occupies bits [i*b, i*b + b) of the code bytes read as a
 *                   little-endian bit string.  record, b = 16: the d FP16 values verbatim.
 *   record size:    d*b/8 + meta_bytes*(d/32) bytes for b in {2,4,8};  2*d bytes for b = 16;
 *                   always a multiple of 16.
 * Wider groups (qkvs_layout_t.group_size = 64 or 128, head_dim 128 or 256).  A group of 64 or 128
 * channels shares one {scale, zero} pair, computed exactly as above over the wider group; a record
 * then carries d/group pairs followed by zero bytes up to the next multiple of 16, then the codes:
 *                   d*b/8 + round_up_16(meta_bytes*(d/group)) bytes.
 * At head_dim 128 that is 80 bytes at 4 bits for every wide combination (5 bits per element, the
 * same as FP16 pairs on groups of 32, because of the padding); at head_dim 256, one FP16 or fp32
 * pair per 128 channels gives 144 bytes (4.5 bits per element).  The wider the group, the larger
 * the range one scale has to cover: channel-wise key outliers then cost every channel of the
 * group precision.  Card creation, injection and attention from the card (head_dim 128) support it.
 *
 * All entry points return a qkvs_status_t.  Unless stated otherwise a pointer named *_dev is a
 * device pointer, anything else is a host pointer.  The library allocates no device memory and
 * every buffer belongs to the caller.  What it keeps between calls is small and per device: how
 * many CTAs of each kernel the device holds at once (looked up at a kernel's first launch), and,
 * for qkvs_card_inject_noalloc, the device address of its built-in counter array together with
 * that array's content (see there).  Both are remembered for the life of the process; a
 * cudaDeviceReset() invalidates the remembered address, so do not reset a device between calls.
 * Launches are asynchronous on the given CUDA stream (a cudaStream_t passed as void*; NULL is the
 * default stream).
 *
 * Non-finite input.  The quantiser is defined for finite values.  A NaN or an infinity inside a
 * token that is quantised (b < 16) gives unspecified scale, zero and codes for its group -- the
 * codes of one group may then spill into each other inside the group's own code bytes -- but
 * every access stays inside the record, the card and the cache: memory-safe, not meaningful.
 * Tokens kept at 16 bits carry any bit pattern through unchanged.
 *
 * Scratch block.  qkvs_card_create and qkvs_card_inject take an optional `workspace_dev`: a
 * device buffer of QKVS_WORKSPACE_BYTES bytes, 16-byte aligned, owned by the caller.  Its content
 * on entry does not matter (each call clears it on its stream).  The kernels keep in it the
 * counters from which their warps draw work -- with them, SMs that run faster simply take more of
 * it -- and, for injection, the status word described there.  Without a block (NULL) the work is
 * split evenly in advance, which is a few percent slower, and injection reports no status.
 * Two calls that may run on the GPU at the same time must not share a block.
 */
#ifndef QKVSHARE_H_
#define QKVSHARE_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define QKVS_API __attribute__((visibility("default")))
#else
#define QKVS_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

#define QKVS_WORKSPACE_BYTES 256

typedef enum {
    QKVS_OK = 0,
    QKVS_ERR_INVALID_ARG = 1,      /* null pointer, negative size, misaligned pointer or stride */
    QKVS_ERR_UNSUPPORTED_SHAPE = 2,/* head_dim not in {64,128,192,256}, group_size not in {32,64,128}
                                      (64 and 128 need head_dim 128 or 256), compact metadata on
                                      groups of 32 with a head_dim that is not a multiple of 128 */
    QKVS_ERR_BAD_BITS = 3,         /* a bit-width outside {2,4,8,16} */
    QKVS_ERR_BUFFER_TOO_SMALL = 4, /* card capacity below what the bit-widths need */
    QKVS_ERR_BAD_CARD = 5,         /* header magic/version/shape/status/size does not check out */
    QKVS_ERR_CUDA = 6,             /* a CUDA runtime call or launch failed */
    QKVS_ERR_TIMEOUT = 7           /* a bounded wait inside a kernel gave up */
} qkvs_status_t;

/* One agent's KV cache: per layer one K and one V block of FP16, HuggingFace layout
 * [1, n_kv_heads, tokens, head_dim] (Section 4.2.2), addressed as
 * base + head*head_stride + token*token_stride + channel (strides in elements). */
typedef struct {
    int32_t n_layers;
    int32_t n_kv_heads;
    int32_t head_dim;     /* 64, 128, 192 or 256 */
    int32_t n_tokens;     /* tokens in the card (sequence length, Section 4.2.1) */
    int32_t group_size;   /* channels per quantisation group: 32, or 64 / 128 (see above) */
    int32_t bits_mode;    /* 0: one bits[n_tokens] for the whole model (the paper's token-level
                             vector); 1: bits[n_layers*n_kv_heads][n_tokens] */
    int64_t head_stride;  /* elements between heads; multiple of 8 */
    int64_t token_stride; /* elements between tokens; >= head_dim, multiple of 8 */
    int32_t meta_bytes;   /* bytes of {scale, zero} per group in the card: 8 (or 0) = two fp32,
                             4 = two FP16 (compact variant above).  A card is read back with the
                             value it was made with: the header records it and a mismatch is a
                             BAD_CARD. */
    int32_t reserved_;    /* 0 */
} qkvs_layout_t;

/* Identifiers carried in the card (Section 4.2.1).  position_offset is the placeholder the
 * paper reserves for cross-prefix alignment; it is stored and returned, never interpreted. */
typedef struct {
    uint64_t model_id;
    uint64_t sender_id;
    int64_t position_offset;
} qkvs_card_meta_t;

/* The first 256 bytes of every card. */
typedef struct {
    uint32_t magic;                /* 0x53564B51, "QKVS" */
    uint32_t version;              /* 1 */
    uint32_t status;               /* qkvs_status_t recorded on the device; 0 = usable card */
    uint32_t bits_mode;
    int32_t n_layers, n_kv_heads, head_dim, n_tokens, group_size;
    uint32_t meta_bytes_per_group; /* 8 or 4 */
    uint64_t model_id;
    uint64_t sender_id;
    int64_t position_offset;
    uint64_t sum_bits;             /* sum of b(t) over all segments and tokens */
    float avg_code_bits;           /* (float)sum_bits / (float)(segments * n_tokens) (Section 4.2.1) */
    uint32_t pad0_;
    uint64_t bits_off, offs_off, payload_off;
    uint64_t stream_bytes;         /* bits_mode 0: bytes of one stream; bits_mode 1: 0 */
    uint64_t total_bytes;          /* header + tables + payload */
    uint64_t sbase_off;            /* bits_mode 1: offset of the stream-base table; else 0 */
    uint8_t reserved_[128];
} qkvs_card_header_t;

/* Record size in bytes of one token row of `head_dim` channels at bit-width b with meta_bytes
 * (8, 0 for 8, or 4) of scale and zero per group of 32 channels; 0 if b is not one of {2,4,8,16} or the
 * combination of head_dim and meta_bytes is not supported.  Host only.  (Closed form above;
 * Section 3.1 for the code bytes.) */
QKVS_API size_t qkvs_record_bytes(int32_t head_dim, int32_t b, int32_t meta_bytes);

/* Exact size of the card for a bit-width vector (Section 4.2.1: the card is variable-length,
 * its size follows from b(t)).  Host only, no GPU work.
 *   bits_host  host array, n_tokens entries (mode 0) or n_layers*n_kv_heads*n_tokens (mode 1);
 *              NULL gives the worst case (every token FP16).
 *   out_bytes  receives header + tables + payload.
 * Strides of `layout` are not looked at.  Errors: INVALID_ARG, UNSUPPORTED_SHAPE, BAD_BITS. */
QKVS_API qkvs_status_t qkvs_card_size(const qkvs_layout_t *layout, const uint8_t *bits_host,
                             size_t *out_bytes);

/* Bytes in front of the payload (header + bits + offsets [+ stream bases]); a card buffer must
 * hold at least this much for qkvs_card_create to start.  Host only. */
QKVS_API qkvs_status_t qkvs_card_prefix_size(const qkvs_layout_t *layout, size_t *out_bytes);

/* Bit-widths from importance scores (the step in front of card creation; Section 3.3: tokens
 * that matter more get more bits; Section 4.1.2: b(t) in {2, 4, 8, 16}).  The paper's controller
 * is a trained network; this is the rank rule of an adaptive budget: order the tokens of a
 * segment by score, highest first, equal scores by lower token index first; the first n_fp16 keep
 * FP16, the next n_8bit get 8 bits, the next n_4bit get 4 bits, the rest 2 bits.
 *   scores_dev   device float32 [n_segments][n_tokens], finite values
 *   bits_dev     device uint8  [n_segments][n_tokens]: ready to be passed to qkvs_card_create
 *                (n_segments = 1 for bits_mode 0, n_layers * n_kv_heads for bits_mode 1)
 * The result is exact (integer ranks).  n_tokens up to 2^20.  Asynchronous on `stream`.  One CTA per
 * segment finds the scores at the three cuts by selection (a byte of the key per pass), equal
 * scores are told apart by a prefix count in index order; nothing is sorted. */
QKVS_API qkvs_status_t qkvs_bits_from_scores(const float *scores_dev, int32_t n_segments,
                                    int32_t n_tokens, int32_t n_fp16, int32_t n_8bit,
                                    int32_t n_4bit, uint8_t *bits_dev, void *stream);

/* Bit-widths under a byte budget (Section 3.3: minimise sum_t eps(t, b(t)) * S(t) subject to
 * sum_t b(t) * d <= M).  The paper prints the objective and no solver; this is the greedy solution
 * of that knapsack by worth per byte, stated so that the result is unique:
 *   - every token starts at 2 bits; raising a token one rung up the ladder 2 -> 4 -> 8 -> 16 is an
 *     upgrade i = 0, 1, 2 whose cost is the difference of the two record sizes (metadata included)
 *     and whose worth per byte is  key = fl32(S(t) * upgrade_weight[i]);
 *   - all 3 * n_tokens upgrades are ordered by key, larger first, equal keys by lower rung, then by
 *     lower token index (with non-negative scores and non-increasing weights a token's own upgrades
 *     come in rung order);
 *   - upgrades are granted in that order while their cost fits into what the budget leaves after
 *     2 bits for everybody; the first one that does not fit ends the procedure.
 *   scores_dev      device float32 [n_segments][n_tokens], finite and non-negative
 *   head_dim, meta_bytes   fix the record sizes (as in qkvs_record_bytes)
 *   budget_bytes    bound on the bytes of ONE stream: sum_t record(b(t)) <= budget_bytes
 *   upgrade_weight  host array of three positive, non-increasing floats, or NULL for 2^-9, 2^-14,
 *                   2^-23 -- the powers of two next to what a quantisation-noise model
 *                   eps(b) = 4^-b gives per byte at head_dim 128
 *   bits_dev        device uint8 [n_segments][n_tokens]
 *   offsets_dev     optional device uint32 [n_segments][n_tokens + 1]: the exclusive prefix sum of
 *                   the record sizes the bit-widths imply, i.e. the offset table of a card, from
 *                   the same launch
 *   status_dev      optional device int32, cleared by the call; raised to INVALID_ARG by a negative
 *                   or non-finite score (every token of that segment then gets 2 bits)
 * Errors on the host: INVALID_ARG, UNSUPPORTED_SHAPE, BUFFER_TOO_SMALL (the budget does not hold
 * 2 bits per token), CUDA.  Exact; n_tokens up to 2^20; asynchronous on `stream`. */
QKVS_API qkvs_status_t qkvs_bits_from_scores_budget(const float *scores_dev, int32_t n_segments, int32_t n_tokens,
                                                    int32_t head_dim, int32_t meta_bytes, uint64_t budget_bytes,
                                                    const float *upgrade_weight, uint8_t *bits_dev,
                                                    uint32_t *offsets_dev, int32_t *status_dev, void *stream);

/* The combined importance score of Section 3.3, S(t) = alpha * I(t) + (1 - alpha) * T(t): local
 * importance I and transferability T weighed by alpha in [0, 1], the quantity the bit-widths are
 * assigned from.  How I and T are obtained (attention statistics, agent topology) is outside this
 * library; this is the combination itself, elementwise, feeding qkvs_bits_from_scores.
 * Arithmetic: binary32, each step rounded to nearest, nothing fused:
 *     S = fl( fl(alpha * I) + fl( fl(1 - alpha) * T ) ).
 *   importance_dev, transfer_dev   device float32 [n]
 *   scores_dev                     device float32 [n]; may be one of the inputs
 * Asynchronous on `stream`.  Errors: INVALID_ARG (null or misaligned pointer, negative n, alpha
 * outside [0, 1] or not a number), CUDA. */
QKVS_API qkvs_status_t qkvs_combine_scores(const float *importance_dev, const float *transfer_dev,
                                  float alpha, int64_t n, float *scores_dev, void *stream);

/* Bit-widths from the controller of Section 4.1.2: a two-layer perceptron over six features per
 * token (frequency, quality, attention variance, entropy, downstream demand, segment type) with
 * one output per bit-width; the paper gives the shape (6 -> hidden -> 4, 512 parameters, trained)
 * and no formula or weights, so the caller supplies the parameters and the arithmetic is fixed as
 *     hidden_j = max(0, b1[j] + sum_i W1[j][i] * x[i]),   out_k = b2[k] + sum_j W2[k][j] * hidden_j,
 * sums starting from the bias and taking the terms in index order, every product and every sum
 * rounded to binary32 on its own; b(t) = 2, 4, 8, 16 for the largest of out_0..3, equal outputs
 * going to the fewer bits.  How the features are obtained is outside this library.
 *   features_dev  device float32 [n_tokens][6]
 *   hidden        1..128 (46 gives 510 parameters, the size of this shape nearest to 512)
 *   params_dev    device float32: W1 [hidden][6], b1 [hidden], W2 [4][hidden], b2 [4], in this order
 *   bits_dev      device uint8 [n_tokens]: ready to be passed to qkvs_card_create
 *   outputs_dev   optional device float32 [n_tokens][4]: the four outputs per token
 * Asynchronous on `stream`.  Errors: INVALID_ARG (null or misaligned pointer, negative n_tokens,
 * hidden < 1), UNSUPPORTED_SHAPE (hidden > 128), CUDA. */
QKVS_API qkvs_status_t qkvs_bits_from_features(const float *features_dev, int64_t n_tokens, int32_t hidden,
                                      const float *params_dev, uint8_t *bits_dev, float *outputs_dev,
                                      void *stream);

/* Card creation (Section 4.2.1): offset scan over the bit-widths, then fused
 * min/max -> scale/zero -> quantise -> bit-pack of every (layer, K|V, head) stream.
 *   K_layers, V_layers  HOST arrays of n_layers DEVICE pointers to FP16 blocks (16-byte aligned)
 *   bits_dev            device array of bit-widths (see qkvs_card_size for its length)
 *   meta                identifiers to store; NULL stores zeros
 *   card_dev            device buffer, 16-byte aligned, written from byte 0
 *   card_capacity       its size in bytes; must cover at least the prefix
 *   workspace_dev       scratch block (see above) or NULL
 * Returns after enqueueing on `stream`.  Problems visible on the host (arguments, shape,
 * alignment, capacity below the prefix) are returned at once and nothing is launched.
 * Problems only the device can see -- a bit-width outside {2,4,8,16}, or a payload that does
 * not fit card_capacity -- are recorded in the card header's `status` (BAD_BITS,
 * BUFFER_TOO_SMALL); the payload is then not written and nothing outside the buffer is touched.
 * Read the outcome with qkvs_card_info.  The card's bytes are fully determined by the inputs.
 * A card of part of a cache -- say, only the tokens a hop appended since its last card -- is made
 * by passing pointers to the first row to encode (base + first * token_stride elements, which
 * keeps the alignment) with n_tokens rows to take and the strides unchanged; records do not
 * depend on where a token sits, so such a card's streams equal the matching slices of the whole
 * cache's card, and qkvs_card_inject places it with dst_token_offset. */
QKVS_API qkvs_status_t qkvs_card_create(const qkvs_layout_t *layout, const void *const *K_layers,
                               const void *const *V_layers, const uint8_t *bits_dev,
                               const qkvs_card_meta_t *meta, void *card_dev,
                               size_t card_capacity, void *workspace_dev, void *stream);

/* Receiver-side injection (Section 4.2.2): unpack, dequantise and write FP16 rows so that
 * token t of the card lands on row dst_token_offset + t of every head of every layer.
 *   card_dev, card_bytes   the card and the number of valid bytes behind the pointer
 *   dst                    shape and strides of the destination; n_layers, n_kv_heads, head_dim
 *                          and n_tokens must equal the card's (checked on the device), and
 *                          (dst_token_offset + n_tokens - 1)*token_stride + head_dim <= head_stride
 *   K_layers_out, V_layers_out   HOST arrays of n_layers DEVICE pointers (16-byte aligned)
 *   workspace_dev          scratch block (see above) or NULL.  Its first 4 bytes are an int32
 *                          status word: 0 after a clean run, raised to BAD_CARD by the kernel if
 *                          the header or its tables do not check out (rows whose table entries
 *                          are inconsistent are not written; with a bad header no row is), or to
 *                          TIMEOUT if a bounded wait gave up
 * Bytes of the destination outside the injected rows and channels are left untouched. */
QKVS_API qkvs_status_t qkvs_card_inject(const void *card_dev, size_t card_bytes, const qkvs_layout_t *dst,
                               void *const *K_layers_out, void *const *V_layers_out,
                               int64_t dst_token_offset, void *workspace_dev, void *stream);

/* Injection for callers that cannot give the library a scratch block.  (The paper has no
 * counterpart; this entry point exists for how the library gets embedded.)  Think of a receiver
 * inside a serving engine that has handed every free byte of the GPU to its KV-cache pool and
 * forbids its components to call cudaMalloc -- there is nothing left to allocate, and an
 * allocation would stall the whole device in the middle of serving -- yet still wants the evenly
 * loaded SMs that the work counters buy.  Same inputs, outputs and results as qkvs_card_inject;
 * the work counters live in a small array inside the library's own device image (256 bytes,
 * present on every GPU that has loaded the library, until the process exits).
 *   status_dev   optional device int32 (4-byte aligned), cleared by the call; the kernel raises it
 *                to BAD_CARD / TIMEOUT exactly like the status word of qkvs_card_inject
 * Limits and rules:
 *   - at most QKVS_NOALLOC_MAX_LAYERS layers per call (the array has 64 counters, one per 64
 *     layers); more are refused with QKVS_ERR_UNSUPPORTED_SHAPE and nothing is launched;
 *   - the call allocates and frees nothing, neither host-side nor on the device;
 *   - all calls on a device share the one array, which still holds what the previous call left
 *     there; each call clears it on its stream before its kernels run.  Two calls that may
 *     execute at the same time on one GPU (different streams, or different host threads) would
 *     disturb each other's counters: run them one after the other, or give the concurrent ones
 *     qkvs_card_inject with blocks of their own;
 *   - the first call on each device asks the runtime for the array's device address (with that
 *     device current) and remembers it; make that first call outside of any stream capture. */
#define QKVS_NOALLOC_MAX_LAYERS 4096
QKVS_API qkvs_status_t qkvs_card_inject_noalloc(const void *card_dev, size_t card_bytes,
                                       const qkvs_layout_t *dst, void *const *K_layers_out,
                                       void *const *V_layers_out, int64_t dst_token_offset,
                                       int32_t *status_dev, void *stream);

/* Hands a card to another GPU (Section 3.2: agents are the nodes of a graph and a handoff travels
 * along an edge; Section 4.2.1: the prototype hands the card over in memory, inside one runtime,
 * and fixes no wire format).  A card is one position-independent blob -- every offset in it is
 * relative to its first byte -- so the handoff is a plain copy of card_bytes bytes into a buffer
 * on the receiver's GPU, over NVLink when the two devices can reach each other; the receiver then
 * calls qkvs_card_inject (or qkvs_card_attend) on its own copy, on its own device.  No kernel of
 * this library ever reads another GPU's memory.
 *   card_dev, card_bytes   the card on the sender's GPU (device src_device); card_bytes is the
 *                          header's total_bytes (qkvs_card_info) or any size that covers it
 *   dst_dev, dst_capacity  buffer on device dst_device, 16-byte aligned, at least card_bytes
 *   stream                 a stream of the CURRENT device, which must be src_device or dst_device;
 *                          the copy is ordered after the work already in it (the create that made
 *                          the card) and the receiver orders its injection after the copy, e.g.
 *                          with an event recorded in this stream
 * src_device == dst_device makes an ordinary device-to-device copy.  With two devices the call
 * first turns on peer access from the current device to the other one if the hardware allows it
 * and it is not on yet (a per-process switch that stays on); without it the runtime stages the
 * copy through host memory, slower but equally correct.
 * Errors: INVALID_ARG (null or misaligned pointer, negative or unknown device), BAD_CARD
 * (card_bytes below a header), BUFFER_TOO_SMALL, CUDA.  Asynchronous on `stream`. */
QKVS_API qkvs_status_t qkvs_card_send(const void *card_dev, size_t card_bytes, int32_t src_device,
                                      void *dst_dev, size_t dst_capacity, int32_t dst_device, void *stream);

/* Decode-step attention straight from a card (Section 4.3 names consuming the quantised cache
 * inside attention as the goal; the FP16 cache of Section 4.2.2 is never rebuilt).  One query
 * token per layer attends to all n_tokens of the card, with grouped queries: query head j reads
 * KV head j / (n_q_heads / n_kv_heads):
 *     s_t = softmax_scale * q_j . K^_t,   p = softmax_t(s),   out_j = sum_t p_t V^_t
 * where K^, V^ are the values the records stand for, code * scale + zero (an FP16 token: its
 * values), without the rounding to FP16 that injection ends with: that rounding belongs to
 * handing an FP16 cache to the receiving framework (Section 4.2.2), which is not done here.
 * Products run on the tensor cores with FP16 inputs (the integer codes, exact in FP16, and the
 * probabilities times the scales, rounded to FP16) and FP32 accumulation; scale and zero are
 * applied outside the products.
 *   layout        n_layers, n_kv_heads, head_dim, n_tokens, meta_bytes and group_size of the card
 *                 (checked against its header on the device); head_dim must be 128; strides are
 *                 not looked at
 *   n_q_heads     multiple of n_kv_heads, at most 8 query heads per KV head.  The products have
 *                 eight columns per KV head whatever is used of them, so a model with four query
 *                 heads per KV head can pass the queries of two new tokens as eight heads per KV
 *                 head (row kv * 8 + token * 4 + head) and have both attended in the time of one
 *   q_dev         FP16 [n_layers][n_q_heads][head_dim], 16-byte aligned
 *   out_dev       FP32 [n_layers][n_q_heads][head_dim], 16-byte aligned; all zeros if n_tokens is
 *                 0 or the card does not check out
 *   scratch_dev   device buffer of at least qkvs_attend_scratch_size() bytes, 16-byte aligned,
 *                 content irrelevant on entry; afterwards its first int32 is the status word
 *                 (0, BAD_CARD or TIMEOUT, as for qkvs_card_inject).  Holds the work counter and
 *                 the per-item partial results that a second kernel merges
 * Asynchronous on `stream`.  Errors visible on the host: INVALID_ARG, UNSUPPORTED_SHAPE,
 * BAD_CARD (card_bytes below a header), BUFFER_TOO_SMALL (scratch), CUDA. */
QKVS_API qkvs_status_t qkvs_attend_scratch_size(const qkvs_layout_t *layout, int32_t n_q_heads,
                                                size_t *out_bytes);
QKVS_API qkvs_status_t qkvs_card_attend(const void *card_dev, size_t card_bytes,
                               const qkvs_layout_t *layout, int32_t n_q_heads, const void *q_dev,
                               float softmax_scale, float *out_dev, void *scratch_dev,
                               size_t scratch_bytes, void *stream);

/* Synchronises `stream`, copies the card's header to the host and returns its recorded status
 * (or BAD_CARD if magic/version are wrong, or CUDA on a runtime error). */
QKVS_API qkvs_status_t qkvs_card_info(const void *card_dev, void *stream, qkvs_card_header_t *out_host);

/* Self-test of the arithmetic shortcuts inside card creation.  The quantiser needs
 * (max-min)/qmax and qmax/(max-min) correctly rounded; the kernels compute them without the
 * generic division routine.  This call compares both shortcuts with the IEEE division for every
 * binary32 value a difference of two FP16 numbers can take (2^-24 .. 131008) and qmax in
 * {3, 15, 255}.  (The paper has no counterpart; Section 4.2.1 only says "quantized groups".)
 *   mismatches_dev  device array of two uint64 (8-byte aligned), zeroed by the call;
 *                   [0] counts mismatches of qmax/range, [1] of range/qmax.  Both must read 0.
 * Asynchronous on `stream`; about 10^9 divisions, a few milliseconds. */
QKVS_API qkvs_status_t qkvs_selftest_division(uint64_t *mismatches_dev, void *stream);

/* Self-test of the bounded waits.  Inside the kernels a warp only ever waits for its own
 * asynchronous copies, and every such wait gives up after a time limit (two seconds): the warp then
 * raises QKVS_ERR_TIMEOUT in the status word, gives the copies it still has in flight the same
 * bounded time to land, and returns, so that a wedged copy engine costs a call, not the GPU.  This
 * entry point runs that wait on a barrier nothing will ever complete (one warp, no copy issued,
 * nothing in flight) with a limit of `limit_us` microseconds (1 .. 1 000 000) and checks that it
 * comes back.  (The paper has no counterpart.)
 *   status_dev     device int32 (4-byte aligned), cleared by the call; reads QKVS_ERR_TIMEOUT afterwards
 *   waited_ns_dev  optional device uint64 (8-byte aligned): how long the warp waited, in nanoseconds
 * Asynchronous on `stream`; the context stays usable. */
QKVS_API qkvs_status_t qkvs_selftest_bounded_wait(uint32_t limit_us, int32_t *status_dev,
                                                  uint64_t *waited_ns_dev, void *stream);

QKVS_API const char *qkvs_status_string(qkvs_status_t status);

/* Library version, major*100 + minor. */
QKVS_API int32_t qkvs_version(void);

#ifdef __cplusplus
}
#endif
#endif /* QKVSHARE_H_ */
