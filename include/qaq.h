/*
 * libqaq -- quality-adaptive KV-cache quantization and attention over the packed
 * cache (QAQ, arXiv 2403.04643), CUDA kernels for sm_100a behind a C ABI.
 *
 * Conventions that hold for every entry point unless its comment says otherwise:
 *   - Pointers are DEVICE pointers owned by the caller ("host" is said explicitly).
 *   - Work is enqueued on the caller's stream (a cudaStream_t passed as void*; NULL
 *     is the default stream) and the call returns without synchronising.
 *   - The return value is a qaq_status; nothing throws or aborts.  Argument and
 *     shape errors are found on the host before anything is launched.
 *   - Dense K/V inputs are binary16, logical shape [batch, heads, tokens, head_dim],
 *     head_dim contiguous, with element strides for batch, head and token.
 *   - "(b,h)" is one batch element of one head; all (b,h) are independent problems
 *     (Section 2.1 of the paper: Q in R^{1xD}, K,V in R^{TxD} "within each head").
 */
#ifndef QAQ_H
#define QAQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    QAQ_OK = 0,
    QAQ_ERR_INVALID_ARG = 1,       /* null pointer, negative size, bad enum */
    QAQ_ERR_UNSUPPORTED_SHAPE = 2, /* head_dim not in {32,64,128}, widths outside 1..8, ... */
    QAQ_ERR_CAPACITY = 3,          /* token or outlier capacity of the cache exceeded */
    QAQ_ERR_CUDA = 4,              /* a CUDA runtime call failed */
    QAQ_ERR_WORKSPACE = 5          /* workspace too small or misaligned */
} qaq_status;

const char* qaq_status_string(qaq_status s);

/* Tokens are stored in groups ("tiles") of this many consecutive tokens. */
#define QAQ_TILE_TOKENS 64

typedef struct {
    int batch, heads, head_dim; /* head_dim in {32, 64, 128} */
    int max_tokens;             /* capacity per (b,h) */
    int bits_min, bits_max;     /* allowed widths, 1 <= bits_min <= bits_max <= 8 */
    int window;                 /* attention window n (Section 4.2); 1 = no window */
    double outlier_frac;        /* alpha: proportion of values treated as outliers, both tails */
    long max_outliers_per_bh;   /* per tensor; <= 0: derived from outlier_frac with slack */
} qaq_config;

/* Scalars of the bit-width rules (Section 4.1), see qaq_policy_from_hyper. */
typedef struct {
    float cK; /* keys:   B = min{b : range       <= cK * 2^b} */
    float cV; /* values: B = min{b : range * S_t <= cV * 2^b} */
} qaq_policy;

typedef struct {
    long tokens;              /* tokens cached per (b,h) */
    long code_bytes[2];       /* packed code bytes, all (b,h): [0]=K, [1]=V */
    long outliers[2];         /* stored outliers, all (b,h) */
    long hist[2][9];          /* hist[x][b] = tokens of tensor x at width b */
    long resident_bytes;      /* codes + per-token metadata + tile tables + outliers in use */
    double cr_paper;          /* 16*2*T*D*BH / (code bits + 16 bits per outlier): memory
                                 "calculated by the quantized bit" (Sections 2.1, 5.2) */
    double cr_total;          /* fp16 bytes / resident_bytes */
    int device_status;        /* sticky qaq_status raised on the device (capacity) */
} qaq_stats;

typedef struct qaq_cache qaq_cache; /* opaque; owns its device memory */

/* Allocates (cudaMalloc on the current device) an empty cache.  host in, host out. */
qaq_status qaq_cache_create(const qaq_config* cfg, qaq_cache** out);
qaq_status qaq_cache_destroy(qaq_cache* c);
/* Forgets all tokens (asynchronous on `stream`). */
qaq_status qaq_cache_reset(qaq_cache* c, void* stream);
/* Tokens currently cached per (b,h) (host counter). */
long qaq_cache_tokens(const qaq_cache* c);

/* Name of the CUDA error behind the most recent QAQ_ERR_CUDA returned in this process
 * ("cudaSuccess" if there was none).  Host function. */
const char* qaq_last_cuda_error(void);

/*
 * Bit-width rule scalars from the paper's hyper-parameters (Section 4.1):
 *   key bound    sigma2(K_t) <= log(T^3/(T-1) * sigmaS_max^2 + 1) / qnorm2
 *   value bound  sigma(V_t)  <= sigmaX_max / (sqrt(T) * |S_t|)
 *   bit count    B = ceil(log2((max - min) / (2 sqrt(3) sigma)))
 * give cK = 2 sqrt(3) sigmaK and cV = 2 sqrt(3) sigmaX_max / sqrt(T) (binary64, rounded
 * once to binary32).  qnorm2 is the caller's quantile of sum_d (Q_d)^2 (the paper uses
 * the upper 10% quantile), T the number of cached tokens.  T < 2 or qnorm2 <= 0 gives
 * cK = 0, which makes every key take bits_max.  Pure host function; host_out is host memory.
 */
qaq_status qaq_policy_from_hyper(double sigmaS_max, double sigmaX_max, double qnorm2, long T,
                                 qaq_policy* host_out);

/*
 * Outlier thresholds (Section 4.2 "Outliers": values beyond the alpha% quantile at the
 * maximum and minimum ends).  Per (b,h) and tensor, over the N = T*head_dim non-NaN
 * values: k = floor(alpha*N/2), lo = k-th smallest, hi = k-th largest (exact order
 * statistics).  thr is [batch*heads][4] binary32 = {loK, hiK, loV, hiV}.  An entry x is
 * later an outlier iff !(lo <= x && x <= hi).  ws: qaq_thresholds_workspace_bytes bytes,
 * 16-byte aligned, overwritten.
 */
qaq_status qaq_thresholds_workspace_bytes(const qaq_config* cfg, size_t* host_out);
qaq_status qaq_outlier_thresholds(const qaq_config* cfg, const void* K, const void* V, long stride_b,
                                  long stride_h, long stride_t, int n_tokens, float* thr, void* ws,
                                  size_t ws_bytes, void* stream);

/*
 * S1: per-token widths (Section 4.1 rules, Section 4.2 attention window).
 *   S_hat_t = max of the nvalid[t] valid rows of the score window for token t
 *             (nvalid[t] == 0: no score seen yet, the value takes bits_max);
 *   [min,max] of a token = range of its non-outlier entries (thr as above);
 *   bitsK[t] = min{b in [bits_min,bits_max] : (max-min)          <= cK * 2^b}, else bits_max
 *   bitsV[t] = min{b in [bits_min,bits_max] : (max-min) * S_hat_t <= cV * 2^b}, else bits_max
 * score_ring: binary32 [batch*heads][window][n_tokens]; nvalid: u8 [batch*heads][n_tokens];
 * bitsK, bitsV: u8 [batch*heads][n_tokens] (outputs).
 */
qaq_status qaq_select_bits(const qaq_config* cfg, const qaq_policy* policy, const void* K, const void* V,
                           long stride_b, long stride_h, long stride_t, int n_tokens,
                           const float* score_ring, const uint8_t* nvalid, const float* thr,
                           uint8_t* bitsK, uint8_t* bitsV, void* stream);

/*
 * Score window right after a prefill (Section 4.2, "Attention score prediction": the predicted
 * score of a token is the maximum over the scores of the preceding n queries; n = cfg->window,
 * at most 64).  From the last n queries of a prefill of n_tokens tokens and the unquantized keys:
 *   row of query i (position n_tokens-n+i) = softmax over the tokens t <= n_tokens-n+i of
 *   softmax_scale * q_i . k_t   (binary16 inputs, tensor-core products, binary32 sums),
 * written newest first: score_ring[bh][r][t] with r = n-1-i, so the rows in which token t exists
 * are 0..nvalid[t]-1, nvalid[t] = min(n, n_tokens-t); entries a query cannot see are 0.  This is
 * the layout qaq_select_bits / qaq_quantize_append / qaq_requantize_down take.  With fewer than n
 * tokens the queries that do not exist are ignored.
 * Q: binary16 [batch*heads][n][head_dim], 16-byte aligned; K as in qaq_outlier_thresholds;
 * score_ring: binary32 [batch*heads][n][n_tokens]; nvalid: u8 [batch*heads][n_tokens];
 * qnorm2: NULL or binary32 [batch*heads][n] receiving sum_d (softmax_scale * q_d)^2 per query
 * (the caller takes the quantile it wants for qaq_policy_from_hyper); ws:
 * qaq_prefill_window_workspace_bytes bytes, 8-byte aligned.  Device pointers, asynchronous on
 * stream.  Errors: QAQ_ERR_INVALID_ARG, QAQ_ERR_UNSUPPORTED_SHAPE (window > 64), QAQ_ERR_WORKSPACE.
 */
qaq_status qaq_prefill_window_workspace_bytes(const qaq_config* cfg, int n_tokens, size_t* host_out);
qaq_status qaq_prefill_window(const qaq_config* cfg, const void* Q, const void* K, long stride_b, long stride_h,
                              long stride_t, int n_tokens, float softmax_scale, float* score_ring,
                              uint8_t* nvalid, float* qnorm2, void* ws, size_t ws_bytes, void* stream);

/*
 * The scalar `qnorm2` of qaq_policy_from_hyper from a set of queries (Section 4.1, end of "Key cache
 * quantization": the distribution of the squared norm of the queries is taken beforehand and its upper
 * 10 % quantile stands for sum_d Q_d^2 in the key rule).  values: binary32 [n] on the device, e.g. the
 * qnorm2 array of qaq_prefill_window or a longer history kept by the caller; NaNs are not counted.
 * With N counted values sorted ascending the result is sorted[N-1-floor(upper_frac*N)], i.e. at most
 * upper_frac*N values lie above it (0 if N = 0).  out: one binary32 on the device, written
 * asynchronously on stream.  Exact (radix select by one CTA: meant for up to a few million values).
 * Errors: QAQ_ERR_INVALID_ARG (null pointer, n < 1, upper_frac outside [0,1)).
 */
qaq_status qaq_qnorm2_quantile(const float* values, long n, double upper_frac, float* out, void* stream);

/*
 * S2+S3: append n_new tokens per (b,h) to the cache: outlier split (entries outside
 * [lo,hi] are kept as binary16 in a sparse side list and take code 0), uniform
 * quantization of each token at its width (Section 4.1: the range [min,max] of the
 * non-outlier entries is cut into 2^B equal segments, each value is represented by the
 * midpoint of its segment) and bit-packing.
 *   step = (max-min) * 2^-B;  code = min(2^B-1, floor((x-min) * (1/step)))  in binary32.
 * bitsK/bitsV: u8 [batch*heads][n_new], or both NULL to choose the widths inside the
 * same kernel exactly as qaq_select_bits would (then policy, score_ring, nvalid are
 * required; score_ring is [batch*heads][window][n_new] for the new tokens, and the
 * policy scalars should have been made for the token count after the append).
 * thr: [batch*heads][4].  Returns QAQ_ERR_CAPACITY (nothing appended) if the token
 * capacity would be exceeded; an outlier-list overflow is detected on the device, drops
 * the surplus outliers and is reported by qaq_cache_stats().device_status.
 */
qaq_status qaq_quantize_append(qaq_cache* c, const void* K_new, const void* V_new, long stride_b,
                               long stride_h, long stride_t, int n_new, const uint8_t* bitsK,
                               const uint8_t* bitsV, const qaq_policy* policy, const float* score_ring,
                               const uint8_t* nvalid, const float* thr, void* stream);

/*
 * Further quantization of the cached tokens to lower widths (Section 4.2, "Integration in
 * text generation process": each step the widths of all existing tokens are computed again
 * and tokens whose new width is lower are quantized further).  For every cached token and
 * both tensors: new width = min(current width, w), where w is
 *   - bitsK/bitsV[bh][t] (values below 1 count as 1) when both are given, else
 *   - the width qaq_select_bits would choose now: the token's range max-min is taken from
 *     its stored metadata, the score window and the policy scalars are the caller's current
 *     ones (policy made for the current token count).
 * A lowered token keeps min, max and its outliers; its codes lose their low bits
 * (code >>= old-new, so step doubles per dropped bit), which equals quantizing the original
 * values at the new width.  Widths are never raised (that needs the unquantized values).
 * bitsK, bitsV: u8 [batch*heads][n_cols] or both NULL; score_ring: binary32
 * [batch*heads][window][n_cols]; nvalid: u8 [batch*heads][n_cols]; n_cols >= cached tokens.
 * Tiles are rewritten in place: the bytes read by qaq_decode_attention and the counters of
 * qaq_cache_stats shrink; pool space inside closed tiles is not handed back to later appends.
 * One exception: the values of a tile are stored in groups of four tokens per piece width, and a
 * tile whose lowered widths need more group padding than before can come out a few bytes larger;
 * it is then placed anew at the end of its pool like a raised tile (see qaq_requantize).  A caller
 * that lowers widths every step gives the cache some room beyond the tokens it will hold and calls
 * qaq_cache_compact now and then; without room the tile stays as it was and the device status
 * reports QAQ_ERR_CAPACITY.
 * Device pointers; asynchronous on stream.  Errors: QAQ_ERR_INVALID_ARG (missing arrays,
 * n_cols too small), QAQ_ERR_UNSUPPORTED_SHAPE, QAQ_ERR_CUDA; an empty cache is a no-op.
 */
qaq_status qaq_requantize_down(qaq_cache* c, const uint8_t* bitsK, const uint8_t* bitsV,
                               const qaq_policy* policy, const float* score_ring, const uint8_t* nvalid,
                               long n_cols, void* stream);

/*
 * Re-quantization in both directions (Section 4.2, "Integration in text generation process":
 * tokens whose new width is lower are quantized further, the others are recomputed at the
 * width they need from the unquantized copy that the caller keeps, in CPU memory in the paper).
 * K_full, V_full: the unquantized binary16 values of the cached tokens, [batch][heads][>=tokens]
 * [head_dim] with element strides as in qaq_outlier_thresholds, in any memory the GPU can read:
 * device memory, or pinned host memory that is mapped into the device's address space (then only
 * the rows of the raised tokens cross the bus).  Pageable host memory is refused.  Both NULL:
 * exactly qaq_requantize_down.  thr: the thresholds the tokens were appended with.
 * New widths as in qaq_requantize_down (given, clamped to 1..8, or by the rules), but taken as
 * they are: a raised token keeps its min, max and outliers and gets the codes an append at the
 * new width would have produced, so after the call the cache equals one filled at the new widths.
 * A closed tile that grows is moved to the end of its (b,h) pool and its old bytes stay unused
 * until qaq_cache_compact (or qaq_cache_reset); if the pool has no room left the tile is left as it was and
 * qaq_cache_stats().device_status reports QAQ_ERR_CAPACITY.
 */
qaq_status qaq_requantize(qaq_cache* c, const void* K_full, const void* V_full, long stride_b, long stride_h,
                          long stride_t, const float* thr, const uint8_t* bitsK, const uint8_t* bitsV,
                          const qaq_policy* policy, const float* score_ring, const uint8_t* nvalid, long n_cols,
                          void* stream);

/*
 * S4+S5: decode attention over the packed cache (Section 2.1, Figure 1):
 *   S = Softmax(softmax_scale * q Khat^T),  X = S Vhat,
 * Khat/Vhat = midpoint reconstruction min + (code + 1/2) * step with the stored outliers
 * put back.  q: binary16 [batch*heads][head_dim]; out: binary32 [batch*heads][head_dim];
 * scores_out: NULL or binary32 [batch*heads][tokens] receiving S (one row of the attention
 * window).  ws: qaq_decode_workspace_bytes bytes, 16-byte aligned (split partials).
 */
qaq_status qaq_decode_workspace_bytes(const qaq_cache* c, size_t* host_out);
qaq_status qaq_decode_attention(const qaq_cache* c, const void* q, float softmax_scale, float* out,
                                float* scores_out, void* ws, size_t ws_bytes, void* stream);

/*
 * The same two steps with HOST buffers (pinned memory recommended): inputs are copied to
 * device staging owned by the cache, the kernels run, and results are copied back, all on
 * `stream`; the call returns after the stream has been synchronised.  K_new/V_new are
 * contiguous [batch*heads][n_new][head_dim]; other arguments as above but in host memory.
 */
qaq_status qaq_quantize_append_host(qaq_cache* c, const void* K_new, const void* V_new, int n_new,
                                    const qaq_policy* policy, const float* score_ring,
                                    const uint8_t* nvalid, const float* thr, void* stream);
qaq_status qaq_decode_attention_host(qaq_cache* c, const void* q, float softmax_scale, float* out,
                                     void* stream);

/*
 * Decode attention for several queries per (b,h) in one call (Section 4.2, "Integration in text generation
 * process"; the packed cache is what every query reads).  Per query the result is what qaq_decode_attention
 * returns for it, within the same tolerance; up to four queries share one pass over the packed cache (a tile is
 * staged and taken apart once, the queries are columns of the tensor-core operand), so n_q = 5..8 takes two passes;
 * a pass left with one or two queries runs the single-query kernel on each of them (it is cheaper there).
 * q: binary16 [batch*heads][n_q][head_dim]; out: binary32 [batch*heads][n_q][head_dim]; 1 <= n_q <= 8;
 * ws: qaq_decode_multi_workspace_bytes bytes, 16-byte aligned.  Device pointers, asynchronous on stream.
 * Errors: QAQ_ERR_INVALID_ARG (null pointer, empty cache, n_q outside 1..8), QAQ_ERR_WORKSPACE.
 */
qaq_status qaq_decode_multi_workspace_bytes(const qaq_cache* c, size_t* host_out);
qaq_status qaq_decode_attention_multi(const qaq_cache* c, const void* q, int n_q, float softmax_scale, float* out,
                                      void* ws, size_t ws_bytes, void* stream);

/*
 * The generation step with the token count kept in device memory (Section 4.2, "Integration in text generation
 * process": every step appends the new token's K and V rows to the quantized cache and attends over the whole of it).
 * The calls above take the token count from the host-side handle, so each step needs the host to issue launches that
 * depend on it.  Between qaq_stream_begin and qaq_stream_end the count lives in the cache's device memory instead:
 * qaq_stream_append reads it, stores one token per (b,h) behind it and advances it; qaq_stream_decode attends over as
 * many tokens as it says.  Neither touches host state, and their launch shapes do not depend on the count, so one
 * append + decode pair can be captured in a CUDA graph once and replayed for every step (the buffers behind the
 * pointers must then stay where they are; their contents are read at replay time).  While the count is on the device
 * the host-side count is stale: call no other function on the cache until qaq_stream_end has brought it back.
 *
 * qaq_stream_begin: writes the host count to the device (asynchronous on stream).
 * qaq_stream_append: k_new / v_new binary16, one row of head_dim per (b,h), element strides between batches and heads
 *   given; the other arguments as for qaq_quantize_append with n_new = 1 (score_col: [batch*heads][window][1],
 *   nvalid: [batch*heads][1]; or given widths bitK / bitV [batch*heads][1]).  A cache that is full keeps its count
 *   and sets the device status to QAQ_ERR_CAPACITY (read by qaq_cache_stats).
 * qaq_stream_decode: as qaq_decode_attention; rows of scores_out lie scores_stride >= max_tokens elements apart.
 *   A count of zero yields zeros.
 * qaq_stream_end: copies the count back and waits for the stream (the one call of the four that synchronises).
 * Errors: QAQ_ERR_INVALID_ARG, QAQ_ERR_WORKSPACE, QAQ_ERR_UNSUPPORTED_SHAPE, QAQ_ERR_CUDA as above.
 */
qaq_status qaq_stream_begin(qaq_cache* c, void* stream);
qaq_status qaq_stream_append(qaq_cache* c, const void* k_new, const void* v_new, long stride_b, long stride_h,
                             const uint8_t* bitK, const uint8_t* bitV, const qaq_policy* policy,
                             const float* score_col, const uint8_t* nvalid, const float* thr, void* stream);
qaq_status qaq_stream_decode(const qaq_cache* c, const void* q, float softmax_scale, float* out, float* scores_out,
                             long scores_stride, void* ws, size_t ws_bytes, void* stream);
qaq_status qaq_stream_end(qaq_cache* c, void* stream);

/*
 * Decode attention without a caller-supplied workspace and without any allocation.
 * (No counterpart in the paper: this exists for the sake of the callers, not the method.)
 *
 * Some users of this library sit where asking for device memory is not an option: a
 * serving loop whose whole memory budget was handed out at start-up, or a step that must
 * not trigger the device-wide synchronisation a cudaMalloc/cudaFree can cause.  For them
 * this variant of qaq_decode_attention keeps the split partials in a fixed 4 MiB device
 * array that is part of the library itself (every GPU that loads libqaq holds these 4 MiB
 * until the process exits).  The call performs no cudaMalloc/cudaFree and uses no
 * allocating library routine; q and out are still the caller's buffers, as above.
 *
 *   - Limit: 2 * CTAs * (head_dim+3) * 4 bytes + batch*heads*8 must fit in 4 MiB, where
 *     CTAs is the launch width qaq_decode_attention would use: at most max(592,
 *     batch*heads), and batch*heads when every (b,h) holds fewer than 4 tiles of 64 tokens
 *     (e.g. 256 (b,h) x 4096 tokens x head_dim 128 needs 0.6 MiB; at head_dim 128 up to
 *     3971 (b,h) fit whatever their length).  Larger shapes get QAQ_ERR_WORKSPACE and nothing is
 *     launched -- use qaq_decode_attention with your own workspace.
 *   - The first call on each device looks up the array's device address (once, with that
 *     device current); the CUDA runtime may also load the library's kernels at that moment,
 *     which can take device memory of its own.  Make that first call as a warm-up, outside
 *     any stream capture; later calls take nothing.
 *   - All calls on a device share the one array.  Calls that may overlap on the GPU
 *     (different streams, no ordering between them) race on it and give wrong results;
 *     keep them on one stream or order them yourself.  The array keeps the previous
 *     call's contents; nothing in it needs clearing, every value is written before use.
 *   - No scores_out here; results equal qaq_decode_attention's.
 */
qaq_status qaq_decode_attention_static(const qaq_cache* c, const void* q, float softmax_scale, float* out,
                                       void* stream);

/* Counters and compression ratios (memory accounting of Sections 2.1 and 5.2).
 * Synchronises `stream`.  host_out is host memory. */
qaq_status qaq_cache_stats(const qaq_cache* c, qaq_stats* host_out, void* stream);

/*
 * Canonical copy of one tensor (0 = K, 1 = V) of the cache, for inspection and checks;
 * all outputs are device arrays, any may be NULL:
 *   bits u8 [BH][T]; mn, step binary32 [BH][T]; off u32 [BH][T+1] (byte offsets, prefix
 *   sums of head_dim*bits/8); codes u8 [BH][codes_stride] (tokens concatenated in token
 *   order); rowptr u32 [BH][T+1]; ch u8 / val binary16 [BH][outl_stride] (outliers in
 *   (token, channel) order).  T = qaq_cache_tokens().  Within one token the codes are
 *   stored as "planes": a B-bit code is cut into the power-of-two pieces of B (widest
 *   first, holding the most significant bits); the plane of a w-bit piece has
 *   head_dim*w/8 bytes; channel d = 32p+4r+i sits in little-endian 32-bit word
 *   p*w + r*w/8 of the plane at bit 8*i + w*(r mod 8/w).
 */
qaq_status qaq_cache_export(const qaq_cache* c, int tensor, uint8_t* bits, float* mn, float* step,
                            uint32_t* off, uint8_t* codes, long codes_stride, uint32_t* rowptr,
                            uint8_t* ch, void* val, long outl_stride, void* stream);

/*
 * Housekeeping for caches whose widths are raised (no counterpart in the paper, which keeps its
 * cache in framework tensors).  qaq_requantize places a tile that grows at the end of its (b,h)
 * pool and leaves the old bytes unused; qaq_cache_compact moves the tiles of every pool down
 * until they are contiguous again (order in memory kept, open tile last), so that the space can
 * be appended to.  Contents, widths and outlier lists are unchanged; only tile offsets move.
 * At most 4096 tiles (262144 tokens) per (b,h), else QAQ_ERR_UNSUPPORTED_SHAPE.  Asynchronous
 * on stream.  qaq_cache_pool_use reports the largest pool fill over all (b,h), in bytes, for
 * K (host_used[0]) and V (host_used[1]), and the pool capacity per (b,h); it synchronises stream.
 */
qaq_status qaq_cache_compact(qaq_cache* c, void* stream);
qaq_status qaq_cache_pool_use(const qaq_cache* c, long* host_used, long* host_capacity, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* QAQ_H */
