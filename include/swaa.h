/*
 * swaa.h -- C ABI of the SWAA attention library for NVIDIA B200 (sm_100a).
 *
 * The library computes causal softmax attention under the per-layer mask policy
 * of SWAA ("Sliding Window Attention Adaptation"):
 *
 *     visible(i, j) = j <= i  and  ( is_full  or  j > i - window  or  j < n_sink )
 *
 * with i, j the positions of query and key inside their own sequence.
 *   - window: sliding window attention, each token sees a fixed-size local
 *     window (Sec. 1, App. A); the window counts `window` keys including the
 *     query's own position.
 *   - n_sink: "Keep First k Tokens", every token additionally sees the first k
 *     tokens of its sequence (Sec. 3.2.1, Fig. 1b).
 *   - is_full: full causal attention, used by FA layers of an interleaved stack
 *     (Sec. 3.1.2) and by the decode phase under "FA Decode" (Sec. 3.1.1, Fig. 1a).
 * Grouped-query attention: query head h reads key/value head h / (Hq / Hkv).
 * Arithmetic: bf16 inputs, fp32 accumulation, bf16 outputs.
 *
 * Conventions for every call
 *   - Pointers named "device" are CUDA device pointers on the current device;
 *     the caller owns every buffer.  Tensors are dense and contiguous in the
 *     stated layout, bf16 unless stated, and 16-byte aligned.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Work
 *     is enqueued asynchronously; no call synchronises except
 *     swaa_last_device_status.
 *   - The return value is a swaa_status.  Argument errors are detected on the
 *     host before anything is launched.  Errors only the device can see (bad
 *     cu_seqlens / seqlens contents, a bounded wait that ran out) are recorded in
 *     a per-device status word that swaa_last_device_status reads; a kernel that
 *     records one skips the stores of the affected rows and returns normally.
 *   - The library allocates no device memory.  There is no CPU fallback.
 */
#ifndef SWAA_H_
#define SWAA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SWAA_OK = 0,
    SWAA_ERR_INVALID_ARG = -1, /* null / misaligned pointer, negative size, window < 1 on an SWA call, ... */
    SWAA_ERR_UNSUPPORTED = -2, /* D not in {64, 128}, Hq % Hkv != 0, device is not sm_100 */
    SWAA_ERR_CUDA = -3,        /* a CUDA runtime / driver call failed */
    SWAA_ERR_WORKSPACE = -4,   /* workspace too small or misaligned */
    SWAA_ERR_BAD_SEQLENS = -5, /* device saw inconsistent cu_seqlens / seqlens */
    SWAA_ERR_TIMEOUT = -6      /* a bounded device-side wait ran out */
} swaa_status;

/*
 * Prefill: packed variable-length causal self attention (Sec. 1, 3.1.2, 3.2.1; App. A: cost O(N*W)).
 *
 *   q, out      device, [T, Hq, D]  bf16 (token-major: token, head, channel)
 *   k, v        device, [T, Hkv, D] bf16
 *   cu_seqlens  device, int32 [B+1]; cu[0] = 0, cu[B] = T, non-decreasing.  Sequence b owns packed
 *               tokens cu[b] .. cu[b+1]-1; positions (and the n_sink first tokens) are per sequence.
 *   B, T        number of sequences, total packed tokens.  T == 0 or B == 0 is a no-op (SWAA_OK).
 *   max_seqlen  upper bound on any sequence length (sizes the launch); a longer sequence is reported
 *               as SWAA_ERR_BAD_SEQLENS through the status word and its rows are not written.
 *   Hq, Hkv, D  head counts and head size; Hq % Hkv == 0; D in {64, 128}.
 *   window      >= 1 unless is_full; n_sink >= 0; is_full != 0 selects full causal attention
 *               (window and n_sink are then ignored).
 *   scale       softmax scale; <= 0 selects 1/sqrt(D).
 *   lse         device, float32 [Hq, T], natural-log sum of exp(scale * q.k) over the visible keys of
 *               each row; may be NULL.
 * Only the key tiles that hold a visible key are visited: the sink tiles and the diagonal band.
 */
int swaa_prefill(const void* q, const void* k, const void* v, void* out, const int32_t* cu_seqlens, int B, int T,
                 int max_seqlen, int Hq, int Hkv, int D, int window, int n_sink, int is_full, float scale,
                 float* lse, void* stream);

/*
 * Chunked prefill: the queries of sequence b are the LAST len_q tokens of a context of len_k >= len_q
 * tokens whose keys and values are all supplied (Sec. 3.1.1 / Fig. 1a: tokens that come later attend to the
 * stored context under the layer's mask; a serving engine feeds a long prompt in chunks).  Query i of the
 * chunk sits at position len_k - len_q + i of its sequence; window and n_sink are measured in sequence
 * positions, not inside the chunk.  With len_q == len_k for every sequence this is swaa_prefill.
 *
 *   q, out        device, [Tq, Hq, D] bf16, packed by cu_seqlens_q (int32 [B+1], cu[0] = 0, cu[B] = Tq)
 *   k, v          device, [Tk, Hkv, D] bf16, packed by cu_seqlens_k (int32 [B+1], cu[0] = 0, cu[B] = Tk)
 *   max_seqlen_q  upper bound on any len_q (sizes the launch); max_seqlen_k upper bound on any len_k.
 *   lse           device, float32 [Hq, Tq]; may be NULL.
 * A sequence with len_q > len_k, or longer than the stated bounds, is reported as SWAA_ERR_BAD_SEQLENS
 * through the status word and its rows are not written.  Other arguments as for swaa_prefill.
 */
int swaa_prefill_chunked(const void* q, const void* k, const void* v, void* out, const int32_t* cu_seqlens_q,
                         const int32_t* cu_seqlens_k, int B, int Tq, int Tk, int max_seqlen_q, int max_seqlen_k,
                         int Hq, int Hkv, int D, int window, int n_sink, int is_full, float scale, float* lse,
                         void* stream);

/*
 * Backward pass of swaa_prefill under the same mask policy (Sec. 3.2.2: fine-tuning under SWA uses the mask
 * the model will be served with).  Given the forward inputs, the forward output `out`, its log-sum-exp
 * rows `lse` (as written by swaa_prefill) and the gradient `dout` of the loss with respect to `out`, writes
 * the gradients with respect to q, k and v (dk, dv summed over the query heads of each GQA group).
 * Work is O(L * window) per head like the forward pass: a key tile only meets the query tiles that see it.
 *
 *   q, out, dout, dq  device, [T, Hq, D] bf16;  k, v, dk, dv  device, [T, Hkv, D] bf16
 *   lse               device, float32 [Hq, T]
 *   workspace         device, at least swaa_prefill_backward_workspace_size(B, T, Hq, Hkv, D, n_sink) bytes,
 *                     256-byte aligned; contents need not be initialised (fp32 accumulators for dq and for the
 *                     dk, dv rows of the sink key tiles, and the row terms dout.out and lse * log2(e))
 * Other arguments and status codes as for swaa_prefill: a sequence longer than max_seqlen (or running past T) is
 * reported as SWAA_ERR_BAD_SEQLENS through the status word; its dk and dv rows are not written and its dq rows are
 * zero.  fp32 accumulation throughout; P and dS are rounded to bf16 for the tensor-core products, as in the
 * forward pass.
 */
size_t swaa_prefill_backward_workspace_size(int B, int T, int Hq, int Hkv, int D, int n_sink);

int swaa_prefill_backward(const void* q, const void* k, const void* v, const void* out, const void* dout,
                          const float* lse, const int32_t* cu_seqlens, int B, int T, int max_seqlen, int Hq, int Hkv,
                          int D, int window, int n_sink, int is_full, float scale, void* dq, void* dk, void* dv,
                          void* workspace, size_t workspace_bytes, void* stream);

/*
 * Chunked prefill against a paged KV cache (the two needs of a serving engine that mixes prefill chunks and
 * decode steps, Sec. 4.1.1): queries as in swaa_prefill_chunked, keys and values as in swaa_decode_paged.
 *
 *   q, out          device, [Tq, Hq, D] bf16, packed by cu_seqlens_q (int32 [B+1])
 *   kpages, vpages  device, [num_pages, page_size, Hkv, D] bf16; page_size is a multiple of 128.
 *   seqlens_k       device, int32 [B]; keys of sequence b INCLUDING the chunk's own tokens, len_q <= len_k <=
 *                   max_blocks * page_size.
 *   block_table     device, int32 [B, max_blocks]; entry j of sequence b lives in page
 *                   block_table[b][j / page_size] at row j % page_size.
 * The rows of a page past a sequence's last key are never used, whatever they hold.  A page index outside
 * [0, num_pages) or len_q > len_k is reported as SWAA_ERR_BAD_SEQLENS through the status word.
 */
int swaa_prefill_paged(const void* q, const void* kpages, const void* vpages, void* out, const int32_t* cu_seqlens_q,
                       const int32_t* seqlens_k, const int32_t* block_table, int B, int Tq, int max_seqlen_q,
                       int max_blocks, int num_pages, int page_size, int Hq, int Hkv, int D, int window, int n_sink,
                       int is_full, float scale, float* lse, void* stream);

/*
 * Mixed batch: swaa_prefill_chunked / swaa_prefill_paged with a mask policy PER SEQUENCE, so that one launch serves
 * sequences in different phases (Fig. 1a: prompt tokens under the SWA mask next to generated tokens under full
 * attention; App. "Inference Efficiency": a serving engine batches prefill chunks and decode tokens together).
 *   is_full_seq   device, uint8 [B]; sequence b runs full causal attention iff is_full_seq[b] != 0, else the
 *                 window + n_sink mask.  window >= 1 is required.
 * Everything else as for swaa_prefill_chunked / swaa_prefill_paged.
 */
int swaa_prefill_chunked_mixed(const void* q, const void* k, const void* v, void* out, const int32_t* cu_seqlens_q,
                               const int32_t* cu_seqlens_k, const uint8_t* is_full_seq, int B, int Tq, int Tk,
                               int max_seqlen_q, int max_seqlen_k, int Hq, int Hkv, int D, int window, int n_sink,
                               float scale, float* lse, void* stream);
int swaa_prefill_paged_mixed(const void* q, const void* kpages, const void* vpages, void* out,
                             const int32_t* cu_seqlens_q, const int32_t* seqlens_k, const int32_t* block_table,
                             const uint8_t* is_full_seq, int B, int Tq, int max_seqlen_q, int max_blocks, int num_pages,
                             int page_size, int Hq, int Hkv, int D, int window, int n_sink, float scale, float* lse,
                             void* stream);

/*
 * Context-parallel SWA prefill: the compute step of one participant that owns a contiguous stretch of every
 * sequence (App. A: SWA prefill costs O(N * W) because a token only looks at the window before it; Sec. 3.2.1: and
 * at the first k tokens).  Before the call the participant has, in its own memory,
 *   k_local, v_local  device, [Tk, Hkv, D] bf16 packed by cu_seqlens_k: for sequence b the keys at positions
 *                     key_pos0[b] .. key_pos0[b] + len_k - 1, i.e. a halo of earlier keys followed by its stretch;
 *   q, out            device, [Tq, Hq, D] bf16 packed by cu_seqlens_q: the LAST len_q of those positions (its stretch);
 *   sink_k, sink_v    device, [B, sink_rows, Hkv, D] bf16: the keys at positions 0 .. sink_rows-1 of every sequence
 *                     (finite values in every row); may be NULL with sink_rows == 0 when n_sink == 0 or every
 *                     key_pos0 is 0;
 *   key_pos0          device, int32 [B].
 * How halo and sink rows get there (a neighbour copy and a broadcast) is the caller's business; the kernel reads
 * local memory only.  A query at position i sees positions j <= i with j > i - window or j < n_sink: positions
 * >= key_pos0[b] are taken from the local keys, sink positions below it from the sink rows.  The halo must hold
 * the window of the stretch's first query: key_pos0[b] == 0 or len_k - len_q >= window - 1, and n_sink <= sink_rows
 * when key_pos0[b] > 0; a sequence that violates this is reported as SWAA_ERR_BAD_SEQLENS through the status word
 * and its rows are not written.  With every key_pos0 == 0 this is swaa_prefill_chunked with the SWA mask.
 * Layers with full attention need all earlier keys, i.e. an all-gather of K and V and then swaa_prefill_chunked.
 * Other arguments as for swaa_prefill_chunked.
 */
int swaa_prefill_context_parallel(const void* q, const void* k_local, const void* v_local, const void* sink_k,
                                  const void* sink_v, void* out, const int32_t* cu_seqlens_q,
                                  const int32_t* cu_seqlens_k, const int32_t* key_pos0, int B, int Tq, int Tk,
                                  int max_seqlen_q, int max_seqlen_k, int sink_rows, int Hq, int Hkv, int D, int window,
                                  int n_sink, float scale, float* lse, void* stream);

/*
 * Lazy ratio of a layer (App. "Results of LightTransfer": layer selection by how much of the attention of the
 * tokens at the end of a sequence goes to recent tokens rather than to the rest of the context; the paper
 * uses the last 64 tokens and a recent window of 1024).  For the queries given (the last len_q tokens of each
 * len_k-token context, packed like swaa_prefill_chunked) and each query head h:
 *     ratio[h] = mean over the queries of  sum_{j recent or sink} p(i, j),
 * p = softmax of scale * q.k over ALL keys j <= i (full causal attention), "recent" = the last `recent` keys
 * ending at the query, "sink" = the first n_sink keys of the sequence.  A value near 1 marks a layer that an SWA
 * mask would hardly change.  The mass is obtained from two log-sum-exp passes (windowed and full) of a prefill
 * kernel instance that forms only the row sums (no values fetched, no P V product, no output) and a small
 * reduction kernel.
 *
 *   ratio        device, float32 [Hq]
 *   scratch_lse  device, float32 [2, Hq, Tq], overwritten.
 *   v, scratch_out  not used (the probe needs no values and writes no attention output); may be NULL.
 * Other arguments, status codes and errors as for swaa_prefill_chunked (recent >= 1, n_sink >= 0).
 */
int swaa_lazy_ratio(const void* q, const void* k, const void* v, const int32_t* cu_seqlens_q,
                    const int32_t* cu_seqlens_k, int B, int Tq, int Tk, int max_seqlen_q, int max_seqlen_k, int Hq,
                    int Hkv, int D, int recent, int n_sink, float scale, float* ratio, void* scratch_out,
                    float* scratch_lse, void* stream);

/*
 * Decode: one query token per sequence against a dense KV cache (Sec. 3.1.1 "FA Decode": with is_full
 * the generated token sees the whole context; App. A: the full-context cache is retained).
 *
 *   q, out          device, [B, Hq, D] bf16
 *   kcache, vcache  device, [B, Lmax, Hkv, D] bf16
 *   seqlens         device, int32 [B]; number of valid cache entries of each sequence INCLUDING the
 *                   current token, 1 <= seqlens[b] <= Lmax; the query sits at position seqlens[b]-1.
 *                   With is_full == 0 it reads the last `window` entries plus the first n_sink.
 *                   A value outside [1, Lmax] is reported as SWAA_ERR_BAD_SEQLENS through the status
 *                   word; that sequence's output rows are zero-filled.
 *   workspace       device scratch of at least swaa_decode_workspace_size(...) bytes for the same
 *                   shape arguments, 256-byte aligned; contents need not be initialised and are
 *                   overwritten.  Two calls that overlap on the GPU must not share a workspace.
 * The visible cache entries of all sequences and heads form one list of 64-entry tiles that is cut
 * evenly over a persistent grid (split-K across blocks wherever a cut falls inside a sequence);
 * partial results are merged by a log-sum-exp combine inside the same launch.  Cache entries past
 * seqlens[b] are never used, whatever they hold.
 */
size_t swaa_decode_workspace_size(int B, int Hq, int Hkv, int D, int Lmax, int window, int n_sink, int is_full);

int swaa_decode(const void* q, const void* kcache, const void* vcache, void* out, const int32_t* seqlens, int B,
                int Lmax, int Hq, int Hkv, int D, int window, int n_sink, int is_full, float scale, void* workspace,
                size_t workspace_bytes, void* stream);

/*
 * Decode against a paged KV cache (the layout of serving engines such as the vLLM integration of Sec. 4.1.1:
 * the cache of a sequence is a list of fixed-size pages anywhere in a common pool).
 *
 *   kpages, vpages  device, [num_pages, page_size, Hkv, D] bf16; page_size is a multiple of 64.
 *   block_table     device, int32 [B, max_blocks]; entry j of sequence b lives in page
 *                   block_table[b][j / page_size] at row j % page_size.  Only the entries that cover
 *                   seqlens[b] are read.  A page index outside [0, num_pages) is reported as
 *                   SWAA_ERR_BAD_SEQLENS through the status word (the page then reads as zeros).
 *   seqlens         device, int32 [B]; 1 <= seqlens[b] <= max_blocks * page_size, as for swaa_decode.
 *   workspace       at least swaa_decode_paged_workspace_size(...) bytes, 256-byte aligned, uninitialised.
 * Same computation, mask policy, status codes and in-launch combine as swaa_decode.
 */
size_t swaa_decode_paged_workspace_size(int B, int Hq, int Hkv, int D, int max_blocks, int page_size, int window,
                                        int n_sink, int is_full);

int swaa_decode_paged(const void* q, const void* kpages, const void* vpages, void* out, const int32_t* block_table,
                      const int32_t* seqlens, int B, int max_blocks, int num_pages, int page_size, int Hq, int Hkv,
                      int D, int window, int n_sink, int is_full, float scale, void* workspace, size_t workspace_bytes,
                      void* stream);

/*
 * Decode with the KV cache cut along the context (App. A: under FA decode the cache of the whole context must be
 * retained, which is what makes spreading it over several devices attractive; Sec. 3.1.1).  A participant holds, for
 * every sequence, the entries at positions key_pos0 .. key_pos0 + Lshard - 1 and computes the partial result of
 * every (sequence, head) row over the visible keys it holds; the partials of all participants (B * Hq * (D + 2)
 * floats each: gather them with any collective or copy) are merged by swaa_decode_combine.  The mask is evaluated
 * on positions of the whole sequence, so the result equals swaa_decode on the uncut cache.
 *
 *   kshard, vshard  device, [B, Lshard, Hkv, D] bf16; entry at position p of sequence b in row p - key_pos0.
 *                   Rows that lie past a sequence's length are never used, whatever they hold.
 *   seqlens         device, int32 [B]: TOTAL number of valid entries of each sequence (>= 1) including the current
 *                   token; the query sits at position seqlens[b] - 1.  A value < 1 is reported as
 *                   SWAA_ERR_BAD_SEQLENS through the status word.
 *   partial_out     device, float32 [B, Hq, D + 2]: (m, l, o[0..D)) with m = largest visible scaled score held by
 *                   this participant (natural-log units), l = sum of exp(score - m), o = sum of exp(score - m) * v.
 *                   A participant that holds no visible key of a row writes (-inf, 0, 0...).
 *   workspace       at least swaa_decode_partial_workspace_size(...) bytes, 256-byte aligned, uninitialised.
 * Other arguments and status codes as for swaa_decode (same kernel; the split-K merge across thread blocks happens
 * inside the launch as usual and produces the participant's partial).
 *
 * swaa_decode_combine: partials device, float32 [P, B, Hq, D + 2] (participant-major); out device, [B, Hq, D] bf16 =
 * sum_s e^(m_s - M) o_s / sum_s e^(m_s - M) l_s with M = max_s m_s over the non-empty partials (zeros when all are
 * empty).
 */
size_t swaa_decode_partial_workspace_size(int B, int Hq, int Hkv, int D, int Lshard, int window, int n_sink,
                                          int is_full);
int swaa_decode_partial(const void* q, const void* kshard, const void* vshard, float* partial_out,
                        const int32_t* seqlens, int B, int Lshard, int key_pos0, int Hq, int Hkv, int D, int window,
                        int n_sink, int is_full, float scale, void* workspace, size_t workspace_bytes, void* stream);
int swaa_decode_combine(const float* partials, int P, int B, int Hq, int D, void* out, void* stream);

/*
 * Allocation-free decode.  (The paper has no counterpart to this call; it exists for integration.)
 *
 * Same computation and arguments as swaa_decode, but the split-K scratch lives in a fixed array inside
 * the library's device image, so the caller passes no workspace and nothing is allocated, by this
 * call or on its behalf.  It is meant for callers that cannot call cudaMalloc at the point where
 * attention runs: code on a latency-critical serving path, where an allocation would stall the whole
 * device; a plug-in that receives tensors from a host framework but has no handle on that framework's
 * memory pool, and must not take memory behind its back; a process whose device memory is already
 * handed out in full to other owners.
 *
 *   - The scratch array is SWAA_DECODE_STATIC_SCRATCH_BYTES (2 MiB) per GPU, held by every GPU that
 *     loads the library until the process exits.  A shape whose scratch need
 *     (swaa_decode_workspace_size) exceeds it is rejected with SWAA_ERR_WORKSPACE and nothing runs;
 *     use swaa_decode with a caller-owned workspace for those (on a 148-SM device: head size 128
 *     with more than 8 query heads per key/value head, once the batch is large enough to occupy every SM).
 *   - The first call on each device looks up the array's device address (once per device, with that
 *     device current) before it launches.  Make that first call outside any stream capture.
 *   - All calls on one device share the one array, and it keeps whatever the previous call left
 *     there; no part of it has to start at zero (tickets carry a per-call stamp).  Two calls whose kernels can overlap
 *     on the same GPU (different streams, no dependency between them) race on it: serialise them.
 * Returns the same status codes as swaa_decode.
 */
#define SWAA_DECODE_STATIC_SCRATCH_BYTES (2u << 20)
int swaa_decode_static(const void* q, const void* kcache, const void* vcache, void* out, const int32_t* seqlens,
                       int B, int Lmax, int Hq, int Hkv, int D, int window, int n_sink, int is_full, float scale,
                       void* stream);

/*
 * Layer schedule (host only).  Sec. 3.1.2: a fixed-interval subset of layers keeps full attention
 * (Table 1 "FA layers": [1,3,5,...], [0,2,4,...], [1,5,9,...], [1,9,17,...], [3,7,11,...]); Sec. 3.1.1:
 * with FA decode every layer is full while decoding.  Layers are 0-based.
 *   is_full(layer, phase) = (layer in FA set) or (phase == decode and fa_decode)
 * The FA set is {fa_start, fa_start+fa_step, ...}, or, when fa_mask is not NULL, the layers l with fa_mask[l] != 0
 * (a set chosen layer by layer, e.g. by lazy ratio as in App. "Results of LightTransfer"; fa_start and fa_step are
 * then ignored).
 */
typedef struct {
    int n_layers;
    int window;    /* SWA window of the non-FA layers */
    int n_sink;    /* keep-first k */
    int fa_start;  /* first FA layer */
    int fa_step;   /* distance between FA layers; 0 = no FA layers */
    int fa_decode; /* non-zero: full attention in the decode phase on every layer */
    const uint8_t* fa_mask; /* NULL, or host array [n_layers]: explicit FA set (owned by the caller) */
} swaa_policy;

#define SWAA_PHASE_PREFILL 0
#define SWAA_PHASE_DECODE 1

/* Returns 1 / 0, or SWAA_ERR_INVALID_ARG (null policy, layer outside [0, n_layers), bad phase, negative fields). */
int swaa_schedule_is_full(const swaa_policy* policy, int layer, int phase);
/* Fills is_full_out[0 .. n_layers) (host memory) with 0/1.  Returns SWAA_OK or SWAA_ERR_INVALID_ARG. */
int swaa_schedule_fill(const swaa_policy* policy, int phase, uint8_t* is_full_out);
/*
 * FA set from lazy ratios (host only; App. "Results of LightTransfer": layers with a higher lazy ratio are the
 * candidates for SWA, the others keep full attention; the paper also evaluates the opposite assignment).
 *   ratio       host, float32 [n_layers, n_heads]: per layer the output of swaa_lazy_ratio; a layer's ratio is the
 *               mean over its heads.
 *   n_lazy      how many layers count as lazy: those with the highest ratio (equal ratios: lower index first);
 *               the paper takes half of the layers.
 *   fa_on_lazy  0: the non-lazy layers get full attention (the method as proposed); != 0: the lazy ones do.
 *   fa_mask_out host, uint8 [n_layers]: 1 for FA layers; usable as swaa_policy.fa_mask.
 * Returns SWAA_OK or SWAA_ERR_INVALID_ARG (null pointer, n_layers < 0, n_heads < 1, n_lazy outside [0, n_layers],
 * a ratio that is not finite).
 */
int swaa_schedule_select_fa_layers(const float* ratio, int n_layers, int n_heads, int n_lazy, int fa_on_lazy,
                                   uint8_t* fa_mask_out);

/*
 * Key-tile enumeration of the prefill kernel, exposed for host-side verification (App. A: only
 * O(N*W) work).  For the query tile of rows [m*BM, min(L, (m+1)*BM)) of a sequence of length L, the
 * kernel visits key tiles (of BN keys) 0 .. *n_sink_tiles-1 and *n_lo .. *n_hi.  Returns SWAA_OK or
 * SWAA_ERR_INVALID_ARG.  swaa_prefill_tile_needs_mask returns 1 when some (row, key) pair of the
 * tile is not visible (the kernel then applies the element predicate), 0 when every pair is visible.
 */
int swaa_prefill_tile_range(int L, int m, int BM, int BN, int window, int n_sink, int is_full, int* n_sink_tiles,
                            int* n_lo, int* n_hi);
int swaa_prefill_tile_needs_mask(int L, int m, int n, int BM, int BN, int window, int n_sink, int is_full);
/* Tile sizes the prefill kernel uses (rows per query tile, keys per key tile). */
int swaa_prefill_block_m(void);
int swaa_prefill_block_n(void);

/* Number of thread blocks swaa_decode cuts the visible cache entries over, for these arguments on the
 * current device (>= 1). */
int swaa_decode_num_blocks(int B, int Hq, int Hkv, int D, int Lmax, int window, int n_sink, int is_full);

/*
 * Trimmed KV cache of a pure-SWA layer (host only).  App. A: without FA decode an SWA layer never looks
 * at more than the first n_sink tokens and the last `window` tokens, so its cache can be cut to n_sink + window
 * entries: the sinks stay in slots 0 .. n_sink-1 and the later tokens go round a ring of `window` slots.
 *   swaa_trimmed_cache_slot(pos, ...)  slot in which the K/V of the token at position `pos` is stored
 *   swaa_trimmed_cache_len(len, ...)   occupied slots after `len` tokens = min(len, n_sink + window)
 * After `len` tokens the occupied slots hold exactly the keys an SWA decode step at that length may see, and
 * softmax attention does not depend on the order of the keys, so the decode step of such a layer is
 *   swaa_decode(q, k_trimmed, v_trimmed, out, seqlens = swaa_trimmed_cache_len(len), Lmax = n_sink + window, ...,
 *               is_full = 1)
 * and reads the same bytes as swaa_decode with the SWA mask on the untrimmed cache.
 * Both return -1 on window < 1, n_sink < 0 or a negative position / length.
 */
long long swaa_trimmed_cache_slot(long long pos, int window, int n_sink);
long long swaa_trimmed_cache_len(long long len, int window, int n_sink);

/* Static string for a swaa_status value. */
const char* swaa_status_str(int status);
/*
 * Waits for `stream` to drain, then returns and clears the current device's status word: SWAA_OK, or
 * the first device-detected error since the last call (SWAA_ERR_BAD_SEQLENS, SWAA_ERR_TIMEOUT), or
 * SWAA_ERR_CUDA if the stream itself reports an error.
 */
int swaa_last_device_status(void* stream);
/* Kernels launched by this library in this process so far (all devices, all streams). */
uint64_t swaa_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SWAA_H_ */
