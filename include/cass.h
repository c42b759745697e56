/*
 * cass.h -- C boundary of the B200-native Cassandra self-speculative decode step.
 *
 * One draft pass reads only the speculation data (pruned, mantissa-truncated weights and KV cache with
 * compressed exponents: unary-coded, or MX-shared for the weights; Sec. 4.1-4.2 of the paper), decodes it in
 * registers and runs low-batch (1 to 8 sequences) GEMV and grouped-query decode attention on it; a bf16
 * verification pass over the gamma+1 drafted rows of every sequence (tensor cores) and a greedy accept/rollback
 * per sequence close each step (Sec. 2.2).
 *
 * Conventions
 *   - Every entry point returns 0 (CASS_OK) or a negative CASS_ERR_* code; nothing throws.
 *   - Pointers are DEVICE pointers unless the name starts with h_ (host).  The caller owns every buffer.
 *   - No entry point allocates or frees device memory; size queries say how much the caller must provide.
 *   - `stream` is a cudaStream_t passed as void*; work is enqueued on it and the call returns without
 *     synchronising, except where a comment says that the call synchronises.
 *   - Kernels are built for sm_100a only.  On any other device the first launch fails and the call
 *     returns CASS_ERR_CUDA (there is no fallback path).
 *   - Device-side problems (capacity exceeded, bounded wait ran out) are recorded in the session's
 *     status word, readable with cass_session_status().
 *   - Two environment variables, read once per process, are debugging aids:
 *     CASS_NO_PDL=1 launches every kernel in plain stream order (no programmatic dependent launch), so that
 *     a trace shows per-kernel times without overlap; CASS_SIMT_VERIFY_ATTN=1 makes cass_verify keep its
 *     fp32-pipe attention kernel where the tensor-core one would run (results then differ by the bf16
 *     rounding of the attention probabilities that the tensor-core kernel applies).
 */
#ifndef CASS_H_
#define CASS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    CASS_OK = 0,
    CASS_ERR_INVALID_ARG = -1,
    CASS_ERR_CAPACITY = -2,
    CASS_ERR_UNSUPPORTED = -3,
    CASS_ERR_TIMEOUT = -4,
    CASS_ERR_CUDA = -5
};

enum { CASS_KV_BF16 = 1, CASS_KV_COMPRESSED = 2 };

/* Format parameters.  p = pruning ratio in per-mille, t = number of LOW mantissa bits removed from the
 * speculation data (Eq. 2's w_t / kv_t; 7 - t mantissa bits remain).  Paper default: 400 / 4 (Sec. 6.1, 7.2).
 * w_seg_cols / w_chunk_cols: columns per superblock and per decode chunk (0 = 2048 / 256). */
typedef struct cass_format {
    int mode;                /* weights: 1 = Cassandra-1 (unary exponent code, lossless for the kept bits),
                              * 2 = Cassandra-2 (Sec. 4.2: MX, blocks of 32 kept values share an exponent, MXINT
                              * elements; see cass_encode_weights). */
    int w_prune_permille, w_trunc_bits;
    int kv_prune_permille, kv_trunc_bits;
    int w_seg_cols, w_chunk_cols;
    int kv_mode;             /* compressed KV cache: 0 or 1 = Cassandra-1 records (unary exponent code), 2 = Cassandra-2
                              * records (Sec. 4.2: the kept values among 32 consecutive channels of a head share one
                              * exponent byte; elements as for the weights); see cass_kv_append */
} cass_format;

typedef struct cass_model_desc {
    int n_layers, hidden, n_q_heads, n_kv_heads, head_dim, ffn, vocab;
    int max_seq;             /* KV positions per sequence (>= 32); the committed length stays <= max_seq - 16 */
    int max_batch;           /* sequences decoded together: 1, 2, 4 or 8; every step-level call handles all of them */
    int gamma_max;           /* largest draft length (<= 15); max_batch * (gamma_max + 1) <= 64 */
    float rope_theta, rms_eps;
} cass_model_desc;

/* Device pointers to the bf16 target model.  Per layer: wqkv [(n_q+2 n_kv) d, hidden] (q rows, then k rows,
 * then v rows), wo [hidden, n_q d], wgu [2 ffn, hidden] (gate rows, then up rows), wd [hidden, ffn],
 * two RMSNorm gains [hidden].  All row-major, rows = output features. */
typedef struct cass_layer_weights {
    const void *wqkv, *wo, *wgu, *wd, *norm_attn, *norm_ffn;
} cass_layer_weights;

typedef struct cass_model_weights {
    const cass_layer_weights* h_layers;   /* HOST array [n_layers] of device pointers */
    const void *embed, *lm_head, *norm_final;
} cass_model_weights;

/* Device pointers to the encoded speculation data of the same matrices (cass_encode_weights output). */
typedef struct cass_layer_blobs { const void *wqkv, *wo, *wgu, *wd; } cass_layer_blobs;
typedef struct cass_model_blobs {
    const cass_layer_blobs* h_layers;     /* HOST array [n_layers] */
    const void* lm_head;
} cass_model_blobs;

/* ------------------------------------------------------------------------------------------------------
 * Offline weight encoder (Sec. 4.2 "Unstructured Value Pruning" with the Wanda score, "Mantissa
 * Truncation", "Exponent Compression" by unary coding; Sec. 5.1 encoder; Sec. 5.3 superblocks).
 * ---------------------------------------------------------------------------------------------------- */

/* Upper bound of the blob size this library accepts for a rows x cols matrix (allows a mean code length of
 * 8 bits per kept value), and the scratch the encoder needs.  Host-only arithmetic. */
int cass_encoded_weight_bytes(const cass_format* fmt, int rows, int cols, size_t* h_blob_bound,
                              size_t* h_workspace_bytes);

/* Encode W (bf16 [rows][cols], row-major) into `blob`.  act_norm: fp32 [cols] per-input-channel L2 norms of
 * calibration activations, or NULL for all ones.  Per row the floor(cols*p/1000) lowest scores
 * fp32(|W_ij|) * act_norm[j] are pruned (ties: lower column first); NaN scores are not supported.
 * blob must be 128-byte aligned.  workspace: scratch of the size the query returned.  d_status: device int32,
 * set to CASS_ERR_CAPACITY if blob_cap is too small (blob contents are then undefined), else left alone.
 * The total size is also stored in the blob header (see cass_weight_blob_info). */
int cass_encode_weights(const cass_format* fmt, const void* W_bf16, const float* act_norm, int rows, int cols,
                        void* blob, size_t blob_cap, void* workspace, size_t workspace_bytes,
                        int32_t* d_status, void* stream);

typedef struct cass_blob_info {
    int rows, cols, prune_permille, trunc_bits, seg_cols, chunk_cols, n_seg, n_rowblocks, kept_per_row;
    int max_superblock_bytes;
    int mode, reserved;      /* 1 = Cassandra-1 (unary exponent code), 2 = Cassandra-2 (shared MX exponents) */
    uint64_t total_bytes;
} cass_blob_info;

/* With fmt->mode = 2 the same call produces Cassandra-2 speculation data (Sec. 4.2, exponent compression by the MX
 * format; Sec. 5.1, MX decoder): pruning, bitmap and truncation as above, but instead of a unary codeword per value
 * every block of 32 consecutive kept values of a row (within one column segment) shares one exponent byte E = the
 * largest exponent of the block, and a field holds the sign and the high 7-t bits of the 7-bit magnitude
 * (0x80 | mantissa) >> (1 + E - e) (an MXINT8 element in sign-magnitude form, truncated toward zero; 0 when the value
 * lies 7 or more binades below the block maximum, when it is zero or denormal, or when E < 7).  The draft value is
 * (-1)^s (magnitude >> t << t) 2^(E-133).  Unlike mode 1 this loses exponent information (the paper's "minor
 * accuracy loss"); verification stays bf16, so the token stream stays lossless.  cass_draft_gemv,
 * cass_draft_gemv_batch, cass_decode_weights, cass_weight_blob_stats (code_bits = exponent bits) and the session
 * take blobs of either mode. */

/* Reads the blob header back to the host.  SYNCHRONISES `stream`. */
int cass_weight_blob_info(const void* blob, cass_blob_info* h_info, void* stream);

/* Bits of speculation data in a blob, by kind (Sec. 4.2: one bitmap bit per value, sign + kept mantissa bits and
 * one unary codeword per kept value), and what the physical layout adds around them (chunk tables, masks, padding,
 * header, codebook, directory).  d_scratch: device memory of at least 8 bytes, 8-byte aligned.  SYNCHRONISES `stream`. */
typedef struct cass_blob_stats {
    uint64_t bitmap_bits, field_bits, code_bits;    /* content: rows*cols, rows*kept*(8-t), sum of codeword lengths */
    uint64_t total_bits;                            /* whole blob */
} cass_blob_stats;
int cass_weight_blob_stats(const void* blob, const cass_blob_info* h_info, void* d_scratch, cass_blob_stats* h_stats,
                           void* stream);

/* Test hook: zero-padded reconstruction (Sec. 4.1, draft inference) of a whole blob into bf16 [rows][cols]. */
int cass_decode_weights(const void* blob, const cass_blob_info* h_info, void* W_bf16_out, void* stream);

/* Verification data of a Cassandra-1 blob (Sec. 4.1 target inference: the target model reads speculation and
 * verification data and concatenates them; Sec. 5.1 encoder: the verification group is stored without transformation):
 * the low t mantissa bits of every kept value and the pruned values as they are.  Layout: 8 header words {'CASV', 1,
 * rows, cols, kept per row, t, words per row, 0}; per row ceil(kept*t/32) words of t-bit groups (column order, MSB
 * first), then the pruned values (column order) as 16-bit little-endian halfwords, padded to a word.  The bitmap is the
 * blob's.  cass_decode_full rebuilds the bf16 matrix from the two parts, bit for bit (one pass, every value written
 * once).  By default the verification pass reads a bf16 copy; cass_session_verify_from_parts makes it read the two parts.
 * Mode 1 blobs only (CASS_ERR_UNSUPPORTED otherwise).  h_bytes: host; vdata: device, 4-byte aligned. */
int cass_verification_data_bytes(const cass_blob_info* h_info, size_t* h_bytes);
int cass_encode_verification_data(const void* blob, const cass_blob_info* h_info, const void* W_bf16, void* vdata,
                                  size_t vdata_bytes, void* stream);
int cass_decode_full(const void* blob, const cass_blob_info* h_info, const void* vdata, void* W_bf16_out, void* stream);

/* ------------------------------------------------------------------------------------------------------
 * Draft GEMV on speculation data (Sec. 4.1 draft inference; decoder dataflow of Sec. 5.1 / Algorithm 1).
 *   y[r] = sum_c decode(blob)[r][c] * x[c], fp32 accumulation, y rounded to bf16 (y_bf16) and/or kept fp32.
 * x: bf16 [cols].  partial: fp32 scratch [n_seg][n_rowblocks*32], which receives the per-segment sums.  Either
 * output pointer may be NULL; with both NULL only `partial` is produced.
 * h_info is what cass_weight_blob_info returned for this blob (that call synchronises, so the blob is complete: the
 * kernel starts reading the blob before earlier work on the stream has finished).  The blob buffer holds at least
 * h_info->total_bytes bytes; nothing beyond them is read, and a directory entry that points outside, like a header
 * that differs from h_info, is refused through d_status (CASS_ERR_INVALID_ARG) instead of being followed.
 * ---------------------------------------------------------------------------------------------------- */
int cass_draft_gemv(const void* blob, const cass_blob_info* h_info, const void* x_bf16, float* partial,
                    void* y_bf16, float* y_f32, int32_t* d_status, void* stream);

/* The same for n_vec = 1, 2, 4 or 8 vectors (the low-batch regime of Sec. 2.1: one pass over the speculation data,
 * every decoded weight used n_vec times).  x: bf16 [n_vec][cols]; partial: fp32 scratch [n_vec][n_seg][n_rowblocks*32];
 * outputs [n_vec][rows].  Vector b's result equals what cass_draft_gemv gives for x[b] alone, bit for bit. */
int cass_draft_gemv_batch(const void* blob, const cass_blob_info* h_info, const void* x_bf16, int n_vec, float* partial,
                          void* y_bf16, float* y_f32, int32_t* d_status, void* stream);

/* Draft GEMV without a scratch argument (the paper has no counterpart; this is a convenience of this library).
 * Some callers cannot obtain device memory at the point where they call: code running between the capture-safe
 * parts of an inference server, plug-ins that are handed only their input and output tensors, or hosts whose
 * memory pool is closed after start-up.  For them the split-K partial sums go to an array built into the library
 * image (CASS_STATIC_PARTIAL_FLOATS floats = 2 MiB, resident on every GPU that loads the library until the
 * process exits) instead of a caller-provided `partial`.  The call allocates and frees nothing.
 *   - Limit: n_seg * n_rowblocks * 32 <= CASS_STATIC_PARTIAL_FLOATS, else CASS_ERR_CAPACITY (nothing is launched).
 *     The largest matrix of the Llama-3-8B shape (lm_head 128256 x 4096: 2 x 128256 floats) fits.
 *   - At least one of y_bf16 / y_f32 must be given; results equal those of cass_draft_gemv.
 *   - The first call on a device looks up the array's device address (with that device current) and keeps it;
 *     make that first call outside any stream capture.
 *   - All calls on one GPU share the array, which keeps the previous call's sums: every value a call reads it has
 *     written itself first, so nothing needs clearing, but two calls that overlap on the GPU (different streams)
 *     race on it.  Serialise them on one stream or with events. */
#define CASS_STATIC_PARTIAL_FLOATS (512 * 1024)
int cass_draft_gemv_static(const void* blob, const cass_blob_info* h_info, const void* x_bf16, void* y_bf16,
                           float* y_f32, int32_t* d_status, void* stream);

/* ------------------------------------------------------------------------------------------------------
 * Session: model, KV caches (bf16 and compressed), activations and step state in caller-provided memory.
 * ---------------------------------------------------------------------------------------------------- */
int cass_session_bytes(const cass_model_desc* desc, const cass_format* fmt, size_t* h_bytes);

/* mem: device memory of at least cass_session_bytes, 256-byte aligned; it is zeroed here.  blobs may be NULL
 * and supplied later with cass_session_set_blobs (after calibration).  *h_session is a host handle released
 * with cass_session_destroy (which frees host memory only).  SYNCHRONISES `stream`. */
int cass_session_init(void* mem, size_t bytes, const cass_model_desc* desc, const cass_format* fmt,
                      const cass_model_weights* weights, const cass_model_blobs* blobs, void** h_session,
                      void* stream);
int cass_session_set_blobs(void* session, const cass_model_blobs* blobs, void* stream);   /* SYNCHRONISES */
int cass_session_destroy(void* session);

/* Verification from the two parts (Sec. 4.1 target inference: "both the speculation and verification data are loaded and
 * fully reconstructed"; Sec. 7.2: no bf16 copy has to stay resident).  vdata: device pointers to the verification data
 * (cass_encode_verification_data) of the matrices whose speculation data the session already has (Cassandra-1 blobs).
 * From then on cass_verify rebuilds each matrix -- kept values with their low mantissa bits appended, pruned values as
 * stored, bit for bit the original -- into `scratch_bf16` right before the projection that reads it, and never touches
 * the bf16 matrices given at cass_session_init again (the caller may free them; embeddings and norm gains are still
 * read).  Results are bit-identical to verification from the bf16 copy.  scratch_bf16: device, 16-byte aligned, at
 * least cass_verify_from_parts_scratch_bytes (the largest matrix).  vdata = NULL switches back to the bf16 copy. */
typedef struct cass_layer_vdata { const void *wqkv, *wo, *wgu, *wd; } cass_layer_vdata;
typedef struct cass_model_vdata {
    const cass_layer_vdata* h_layers;     /* HOST array [n_layers] */
    const void* lm_head;
} cass_model_vdata;
size_t cass_verify_from_parts_scratch_bytes(const cass_model_desc* desc);
int cass_session_verify_from_parts(void* session, const cass_model_vdata* vdata, void* scratch_bf16, size_t scratch_bytes);

/* Forget all sequences: committed length 0, no draft in flight, KV codebooks cleared. */
int cass_session_reset(void* session, void* stream);

/* Reads the device status word and the committed length of sequence 0.  SYNCHRONISES `stream`. */
int cass_session_status(void* session, int32_t* h_status, int32_t* h_len, void* stream);
/* Committed lengths of all sequences: h_lens[max_batch].  SYNCHRONISES `stream`. */
int cass_session_lens(void* session, int32_t* h_lens, void* stream);
/* Rows (over all sequences) one cass_verify call can take for this description: 16, 32 or 64; negative on a bad
 * description.  Prefill feeds max_batch * (g+1) <= that many rows per call.  Host-only arithmetic. */
int cass_session_rows(const cass_model_desc* desc);

/* Wanda calibration (Sec. 4.2, Sec. 7.2 "Pre-Computation Cost"): while enabled, cass_verify accumulates the
 * per-input-channel sums of squares of the activations entering each projection.  cass_calib_norms writes
 * their square roots: fp32 [n_layers][4][max(hidden, ffn)] (inputs of wqkv, wo, wgu, wd) followed by
 * fp32 [hidden] (input of lm_head). */
int cass_calib_enable(void* session, int on, void* stream);
int cass_calib_norms(void* session, float* norms_out, void* stream);
size_t cass_calib_norms_count(const cass_model_desc* desc);

/* Online KV encoder (Sec. 4.2 per-token magnitude pruning; Sec. 5.1 encoder).  Writes n_new tokens of one
 * layer, starting at position start_pos of sequence `seq`, into the bf16 cache and/or the compressed cache
 * (flags).  K, V: bf16 [n_new][n_kv_heads][head_dim]; K is expected post-RoPE.  Per token and head the
 * floor(d*p/1000) smallest |x| are pruned (ties: lower channel first).  Positions must be appended in
 * order: start_pos may not exceed the number of positions already in the compressed cache of that layer.
 * The compressed cache uses the layer's frozen codebooks (cass_kv_build_codebook).
 * Record of one (token, head, K|V) in the compressed cache, kv_mode 1: entry words (a 10-bit code-bit offset for every
 * 32-channel slice after the first, three per word from bit 29 down: a decoder can enter a record at any slice;
 * bit 31 of the first word = raw flag), bitmap, sign+mantissa fields, and in the arena the unary exponent stream -- or,
 * when that stream would take more than min(8 * kept, 1023) bits, the kept exponents as raw bytes, so that a record
 * never takes more than ceil(8 * kept / 32) arena words and the arena is sized for that: a codebook that fits the later
 * tokens badly costs bytes, never capacity.  kv_mode 2: bitmap, fields (sign + high 7-t bits of the MXINT magnitude)
 * and one shared exponent byte per 32-channel slice; fixed size, no arena use, no codebook. */
int cass_kv_append(void* session, int seq, int layer, const void* K_bf16, const void* V_bf16, int start_pos, int n_new,
                   int flags, void* stream);

/* Builds the exponent codebooks of every sequence and layer (one for K, one for V) from the kept values of the
 * first n_tokens positions of that sequence's bf16 cache, freezes them, and encodes those positions into the
 * compressed cache. */
int cass_kv_build_codebook(void* session, int n_tokens, void* stream);

/* Sets the committed length of every sequence to len (after prefill through cass_verify, or to roll back);
 * cass_set_lens gives each sequence its own (h_lens: HOST [max_batch]).  len + 16 <= max_seq, so that the rows of
 * the next call still fit.  Both clear the drafts in flight and SYNCHRONISE `stream`. */
int cass_set_len(void* session, int len, void* stream);
int cass_set_lens(void* session, const int32_t* h_lens, void* stream);

/* One draft token per sequence (Sec. 4.1 draft inference).  Reads the token id tok_in[b * tok_stride] of each
 * sequence b, runs the draft model for it at position len_b + (tokens drafted since the last accept), appends that
 * position's K/V to the sequence's compressed cache only, and writes the greedy next token to
 * tok_out[b * tok_stride] (lowest index on ties).  tok_stride = 1 for packed arrays, g+1 when the tokens sit in the
 * [max_batch][g+1] array that cass_verify reads.  The weights' speculation data is read and decoded once for all
 * sequences.  logits_opt: fp32 [max_batch][vocab] or NULL.  At most gamma_max calls between two accepts (or
 * cass_set_len / cass_set_lens / cass_session_reset): one more returns CASS_ERR_INVALID_ARG and launches nothing. */
int cass_draft_step(void* session, const int32_t* tok_in, int32_t* tok_out, int tok_stride, float* logits_opt,
                    void* stream);

/* Target pass over g+1 rows of every sequence (Sec. 2.2 verification; Sec. 4.1 target inference):
 * toks[b][i] sits at position len_b + i of sequence b; causal among a sequence's rows; K/V of those positions are
 * (over)written in both caches; the greedy token of row (b, i) goes to target_argmax[b][i].  g+1 <= 16 and
 * max_batch * (g+1) <= cass_session_rows().  g = 0 is plain autoregressive decoding.  Does not move len.
 * logits_opt: fp32 [max_batch][g+1][vocab] or NULL.  Row results do not depend on how many rows the call has. */
int cass_verify(void* session, const int32_t* toks, int g, int32_t* target_argmax, float* logits_opt,
                void* stream);

/* Stand-alone draft attention of one layer (Sec. 4.1 draft inference over the KV speculation data of Sec. 4.2):
 * q: bf16 [max_batch][n_q_heads][head_dim] (post-RoPE); sequence b's query sees the first len_b + 1 positions of its
 * compressed cache of that layer (len = committed length, see cass_set_len; no draft in flight);
 * out: bf16 [max_batch][n_q_heads][head_dim].  Returns CASS_ERR_UNSUPPORTED for KV truncations other than 0 and 4,
 * more than 8 query heads per KV head, or a head size that is not a multiple of 32 (cass_draft_step likewise). */
int cass_draft_attention(void* session, int layer, const void* q_bf16, void* out_bf16, void* stream);

/* Stand-alone verification projection (Sec. 2.2: the gamma+1 rows are processed as one small batch, bound by
 * the bf16 weight bytes): Y[r][j] = sum_c W[j][c] X[r][c] for r < rows <= 64, fp32 accumulation on the tensor
 * cores.  W: bf16 [n][k] row-major, 16-byte aligned, k a multiple of 8.  X: bf16 buffer of 16, 32 or 64 rows (the
 * smallest of these >= rows) of k values, 16-byte aligned (rows beyond `rows` are read but do not influence the
 * result).  scratch: device memory of
 * cass_verify_gemm_scratch_bytes(n, k).  Outputs [rows][n]; either may be NULL.  A row's result does not depend
 * on `rows`.  d_status (required) receives CASS_ERR_TIMEOUT if a bounded device wait runs out. */
size_t cass_verify_gemm_scratch_bytes(int n, int k);
int cass_verify_gemm(const void* W_bf16, const void* X_bf16, int rows, int n, int k, void* scratch, size_t scratch_bytes,
                     void* y_bf16, float* y_f32, int32_t* d_status, void* stream);

/* Greedy acceptance (Sec. 2.2; Eq. 1 with p/q in {0,1}), per sequence b, with draft_b[i] = draft[b * draft_stride + i]:
 * a = min({i-1 : draft_b[i-1] != target_argmax[b][i-1]} U {g});
 * out_tokens[b][0..a] = draft_b[0..a-1], target_argmax[b][a] (the rest -1); len_b += a + 1 (both caches are trimmed
 * by that); the draft-in-flight counter returns to 0; next_tok[b * next_stride] = target_argmax[b][a].
 * draft_stride >= g (g for a packed [max_batch][g] array; g+1 with draft = toks + 1 of the verification array);
 * target_argmax and out_tokens: [max_batch][g+1]; n_accepted: [max_batch]; all device.
 * A sequence that would come within 16 positions of max_seq keeps its length and the status word is set to
 * CASS_ERR_CAPACITY (tokens are still reported). */
int cass_accept(void* session, const int32_t* draft, int draft_stride, const int32_t* target_argmax, int g,
                int32_t* n_accepted, int32_t* out_tokens, int32_t* next_tok, int next_stride, void* stream);

/* Acceptance by rejection sampling (Sec. 2.2, Eq. 1), for decoding with sampling instead of greedy choice.  Per
 * sequence b, with x_i = draft[b * draft_stride + i - 1] the i-th drafted token (drawn from the draft's distribution
 * q_i), p_i the target's distribution at the same row and r_i a uniform number in (0, 1):
 *   n = min({i-1 : 1 <= i <= g, r_i > p_i(x_i) / q_i(x_i)} U {g})                                        (Eq. 1)
 * and the step emits one more token, drawn with the uniform number u_b by inverse CDF (lowest index whose cumulative
 * weight exceeds u_b times the total): from the normalised positive part of p_{n+1} - q_{n+1} after a rejection, from
 * p_{g+1} when all g drafts were accepted.  (The paper states the guarantee -- outputs distributed exactly as the
 * target's -- and cites speculative sampling for the procedure; this is that procedure's correction step.)
 * p_target: fp32 [n_seq][g+1][vocab], q_draft: fp32 [n_seq][g][vocab] (probabilities, see cass_softmax);
 * r_uniform: fp32 [n_seq][g]; u_uniform: fp32 [n_seq]; the library draws no random numbers itself.
 * Outputs as cass_accept: n_accepted [n_seq], out_tokens [n_seq][g+1] (n drafts, the extra token, then -1),
 * next_tok[b * next_stride] = the extra token.  With a session (n_seq must equal its max_batch, vocab its vocab) the
 * lengths move by n+1 and the draft counters are cleared exactly as in cass_accept; session may be NULL, then only
 * the outputs are produced (any n_seq).  A drafted token outside [0, vocab) is rejected. */
int cass_accept_sampling(void* session, int n_seq, const int32_t* draft, int draft_stride, const float* p_target,
                         const float* q_draft, int vocab, const float* r_uniform, const float* u_uniform, int g,
                         int32_t* n_accepted, int32_t* out_tokens, int32_t* next_tok, int next_stride, void* stream);

/* Helpers for sampled decoding (Sec. 2.2).  cass_softmax: probs[r][v] = softmax(logits[r][.] / temperature), fp32
 * [rows][vocab] both, temperature > 0 (the fp32 logits are what cass_draft_step / cass_verify return in logits_opt).
 * cass_sample: tokens[r * tok_stride] = inverse-CDF draw from probs[r][.] (non-negative weights; need not be
 * normalised) with the uniform number u[r] in [0, 1). */
int cass_softmax(const float* logits, int rows, int vocab, float temperature, float* probs, void* stream);
int cass_sample(const float* probs, int rows, int vocab, const float* u, int32_t* tokens, int tok_stride, void* stream);

/* Geometry of the compressed KV cache of (sequence, layer, kind 0=K 1=V, head) for tests: device pointers to the
 * fixed-part blocks, the unary arena and the per-token word offsets, plus words per token in the fixed part. */
typedef struct cass_kv_view {
    const uint32_t* fixed; const uint32_t* arena; const uint32_t* offsets; const uint8_t* codebook;
    const void* k_or_v_bf16;
    int fixed_words_per_token, bitmap_words, arena_words;
} cass_kv_view;
int cass_kv_query(void* session, int seq, int layer, int kind, int head, cass_kv_view* h_view);

/* Standalone draft attention / verify kernels are reached through cass_draft_step / cass_verify; the
 * activations of the last call can be inspected for tests: which = 0 hidden state after the last layer
 * (bf16 [rows][hidden]), 1 = the last layer's attention output (bf16 [rows][n_q d]), 2 = the last layer's rotated
 * q, k, v rows (bf16 [rows][(n_q + 2 n_kv) d]).  *h_rows is the buffer's row capacity. */
int cass_debug_activation(void* session, int which, const void** d_ptr, int* h_rows, int* h_cols);

const char* cass_version(void);

#ifdef __cplusplus
}
#endif
#endif /* CASS_H_ */
