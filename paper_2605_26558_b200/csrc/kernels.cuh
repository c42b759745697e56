// Internal launchers shared between the translation units of the library.
#pragma once

#include <type_traits>

#include "common.cuh"

namespace cass {

// Device-resident step state of the session's sequences; kernels read positions from here so that a captured
// graph of launches can be replayed without host-side position arguments.
struct DevState {
    int32_t len[kMaxBatch];        // committed KV positions of each sequence
    int32_t inflight[kMaxBatch];   // draft tokens appended since the last accept
    int32_t status;     // first device-side error (CASS_ERR_*), 0 if none
    int32_t calib_on;
    int32_t max_seq;    // KV positions per sequence; len never moves past max_seq - kMaxVerifyRows
};

// Row r of a call with `rps` rows per sequence belongs to sequence r / rps and is its (r % rps)-th new row.

// Compressed KV cache of one (layer, K|V): per head a fixed part (32-token blocks interleaved word by word), an
// append-only arena of exponent words and per-token word offsets.
// Cassandra-1 record (mode 1): fixed part = entry words | bitmap | fields (rotated, as in the weight blobs); the arena
// holds the record's unary exponent stream or, when that would take more than min(8 * kept, 1023) bits, the kept
// values' exponents as raw bytes (four per word from the top; bit 31 of the first entry word says so).  Entry words:
// a 10-bit code-bit offset for every 32-channel slice after the first, three per word from bit 29 down, so that the
// d/32 slices of a record can be decoded side by side.
// Cassandra-2 record (mode 2): fixed part = bitmap | fields (sign + magnitude, packed from the top) | one shared
// exponent byte per 32-channel slice (four per word from the top); no arena use.
struct KvComp {
    uint32_t* fixed;        // [n_kv][n_blocks][wpt][32]
    uint32_t* arena;        // [n_kv][arena_words]
    uint32_t* off;          // [n_kv][max_seq + 1]
    uint8_t* rank_to_exp;   // [256]
    uint8_t* exp_to_rank;   // [256]
    unsigned long long* hist;   // [256]
};

constexpr uint32_t kKvRawFlag = 0x80000000u;
struct KvGeom {
    int n_kv, d, max_seq, n_blocks, wpt, bm_words, f_words, kept, n_prune, t, arena_words;
    int mode;               // 1 = Cassandra-1 records, 2 = Cassandra-2 (MX) records
    int e_words;            // entry words in front of the bitmap (mode 1), 0 in mode 2
    int x_words;            // exponent words behind the fields (mode 2), 0 in mode 1
    int rec_words_max;      // most arena words one record can take
    size_t seq_stride;      // bytes between the KV storage (both caches, all layers) of consecutive sequences
};

// The same object of sequence b: every sequence's KV storage has the same internal layout.
template <class P>
__host__ __device__ __forceinline__ P* of_seq(P* p, int b, size_t seq_stride) {
    using Byte = typename std::conditional<std::is_const<P>::value, const char, char>::type;
    return reinterpret_cast<P*>(reinterpret_cast<Byte*>(p) + (size_t)b * seq_stride);     // pointer arithmetic: stays a global-memory pointer
}
__host__ __device__ inline int kv_entry_words(int d) { int n = (d / 32 - 1 + 2) / 3; return n < 1 ? 1 : n; }
__host__ __device__ inline int kv_code_budget(int kept) { return 8 * kept < 1023 ? 8 * kept : 1023; }
// Positions one CTA of the draft attention handles: one 64-token chunk, doubled while the grid would exceed about four
// CTAs per SM.  The kernel and its merge compute it from the same visible length, so they agree without host involvement.
__host__ __device__ inline int tc_run_tokens(int visible, int heads_x_seqs) {
    int t = 64;
    while (t < 2048 && ceil_div(visible, t) * heads_x_seqs > 592) t *= 2;
    return t;
}
__host__ __device__ __forceinline__ KvComp of_seq(const KvComp& c, int b, size_t seq_stride) {
    KvComp r;
    r.fixed = of_seq(c.fixed, b, seq_stride); r.arena = of_seq(c.arena, b, seq_stride); r.off = of_seq(c.off, b, seq_stride);
    r.rank_to_exp = of_seq(c.rank_to_exp, b, seq_stride); r.exp_to_rank = of_seq(c.exp_to_rank, b, seq_stride);
    r.hist = of_seq(c.hist, b, seq_stride);
    return r;
}

// fp32 split-K partial sums of a projection: element (row r, feature i) of part s sits at p[s * seg_stride + r * row_stride + i];
// consumers add the parts in order and round to bf16 where the projection output is a bf16 activation.
struct Partials {
    const float* p;
    int n_seg;
    size_t seg_stride, row_stride;
};

// Sum of the parts at element offset `off` (row and feature already applied), added in part order.  The loads of up to
// eight parts are issued before the first addition, so that a sum costs one round trip to L2 instead of one per part.
constexpr int kPartBatch = 8;
__device__ __forceinline__ float parts_sum(const Partials& pp, size_t off) {
    float acc = 0.f;
    const float* p = pp.p + off;
    for (int s0 = 0; s0 < pp.n_seg; s0 += kPartBatch) {
        float v[kPartBatch];
#pragma unroll
        for (int i = 0; i < kPartBatch; ++i) v[i] = s0 + i < pp.n_seg ? __ldcg(p + (size_t)(s0 + i) * pp.seg_stride) : 0.f;
#pragma unroll
        for (int i = 0; i < kPartBatch; ++i)
            if (s0 + i < pp.n_seg) acc += v[i];
    }
    return acc;
}
// Four consecutive elements (16-byte loads; `off` a multiple of 4 elements, strides too), four parts per batch.
__device__ __forceinline__ float4 parts_sum4(const Partials& pp, size_t off) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    const float* p = pp.p + off;
    for (int s0 = 0; s0 < pp.n_seg; s0 += 4) {
        float4 v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
            v[i] = s0 + i < pp.n_seg ? __ldcg(reinterpret_cast<const float4*>(p + (size_t)(s0 + i) * pp.seg_stride)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (s0 + i < pp.n_seg) { acc.x += v[i].x; acc.y += v[i].y; acc.z += v[i].z; acc.w += v[i].w; }
    }
    return acc;
}
// The same for N offsets at once: all loads of a batch of parts travel together.
template <int N>
__device__ __forceinline__ void parts_sum_n(const Partials& pp, const size_t (&off)[N], const bool (&on)[N], float (&acc)[N]) {
    constexpr int B = N >= 8 ? 2 : (N >= 4 ? 4 : 8);                  // parts per batch: at most 16-32 loads in flight per thread
#pragma unroll
    for (int j = 0; j < N; ++j) acc[j] = 0.f;
    for (int s0 = 0; s0 < pp.n_seg; s0 += B) {
        float v[N][B];
#pragma unroll
        for (int j = 0; j < N; ++j)
#pragma unroll
            for (int i = 0; i < B; ++i)
                v[j][i] = (on[j] && s0 + i < pp.n_seg) ? __ldcg(pp.p + (size_t)(s0 + i) * pp.seg_stride + off[j]) : 0.f;
#pragma unroll
        for (int j = 0; j < N; ++j)
#pragma unroll
            for (int i = 0; i < B; ++i)
                if (on[j] && s0 + i < pp.n_seg) acc[j] += v[j][i];
    }
}

constexpr int kAttnChunk = 64;       // split-K granularity over the sequence (fixed absolute boundaries)

size_t gemv_smem_bytes(const cass_blob_info& bi, int nb);
// x: bf16 [nb][cols], nb in {1, 2, 4, 8} vectors multiplied in one pass over the blob.
// partial: fp32 [nb][n_seg][n_rowblocks*32]; the caller sums the segments (fixed order) afterwards.
int launch_draft_gemv(const void* blob, const cass_blob_info& bi, const void* x_bf16, int nb, float* partial,
                      int32_t* d_status, cudaStream_t stream);
inline Partials draft_gemv_partials(const float* partial, const cass_blob_info& bi) {
    const size_t n_pad = (size_t)bi.n_rowblocks * kRowsPerBlock;
    return Partials{partial, bi.n_seg, n_pad, (size_t)bi.n_seg * n_pad};
}

// ---- small ops (ops.cu) -------------------------------------------------------------------------------
int launch_rope_table(float* cos_t, float* sin_t, int max_seq, int d, float theta, cudaStream_t s);
// row r takes token toks[r * tok_stride]
int launch_embed(const int32_t* toks, int tok_stride, const uint16_t* embed, uint16_t* h, int rows, int hidden, cudaStream_t s);
int launch_rmsnorm(const uint16_t* h, const uint16_t* gain, uint16_t* out, int rows, int hidden, float eps,
                   cudaStream_t s);
// h = bf16(h + y); out = rmsnorm(h) * gain.  y comes either as bf16 [rows][hidden] or (rows == 1) as fp32 split-K
// partials [n_seg][n_pad] that are summed in segment order and rounded to bf16 first.
int launch_residual_rmsnorm(uint16_t* h, const uint16_t* y_bf16, Partials pp,
                            const uint16_t* gain, uint16_t* out, int rows, int hidden, float eps, cudaStream_t s);
// q and k of qkv (bf16 [rows][qkv_dim]) rotated in place at the row's position: len (+ inflight when use_inflight)
// of its sequence + its index among the sequence's rps rows.  With partials, qkv is first formed from them.
int launch_qkv_rope(uint16_t* qkv, Partials pp, const float* cos_t, const float* sin_t,
                    const DevState* st, int use_inflight, int rows, int rps, int n_q, int n_kv, int d, cudaStream_t s);
int launch_swiglu(const uint16_t* gu_bf16, Partials pp, uint16_t* act, int rows,
                  int ffn, cudaStream_t s);
// logits (fp32 [rows][vocab], or formed from partials) -> lowest-index argmax per row; optional copy
// of the logits; bump_inflight adds 1 to the draft counter of sequence r (one row per sequence) afterwards.
// tmp_v / tmp_i: scratch of kMaxRows x 128 entries each.
// Row r's token goes to out[r * out_stride].
int launch_argmax(const float* logits, Partials pp, int rows, int vocab, int32_t* out, int out_stride,
                  float* logits_copy, float* tmp_v, int32_t* tmp_i, DevState* st, int bump_inflight, cudaStream_t s);
int launch_accept(DevState* st, int n_seq, const int32_t* draft, int draft_stride, const int32_t* target, int g, int32_t* n_acc,
                  int32_t* out_tokens, int32_t* next_tok, int next_stride, cudaStream_t s);
// Sampling-based acceptance (sampling.cu): p [n_seq][g+1][vocab], q [n_seq][g][vocab] probabilities, r [n_seq][g] and
// u [n_seq] uniform numbers; st may be null (no lengths to move).
int launch_accept_sampling(DevState* st, int n_seq, const int32_t* draft, int draft_stride, const float* p, const float* q,
                           int vocab, const float* r, const float* u, int g, int32_t* n_acc, int32_t* out_tokens,
                           int32_t* next_tok, int next_stride, cudaStream_t s);
int launch_calib_accum(const uint16_t* x, int rows, int cols, float* sumsq, const DevState* st, cudaStream_t s);
int launch_sqrt(const float* in, float* out, size_t n, cudaStream_t s);

// ---- KV encoder (kv.cu) -------------------------------------------------------------------------------
// Appends n_new tokens to each of the n_seq sequences seq0 .. seq0 + n_seq - 1 (caches given for sequence 0).
// src_k/src_v: bf16 rows with `row_stride` elements between tokens and n_kv*d contiguous per token; the rows of the
// i-th sequence of the call start at row i * n_new.
// start_pos < 0: take the position from the state (len, or len + inflight when use_inflight).
int launch_kv_append(const KvGeom& g, const KvComp& ck, const KvComp& cv, uint16_t* k_cache, uint16_t* v_cache,
                     const uint16_t* src_k, const uint16_t* src_v, int row_stride, int start_pos, int use_inflight,
                     int n_new, int flags, DevState* st, int seq0, int n_seq, cudaStream_t s);
// The same fused with what precedes it in a layer: adds the qkv projection's split-K parts, rounds to bf16, applies
// RoPE to q and k at each row's position, writes the bf16 qkv rows (rps per sequence) and appends the K/V of those
// rows at the positions the state gives.  Needs head_dim % 64 == 0 (rope_kv_fusable); otherwise the caller runs
// launch_qkv_rope + launch_kv_append.
bool rope_kv_fusable(const KvGeom& g);
int launch_rope_kv_append(const KvGeom& g, const KvComp& ck, const KvComp& cv, uint16_t* k_cache, uint16_t* v_cache,
                          Partials pp, const float* cos_t, const float* sin_t, uint16_t* qkv, int n_q, int use_inflight,
                          int rps, int flags, DevState* st, int n_seq, cudaStream_t s);
int launch_kv_codebook(const KvGeom& g, const KvComp& ck, const KvComp& cv, const uint16_t* k_cache,
                       const uint16_t* v_cache, int n_tokens, cudaStream_t s);

// ---- attention ----------------------------------------------------------------------------------------
struct AttnScratch {
    float* o;     // [rows*n_q][n_chunks][d]
    float* m;     // [rows*n_q][n_chunks]
    float* l;     // [rows*n_q][n_chunks]
};
// Draft: one query row per sequence (qkv row b, `qkv_stride` elements apart) at position len + inflight over that
// sequence's compressed cache (caches given for sequence 0).
int launch_draft_attn(const KvGeom& g, const KvComp& ck, const KvComp& cv, const uint16_t* qkv, int qkv_stride, int n_q,
                      int n_seq, const DevState* st, const AttnScratch& sc, uint16_t* out, cudaStream_t s);
// Verify: rps rows per sequence at positions len + i over that sequence's bf16 cache, causal.
int launch_verify_attn(const KvGeom& g, const uint16_t* k_cache, const uint16_t* v_cache, const uint16_t* qkv,
                       int n_seq, int rps, int n_q, const DevState* st, const AttnScratch& sc, uint16_t* out, cudaStream_t s);

// Tensor-core version (verify_attn_tc.cu) for head_dim 128 and rps * (n_q / n_kv) <= 64.  np_cols = 32 or 64: the
// MMA's pair columns (>= rps * group); a pair's result does not depend on it, but a session keeps one value for
// all its decode calls.
bool verify_attn_tc_usable(const KvGeom& g, int rps, int n_q);
int launch_verify_attn_tc(const KvGeom& g, const uint16_t* k_cache, const uint16_t* v_cache, const uint16_t* qkv, int n_seq,
                          int rps, int n_q, int np_cols, const DevState* st, const AttnScratch& sc, uint16_t* out,
                          int32_t* d_status, cudaStream_t s);

// ---- verification GEMM (verify_gemm.cu): Y[r][n] = sum_k W[n][k] X[r][k], bf16 in, fp32 accumulate (tcgen05) ----
// X is a buffer of `bn` rows of k values (bn = 16, 32 or 64 token columns of the MMA; the first `rows` are used);
// partial: fp32 scratch of verify_gemm_partial_floats.
// With both outputs null only the partial sums are produced: [splits][bn][n], see verify_gemm_partials().
inline int verify_gemm_bn(int rows) { return rows <= 16 ? 16 : rows <= 32 ? 32 : 64; }
size_t verify_gemm_partial_floats(int n, int k, int bn);
Partials verify_gemm_partials(const float* partial, int n, int k, int bn);
// w_static: W is not the output of a kernel that may still be running when this one is scheduled (the bf16 matrices of
// a session); its first tiles are then requested before the wait for the predecessor.
int launch_verify_gemm(const uint16_t* W, const uint16_t* X, int rows, int bn, int n, int k, float* partial, uint16_t* y_bf16,
                       float* y_f32, int32_t* d_status, cudaStream_t s, int w_static = 0);

}  // namespace cass
