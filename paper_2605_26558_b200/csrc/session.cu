// Session: device memory plan, model pointers, and the three step-level entry points
// (draft step, verification pass, greedy accept) built from the library's kernels.
#include <cstddef>
#include <cstdlib>
#include <new>
#include <vector>

#include "kernels.cuh"

namespace cass {

struct LayerDev {
    cass_layer_weights w;
    const void* vdata[4];    // verification data of wqkv, wo, wgu, wd (only when verifying from the two parts)
    const void* blob[4];
    cass_blob_info bi[4];
    uint16_t *kc, *vc;       // bf16 caches [max_seq][n_kv][d]
    KvComp ck, cv;
    float* calib[4];         // sums of squares of the inputs of wqkv, wo, wgu, wd
};

struct Session {
    cass_model_desc d;
    cass_format f;
    KvGeom kg;
    uint8_t* base;
    size_t bytes;
    DevState* st;
    float *cos_t, *sin_t;
    std::vector<LayerDev> layers;
    const void *embed, *lm_head, *norm_final;
    const void* lm_blob;
    cass_blob_info lm_bi;
    float* calib_lm;
    float* calib_all;        // start of the calibration block
    size_t calib_count;
    int calib_kmax;
    int B, R;                // sequences; row capacity of one call (16, 32 or 64 = token columns of the verification MMA)
    // activations (R rows)
    uint16_t *h, *xn, *qkv, *attn, *y, *gu, *act;
    float *logits, *partial, *vg_partial;
    size_t partial_floats;
    AttnScratch asc;
    int32_t* argmax_tmp;
    float* argmax_val;
    bool have_blobs, codebooks_ready, calib_host;
    int qkv_dim, kmax;
    int drafts_pending;      // cass_draft_step calls since the last accept / set_len / reset (host-side count)
    bool from_parts;         // verification rebuilds each matrix from speculation + verification data into vscratch
    const void* lm_vdata;
    uint16_t* vscratch;
};

struct Plan {
    size_t off = 0;
    size_t take(size_t b) { size_t o = off; off = align_up(off + b, 256); return o; }
};

static int check_desc(const cass_model_desc* d, const cass_format* f) {
    if (!d || !f) return CASS_ERR_INVALID_ARG;
    if (f->mode != 1 && f->mode != 2) return CASS_ERR_UNSUPPORTED;     // weights: Cassandra-1 or Cassandra-2; KV: see kv_mode
    if (d->max_batch != 1 && d->max_batch != 2 && d->max_batch != 4 && d->max_batch != 8) return CASS_ERR_UNSUPPORTED;
    if (d->n_layers <= 0 || d->hidden <= 0 || d->n_q_heads <= 0 || d->n_kv_heads <= 0 || d->head_dim <= 0 ||
        d->ffn <= 0 || d->vocab <= 0 || d->max_seq < 2 * kMaxVerifyRows)
        return CASS_ERR_INVALID_ARG;
    if (d->n_q_heads % d->n_kv_heads || d->head_dim % 32 || d->head_dim > 256 || d->n_q_heads / d->n_kv_heads > 8)
        return CASS_ERR_UNSUPPORTED;
    if (d->hidden % 8 || d->ffn % 8 || (d->n_q_heads * d->head_dim) % 8) return CASS_ERR_UNSUPPORTED;
    if (d->gamma_max < 0 || d->gamma_max + 1 > kMaxVerifyRows) return CASS_ERR_INVALID_ARG;
    if (d->max_batch * (d->gamma_max + 1) > kMaxRows) return CASS_ERR_INVALID_ARG;
    if (f->kv_prune_permille < 0 || f->kv_prune_permille > 999 || f->kv_trunc_bits < 0 || f->kv_trunc_bits > 7)
        return CASS_ERR_INVALID_ARG;
    if (f->kv_trunc_bits != 0 && f->kv_trunc_bits != 4) return CASS_ERR_UNSUPPORTED;    // draft attention walks t = 0 or 4 records
    if (f->kv_mode < 0 || f->kv_mode > 2) return CASS_ERR_INVALID_ARG;
    return CASS_OK;
}

static KvGeom make_kv_geom(const cass_model_desc& d, const cass_format& f) {
    KvGeom g;
    g.n_kv = d.n_kv_heads; g.d = d.head_dim; g.max_seq = d.max_seq;
    g.n_blocks = ceil_div(d.max_seq, 32);
    g.n_prune = (d.head_dim * f.kv_prune_permille) / 1000;
    g.kept = d.head_dim - g.n_prune;
    g.t = f.kv_trunc_bits;
    g.mode = f.kv_mode == 2 ? 2 : 1;
    int per = 32 / (8 - g.t);
    g.bm_words = d.head_dim / 32;
    g.f_words = ceil_div(g.kept, per);
    g.e_words = g.mode == 1 ? kv_entry_words(d.head_dim) : 0;
    g.x_words = g.mode == 2 ? ceil_div(g.bm_words, 4) : 0;
    g.wpt = g.e_words + g.bm_words + g.f_words + g.x_words;
    // arena: the most a record can take (raw exponents: one byte per kept value), so that only the end of the cache
    // itself can exhaust it; Cassandra-2 records have no variable part
    g.rec_words_max = g.mode == 1 ? ceil_div(8 * g.kept, 32) : 0;
    g.arena_words = g.mode == 1 ? d.max_seq * (g.rec_words_max < 1 ? 1 : g.rec_words_max) : 32;
    return g;
}

// Lays the session out in `base` (base may be null: sizes only).
static int row_capacity(const cass_model_desc& d) {
    int r = d.max_batch * (d.gamma_max + 1);
    return verify_gemm_bn(r < kMaxVerifyRows ? kMaxVerifyRows : r);
}

static size_t layout(Session* s, uint8_t* base) {
    const cass_model_desc& d = s->d;
    KvGeom& g = s->kg;
    s->B = d.max_batch;
    s->R = row_capacity(d);
    Plan p;
    auto at = [&](size_t o) { return base ? base + o : nullptr; };
    s->st = (DevState*)at(p.take(sizeof(DevState)));
    size_t rt = (size_t)d.max_seq * (d.head_dim / 2) * 4;
    s->cos_t = (float*)at(p.take(rt));
    s->sin_t = (float*)at(p.take(rt));
    s->qkv_dim = (d.n_q_heads + 2 * d.n_kv_heads) * d.head_dim;
    s->kmax = d.hidden;
    if (d.ffn > s->kmax) s->kmax = d.ffn;
    if (d.n_q_heads * d.head_dim > s->kmax) s->kmax = d.n_q_heads * d.head_dim;
    s->calib_kmax = s->kmax;
    s->calib_count = (size_t)d.n_layers * 4 * s->kmax + d.hidden;
    s->calib_all = (float*)at(p.take(s->calib_count * 4));
    s->calib_lm = s->calib_all ? s->calib_all + (size_t)d.n_layers * 4 * s->kmax : nullptr;
    const int R = s->R;
    s->h = (uint16_t*)at(p.take((size_t)R * d.hidden * 2));
    s->xn = (uint16_t*)at(p.take((size_t)R * d.hidden * 2));
    s->qkv = (uint16_t*)at(p.take((size_t)R * s->qkv_dim * 2));
    s->attn = (uint16_t*)at(p.take((size_t)R * d.n_q_heads * d.head_dim * 2));
    s->y = (uint16_t*)at(p.take((size_t)R * d.hidden * 2));
    s->gu = (uint16_t*)at(p.take((size_t)R * 2 * d.ffn * 2));
    s->act = (uint16_t*)at(p.take((size_t)R * d.ffn * 2));
    s->logits = (float*)at(p.take((size_t)R * d.vocab * 4));
    // split-K partials of the draft GEMVs: segments (<= ceil(K/256)) x padded rows
    size_t nmax = (size_t)d.vocab;
    if ((size_t)2 * d.ffn > nmax) nmax = 2 * (size_t)d.ffn;
    if ((size_t)s->qkv_dim > nmax) nmax = s->qkv_dim;
    size_t segmax = (size_t)ceil_div(s->kmax, 256) + 1;
    size_t pf = 0;
    {   // exact bound: max over the five matrix shapes of ceil(K/256) * pad32(N) (smallest legal segment is one chunk)
        auto need = [&](size_t n, size_t k) { return (size_t)ceil_div((int)k, 256) * align_up(n, 32); };
        size_t c[5] = {need(s->qkv_dim, d.hidden), need(d.hidden, (size_t)d.n_q_heads * d.head_dim), need(2 * (size_t)d.ffn, d.hidden),
                       need(d.hidden, d.ffn), need(d.vocab, d.hidden)};
        for (size_t v : c) if (v > pf) pf = v;
    }
    (void)segmax; (void)nmax;
    s->partial_floats = pf;                                   // per vector of a draft GEMV
    s->partial = (float*)at(p.take(pf * 4 * s->B));
    {   // split-K scratch of the verification GEMMs
        size_t c[5] = {verify_gemm_partial_floats(s->qkv_dim, d.hidden, R), verify_gemm_partial_floats(d.hidden, d.n_q_heads * d.head_dim, R),
                       verify_gemm_partial_floats(2 * d.ffn, d.hidden, R), verify_gemm_partial_floats(d.hidden, d.ffn, R),
                       verify_gemm_partial_floats(d.vocab, d.hidden, R)};
        size_t m = 0;
        for (size_t v : c) if (v > m) m = v;
        s->vg_partial = (float*)at(p.take(m * 4));
    }
    const int n_chunks = ceil_div(d.max_seq, kAttnChunk);
    size_t pairs = (size_t)R * d.n_q_heads;
    s->asc.o = (float*)at(p.take(pairs * n_chunks * d.head_dim * 4));
    s->asc.m = (float*)at(p.take(pairs * n_chunks * 4));
    s->asc.l = (float*)at(p.take(pairs * n_chunks * 4));
    s->argmax_tmp = (int32_t*)at(p.take((size_t)R * 128 * 4));
    s->argmax_val = (float*)at(p.take((size_t)R * 128 * 4));
    s->layers.resize(d.n_layers);
    // KV storage: the block of sequence 0 (all layers, both caches), then identical blocks for the other sequences
    const size_t kv_begin = p.off;
    for (int l = 0; l < d.n_layers; ++l) {
        LayerDev& L = s->layers[l];
        size_t kvb = (size_t)d.max_seq * g.n_kv * g.d * 2;
        L.kc = (uint16_t*)at(p.take(kvb));
        L.vc = (uint16_t*)at(p.take(kvb));
        for (int kind = 0; kind < 2; ++kind) {
            KvComp& c = kind ? L.cv : L.ck;
            c.fixed = (uint32_t*)at(p.take((size_t)g.n_kv * g.n_blocks * g.wpt * 32 * 4));
            c.arena = (uint32_t*)at(p.take((size_t)g.n_kv * g.arena_words * 4));
            c.off = (uint32_t*)at(p.take((size_t)g.n_kv * (g.max_seq + 1) * 4));
            c.rank_to_exp = (uint8_t*)at(p.take(256));
            c.exp_to_rank = (uint8_t*)at(p.take(256));
            c.hist = (unsigned long long*)at(p.take(256 * 8));
        }
        for (int i = 0; i < 4; ++i) L.calib[i] = s->calib_all ? s->calib_all + ((size_t)l * 4 + i) * s->kmax : nullptr;
    }
    g.seq_stride = p.off - kv_begin;
    p.off += g.seq_stride * (size_t)(s->B - 1);
    return p.off;
}

static int read_blob_infos(Session* s, const cass_model_blobs* blobs, cudaStream_t stream) {
    for (int l = 0; l < s->d.n_layers; ++l) {
        const cass_layer_blobs& b = blobs->h_layers[l];
        const void* ptr[4] = {b.wqkv, b.wo, b.wgu, b.wd};
        const int rows[4] = {s->qkv_dim, s->d.hidden, 2 * s->d.ffn, s->d.hidden};
        const int cols[4] = {s->d.hidden, s->d.n_q_heads * s->d.head_dim, s->d.hidden, s->d.ffn};
        for (int i = 0; i < 4; ++i) {
            if (!ptr[i]) return CASS_ERR_INVALID_ARG;
            int rc = cass_weight_blob_info(ptr[i], &s->layers[l].bi[i], stream);
            if (rc) return rc;
            if (s->layers[l].bi[i].rows != rows[i] || s->layers[l].bi[i].cols != cols[i]) return CASS_ERR_INVALID_ARG;
            if (gemv_smem_bytes(s->layers[l].bi[i], s->B) > 227 * 1024) return CASS_ERR_CAPACITY;
            if ((size_t)s->layers[l].bi[i].n_seg * s->layers[l].bi[i].n_rowblocks * 32 > s->partial_floats) return CASS_ERR_CAPACITY;
            s->layers[l].blob[i] = ptr[i];
        }
    }
    if (!blobs->lm_head) return CASS_ERR_INVALID_ARG;
    int rc = cass_weight_blob_info(blobs->lm_head, &s->lm_bi, stream);
    if (rc) return rc;
    if (s->lm_bi.rows != s->d.vocab || s->lm_bi.cols != s->d.hidden) return CASS_ERR_INVALID_ARG;
    if ((size_t)s->lm_bi.n_seg * s->lm_bi.n_rowblocks * 32 > s->partial_floats) return CASS_ERR_CAPACITY;
    s->lm_blob = blobs->lm_head;
    s->have_blobs = true;
    return CASS_OK;
}

}  // namespace cass

using namespace cass;

extern "C" int cass_session_bytes(const cass_model_desc* desc, const cass_format* fmt, size_t* h_bytes) {
    int rc = check_desc(desc, fmt);
    if (rc) return rc;
    if (!h_bytes) return CASS_ERR_INVALID_ARG;
    Session s{};
    s.d = *desc; s.f = *fmt; s.kg = make_kv_geom(*desc, *fmt);
    *h_bytes = layout(&s, nullptr);
    return CASS_OK;
}

extern "C" int cass_session_init(void* mem, size_t bytes, const cass_model_desc* desc, const cass_format* fmt,
                                 const cass_model_weights* weights, const cass_model_blobs* blobs, void** h_session,
                                 void* stream_) {
    int rc = check_desc(desc, fmt);
    if (rc) return rc;
    if (!mem || !weights || !weights->h_layers || !h_session || ((uintptr_t)mem & 255)) return CASS_ERR_INVALID_ARG;
    Session* s = new (std::nothrow) Session{};
    if (!s) return CASS_ERR_CAPACITY;
    s->d = *desc; s->f = *fmt; s->kg = make_kv_geom(*desc, *fmt);
    size_t need = layout(s, (uint8_t*)mem);
    if (bytes < need) { delete s; return CASS_ERR_CAPACITY; }
    s->base = (uint8_t*)mem; s->bytes = need;
    cudaStream_t stream = (cudaStream_t)stream_;
    for (int l = 0; l < desc->n_layers; ++l) s->layers[l].w = weights->h_layers[l];
    s->embed = weights->embed; s->lm_head = weights->lm_head; s->norm_final = weights->norm_final;
    if (cudaMemsetAsync(mem, 0, need, stream) != cudaSuccess) { delete s; return CASS_ERR_CUDA; }
    if (cudaMemcpyAsync(&s->st->max_seq, &s->d.max_seq, 4, cudaMemcpyHostToDevice, stream) != cudaSuccess) { delete s; return CASS_ERR_CUDA; }
    rc = launch_rope_table(s->cos_t, s->sin_t, desc->max_seq, desc->head_dim, desc->rope_theta, stream);
    if (!rc && blobs) rc = read_blob_infos(s, blobs, stream);
    if (!rc && cudaStreamSynchronize(stream) != cudaSuccess) rc = CASS_ERR_CUDA;
    if (rc) { delete s; return rc; }
    *h_session = s;
    return CASS_OK;
}

extern "C" int cass_session_set_blobs(void* session, const cass_model_blobs* blobs, void* stream_) {
    if (!session || !blobs || !blobs->h_layers) return CASS_ERR_INVALID_ARG;
    return read_blob_infos((Session*)session, blobs, (cudaStream_t)stream_);
}

extern "C" int cass_session_destroy(void* session) {
    if (!session) return CASS_ERR_INVALID_ARG;
    delete (Session*)session;
    return CASS_OK;
}

extern "C" int cass_session_reset(void* session, void* stream_) {
    if (!session) return CASS_ERR_INVALID_ARG;
    Session* s = (Session*)session;
    cudaStream_t stream = (cudaStream_t)stream_;
    CASS_CUDA_CHECK(cudaMemsetAsync(s->st, 0, sizeof(DevState), stream));
    CASS_CUDA_CHECK(cudaMemcpyAsync(&s->st->max_seq, &s->d.max_seq, 4, cudaMemcpyHostToDevice, stream));
    CASS_CUDA_CHECK(cudaMemsetAsync(s->calib_all, 0, s->calib_count * 4, stream));
    for (auto& L : s->layers)
        for (int kind = 0; kind < 2; ++kind)
            for (int b = 0; b < s->B; ++b) {
                KvComp c = of_seq(kind ? L.cv : L.ck, b, s->kg.seq_stride);
                CASS_CUDA_CHECK(cudaMemsetAsync(c.off, 0, (size_t)s->kg.n_kv * (s->kg.max_seq + 1) * 4, stream));
            }
    s->codebooks_ready = false;
    s->drafts_pending = 0;
    return CASS_OK;
}

extern "C" int cass_session_status(void* session, int32_t* h_status, int32_t* h_len, void* stream_) {
    if (!session) return CASS_ERR_INVALID_ARG;
    Session* s = (Session*)session;
    cudaStream_t stream = (cudaStream_t)stream_;
    DevState st;
    CASS_CUDA_CHECK(cudaMemcpyAsync(&st, s->st, sizeof(st), cudaMemcpyDeviceToHost, stream));
    CASS_CUDA_CHECK(cudaStreamSynchronize(stream));
    if (h_status) *h_status = st.status;
    if (h_len) *h_len = st.len[0];
    return CASS_OK;
}

extern "C" int cass_session_lens(void* session, int32_t* h_lens, void* stream_) {
    if (!session || !h_lens) return CASS_ERR_INVALID_ARG;
    Session* s = (Session*)session;
    cudaStream_t stream = (cudaStream_t)stream_;
    DevState st;
    CASS_CUDA_CHECK(cudaMemcpyAsync(&st, s->st, sizeof(st), cudaMemcpyDeviceToHost, stream));
    CASS_CUDA_CHECK(cudaStreamSynchronize(stream));
    for (int b = 0; b < s->B; ++b) h_lens[b] = st.len[b];
    return CASS_OK;
}

extern "C" int cass_session_rows(const cass_model_desc* desc) {
    if (!desc || desc->max_batch < 1 || desc->gamma_max < 0) return CASS_ERR_INVALID_ARG;
    if (desc->max_batch * (desc->gamma_max + 1) > kMaxRows) return CASS_ERR_INVALID_ARG;
    return row_capacity(*desc);
}

extern "C" int cass_calib_enable(void* session, int on, void* stream_) {
    if (!session) return CASS_ERR_INVALID_ARG;
    Session* s = (Session*)session;
    int32_t v = on ? 1 : 0;
    CASS_CUDA_CHECK(cudaMemcpyAsync(&s->st->calib_on, &v, 4, cudaMemcpyHostToDevice, (cudaStream_t)stream_));
    CASS_CUDA_CHECK(cudaStreamSynchronize((cudaStream_t)stream_));
    s->calib_host = on != 0;
    return CASS_OK;
}

extern "C" size_t cass_calib_norms_count(const cass_model_desc* d) {
    if (!d) return 0;
    int kmax = d->hidden;
    if (d->ffn > kmax) kmax = d->ffn;
    if (d->n_q_heads * d->head_dim > kmax) kmax = d->n_q_heads * d->head_dim;
    return (size_t)d->n_layers * 4 * kmax + d->hidden;
}

extern "C" int cass_calib_norms(void* session, float* norms_out, void* stream_) {
    if (!session || !norms_out) return CASS_ERR_INVALID_ARG;
    Session* s = (Session*)session;
    return launch_sqrt(s->calib_all, norms_out, s->calib_count, (cudaStream_t)stream_);
}

extern "C" int cass_set_len(void* session, int len, void* stream_) {
    if (!session) return CASS_ERR_INVALID_ARG;
    Session* s = (Session*)session;
    if (len < 0 || len + kMaxVerifyRows > s->d.max_seq) return CASS_ERR_INVALID_ARG;      // room for one more call's rows
    int32_t v[2 * kMaxBatch];
    for (int b = 0; b < kMaxBatch; ++b) { v[b] = len; v[kMaxBatch + b] = 0; }
    static_assert(offsetof(DevState, inflight) == sizeof(int32_t) * kMaxBatch, "len[] then inflight[]");
    CASS_CUDA_CHECK(cudaMemcpyAsync(s->st->len, v, sizeof(v), cudaMemcpyHostToDevice, (cudaStream_t)stream_));
    CASS_CUDA_CHECK(cudaStreamSynchronize((cudaStream_t)stream_));
    s->drafts_pending = 0;
    return CASS_OK;
}

extern "C" int cass_set_lens(void* session, const int32_t* h_lens, void* stream_) {
    if (!session || !h_lens) return CASS_ERR_INVALID_ARG;
    Session* s = (Session*)session;
    int32_t v[2 * kMaxBatch] = {0};
    for (int b = 0; b < s->B; ++b) {
        if (h_lens[b] < 0 || h_lens[b] + kMaxVerifyRows > s->d.max_seq) return CASS_ERR_INVALID_ARG;
        v[b] = h_lens[b];
    }
    CASS_CUDA_CHECK(cudaMemcpyAsync(s->st->len, v, sizeof(v), cudaMemcpyHostToDevice, (cudaStream_t)stream_));
    CASS_CUDA_CHECK(cudaStreamSynchronize((cudaStream_t)stream_));
    s->drafts_pending = 0;
    return CASS_OK;
}

extern "C" int cass_kv_append(void* session, int seq, int layer, const void* K_bf16, const void* V_bf16, int start_pos,
                              int n_new, int flags, void* stream_) {
    if (!session || !K_bf16 || !V_bf16) return CASS_ERR_INVALID_ARG;
    Session* s = (Session*)session;
    if (seq < 0 || seq >= s->B || layer < 0 || layer >= s->d.n_layers || start_pos < 0 || n_new < 0 ||
        start_pos + n_new > s->d.max_seq)
        return CASS_ERR_INVALID_ARG;
    if (!(flags & (CASS_KV_BF16 | CASS_KV_COMPRESSED))) return CASS_ERR_INVALID_ARG;
    LayerDev& L = s->layers[layer];
    return launch_kv_append(s->kg, L.ck, L.cv, L.kc, L.vc, (const uint16_t*)K_bf16, (const uint16_t*)V_bf16,
                            s->kg.n_kv * s->kg.d, start_pos, 0, n_new, flags, s->st, seq, 1, (cudaStream_t)stream_);
}

extern "C" int cass_kv_build_codebook(void* session, int n_tokens, void* stream_) {
    if (!session) return CASS_ERR_INVALID_ARG;
    Session* s = (Session*)session;
    if (n_tokens < 0 || n_tokens > s->d.max_seq) return CASS_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)stream_;
    const size_t ss = s->kg.seq_stride;
    for (auto& L : s->layers)
        for (int b = 0; b < s->B; ++b) {       // every sequence has its own codebooks, built from its own prompt
            const uint16_t *kc = of_seq(L.kc, b, ss), *vc = of_seq(L.vc, b, ss);
            int rc = launch_kv_codebook(s->kg, of_seq(L.ck, b, ss), of_seq(L.cv, b, ss), kc, vc, n_tokens, stream);
            if (rc) return rc;
            rc = launch_kv_append(s->kg, L.ck, L.cv, L.kc, L.vc, kc, vc, s->kg.n_kv * s->kg.d, 0, 0, n_tokens,
                                  CASS_KV_COMPRESSED, s->st, b, 1, stream);
            if (rc) return rc;
        }
    s->codebooks_ready = true;
    return CASS_OK;
}

extern "C" int cass_kv_query(void* session, int seq, int layer, int kind, int head, cass_kv_view* v) {
    if (!session || !v) return CASS_ERR_INVALID_ARG;
    Session* s = (Session*)session;
    if (seq < 0 || seq >= s->B || layer < 0 || layer >= s->d.n_layers || kind < 0 || kind > 1 || head < 0 || head >= s->kg.n_kv)
        return CASS_ERR_INVALID_ARG;
    const KvGeom& g = s->kg;
    LayerDev& L = s->layers[layer];
    const KvComp c = of_seq(kind ? L.cv : L.ck, seq, g.seq_stride);
    v->fixed = c.fixed + (size_t)head * g.n_blocks * g.wpt * 32;
    v->arena = c.arena + (size_t)head * g.arena_words;
    v->offsets = c.off + (size_t)head * (g.max_seq + 1);
    v->codebook = c.rank_to_exp;
    v->k_or_v_bf16 = of_seq(kind ? L.vc : L.kc, seq, g.seq_stride);
    v->fixed_words_per_token = g.wpt;
    v->bitmap_words = g.bm_words;
    v->arena_words = g.arena_words;
    return CASS_OK;
}

extern "C" int cass_draft_attention(void* session, int layer, const void* q_bf16, void* out_bf16, void* stream_) {
    if (!session || !q_bf16 || !out_bf16) return CASS_ERR_INVALID_ARG;
    Session* s = (Session*)session;
    if (layer < 0 || layer >= s->d.n_layers) return CASS_ERR_INVALID_ARG;
    LayerDev& L = s->layers[layer];
    return launch_draft_attn(s->kg, L.ck, L.cv, (const uint16_t*)q_bf16, s->d.n_q_heads * s->d.head_dim, s->d.n_q_heads, s->B,
                             s->st, s->asc, (uint16_t*)out_bf16, (cudaStream_t)stream_);
}

extern "C" int cass_debug_activation(void* session, int which, const void** d_ptr, int* h_rows, int* h_cols) {
    if (!session || !d_ptr) return CASS_ERR_INVALID_ARG;
    Session* s = (Session*)session;
    if (which == 0) { *d_ptr = s->h; if (h_cols) *h_cols = s->d.hidden; }
    else if (which == 1) { *d_ptr = s->attn; if (h_cols) *h_cols = s->d.n_q_heads * s->d.head_dim; }
    else if (which == 2) { *d_ptr = s->qkv; if (h_cols) *h_cols = s->qkv_dim; }
    else return CASS_ERR_INVALID_ARG;
    if (h_rows) *h_rows = s->R;
    return CASS_OK;
}

#define RC(expr) do { int _rc = (expr); if (_rc) return _rc; } while (0)

extern "C" int cass_verify(void* session, const int32_t* toks, int g, int32_t* target_argmax, float* logits_opt,
                           void* stream_) {
    if (!session || !toks || !target_argmax) return CASS_ERR_INVALID_ARG;
    Session* s = (Session*)session;
    const int rps = g + 1, B = s->B, bn = s->R;      // rows per sequence; the MMA's token columns are fixed per session
    const int rows = B * rps;
    if (g < 0 || rps > kMaxVerifyRows || rows > s->R) return CASS_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream_;
    const cass_model_desc& d = s->d;
    auto vparts = [&](int n, int k) { return verify_gemm_partials(s->vg_partial, n, k, bn); };
    const bool fused = rope_kv_fusable(s->kg);       // RoPE and the KV append in one kernel
    // tensor-core attention where the shape allows (head_dim 128, rows x group <= 64); CASS_SIMT_VERIFY_ATTN=1 keeps
    // the fp32-pipe kernel.  For a given model shape every decode call of a session takes the same path.
    static const bool simt_env = [] { const char* e = std::getenv("CASS_SIMT_VERIFY_ATTN"); return e && e[0] == '1'; }();
    const int grp = d.n_q_heads / d.n_kv_heads;
    // decode calls (rps <= gamma_max + 1) are classed by gamma_max, so that plain and speculative decoding agree
    const bool attn_tc = !simt_env && verify_attn_tc_usable(s->kg, rps <= d.gamma_max + 1 ? d.gamma_max + 1 : rps, d.n_q_heads);
    // decode calls (rps <= gamma_max + 1) all use the column count the session's gamma_max needs; longer prefill chunks 64
    const int np_cols = (rps <= d.gamma_max + 1 && (d.gamma_max + 1) * grp <= 32) ? 32 : 64;
    const int qd = d.n_q_heads * d.head_dim;
    // The matrix a projection multiplies with: the caller's bf16 copy, or -- Sec. 4.1 target inference -- the exact
    // reconstruction from speculation + verification data, rebuilt into the session's scratch right before its use.
    int w_rc = CASS_OK;
    auto weight = [&](const void* bf16, const void* blob, const cass_blob_info& bi, const void* vd) -> const uint16_t* {
        if (!s->from_parts) return (const uint16_t*)bf16;
        const int rc = cass_decode_full(blob, &bi, vd, s->vscratch, stream_);
        if (rc) w_rc = rc;
        return s->vscratch;
    };
    RC(launch_embed(toks, 1, (const uint16_t*)s->embed, s->h, rows, d.hidden, st));
    RC(launch_rmsnorm(s->h, (const uint16_t*)s->layers[0].w.norm_attn, s->xn, rows, d.hidden, d.rms_eps, st));
    const int kv_flags = CASS_KV_BF16 | (s->codebooks_ready ? CASS_KV_COMPRESSED : 0);
    const bool calib = s->calib_host;           // the accumulation kernels are only launched while calibration is on
    int32_t* status = &s->st->status;
    // every projection leaves fp32 split-K parts in vg_partial; the kernel that consumes the projection adds them
    for (int l = 0; l < d.n_layers; ++l) {
        LayerDev& L = s->layers[l];
        if (calib) RC(launch_calib_accum(s->xn, rows, d.hidden, L.calib[0], s->st, st));
        RC(launch_verify_gemm(weight(L.w.wqkv, L.blob[0], L.bi[0], L.vdata[0]), s->xn, rows, bn, s->qkv_dim, d.hidden, s->vg_partial, nullptr, nullptr, status, st, s->from_parts ? 0 : 1));
        if (fused) {
            RC(launch_rope_kv_append(s->kg, L.ck, L.cv, L.kc, L.vc, vparts(s->qkv_dim, d.hidden), s->cos_t, s->sin_t, s->qkv,
                                     d.n_q_heads, 0, rps, kv_flags, s->st, B, st));
        } else {
            RC(launch_qkv_rope(s->qkv, vparts(s->qkv_dim, d.hidden), s->cos_t, s->sin_t, s->st, 0, rows, rps,
                               d.n_q_heads, d.n_kv_heads, d.head_dim, st));
            RC(launch_kv_append(s->kg, L.ck, L.cv, L.kc, L.vc, s->qkv + qd, s->qkv + qd + d.n_kv_heads * d.head_dim, s->qkv_dim,
                                -1, 0, rps, kv_flags, s->st, 0, B, st));
        }
        if (attn_tc) RC(launch_verify_attn_tc(s->kg, L.kc, L.vc, s->qkv, B, rps, d.n_q_heads, np_cols, s->st, s->asc, s->attn, status, st));
        else RC(launch_verify_attn(s->kg, L.kc, L.vc, s->qkv, B, rps, d.n_q_heads, s->st, s->asc, s->attn, st));
        if (calib) RC(launch_calib_accum(s->attn, rows, qd, L.calib[1], s->st, st));
        RC(launch_verify_gemm(weight(L.w.wo, L.blob[1], L.bi[1], L.vdata[1]), s->attn, rows, bn, d.hidden, qd, s->vg_partial, nullptr, nullptr, status, st, s->from_parts ? 0 : 1));
        RC(launch_residual_rmsnorm(s->h, nullptr, vparts(d.hidden, qd), (const uint16_t*)L.w.norm_ffn, s->xn,
                                   rows, d.hidden, d.rms_eps, st));
        if (calib) RC(launch_calib_accum(s->xn, rows, d.hidden, L.calib[2], s->st, st));
        RC(launch_verify_gemm(weight(L.w.wgu, L.blob[2], L.bi[2], L.vdata[2]), s->xn, rows, bn, 2 * d.ffn, d.hidden, s->vg_partial, nullptr, nullptr, status, st, s->from_parts ? 0 : 1));
        RC(launch_swiglu(nullptr, vparts(2 * d.ffn, d.hidden), s->act, rows, d.ffn, st));
        if (calib) RC(launch_calib_accum(s->act, rows, d.ffn, L.calib[3], s->st, st));
        RC(launch_verify_gemm(weight(L.w.wd, L.blob[3], L.bi[3], L.vdata[3]), s->act, rows, bn, d.hidden, d.ffn, s->vg_partial, nullptr, nullptr, status, st, s->from_parts ? 0 : 1));
        const uint16_t* next_gain = (const uint16_t*)(l + 1 < d.n_layers ? s->layers[l + 1].w.norm_attn : s->norm_final);
        RC(launch_residual_rmsnorm(s->h, nullptr, vparts(d.hidden, d.ffn), next_gain, s->xn, rows, d.hidden,
                                   d.rms_eps, st));
    }
    if (calib) RC(launch_calib_accum(s->xn, rows, d.hidden, s->calib_lm, s->st, st));
    RC(launch_verify_gemm(weight(s->lm_head, s->lm_blob, s->lm_bi, s->lm_vdata), s->xn, rows, bn, d.vocab, d.hidden, s->vg_partial, nullptr, nullptr, status, st, s->from_parts ? 0 : 1));
    RC(launch_argmax(nullptr, vparts(d.vocab, d.hidden), rows, d.vocab, target_argmax, 1, logits_opt,
                     s->argmax_val, s->argmax_tmp, s->st, 0, st));
    return w_rc;
}

extern "C" int cass_draft_step(void* session, const int32_t* tok_in, int32_t* tok_out, int tok_stride, float* logits_opt,
                               void* stream_) {
    if (!session || !tok_in || !tok_out || tok_stride < 1) return CASS_ERR_INVALID_ARG;
    Session* s = (Session*)session;
    if (!s->have_blobs || !s->codebooks_ready) return CASS_ERR_INVALID_ARG;
    // a drafted token sits at position len + (drafts since the last accept); more than gamma_max of them would leave
    // the rows a verification call can take and, at the end of a cache, the cache itself
    if (s->drafts_pending >= s->d.gamma_max) return CASS_ERR_INVALID_ARG;
    s->drafts_pending += 1;
    cudaStream_t st = (cudaStream_t)stream_;
    const cass_model_desc& d = s->d;
    const int qd = d.n_q_heads * d.head_dim;
    int32_t* status = &s->st->status;
    const int B = s->B;
    auto draftp = [&](const cass_blob_info& b) { return draft_gemv_partials(s->partial, b); };
    const bool fused = rope_kv_fusable(s->kg);
    RC(launch_embed(tok_in, tok_stride, (const uint16_t*)s->embed, s->h, B, d.hidden, st));
    RC(launch_rmsnorm(s->h, (const uint16_t*)s->layers[0].w.norm_attn, s->xn, B, d.hidden, d.rms_eps, st));
    for (int l = 0; l < d.n_layers; ++l) {
        LayerDev& L = s->layers[l];
        RC(launch_draft_gemv(L.blob[0], L.bi[0], s->xn, B, s->partial, status, st));
        if (fused) {
            RC(launch_rope_kv_append(s->kg, L.ck, L.cv, L.kc, L.vc, draftp(L.bi[0]), s->cos_t, s->sin_t, s->qkv, d.n_q_heads, 1, 1,
                                     CASS_KV_COMPRESSED, s->st, B, st));
        } else {
            RC(launch_qkv_rope(s->qkv, draftp(L.bi[0]), s->cos_t, s->sin_t, s->st, 1, B, 1, d.n_q_heads, d.n_kv_heads, d.head_dim, st));
            RC(launch_kv_append(s->kg, L.ck, L.cv, L.kc, L.vc, s->qkv + qd, s->qkv + qd + d.n_kv_heads * d.head_dim, s->qkv_dim,
                                -1, 1, 1, CASS_KV_COMPRESSED, s->st, 0, B, st));
        }
        RC(launch_draft_attn(s->kg, L.ck, L.cv, s->qkv, s->qkv_dim, d.n_q_heads, B, s->st, s->asc, s->attn, st));
        RC(launch_draft_gemv(L.blob[1], L.bi[1], s->attn, B, s->partial, status, st));
        RC(launch_residual_rmsnorm(s->h, nullptr, draftp(L.bi[1]), (const uint16_t*)L.w.norm_ffn, s->xn, B, d.hidden, d.rms_eps, st));
        RC(launch_draft_gemv(L.blob[2], L.bi[2], s->xn, B, s->partial, status, st));
        RC(launch_swiglu(nullptr, draftp(L.bi[2]), s->act, B, d.ffn, st));
        RC(launch_draft_gemv(L.blob[3], L.bi[3], s->act, B, s->partial, status, st));
        const uint16_t* next_gain = (const uint16_t*)(l + 1 < d.n_layers ? s->layers[l + 1].w.norm_attn : s->norm_final);
        RC(launch_residual_rmsnorm(s->h, nullptr, draftp(L.bi[3]), next_gain, s->xn, B, d.hidden, d.rms_eps, st));
    }
    RC(launch_draft_gemv(s->lm_blob, s->lm_bi, s->xn, B, s->partial, status, st));
    RC(launch_argmax(nullptr, draftp(s->lm_bi), B, d.vocab, tok_out, tok_stride, logits_opt, s->argmax_val, s->argmax_tmp, s->st, 1, st));
    return CASS_OK;
}

extern "C" int cass_accept(void* session, const int32_t* draft, int draft_stride, const int32_t* target_argmax, int g,
                           int32_t* n_accepted, int32_t* out_tokens, int32_t* next_tok, int next_stride, void* stream_) {
    if (!session || !target_argmax || !n_accepted || !out_tokens || (g > 0 && !draft)) return CASS_ERR_INVALID_ARG;
    if (draft_stride < g || next_stride < 1) return CASS_ERR_INVALID_ARG;
    Session* s = (Session*)session;
    if (g < 0 || g + 1 > kMaxVerifyRows) return CASS_ERR_INVALID_ARG;
    s->drafts_pending = 0;
    return launch_accept(s->st, s->B, draft, draft_stride, target_argmax, g, n_accepted, out_tokens, next_tok, next_stride,
                         (cudaStream_t)stream_);
}

extern "C" int cass_accept_sampling(void* session, int n_seq, const int32_t* draft, int draft_stride, const float* p_target,
                                    const float* q_draft, int vocab, const float* r_uniform, const float* u_uniform, int g,
                                    int32_t* n_accepted, int32_t* out_tokens, int32_t* next_tok, int next_stride,
                                    void* stream_) {
    if (!p_target || !u_uniform || !n_accepted || !out_tokens || (g > 0 && (!draft || !q_draft || !r_uniform)))
        return CASS_ERR_INVALID_ARG;
    if (g < 0 || g + 1 > kMaxVerifyRows || draft_stride < g || next_stride < 1 || vocab <= 0 || n_seq < 1)
        return CASS_ERR_INVALID_ARG;
    DevState* st = nullptr;
    if (session) {
        Session* s = (Session*)session;
        if (n_seq != s->B || vocab != s->d.vocab) return CASS_ERR_INVALID_ARG;
        s->drafts_pending = 0;
        st = s->st;
    }
    return launch_accept_sampling(st, n_seq, draft, draft_stride, p_target, q_draft, vocab, r_uniform, u_uniform, g, n_accepted,
                                  out_tokens, next_tok, next_stride, (cudaStream_t)stream_);
}

extern "C" size_t cass_verify_from_parts_scratch_bytes(const cass_model_desc* d) {
    if (!d) return 0;
    const size_t qkv = (size_t)(d->n_q_heads + 2 * d->n_kv_heads) * d->head_dim;
    size_t m = qkv * d->hidden;
    const size_t c[4] = {(size_t)d->hidden * d->n_q_heads * d->head_dim, (size_t)2 * d->ffn * d->hidden, (size_t)d->hidden * d->ffn,
                         (size_t)d->vocab * d->hidden};
    for (size_t v : c) if (v > m) m = v;
    return m * 2;
}

extern "C" int cass_session_verify_from_parts(void* session, const cass_model_vdata* vdata, void* scratch_bf16, size_t scratch_bytes) {
    if (!session) return CASS_ERR_INVALID_ARG;
    Session* s = (Session*)session;
    if (!vdata) { s->from_parts = false; return CASS_OK; }                 // back to the caller's bf16 matrices
    if (!vdata->h_layers || !vdata->lm_head || !scratch_bf16 || ((uintptr_t)scratch_bf16 & 15)) return CASS_ERR_INVALID_ARG;
    if (!s->have_blobs) return CASS_ERR_INVALID_ARG;                       // the speculation data comes first
    if (scratch_bytes < cass_verify_from_parts_scratch_bytes(&s->d)) return CASS_ERR_CAPACITY;
    if (s->lm_bi.mode != 1) return CASS_ERR_UNSUPPORTED;                   // Cassandra-2 speculation data has no exact complement here
    for (int l = 0; l < s->d.n_layers; ++l) {
        const cass_layer_vdata& v = vdata->h_layers[l];
        const void* p[4] = {v.wqkv, v.wo, v.wgu, v.wd};
        for (int i = 0; i < 4; ++i) {
            if (!p[i]) return CASS_ERR_INVALID_ARG;
            if (s->layers[l].bi[i].mode != 1) return CASS_ERR_UNSUPPORTED;
            s->layers[l].vdata[i] = p[i];
        }
    }
    s->lm_vdata = vdata->lm_head;
    s->vscratch = (uint16_t*)scratch_bf16;
    s->from_parts = true;
    return CASS_OK;
}
