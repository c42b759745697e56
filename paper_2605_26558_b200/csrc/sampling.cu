// Sampling-based acceptance (Sec. 2.2, Eq. 1: rejection sampling against the draft's distribution) and the two
// small operators it needs around it: softmax of logits at a temperature and an inverse-CDF draw.  Random numbers
// are inputs (uniform in [0, 1)); nothing here generates them.
#include <cfloat>

#include "kernels.cuh"

namespace cass {

constexpr int kSampleThreads = 256;

__device__ __forceinline__ float block_reduce(float v, bool is_max, float* s_red) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    v = is_max ? warp_max(v) : warp_sum(v);
    __syncthreads();                                      // s_red may still be read from a previous call
    if (lane == 0) s_red[warp] = v;
    __syncthreads();
    float r = s_red[0];
    for (int w = 1; w < nw; ++w) r = is_max ? fmaxf(r, s_red[w]) : r + s_red[w];      // fixed order
    return r;
}

// probs[r][v] = exp((logits[r][v] - max) / T) / sum
__global__ void __launch_bounds__(kSampleThreads) k_softmax_rows(const float* __restrict__ logits, int vocab, float inv_t,
                                                                 float* __restrict__ probs) {
    __shared__ float s_red[kSampleThreads / 32];
    pdl_wait();
    const float* in = logits + (size_t)blockIdx.x * vocab;
    float* out = probs + (size_t)blockIdx.x * vocab;
    float m = -FLT_MAX;
    for (int v = threadIdx.x; v < vocab; v += blockDim.x) m = fmaxf(m, in[v]);
    m = block_reduce(m, true, s_red);
    float sum = 0.f;
    for (int v = threadIdx.x; v < vocab; v += blockDim.x) {
        const float e = __expf((in[v] - m) * inv_t);
        out[v] = e;
        sum += e;
    }
    sum = block_reduce(sum, false, s_red);
    const float inv = 1.f / sum;
    for (int v = threadIdx.x; v < vocab; v += blockDim.x) out[v] *= inv;
}

// Inverse-CDF draw over weight(v), v in [0, vocab): the lowest index whose cumulative weight exceeds u * total.
// Thread i owns the contiguous indices [i * per, (i + 1) * per); segment sums are scanned in thread order, so the
// result does not depend on scheduling.  Returns the index to every thread (total <= 0: vocab - 1... callers test).
template <class W>
__device__ int block_inverse_cdf(W weight, int vocab, float u, float* s_seg, int* s_pick, float* total_out) {
    const int per = ceil_div(vocab, (int)blockDim.x);
    const int v0 = threadIdx.x * per, v1 = min(vocab, v0 + per);
    float seg = 0.f;
    for (int v = v0; v < v1; ++v) seg += weight(v);
    __syncthreads();
    s_seg[threadIdx.x] = seg;
    if (threadIdx.x == 0) *s_pick = vocab - 1;
    __syncthreads();
    if (threadIdx.x == 0) {                               // exclusive scan of the segment sums, in order
        float run = 0.f;
        for (int i = 0; i < (int)blockDim.x; ++i) { const float s = s_seg[i]; s_seg[i] = run; run += s; }
        s_seg[blockDim.x] = run;
    }
    __syncthreads();
    const float total = s_seg[blockDim.x];
    const float target = u * total;
    const float before = s_seg[threadIdx.x];
    const float after = threadIdx.x + 1 < (int)blockDim.x ? s_seg[threadIdx.x + 1] : total;
    if (before <= target && target < after) {             // exactly one thread: the segment sums are non-negative
        float run = before;
        int pick = v1 - 1;
        for (int v = v0; v < v1; ++v) {
            run += weight(v);
            if (run > target) { pick = v; break; }
        }
        *s_pick = pick;
    }
    __syncthreads();
    if (total_out) *total_out = total;
    return *s_pick;
}

__global__ void __launch_bounds__(kSampleThreads) k_sample_rows(const float* __restrict__ probs, int vocab,
                                                                const float* __restrict__ u, int32_t* __restrict__ tokens,
                                                                int tok_stride) {
    __shared__ float s_seg[kSampleThreads + 1];
    __shared__ int s_pick;
    pdl_wait();
    const float* p = probs + (size_t)blockIdx.x * vocab;
    const int pick = block_inverse_cdf([&](int v) { return p[v]; }, vocab, u[blockIdx.x], s_seg, &s_pick, nullptr);
    if (threadIdx.x == 0) tokens[(size_t)blockIdx.x * tok_stride] = pick;
}

// One block per sequence b.  Eq. 1: n = min({i-1 : r_i > p_i(x_i) / q_i(x_i)} U {g}); then one more token: from the
// normalised positive part of p_{n+1} - q_{n+1} after a rejection, from p_{g+1} after full acceptance.
__global__ void __launch_bounds__(kSampleThreads) k_accept_sampling(DevState* st, const int32_t* __restrict__ draft, int draft_stride,
                                                                    const float* __restrict__ p, const float* __restrict__ q, int vocab,
                                                                    const float* __restrict__ r, const float* __restrict__ u, int g,
                                                                    int32_t* n_acc, int32_t* out_tokens, int32_t* next_tok,
                                                                    int next_stride) {
    __shared__ float s_seg[kSampleThreads + 1];
    __shared__ int s_pick, s_n;
    pdl_wait();
    const int b = blockIdx.x;
    draft += (size_t)b * draft_stride;
    p += (size_t)b * (g + 1) * vocab;
    q += (size_t)b * g * vocab;
    r += (size_t)b * g;
    if (threadIdx.x == 0) {
        int n = 0;
        while (n < g) {
            const int x = draft[n];
            const bool in_range = x >= 0 && x < vocab;
            // r > p/q, written without the division (q(x) = 0 cannot have been drawn; it rejects unless p(x) = 0 too)
            if (!in_range || r[n] * q[(size_t)n * vocab + x] > p[(size_t)n * vocab + x]) break;
            ++n;
        }
        s_n = n;
    }
    __syncthreads();
    const int n = s_n;
    const float* pn = p + (size_t)n * vocab;
    const float* qn = q + (size_t)n * vocab;              // read only when n < g
    float total = 0.f;
    int extra;
    if (n < g) {
        extra = block_inverse_cdf([&](int v) { return fmaxf(pn[v] - qn[v], 0.f); }, vocab, u[b], s_seg, &s_pick, &total);
        if (!(total > 0.f)) extra = block_inverse_cdf([&](int v) { return pn[v]; }, vocab, u[b], s_seg, &s_pick, nullptr);
    } else {
        extra = block_inverse_cdf([&](int v) { return pn[v]; }, vocab, u[b], s_seg, &s_pick, nullptr);
    }
    if (threadIdx.x != 0) return;
    out_tokens += (size_t)b * (g + 1);
    for (int i = 0; i < n; ++i) out_tokens[i] = draft[i];
    out_tokens[n] = extra;
    for (int i = n + 1; i <= g; ++i) out_tokens[i] = -1;
    n_acc[b] = n;
    if (next_tok) next_tok[(size_t)b * next_stride] = extra;
    if (st && b < kMaxBatch) {                            // the same length rule as the greedy accept
        if (st->len[b] + n + 1 + kMaxVerifyRows > st->max_seq) atomicCAS(&st->status, 0, CASS_ERR_CAPACITY);
        else st->len[b] += n + 1;
        st->inflight[b] = 0;
    }
}

int launch_softmax(const float* logits, int rows, int vocab, float temperature, float* probs, cudaStream_t s) {
    CASS_PDL_LAUNCH(k_softmax_rows, dim3(rows), dim3(kSampleThreads), 0, s, logits, vocab, 1.f / temperature, probs);
    return CASS_OK;
}

int launch_sample(const float* probs, int rows, int vocab, const float* u, int32_t* tokens, int tok_stride, cudaStream_t s) {
    CASS_PDL_LAUNCH(k_sample_rows, dim3(rows), dim3(kSampleThreads), 0, s, probs, vocab, u, tokens, tok_stride);
    return CASS_OK;
}

int launch_accept_sampling(DevState* st, int n_seq, const int32_t* draft, int draft_stride, const float* p, const float* q,
                           int vocab, const float* r, const float* u, int g, int32_t* n_acc, int32_t* out_tokens,
                           int32_t* next_tok, int next_stride, cudaStream_t s) {
    CASS_PDL_LAUNCH(k_accept_sampling, dim3(n_seq), dim3(kSampleThreads), 0, s, st, draft, draft_stride, p, q, vocab, r, u, g,
                    n_acc, out_tokens, next_tok, next_stride);
    return CASS_OK;
}

}  // namespace cass

using namespace cass;

extern "C" int cass_softmax(const float* logits, int rows, int vocab, float temperature, float* probs, void* stream) {
    if (!logits || !probs || rows < 0 || vocab <= 0 || !(temperature > 0.f)) return CASS_ERR_INVALID_ARG;
    if (rows == 0) return CASS_OK;
    return launch_softmax(logits, rows, vocab, temperature, probs, (cudaStream_t)stream);
}

extern "C" int cass_sample(const float* probs, int rows, int vocab, const float* u, int32_t* tokens, int tok_stride,
                           void* stream) {
    if (!probs || !u || !tokens || rows < 0 || vocab <= 0 || tok_stride < 1) return CASS_ERR_INVALID_ARG;
    if (rows == 0) return CASS_OK;
    return launch_sample(probs, rows, vocab, u, tokens, tok_stride, (cudaStream_t)stream);
}
