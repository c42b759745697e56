// Small per-token operators of the decoder layer (Sec. 2.1): embedding gather, RMSNorm, RoPE, SwiGLU, residual
// add, greedy argmax, and the greedy accept / rollback step (Sec. 2.2).  Activations are bf16 between
// operators; arithmetic inside an operator is fp32.
#include "kernels.cuh"

namespace cass {

__global__ void k_rope_table(float* __restrict__ cos_t, float* __restrict__ sin_t, int max_seq, int half, float theta) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)max_seq * half) return;
    int pos = (int)(i / half), j = (int)(i % half);
    double inv = pow((double)theta, -2.0 * (double)j / (double)(2 * half));
    double ang = (double)pos * inv;
    cos_t[i] = (float)cos(ang);
    sin_t[i] = (float)sin(ang);
}

__global__ void k_embed(const int32_t* __restrict__ toks, int tok_stride, const uint16_t* __restrict__ embed,
                        uint16_t* __restrict__ h, int hidden) {
    pdl_early<0>();
    pdl_wait();
    int r = blockIdx.x;
    const uint16_t* src = embed + (size_t)toks[(size_t)r * tok_stride] * hidden;
    uint16_t* dst = h + (size_t)r * hidden;
    if ((hidden & 7) == 0 && (((uintptr_t)src | (uintptr_t)dst) & 15) == 0) {
        // 16 bytes per load, two loads in flight per thread: the row costs one or two round trips
        const uint4* s4 = reinterpret_cast<const uint4*>(src);
        uint4* d4 = reinterpret_cast<uint4*>(dst);
        const int n16 = hidden / 8;
        for (int i = threadIdx.x; i < n16; i += 2 * blockDim.x) {
            const int j = i + blockDim.x;
            const uint4 a = s4[i];
            uint4 b = make_uint4(0u, 0u, 0u, 0u);
            if (j < n16) b = s4[j];
            d4[i] = a;
            if (j < n16) d4[j] = b;
        }
        return;
    }
    for (int i = threadIdx.x; i < hidden; i += blockDim.x) dst[i] = src[i];
}

__device__ __forceinline__ float block_sum(float v, float* s_red) {
    v = warp_sum(v);
    int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    __syncthreads();
    if (lane == 0) s_red[warp] = v;
    __syncthreads();
    float t = 0.f;
    for (int i = 0; i < nw; ++i) t += s_red[i];
    return t;
}

// h (+= y) then out = h * rsqrt(mean(h^2) + eps) * gain, all rounded to bf16 where stored.  Four values per thread
// and iteration (16-byte loads of the fp32 partial sums); the updated values stay in registers for the second pass.
constexpr int kNormMaxIter = 8;          // hidden <= 8 * 4 * blockDim.x

template <int ITERS>          // rounds of 4 x blockDim.x values: hidden <= ITERS * 4 * blockDim.x
__global__ void __launch_bounds__(1024) k_residual_rmsnorm(uint16_t* __restrict__ h, const uint16_t* __restrict__ y_bf16,
                                                           Partials pp,
                                                           const uint16_t* __restrict__ gain, uint16_t* __restrict__ out,
                                                           int hidden, float eps) {
    __shared__ float s_red[32];
    // the gains are weights: they are requested ahead of the wait for the predecessor
    uint2 gvs[ITERS];
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
        const int i = threadIdx.x * 4 + it * (int)blockDim.x * 4;
        gvs[it] = (out && i < hidden) ? __ldg(reinterpret_cast<const uint2*>(gain + i)) : make_uint2(0u, 0u);
    }
    pdl_early<0>();
    pdl_wait();
    const int r = blockIdx.x;
    uint16_t* hr = h + (size_t)r * hidden;
    float vals[ITERS][4];
    float ss = 0.f;
    const int step = blockDim.x * 4;
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
        const int i = threadIdx.x * 4 + it * step;
        if (i < hidden) {
            const uint2 hv = *reinterpret_cast<const uint2*>(hr + i);
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            if (pp.p) acc = parts_sum4(pp, (size_t)r * pp.row_stride + i);       // requested before hv is first used: one round trip for both
            float v[4] = {__uint_as_float(hv.x << 16), __uint_as_float(hv.x & 0xFFFF0000u), __uint_as_float(hv.y << 16),
                          __uint_as_float(hv.y & 0xFFFF0000u)};
            if (y_bf16 || pp.p) {
                float y[4];
                if (pp.p) {
                    y[0] = round_bf16(acc.x); y[1] = round_bf16(acc.y); y[2] = round_bf16(acc.z); y[3] = round_bf16(acc.w);
                } else {
                    const uint2 yv = *reinterpret_cast<const uint2*>(y_bf16 + (size_t)r * hidden + i);
                    y[0] = __uint_as_float(yv.x << 16); y[1] = __uint_as_float(yv.x & 0xFFFF0000u);
                    y[2] = __uint_as_float(yv.y << 16); y[3] = __uint_as_float(yv.y & 0xFFFF0000u);
                }
#pragma unroll
                for (int q = 0; q < 4; ++q) v[q] = round_bf16(v[q] + y[q]);
                uint2 o;
                o.x = (uint32_t)float_to_bf16_bits(v[0]) | ((uint32_t)float_to_bf16_bits(v[1]) << 16);
                o.y = (uint32_t)float_to_bf16_bits(v[2]) | ((uint32_t)float_to_bf16_bits(v[3]) << 16);
                *reinterpret_cast<uint2*>(hr + i) = o;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) { vals[it][q] = v[q]; ss += v[q] * v[q]; }
        }
    }
    ss = block_sum(ss, s_red);
    const float inv = 1.0f / sqrtf(ss / (float)hidden + eps);
    if (out) {
#pragma unroll
        for (int it = 0; it < ITERS; ++it) {
            const int i = threadIdx.x * 4 + it * step;
            if (i < hidden) {
                const uint2 gv = gvs[it];
                const float gq[4] = {__uint_as_float(gv.x << 16), __uint_as_float(gv.x & 0xFFFF0000u), __uint_as_float(gv.y << 16),
                                     __uint_as_float(gv.y & 0xFFFF0000u)};
                uint32_t ob[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) ob[q] = float_to_bf16_bits(vals[it][q] * inv * gq[q]);
                uint2 o;
                o.x = ob[0] | (ob[1] << 16);
                o.y = ob[2] | (ob[3] << 16);
                *reinterpret_cast<uint2*>(out + (size_t)r * hidden + i) = o;
            }
        }
    }
}

__global__ void k_qkv_rope(uint16_t* __restrict__ qkv, Partials pp,
                           const float* __restrict__ cos_t, const float* __restrict__ sin_t,
                           const DevState* __restrict__ st, int use_inflight, int rps, int n_q, int n_kv, int d) {
    pdl_early<0>();
    pdl_wait();
    const int r = blockIdx.y, half = d / 2;
    const int qkv_dim = (n_q + 2 * n_kv) * d;
    const int b = r / rps;
    const int pos = st->len[b] + (use_inflight ? st->inflight[b] : 0) + r % rps;
    uint16_t* row = qkv + (size_t)r * qkv_dim;
    const int n_rot = (n_q + n_kv) * half;             // rotated pairs
    const int n_items = n_rot + n_kv * d;              // + plain v elements
    auto load = [&](int i) -> float {
        if (pp.p) {
            return round_bf16(parts_sum(pp, (size_t)r * pp.row_stride + i));
        }
        return bf16_bits_to_float(row[i]);
    };
    for (int it = blockIdx.x * blockDim.x + threadIdx.x; it < n_items; it += gridDim.x * blockDim.x) {
        if (it < n_rot) {
            int head = it / half, j = it % half;
            int ia = head * d + j, ib = ia + half;
            float a = load(ia), b = load(ib);
            float c = cos_t[(size_t)pos * half + j], s = sin_t[(size_t)pos * half + j];
            row[ia] = float_to_bf16_bits(a * c - b * s);
            row[ib] = float_to_bf16_bits(b * c + a * s);
        } else if (pp.p) {
            int i = (n_q + n_kv) * d + (it - n_rot);
            row[i] = float_to_bf16_bits(load(i));
        }
    }
}

__global__ void k_swiglu(const uint16_t* __restrict__ gu, Partials pp,
                         uint16_t* __restrict__ act, int ffn) {
    pdl_early<0>();
    pdl_wait();
    const int r = blockIdx.y;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < ffn; i += gridDim.x * blockDim.x) {
        float g, u;
        if (pp.p) {
            const size_t offs[2] = {(size_t)r * pp.row_stride + i, (size_t)r * pp.row_stride + ffn + i};
            const bool on2[2] = {true, true};
            float gu2[2];
            parts_sum_n<2>(pp, offs, on2, gu2);
            g = round_bf16(gu2[0]);
            u = round_bf16(gu2[1]);
        } else {
            g = bf16_bits_to_float(gu[(size_t)r * 2 * ffn + i]);
            u = bf16_bits_to_float(gu[(size_t)r * 2 * ffn + ffn + i]);
        }
        float silu = g / (1.0f + expf(-g));
        act[(size_t)r * ffn + i] = float_to_bf16_bits(silu * u);
    }
}

// Greedy token of each row, lowest index on ties, in two levels: slices of the vocabulary, then the slices' winners.
constexpr int kArgmaxSlices = 128;

__device__ __forceinline__ void argmax_combine(float& best, int& best_i, float ov, int oi) {
    if (ov > best || (ov == best && oi < best_i)) { best = ov; best_i = oi; }
}

__global__ void __launch_bounds__(256) k_argmax_part(const float* __restrict__ logits, Partials pp, int vocab, float* __restrict__ tmp_v,
                                                     int32_t* __restrict__ tmp_i, float* __restrict__ logits_copy) {
    __shared__ float s_v[8];
    __shared__ int s_i[8];
    pdl_early<0>();
    pdl_wait();
    const int r = blockIdx.y, nsl = gridDim.x;
    const int per = ceil_div(vocab, nsl);
    const int lo = blockIdx.x * per, hi = min(vocab, lo + per);
    float best = -INFINITY;
    int best_i = 0x7fffffff;
    for (int i = lo + threadIdx.x; i < hi; i += blockDim.x) {
        float v;
        if (pp.p) {
            v = parts_sum(pp, (size_t)r * pp.row_stride + i);
        } else {
            v = logits[(size_t)r * vocab + i];
        }
        if (logits_copy) logits_copy[(size_t)r * vocab + i] = v;
        argmax_combine(best, best_i, v, i);
    }
    for (int o = 16; o > 0; o >>= 1) {
        float ov = __shfl_xor_sync(0xffffffffu, best, o);
        int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
        argmax_combine(best, best_i, ov, oi);
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { s_v[warp] = best; s_i[warp] = best_i; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w) argmax_combine(best, best_i, s_v[w], s_i[w]);
        tmp_v[r * nsl + blockIdx.x] = best;
        tmp_i[r * nsl + blockIdx.x] = best_i;
    }
}

__global__ void __launch_bounds__(kArgmaxSlices) k_argmax_final(const float* __restrict__ tmp_v, const int32_t* __restrict__ tmp_i,
                                                                int nsl, int32_t* __restrict__ out, int out_stride, DevState* st,
                                                                int bump_inflight) {
    __shared__ float s_v[kArgmaxSlices / 32];
    __shared__ int s_i[kArgmaxSlices / 32];
    pdl_early<0>();
    pdl_wait();
    const int r = blockIdx.x;
    float best = -INFINITY;
    int best_i = 0x7fffffff;
    if ((int)threadIdx.x < nsl) { best = tmp_v[r * nsl + threadIdx.x]; best_i = tmp_i[r * nsl + threadIdx.x]; }
    for (int o = 16; o > 0; o >>= 1) {
        float ov = __shfl_xor_sync(0xffffffffu, best, o);
        int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
        argmax_combine(best, best_i, ov, oi);
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { s_v[warp] = best; s_i[warp] = best_i; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kArgmaxSlices / 32; ++w) argmax_combine(best, best_i, s_v[w], s_i[w]);
        out[(size_t)r * out_stride] = best_i == 0x7fffffff ? 0 : best_i;
        if (bump_inflight && r < kMaxBatch) {
            // the draft counter never passes the margin kept free at the end of a cache (positions len .. len + 15)
            if (st->inflight[r] < kMaxVerifyRows - 1) st->inflight[r] += 1;
            else atomicCAS(&st->status, 0, CASS_ERR_INVALID_ARG);
        }
    }
}

// Greedy acceptance: a = min({i-1 : draft_i != target_{i-1}} U {g}); emit draft_1..draft_a and target_a.
// One block per sequence b: draft[b * draft_stride + i], target[b][g+1] -> n_acc[b], out_tokens[b][g+1],
// next_tok[b * next_stride].
__global__ void k_accept(DevState* st, const int32_t* __restrict__ draft, int draft_stride, const int32_t* __restrict__ target, int g,
                         int32_t* n_acc, int32_t* out_tokens, int32_t* next_tok, int next_stride) {
    pdl_early<0>();
    pdl_wait();
    if (threadIdx.x != 0) return;
    const int b = blockIdx.x;
    draft += (size_t)b * draft_stride;
    target += (size_t)b * (g + 1);
    out_tokens += (size_t)b * (g + 1);
    n_acc += b;
    if (next_tok) next_tok += (size_t)b * next_stride;
    int a = 0;
    while (a < g && draft[a] == target[a]) ++a;
    for (int i = 0; i < a; ++i) out_tokens[i] = draft[i];
    out_tokens[a] = target[a];
    for (int i = a + 1; i <= g; ++i) out_tokens[i] = -1;
    *n_acc = a;
    if (next_tok) *next_tok = target[a];
    // Every later call touches positions up to len + 15 at most; a sequence that would come closer than that to
    // the end of its cache stops growing and the status word says so.
    if (st->len[b] + a + 1 + kMaxVerifyRows > st->max_seq) atomicCAS(&st->status, 0, CASS_ERR_CAPACITY);
    else st->len[b] += a + 1;
    st->inflight[b] = 0;
}

__global__ void k_calib_accum(const uint16_t* __restrict__ x, int rows, int cols, float* __restrict__ sumsq,
                              const DevState* __restrict__ st) {
    pdl_early<0>();
    pdl_wait();
    if (!st->calib_on) return;
    int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= cols) return;
    float acc = sumsq[c];
    for (int r = 0; r < rows; ++r) {
        float v = bf16_bits_to_float(x[(size_t)r * cols + c]);
        acc += v * v;
    }
    sumsq[c] = acc;
}

__global__ void k_sqrt(const float* __restrict__ in, float* __restrict__ out, size_t n) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = sqrtf(in[i]);
}

int launch_rope_table(float* cos_t, float* sin_t, int max_seq, int d, float theta, cudaStream_t s) {
    size_t n = (size_t)max_seq * (d / 2);
    k_rope_table<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(cos_t, sin_t, max_seq, d / 2, theta);
    CASS_LAUNCH_CHECK();
    return CASS_OK;
}

int launch_embed(const int32_t* toks, int tok_stride, const uint16_t* embed, uint16_t* h, int rows, int hidden, cudaStream_t s) {
    CASS_PDL_LAUNCH(k_embed, dim3(rows), dim3(256), 0, s, toks, tok_stride, embed, h, hidden);
    return CASS_OK;
}

static int norm_threads(int hidden) {
    int t = ceil_div(ceil_div(hidden, 4), 32) * 32;
    return t > 1024 ? 1024 : t;
}

static int norm_iters(int hidden, int threads) {
    const int it = ceil_div(hidden, 4 * threads);
    return it <= 1 ? 1 : (it <= 2 ? 2 : (it <= 4 ? 4 : 8));
}

int launch_residual_rmsnorm(uint16_t* h, const uint16_t* y_bf16, Partials pp,
                            const uint16_t* gain, uint16_t* out, int rows, int hidden, float eps, cudaStream_t s) {
    if (hidden % 4 || hidden > kNormMaxIter * 4 * 1024) return CASS_ERR_UNSUPPORTED;
    const int threads = norm_threads(hidden);
    switch (norm_iters(hidden, threads)) {
        case 1: CASS_PDL_LAUNCH(k_residual_rmsnorm<1>, dim3(rows), dim3(threads), 0, s, h, y_bf16, pp, gain, out, hidden, eps); break;
        case 2: CASS_PDL_LAUNCH(k_residual_rmsnorm<2>, dim3(rows), dim3(threads), 0, s, h, y_bf16, pp, gain, out, hidden, eps); break;
        case 4: CASS_PDL_LAUNCH(k_residual_rmsnorm<4>, dim3(rows), dim3(threads), 0, s, h, y_bf16, pp, gain, out, hidden, eps); break;
        default: CASS_PDL_LAUNCH(k_residual_rmsnorm<8>, dim3(rows), dim3(threads), 0, s, h, y_bf16, pp, gain, out, hidden, eps); break;
    }
    return CASS_OK;
}

int launch_rmsnorm(const uint16_t* h, const uint16_t* gain, uint16_t* out, int rows, int hidden, float eps, cudaStream_t s) {
    return launch_residual_rmsnorm(const_cast<uint16_t*>(h), nullptr, Partials{nullptr, 0, 0, 0}, gain, out, rows, hidden, eps, s);
}

int launch_qkv_rope(uint16_t* qkv, Partials pp, const float* cos_t, const float* sin_t,
                    const DevState* st, int use_inflight, int rows, int rps, int n_q, int n_kv, int d, cudaStream_t s) {
    int items = (n_q + n_kv) * (d / 2) + n_kv * d;
    dim3 grid(ceil_div(items, 256), rows);
    CASS_PDL_LAUNCH(k_qkv_rope, grid, dim3(256), 0, s, qkv, pp, cos_t, sin_t, st, use_inflight, rps, n_q, n_kv, d);
    return CASS_OK;
}

int launch_swiglu(const uint16_t* gu_bf16, Partials pp, uint16_t* act, int rows, int ffn,
                  cudaStream_t s) {
    dim3 grid(ceil_div(ffn, 256), rows);
    CASS_PDL_LAUNCH(k_swiglu, grid, dim3(256), 0, s, gu_bf16, pp, act, ffn);
    return CASS_OK;
}

int launch_argmax(const float* logits, Partials pp, int rows, int vocab, int32_t* out, int out_stride,
                  float* logits_copy, float* tmp_v, int32_t* tmp_i, DevState* st, int bump_inflight, cudaStream_t s) {
    int nsl = ceil_div(vocab, 1024);
    if (nsl > kArgmaxSlices) nsl = kArgmaxSlices;
    dim3 grid(nsl, rows);
    CASS_PDL_LAUNCH(k_argmax_part, grid, dim3(256), 0, s, logits, pp, vocab, tmp_v, tmp_i, logits_copy);
    CASS_PDL_LAUNCH(k_argmax_final, dim3(rows), dim3(kArgmaxSlices), 0, s, (const float*)tmp_v, (const int32_t*)tmp_i, nsl, out, out_stride, st, bump_inflight);
    return CASS_OK;
}

int launch_accept(DevState* st, int n_seq, const int32_t* draft, int draft_stride, const int32_t* target, int g, int32_t* n_acc,
                  int32_t* out_tokens, int32_t* next_tok, int next_stride, cudaStream_t s) {
    CASS_PDL_LAUNCH(k_accept, dim3(n_seq), dim3(32), 0, s, st, draft, draft_stride, target, g, n_acc, out_tokens, next_tok, next_stride);
    return CASS_OK;
}

int launch_calib_accum(const uint16_t* x, int rows, int cols, float* sumsq, const DevState* st, cudaStream_t s) {
    CASS_PDL_LAUNCH(k_calib_accum, dim3(ceil_div(cols, 256)), dim3(256), 0, s, x, rows, cols, sumsq, st);
    return CASS_OK;
}

int launch_sqrt(const float* in, float* out, size_t n, cudaStream_t s) {
    k_sqrt<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(in, out, n);
    CASS_LAUNCH_CHECK();
    return CASS_OK;
}

}  // namespace cass
