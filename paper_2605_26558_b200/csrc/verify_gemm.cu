// Verification projections (Sec. 2.2: the target model processes the gamma+1 drafted rows as one small batch,
// memory-bound on the bf16 weights): Y[r][n] = sum_k W[n][k] X[r][k], bf16 operands, fp32 accumulation.
//
// CUDA-core version: every weight element is read once from HBM (streaming 16-byte loads) and multiplied
// against all rows, which sit in shared memory.  The accumulation order of one output element depends only
// on (n, k) and never on the number of rows in the call, so a row gives bit-identical results whether it is
// verified alone or with others.
#include "kernels.cuh"

namespace cass {

constexpr int kVgWarps = 8, kVgFeat = 4, kVgKT = 1024;

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

template <int RT>
__global__ void __launch_bounds__(256) k_verify_gemm(const uint16_t* __restrict__ W, const uint16_t* __restrict__ X,
                                                     int rows, int n, int k, uint16_t* __restrict__ y_bf16,
                                                     float* __restrict__ y_f32) {
    __shared__ __align__(16) uint16_t xs[RT][kVgKT];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n0 = (blockIdx.x * kVgWarps + warp) * kVgFeat;
    float acc[kVgFeat][RT];
#pragma unroll
    for (int f = 0; f < kVgFeat; ++f)
#pragma unroll
        for (int r = 0; r < RT; ++r) acc[f][r] = 0.f;

    for (int kt = 0; kt < k; kt += kVgKT) {
        __syncthreads();
        for (int i = tid; i < RT * (kVgKT / 8); i += 256) {
            int r = i / (kVgKT / 8), c8 = i % (kVgKT / 8);
            uint4 v = make_uint4(0, 0, 0, 0);
            if (r < rows && kt + c8 * 8 < k) v = *reinterpret_cast<const uint4*>(X + (size_t)r * k + kt + c8 * 8);
            *reinterpret_cast<uint4*>(&xs[r][c8 * 8]) = v;
        }
        __syncthreads();
#pragma unroll
        for (int step = 0; step < kVgKT / 256; ++step) {
            const int kk = (step * 32 + lane) * 8;
            if (kt + kk >= k) continue;
            uint4 wv[kVgFeat];
#pragma unroll
            for (int f = 0; f < kVgFeat; ++f) {
                wv[f] = make_uint4(0, 0, 0, 0);
                if (n0 + f < n) wv[f] = ld_stream(reinterpret_cast<const uint4*>(W + (size_t)(n0 + f) * k + kt + kk));
            }
#pragma unroll
            for (int r = 0; r < RT; ++r) {
                const uint4 xv = *reinterpret_cast<const uint4*>(&xs[r][kk]);
                const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
                for (int f = 0; f < kVgFeat; ++f) {
                    const uint32_t ww[4] = {wv[f].x, wv[f].y, wv[f].z, wv[f].w};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        acc[f][r] = fmaf(__uint_as_float(ww[q] << 16), __uint_as_float(xw[q] << 16), acc[f][r]);
                        acc[f][r] = fmaf(__uint_as_float(ww[q] & 0xFFFF0000u), __uint_as_float(xw[q] & 0xFFFF0000u), acc[f][r]);
                    }
                }
            }
        }
    }
#pragma unroll
    for (int f = 0; f < kVgFeat; ++f)
#pragma unroll
        for (int r = 0; r < RT; ++r) {
            float v = warp_sum(acc[f][r]);
            if (lane == 0 && r < rows && n0 + f < n) {
                if (y_f32) y_f32[(size_t)r * n + n0 + f] = v;
                if (y_bf16) y_bf16[(size_t)r * n + n0 + f] = float_to_bf16_bits(v);
            }
        }
}

int launch_verify_gemm(const uint16_t* W, const uint16_t* X, int rows, int n, int k, uint16_t* y_bf16, float* y_f32,
                       cudaStream_t s) {
    if (rows < 1 || rows > kMaxVerifyRows || (k % 8)) return CASS_ERR_INVALID_ARG;
    dim3 grid(ceil_div(n, kVgWarps * kVgFeat));
#define CASS_VG(RT_) k_verify_gemm<RT_><<<grid, 256, 0, s>>>(W, X, rows, n, k, y_bf16, y_f32)
    if (rows == 1) CASS_VG(1);
    else if (rows <= 3) CASS_VG(3);
    else if (rows <= 5) CASS_VG(5);
    else if (rows <= 7) CASS_VG(7);
    else if (rows <= 9) CASS_VG(9);
    else CASS_VG(16);
#undef CASS_VG
    CASS_LAUNCH_CHECK();
    return CASS_OK;
}

}  // namespace cass
