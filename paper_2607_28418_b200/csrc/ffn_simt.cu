// CUDA-core implementation of the masked FFN (Eq. 3) and masked O-projection (Eq. 2 / Eq. 10)
// for any shape and for fp32 or bf16 inputs, fp32 accumulation.  It works from the bit mask
// alone: a 64-token x 64-channel block of the hidden activation whose (token, group) pairs are
// all inactive is skipped (block-level predicate); inside an active block inactive pairs are
// written as exact zeros.  The tensor-core paths are the fast ones; this is the path for fp32
// data and odd shapes.
#include "internal.h"

namespace {

constexpr int BT = 64;   // tokens per block
constexpr int BC = 64;   // output columns per block
constexpr int BK = 16;

// H[t, c] = M[t, c/G] ? silu(x_t . wg_c) * (x_t . wu_c) : 0
template <typename TIn>
__global__ void __launch_bounds__(256) gateup_kernel(const TIn* __restrict__ x, const TIn* __restrict__ wg,
                                                     const TIn* __restrict__ wu, int T, int D, int Dff, int G,
                                                     const uint32_t* __restrict__ mask_bits, int words,
                                                     TIn* __restrict__ h) {
    __shared__ float xs[BK][BT + 4];
    __shared__ float gs[BK][BC + 4];
    __shared__ float us[BK][BC + 4];
    const int t0 = blockIdx.y * BT, c0 = blockIdx.x * BC;
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;  // thread owns tokens ty*4.., channels tx*4..

    // block-level predicate over every (token, group) pair the block touches
    const int g_lo = c0 / G, g_hi = min(Dff - 1, c0 + BC - 1) / G;
    int any = 0;
    for (int i = tid; i < BT * (g_hi - g_lo + 1); i += 256) {
        const int t = t0 + i % BT, g = g_lo + i / BT;
        if (t < T) any |= wide_mask_bit(mask_bits, words, t, g) ? 1 : 0;
    }
    any = __syncthreads_or(any);

    float accg[4][4], accu[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) accg[i][j] = accu[i][j] = 0.f;

    if (any) {
        for (int k0 = 0; k0 < D; k0 += BK) {
            for (int i = tid; i < BT * BK; i += 256) {
                const int r = i / BK, k = i % BK;
                const int t = t0 + r, c = c0 + r;
                xs[k][r] = (t < T && k0 + k < D) ? wide_to_float(x[static_cast<size_t>(t) * D + k0 + k]) : 0.f;
                const bool ok = c < Dff && k0 + k < D;
                gs[k][r] = ok ? wide_to_float(wg[static_cast<size_t>(c) * D + k0 + k]) : 0.f;
                us[k][r] = ok ? wide_to_float(wu[static_cast<size_t>(c) * D + k0 + k]) : 0.f;
            }
            __syncthreads();
#pragma unroll
            for (int k = 0; k < BK; ++k) {
                float xv[4], gv[4], uv[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    xv[i] = xs[k][ty * 4 + i];
                    gv[i] = gs[k][tx * 4 + i];
                    uv[i] = us[k][tx * 4 + i];
                }
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        accg[i][j] = fmaf(xv[i], gv[j], accg[i][j]);
                        accu[i][j] = fmaf(xv[i], uv[j], accu[i][j]);
                    }
            }
            __syncthreads();
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int t = t0 + ty * 4 + i;
        if (t >= T) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = c0 + tx * 4 + j;
            if (c >= Dff) continue;
            float v = 0.f;
            if (any && wide_mask_bit(mask_bits, words, t, c / G)) {
                const float a = accg[i][j];
                v = a / (1.f + expf(-a)) * accu[i][j];
            }
            wide_store(&h[static_cast<size_t>(t) * Dff + c], v);
        }
    }
}

// C[m, n] = sum_k A'[m, k] * B[n, k];  A' = A with (row, k/G) pairs outside the mask zeroed when
// mask_bits != nullptr.
template <typename TIn, typename TOut>
__global__ void __launch_bounds__(256) gemm_nt_kernel(const TIn* __restrict__ A, const TIn* __restrict__ B,
                                                      TOut* __restrict__ C, int M, int N, int K,
                                                      const uint32_t* __restrict__ mask_bits, int words, int G) {
    __shared__ float as[BK][BT + 4];
    __shared__ float bs[BK][BC + 4];
    const int m0 = blockIdx.y * BT, n0 = blockIdx.x * BC;
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (int k0 = 0; k0 < K; k0 += BK) {
        for (int i = tid; i < BT * BK; i += 256) {
            const int r = i / BK, k = i % BK;
            const int m = m0 + r, n = n0 + r, kk = k0 + k;
            float av = 0.f;
            if (m < M && kk < K) {
                av = wide_to_float(A[static_cast<size_t>(m) * K + kk]);
                if (mask_bits && !wide_mask_bit(mask_bits, words, m, kk / G)) av = 0.f;
            }
            as[k][r] = av;
            bs[k][r] = (n < N && kk < K) ? wide_to_float(B[static_cast<size_t>(n) * K + kk]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            float av[4], bv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                av[i] = as[k][ty * 4 + i];
                bv[i] = bs[k][tx * 4 + i];
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n < N) wide_store(&C[static_cast<size_t>(m) * N + n], acc[i][j]);
        }
    }
}

template <typename TIn>
int run_gemm_nt(wide_ctx* ctx, cudaStream_t s, const TIn* A, const TIn* B, void* C, int out_dtype, int M, int N, int K,
                const uint32_t* mask_bits, int words, int G) {
    if (M == 0) return WIDE_OK;
    dim3 grid((N + BC - 1) / BC, (M + BT - 1) / BT);
    WideLaunch l(ctx, s, "simt_gemm_nt");
    if (out_dtype == WIDE_BF16)
        gemm_nt_kernel<TIn, __nv_bfloat16><<<grid, 256, 0, s>>>(A, B, static_cast<__nv_bfloat16*>(C), M, N, K,
                                                               mask_bits, words, G);
    else
        gemm_nt_kernel<TIn, float><<<grid, 256, 0, s>>>(A, B, static_cast<float*>(C), M, N, K, mask_bits, words, G);
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}

template <typename TIn>
int run_ffn(wide_ctx* ctx, cudaStream_t s, const void* x, const void* wg, const void* wu, const void* wd, int T, int D,
            int Dff, int G, const uint32_t* mask_bits, void* y, int out_dtype, void* h) {
    if (T == 0) return WIDE_OK;
    const int words = (Dff / G + 31) / 32;
    dim3 grid((Dff + BC - 1) / BC, (T + BT - 1) / BT);
    {
        WideLaunch l(ctx, s, "simt_gateup");
        gateup_kernel<TIn><<<grid, 256, 0, s>>>(static_cast<const TIn*>(x), static_cast<const TIn*>(wg),
                                                static_cast<const TIn*>(wu), T, D, Dff, G, mask_bits, words,
                                                static_cast<TIn*>(h));
    }
    if (cudaGetLastError() != cudaSuccess) return WIDE_ERR_CUDA;
    return run_gemm_nt<TIn>(ctx, s, static_cast<const TIn*>(h), static_cast<const TIn*>(wd), y, out_dtype, T, D, Dff,
                            nullptr, 0, 1);
}

}  // namespace

int wide_launch_ffn_simt(wide_ctx* ctx, cudaStream_t s, const void* x, const void* wg, const void* wu, const void* wd,
                         int dtype, int T, int D, int Dff, int G, const uint32_t* mask_bits, void* y,
                         int out_dtype, void* h) {
    if (dtype == WIDE_BF16) return run_ffn<__nv_bfloat16>(ctx, s, x, wg, wu, wd, T, D, Dff, G, mask_bits, y, out_dtype, h);
    return run_ffn<float>(ctx, s, x, wg, wu, wd, T, D, Dff, G, mask_bits, y, out_dtype, h);
}

int wide_launch_oproj_simt(wide_ctx* ctx, cudaStream_t s, const void* a, const void* wo, int dtype, int T, int D,
                           int K, int G, const uint32_t* mask_bits, void* y, int out_dtype) {
    const int words = (K / G + 31) / 32;
    if (dtype == WIDE_BF16)
        return run_gemm_nt<__nv_bfloat16>(ctx, s, static_cast<const __nv_bfloat16*>(a),
                                          static_cast<const __nv_bfloat16*>(wo), y, out_dtype, T, D, K, mask_bits,
                                          words, G);
    return run_gemm_nt<float>(ctx, s, static_cast<const float*>(a), static_cast<const float*>(wo), y, out_dtype, T, D, K,
                              mask_bits, words, G);
}
