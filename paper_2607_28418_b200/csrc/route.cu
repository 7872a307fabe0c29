// wide_route: router scores and per-token group selection (Section 3.1, Eq. 4; fixed-budget
// top-k reading of Appendix A).  The decision is taken on fp64 sums of exact products so that
// it does not depend on summation order.
#include "internal.h"

namespace {

constexpr int kTile = 32;

// C[m, n] = sum_k A[m, k] * B(k, n), fp64 accumulate.  A is row-major [M, K]; B(k, n) lives at
// B[k * sbk + n * sbn].  32x32 output tile per CTA, 256 threads, 4 outputs per thread.
template <typename TA, typename TB>
__global__ void __launch_bounds__(256) gemm_f64_kernel(const TA* __restrict__ A, const TB* __restrict__ B,
                                                       double* __restrict__ C, int M, int N, int K,
                                                       long long sbk, long long sbn) {
    __shared__ double xs[kTile][kTile + 1];
    __shared__ double ws[kTile][kTile + 1];  // ws[k][n]
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;  // ty in 0..7
    const int m0 = blockIdx.y * kTile, n0 = blockIdx.x * kTile;
    double acc[4] = {0.0, 0.0, 0.0, 0.0};
    for (int k0 = 0; k0 < K; k0 += kTile) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = ty + 8 * i;
            const int m = m0 + r, k = k0 + tx;
            xs[r][tx] = (m < M && k < K) ? wide_to_double(A[static_cast<size_t>(m) * K + k]) : 0.0;
            const int n = n0 + r;  // row r of the B tile = output column n, tx walks k
            ws[tx][r] = (n < N && k < K) ? wide_to_double(B[static_cast<long long>(k) * sbk + static_cast<long long>(n) * sbn]) : 0.0;
        }
        __syncthreads();
#pragma unroll 8
        for (int k = 0; k < kTile; ++k) {
            const double w = ws[k][tx];
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[i] = fma(xs[ty + 8 * i][k], w, acc[i]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty + 8 * i, n = n0 + tx;
        if (m < M && n < N) C[static_cast<size_t>(m) * N + n] = acc[i];
    }
}

// One warp per token: rank every group under (score descending, index ascending); bit set iff
// rank < k_t.  Writes the packed mask row and, optionally, fp32 scores.
__global__ void __launch_bounds__(256) topk_select_kernel(const double* __restrict__ scores, int T, int NG,
                                                          int k, const int32_t* __restrict__ k_per_token,
                                                          uint32_t* __restrict__ mask_bits,
                                                          float* __restrict__ scores_out) {
    __shared__ double sh[8][WIDE_MAX_GROUPS];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t = blockIdx.x * 8 + warp;
    if (t >= T) return;
    double* s = sh[warp];
    for (int g = lane; g < NG; g += 32) {
        const double v = scores[static_cast<size_t>(t) * NG + g];
        s[g] = v;
        if (scores_out) scores_out[static_cast<size_t>(t) * NG + g] = static_cast<float>(v);
    }
    __syncwarp();
    const int kt = k_per_token ? k_per_token[t] : k;
    const int words = (NG + 31) >> 5;
    for (int w = 0; w < words; ++w) {
        const int g = w * 32 + lane;
        bool sel = false;
        if (g < NG) {
            const double v = s[g];
            int beats = 0;
            for (int h = 0; h < NG; ++h) {
                const double u = s[h];
                beats += (u > v) || (u == v && h < g);
            }
            sel = beats < kt;
        }
        const unsigned word = __ballot_sync(0xffffffffu, sel);
        if (lane == 0) mask_bits[static_cast<size_t>(t) * words + w] = word;
    }
}

// Eq. 4, inference branch: execute iff logit of class 0 >= logit of class 1.
__global__ void __launch_bounds__(256) pair_select_kernel(const double* __restrict__ logits, int T, int NG,
                                                          uint32_t* __restrict__ mask_bits,
                                                          float* __restrict__ scores_out) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t = blockIdx.x * 8 + warp;
    if (t >= T) return;
    const int words = (NG + 31) >> 5;
    const double* row = logits + static_cast<size_t>(t) * 2 * NG;
    for (int w = 0; w < words; ++w) {
        const int g = w * 32 + lane;
        bool sel = false;
        if (g < NG) {
            const double l0 = row[2 * g], l1 = row[2 * g + 1];
            sel = l0 >= l1;
            if (scores_out) {
                scores_out[static_cast<size_t>(t) * 2 * NG + 2 * g] = static_cast<float>(l0);
                scores_out[static_cast<size_t>(t) * 2 * NG + 2 * g + 1] = static_cast<float>(l1);
            }
        }
        const unsigned word = __ballot_sync(0xffffffffu, sel);
        if (lane == 0) mask_bits[static_cast<size_t>(t) * words + w] = word;
    }
}


// ---------------------------------------------------------------------------- fast path (bf16)
// Scores come from the tensor cores in fp32 (exact products, fp32 accumulation).  Their error is
// bounded by eps_t = kAccumErr * D * ||x_t|| * max_g ||w_g|| (Cauchy-Schwarz on the sum of absolute
// products times a per-step accumulation error).  A group whose fp32 score is further than
// 2*eps_t from the selection boundary keeps its fp32 decision; the few groups inside that band
// get their score recomputed exactly in fp64, and the band is re-ranked on those exact values.
// The result equals the fp64 decision of the slow path.
constexpr float kAccumErr = 5.9604645e-8f;  // 2^-24 per accumulated element

// ||w_g||_2 for every group, one warp per group.
__global__ void __launch_bounds__(256) wnorm_kernel(const __nv_bfloat16* __restrict__ w, int NG, int D,
                                                    float* __restrict__ wnorm) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = blockIdx.x * 8 + warp;
    if (g >= NG) return;
    const uint4* row = reinterpret_cast<const uint4*>(w + static_cast<size_t>(g) * D);
    float acc = 0.f;
    for (int i = lane; i < D / 8; i += 32) {
        const uint4 v = row[i];
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(h[e]);
            acc = fmaf(f.x, f.x, fmaf(f.y, f.y, acc));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) wnorm[g] = sqrtf(acc) * 1.0001f;  // rounded up a little: it feeds a bound
}

// Exact x_t . w_g in fp64 by one warp (bf16 products are exact in fp64).
__device__ __forceinline__ double warp_dot_f64(const __nv_bfloat16* __restrict__ xrow,
                                               const __nv_bfloat16* __restrict__ wrow, int D, int lane) {
    const uint4* xv = reinterpret_cast<const uint4*>(xrow);
    const uint4* wv = reinterpret_cast<const uint4*>(wrow);
    double acc = 0.0;
    for (int i = lane; i < D / 8; i += 32) {
        const uint4 a = xv[i], b = wv[i];
        const __nv_bfloat162* ah = reinterpret_cast<const __nv_bfloat162*>(&a);
        const __nv_bfloat162* bh = reinterpret_cast<const __nv_bfloat162*>(&b);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 fa = __bfloat1622float2(ah[e]), fb = __bfloat1622float2(bh[e]);
            acc = fma(static_cast<double>(fa.x), static_cast<double>(fb.x), acc);
            acc = fma(static_cast<double>(fa.y), static_cast<double>(fb.y), acc);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    return acc;
}

// One warp per token.
__global__ void __launch_bounds__(256) select_band_kernel(const float* __restrict__ scores, int ld,
                                                          const __nv_bfloat16* __restrict__ x,
                                                          const __nv_bfloat16* __restrict__ w,
                                                          const float* __restrict__ wnorm, int T, int NG, int D,
                                                          int k, const int32_t* __restrict__ k_per_token,
                                                          uint32_t* __restrict__ mask_bits,
                                                          float* __restrict__ scores_out) {
    __shared__ float sh_s[8][WIDE_MAX_GROUPS];
    __shared__ double sh_e[8][WIDE_MAX_GROUPS];
    __shared__ float sh_b[8][2];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t = blockIdx.x * 8 + warp;
    if (t >= T) return;
    float* s = sh_s[warp];
    double* ex = sh_e[warp];
    const int words = (NG + 31) >> 5;
    float wmax = 0.f;
    for (int g = lane; g < NG; g += 32) {
        const float v = scores[static_cast<size_t>(t) * ld + g];
        s[g] = v;
        wmax = fmaxf(wmax, wnorm[g]);
        if (scores_out) scores_out[static_cast<size_t>(t) * NG + g] = v;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) wmax = fmaxf(wmax, __shfl_xor_sync(0xffffffffu, wmax, o));
    __syncwarp();
    const int kt = min(max(k_per_token ? k_per_token[t] : k, 0), NG);
    const __nv_bfloat16* xrow = x + static_cast<size_t>(t) * D;

    // fp32 ranks; remember the k-th and (k+1)-th largest
    int rank[WIDE_MAX_GROUPS / 32];
    if (lane == 0) { sh_b[warp][0] = 0.f; sh_b[warp][1] = 0.f; }
    __syncwarp();
#pragma unroll
    for (int w8 = 0; w8 < WIDE_MAX_GROUPS / 32; ++w8) {
        rank[w8] = NG;
        const int g = w8 * 32 + lane;
        if (w8 < words && g < NG) {
            const float v = s[g];
            int beats = 0;
            for (int h = 0; h < NG; ++h) {
                const float u = s[h];
                beats += (u > v) || (u == v && h < g);
            }
            rank[w8] = beats;
            if (beats == kt - 1) sh_b[warp][0] = v;
            if (beats == kt) sh_b[warp][1] = v;
        }
    }
    __syncwarp();
    const bool boundary = kt > 0 && kt < NG;
    const float v_k = sh_b[warp][0], v_k1 = sh_b[warp][1];

    float tau = 0.f;
    if (boundary) {
        // ||x_t||, then the band half-width 2*eps
        float acc = 0.f;
        const uint4* xv = reinterpret_cast<const uint4*>(xrow);
        for (int i = lane; i < D / 8; i += 32) {
            const uint4 a = xv[i];
            const __nv_bfloat162* ah = reinterpret_cast<const __nv_bfloat162*>(&a);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 f = __bfloat1622float2(ah[e]);
                acc = fmaf(f.x, f.x, fmaf(f.y, f.y, acc));
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        tau = 2.f * kAccumErr * static_cast<float>(D) * sqrtf(acc) * 1.0001f * wmax;
    }

    // band membership, exact scores of the band
    unsigned in_band[WIDE_MAX_GROUPS / 32];
    int m_hi = 0;  // band members currently ranked inside the top k
#pragma unroll
    for (int w8 = 0; w8 < WIDE_MAX_GROUPS / 32; ++w8) {
        in_band[w8] = 0u;
        if (w8 >= words) continue;
        const int g = w8 * 32 + lane;
        bool u = false, hi = false;
        if (boundary && g < NG) {
            hi = rank[w8] < kt;
            u = hi ? (s[g] - v_k1 <= tau) : (v_k - s[g] <= tau);
        }
        unsigned vote = __ballot_sync(0xffffffffu, u);
        in_band[w8] = vote;
        m_hi += __popc(__ballot_sync(0xffffffffu, u && hi));
        while (vote) {
            const int b = __ffs(vote) - 1;
            vote &= vote - 1;
            const int gg = w8 * 32 + b;
            const double e = warp_dot_f64(xrow, w + static_cast<size_t>(gg) * D, D, lane);
            if (lane == 0) ex[gg] = e;
        }
    }
    __syncwarp();

    // final decision
#pragma unroll
    for (int w8 = 0; w8 < WIDE_MAX_GROUPS / 32; ++w8) {
        if (w8 >= words) continue;
        const int g = w8 * 32 + lane;
        bool sel = false;
        if (g < NG) {
            if ((in_band[w8] >> lane) & 1u) {
                const double v = ex[g];
                int beats = 0;
                for (int w2 = 0; w2 < words; ++w2) {
                    unsigned bits = in_band[w2];
                    while (bits) {
                        const int b = __ffs(bits) - 1;
                        bits &= bits - 1;
                        const int h = w2 * 32 + b;
                        const double u = ex[h];
                        beats += (u > v) || (u == v && h < g);
                    }
                }
                sel = beats < m_hi;
            } else {
                sel = rank[w8] < kt;
            }
        }
        const unsigned word = __ballot_sync(0xffffffffu, sel);
        if (lane == 0) mask_bits[static_cast<size_t>(t) * words + w8] = word;
    }
}

template <typename TA, typename TB>
void launch_gemm_f64(wide_ctx* ctx, cudaStream_t s, const TA* A, const TB* B, double* C, int M, int N, int K,
                     long long sbk, long long sbn) {
    dim3 grid((N + kTile - 1) / kTile, (M + kTile - 1) / kTile);
    WideLaunch l(ctx, s, "route_scores_f64");
    gemm_f64_kernel<TA, TB><<<grid, 256, 0, s>>>(A, B, C, M, N, K, sbk, sbn);
}

}  // namespace

size_t wide_route_workspace(int T, int NG, int rank) {
    // fp64 scores [T, NG] (TOPK) or logits [T, 2NG] plus bottleneck activations [T, rank] (PAIR);
    // the tensor-core path reuses the first part for fp32 scores [T, roundup(NG, 32)] and keeps
    // the group norms in the tail
    return wide_align_up(static_cast<size_t>(T) * 2 * NG * sizeof(double), 256) +
           wide_align_up(static_cast<size_t>(T) * (rank > 0 ? rank : 1) * sizeof(double), 256) +
           wide_align_up(static_cast<size_t>(T) * 128, 256) + 1024;
}

int wide_launch_route(wide_ctx* ctx, cudaStream_t s, const void* x, int dtype, int T, int D,
                      const void* w_router, const void* w2, int rank, int NG, int mode, int k,
                      const int32_t* k_per_token, uint32_t* mask_bits, float* scores, void* ws, unsigned flags) {
    if (T == 0) return WIDE_OK;
    if (mode == WIDE_ROUTE_TOPK && dtype == WIDE_BF16 && D % 64 == 0 && ctx->encode_tiled &&
        !(flags & WIDE_FLAG_SIMT)) {
        const int ld = (NG + 31) / 32 * 32;
        float* sc32 = static_cast<float*>(ws);
        float* wn = reinterpret_cast<float*>(static_cast<char*>(ws) + wide_route_workspace(T, NG, rank) - 1024);
        {
            WideLaunch l(ctx, s, "route_wnorm");
            wnorm_kernel<<<(NG + 7) / 8, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(w_router), NG, D, wn);
        }
        const int rc = wide_launch_scores_tc(ctx, s, x, w_router, T, NG, ld, D, sc32);
        if (rc != WIDE_OK) return rc;
        WideLaunch l(ctx, s, "route_select_band");
        select_band_kernel<<<(T + 7) / 8, 256, 0, s>>>(sc32, ld, static_cast<const __nv_bfloat16*>(x),
                                                       static_cast<const __nv_bfloat16*>(w_router), wn, T, NG, D, k,
                                                       k_per_token, mask_bits, scores);
        return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
    }
    double* sc = static_cast<double*>(ws);
    double* u = reinterpret_cast<double*>(static_cast<char*>(ws) +
                                          wide_align_up(static_cast<size_t>(T) * 2 * NG * sizeof(double), 256));
    const int sel_blocks = (T + 7) / 8;
    if (mode == WIDE_ROUTE_TOPK) {
        if (dtype == WIDE_BF16)
            launch_gemm_f64(ctx, s, static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(w_router),
                            sc, T, NG, D, 1LL, static_cast<long long>(D));
        else
            launch_gemm_f64(ctx, s, static_cast<const float*>(x), static_cast<const float*>(w_router), sc, T, NG,
                            D, 1LL, static_cast<long long>(D));
        WideLaunch l(ctx, s, "route_topk_select");
        topk_select_kernel<<<sel_blocks, 256, 0, s>>>(sc, T, NG, k, k_per_token, mask_bits, scores);
    } else {
        // u = x W1 (W1 [D, rank]),  l = u W2 (W2 [rank, 2NG])
        if (dtype == WIDE_BF16) {
            launch_gemm_f64(ctx, s, static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(w_router),
                            u, T, rank, D, static_cast<long long>(rank), 1LL);
            launch_gemm_f64(ctx, s, u, static_cast<const __nv_bfloat16*>(w2), sc, T, 2 * NG, rank,
                            static_cast<long long>(2 * NG), 1LL);
        } else {
            launch_gemm_f64(ctx, s, static_cast<const float*>(x), static_cast<const float*>(w_router), u, T, rank,
                            D, static_cast<long long>(rank), 1LL);
            launch_gemm_f64(ctx, s, u, static_cast<const float*>(w2), sc, T, 2 * NG, rank,
                            static_cast<long long>(2 * NG), 1LL);
        }
        WideLaunch l(ctx, s, "route_pair_select");
        pair_select_kernel<<<sel_blocks, 256, 0, s>>>(sc, T, NG, mask_bits, scores);
    }
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------
// wide_route_static: the same routing as wide_route, for callers that cannot provide scratch.
//
// Some hosts of this library are not allowed to allocate device memory at the point where they
// route: a serving loop that has handed the whole device heap to its own pool, a plugin that runs
// inside another framework's allocator lock, or code running under a policy that forbids
// cudaMalloc after start-up.  For them the fp64 score buffer lives in a file-scope device array of
// fixed size instead of a caller-supplied workspace.  Every GPU that loads the library holds these
// WIDE_ROUTE_STATIC_BYTES until the process exits.
//
// In host code the array's name is only a handle for the runtime, not a device address, so the
// address is resolved once per device with cudaGetSymbolAddress while that device is current and
// cached; kernels only ever see the resolved pointer.
static __device__ __align__(256) unsigned char g_route_static_scratch[WIDE_ROUTE_STATIC_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void* g_static_ptr[kMaxDevices] = {nullptr};

// Returns the device address of the static scratch for `device`, resolving it on first use.
// The first use must happen with `device` current and outside stream capture.
int static_scratch_for(int device, void** out) {
    if (device < 0 || device >= kMaxDevices) return WIDE_ERR_INVALID_ARG;
    if (!g_static_ptr[device]) {
        int cur = -1;
        if (cudaGetDevice(&cur) != cudaSuccess) return WIDE_ERR_CUDA;
        if (cur != device) return WIDE_ERR_INVALID_ARG;
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_route_static_scratch) != cudaSuccess || !p) return WIDE_ERR_CUDA;
        g_static_ptr[device] = p;
    }
    *out = g_static_ptr[device];
    return WIDE_OK;
}
}  // namespace

extern "C" int wide_route_static(wide_ctx* ctx, void* stream, const void* x, int dtype, int tokens, int hidden,
                                 const void* w_router, const void* w2, int rank, int n_groups, int mode, int k,
                                 const int32_t* k_per_token, uint32_t* mask_bits, float* scores, unsigned flags) {
    if (!ctx || !x || !w_router || !mask_bits || (dtype != WIDE_BF16 && dtype != WIDE_F32)) return WIDE_ERR_INVALID_ARG;
    if (tokens < 0 || hidden <= 0 || n_groups <= 0) return WIDE_ERR_INVALID_ARG;
    if (mode == WIDE_ROUTE_TOPK) {
        if (w2 || rank != 0) return WIDE_ERR_INVALID_ARG;
        if (!k_per_token && (k < 0 || k > n_groups)) return WIDE_ERR_INVALID_ARG;
    } else if (mode == WIDE_ROUTE_PAIR_ARGMAX) {
        if (!w2 || rank <= 0 || rank > 64) return WIDE_ERR_INVALID_ARG;
    } else {
        return WIDE_ERR_INVALID_ARG;
    }
    if (n_groups > WIDE_MAX_GROUPS || hidden % 8 != 0) return WIDE_ERR_UNSUPPORTED_SHAPE;
    if (!wide_aligned16(x) || !wide_aligned16(w_router) || (w2 && !wide_aligned16(w2))) return WIDE_ERR_ALIGNMENT;
    // the fixed array bounds the problem size: say so instead of overrunning it
    if (wide_route_workspace(tokens, n_groups, rank) > static_cast<size_t>(WIDE_ROUTE_STATIC_BYTES))
        return WIDE_ERR_WORKSPACE;
    void* scratch = nullptr;
    const int rc = static_scratch_for(ctx->device, &scratch);
    if (rc != WIDE_OK) return rc;
    // every byte of the scratch that a call reads is written by that call first, so nothing has to
    // be cleared between calls
    return wide_launch_route(ctx, static_cast<cudaStream_t>(stream), x, dtype, tokens, hidden, w_router, w2, rank,
                             n_groups, mode, k, k_per_token, mask_bits, scores, scratch, flags);
}
