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

constexpr int kSelWarps = 4;   // tokens (warps) per CTA in select_band_kernel
constexpr int kBatch = 4;      // 16-byte loads in flight per lane

// Exact x_t . w_g in fp64 by one warp: x row in shared memory, w row streamed from L2 with
// kBatch loads in flight per lane (bf16 products are exact in fp64).
__device__ __forceinline__ double warp_dot_f64(const uint4* __restrict__ xs, const __nv_bfloat16* __restrict__ wrow,
                                               int nch, int lane) {
    const uint4* wv = reinterpret_cast<const uint4*>(wrow);
    double acc = 0.0;
    for (int base = 0; base < nch; base += 32 * kBatch) {
        uint4 b[kBatch];
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
            const int i = base + lane + 32 * j;
            b[j] = i < nch ? wv[i] : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
            const int i = base + lane + 32 * j;
            if (i < nch) {
                const uint4 a = xs[i];
                const __nv_bfloat162* ah = reinterpret_cast<const __nv_bfloat162*>(&a);
                const __nv_bfloat162* bh = reinterpret_cast<const __nv_bfloat162*>(&b[j]);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 fa = __bfloat1622float2(ah[e]), fb = __bfloat1622float2(bh[e]);
                    acc = fma(static_cast<double>(fa.x), static_cast<double>(fb.x), acc);
                    acc = fma(static_cast<double>(fa.y), static_cast<double>(fb.y), acc);
                }
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    return acc;
}

// One CTA (4 warps) per token.  scores: nsplit partial slabs [nsplit][T, ld] that are summed on
// load.  Thread g ranks group g (and g + 128); the exact re-scoring of the band is spread over
// the four warps.
__global__ void __launch_bounds__(32 * kSelWarps, 12)
select_band_kernel(const float* __restrict__ scores, int nsplit, int ld, const __nv_bfloat16* __restrict__ x,
                   const __nv_bfloat16* __restrict__ w, const float* __restrict__ wnorm, int T, int NG, int D, int k,
                   const int32_t* __restrict__ k_per_token, uint32_t* __restrict__ mask_bits,
                   float* __restrict__ scores_out) {
    extern __shared__ uint4 sh_x[];  // [D / 8]
    __shared__ float s[WIDE_MAX_GROUPS];
    __shared__ __align__(16) unsigned long long skey[WIDE_MAX_GROUPS + 2];  // (ordered score bits, NG - index)
    __shared__ double ex[WIDE_MAX_GROUPS];
    __shared__ int band[WIDE_MAX_GROUPS];
    __shared__ float red[2 * kSelWarps];
    __shared__ float sh_b[2];
    __shared__ int n_band, n_band_hi;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int t = blockIdx.x;
    const int nch = D / 8;
    const int words = (NG + 31) >> 5;
    const size_t slab = static_cast<size_t>(T) * ld;
    constexpr int kThreads = 32 * kSelWarps;
    constexpr int kPer = WIDE_MAX_GROUPS / kThreads;  // groups per thread (2)

    float wmax = 0.f;
#pragma unroll
    for (int q = 0; q < kPer; ++q) {
        const int g = tid + q * kThreads;
        if (g < NG) {
            float v = 0.f;
            for (int ks = 0; ks < nsplit; ++ks) v += scores[ks * slab + static_cast<size_t>(t) * ld + g];
            s[g] = v;
            // total order "score descending, index ascending" as one unsigned 64-bit compare
            const uint32_t u = __float_as_uint(v + 0.0f);  // -0 -> +0
            const uint32_t ord = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
            skey[g] = (static_cast<unsigned long long>(ord) << 32) | static_cast<uint32_t>(NG - g);
            wmax = fmaxf(wmax, wnorm[g]);
            if (scores_out) scores_out[static_cast<size_t>(t) * NG + g] = v;
        } else if (g < NG + 2) {
            skey[g] = 0ull;  // padding: beats nobody
        }
    }
    const int kt = min(max(k_per_token ? k_per_token[t] : k, 0), NG);
    const bool boundary = kt > 0 && kt < NG;

    // x row -> shared memory, partial ||x_t||^2 on the way
    float xsq = 0.f;
    if (boundary) {
        const uint4* xv = reinterpret_cast<const uint4*>(x + static_cast<size_t>(t) * D);
        for (int base = 0; base < nch; base += kThreads * kBatch) {
            uint4 a[kBatch];
#pragma unroll
            for (int j = 0; j < kBatch; ++j) {
                const int i = base + tid + kThreads * j;
                a[j] = i < nch ? xv[i] : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int j = 0; j < kBatch; ++j) {
                const int i = base + tid + kThreads * j;
                if (i < nch) {
                    sh_x[i] = a[j];
                    const __nv_bfloat162* ah = reinterpret_cast<const __nv_bfloat162*>(&a[j]);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 f = __bfloat1622float2(ah[e]);
                        xsq = fmaf(f.x, f.x, fmaf(f.y, f.y, xsq));
                    }
                }
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        xsq += __shfl_xor_sync(0xffffffffu, xsq, o);
        wmax = fmaxf(wmax, __shfl_xor_sync(0xffffffffu, wmax, o));
    }
    if (lane == 0) { red[warp] = xsq; red[kSelWarps + warp] = wmax; }
    if (tid == 0) { sh_b[0] = 0.f; sh_b[1] = 0.f; n_band = 0; n_band_hi = 0; }
    __syncthreads();
    xsq = 0.f;
    wmax = 0.f;
#pragma unroll
    for (int i = 0; i < kSelWarps; ++i) { xsq += red[i]; wmax = fmaxf(wmax, red[kSelWarps + i]); }

    // fp32 ranks; remember the k-th and (k+1)-th largest
    int rank[kPer];
#pragma unroll
    for (int q = 0; q < kPer; ++q) {
        rank[q] = NG;
        const int g = tid + q * kThreads;
        if (g < NG) {
            const float v = s[g];
            const unsigned long long mine = skey[g];
            int beats = 0;
            const ulonglong2* kp = reinterpret_cast<const ulonglong2*>(skey);
#pragma unroll 4
            for (int h = 0; h < (NG + 1) / 2; ++h) {
                const ulonglong2 kk = kp[h];
                beats += (kk.x > mine) + (kk.y > mine);
            }
            rank[q] = beats;
            if (beats == kt - 1) sh_b[0] = v;
            if (beats == kt) sh_b[1] = v;
        }
    }
    __syncthreads();
    const float v_k = sh_b[0], v_k1 = sh_b[1];
    // band half-width 2 * eps_t (a little slack for the fp32 evaluation of the bound itself)
    const float tau = boundary ? 2.f * kAccumErr * static_cast<float>(D) * sqrtf(xsq) * 1.0001f * wmax : 0.f;

    bool in_band[kPer];
#pragma unroll
    for (int q = 0; q < kPer; ++q) {
        in_band[q] = false;
        const int g = tid + q * kThreads;
        if (boundary && g < NG) {
            const bool hi = rank[q] < kt;
            const bool u = hi ? (s[g] - v_k1 <= tau) : (v_k - s[g] <= tau);
            if (u) {
                in_band[q] = true;
                band[atomicAdd(&n_band, 1)] = g;
                if (hi) atomicAdd(&n_band_hi, 1);
            }
        }
    }
    __syncthreads();
    const int nb = n_band, m_hi = n_band_hi;
    for (int i = warp; i < nb; i += kSelWarps) {
        const int gg = band[i];
        const double e = warp_dot_f64(sh_x, w + static_cast<size_t>(gg) * D, nch, lane);
        if (lane == 0) ex[gg] = e;
    }
    __syncthreads();

    // final decision: band members are re-ranked among themselves on the exact scores
#pragma unroll
    for (int q = 0; q < kPer; ++q) {
        const int g = tid + q * kThreads;
        bool sel = false;
        if (g < NG) {
            if (in_band[q]) {
                const double v = ex[g];
                int beats = 0;
                for (int i = 0; i < nb; ++i) {
                    const int h = band[i];
                    const double u = ex[h];
                    beats += (u > v) || (u == v && h < g);
                }
                sel = beats < m_hi;
            } else {
                sel = rank[q] < kt;
            }
        }
        const unsigned word = __ballot_sync(0xffffffffu, sel);
        const int widx = warp + q * kSelWarps;
        if (lane == 0 && widx < words) mask_bits[static_cast<size_t>(t) * words + widx] = word;
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
           wide_align_up(static_cast<size_t>(T) * 128, 256) + wide_align_up(static_cast<size_t>(T) * 2048, 256) + 1024;
}

int wide_launch_route(wide_ctx* ctx, cudaStream_t s, const void* x, int dtype, int T, int D,
                      const void* w_router, const void* w2, int rank, int NG, int mode, int k,
                      const int32_t* k_per_token, uint32_t* mask_bits, float* scores, void* ws, unsigned flags) {
    if (T == 0) return WIDE_OK;
    if (mode == WIDE_ROUTE_TOPK && dtype == WIDE_BF16 && D % 64 == 0 && D <= 16384 && ctx->encode_tiled &&
        !(flags & WIDE_FLAG_SIMT)) {
        const int ld = (NG + 31) / 32 * 32;
        float* sc32 = static_cast<float*>(ws);
        float* wn = reinterpret_cast<float*>(static_cast<char*>(ws) + wide_route_workspace(T, NG, rank) - 1024);
        // as many K-split slabs as the first part of the workspace holds (at most 8)
        const size_t part0 = wide_route_workspace(T, NG, rank) - 1024;
        int max_split = static_cast<int>(part0 / (static_cast<size_t>(T) * ld * sizeof(float)));
        if (max_split > 8) max_split = 8;
        if (max_split < 1) max_split = 1;
        int ksplit = 1;
        const int rc = wide_launch_scores_tc(ctx, s, x, w_router, T, NG, ld, D, sc32, wn, max_split, &ksplit);
        if (rc != WIDE_OK) return rc;
        const int sel_smem = (D / 8) * static_cast<int>(sizeof(uint4));
        WIDE_CUDA_CHECK(cudaFuncSetAttribute(select_band_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, sel_smem));
        WideLaunch l(ctx, s, "route_select_band");
        select_band_kernel<<<T, 32 * kSelWarps, sel_smem, s>>>(
            sc32, ksplit, ld, static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(w_router), wn, T,
            NG, D, k, k_per_token, mask_bits, scores);
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
