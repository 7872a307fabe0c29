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

template <typename TA, typename TB>
void launch_gemm_f64(wide_ctx* ctx, cudaStream_t s, const TA* A, const TB* B, double* C, int M, int N, int K,
                     long long sbk, long long sbn) {
    dim3 grid((N + kTile - 1) / kTile, (M + kTile - 1) / kTile);
    WideLaunch l(ctx, s, "route_scores_f64");
    gemm_f64_kernel<TA, TB><<<grid, 256, 0, s>>>(A, B, C, M, N, K, sbk, sbn);
}

}  // namespace

size_t wide_route_workspace(int T, int NG, int rank) {
    // fp64 scores [T, NG] (TOPK) or logits [T, 2NG] plus bottleneck activations [T, rank] (PAIR)
    return wide_align_up(static_cast<size_t>(T) * 2 * NG * sizeof(double), 256) +
           wide_align_up(static_cast<size_t>(T) * (rank > 0 ? rank : 1) * sizeof(double), 256);
}

int wide_launch_route(wide_ctx* ctx, cudaStream_t s, const void* x, int dtype, int T, int D,
                      const void* w_router, const void* w2, int rank, int NG, int mode, int k,
                      const int32_t* k_per_token, uint32_t* mask_bits, float* scores, void* ws) {
    if (T == 0) return WIDE_OK;
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
    (void)flags;
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
                             n_groups, mode, k, k_per_token, mask_bits, scores, scratch);
}
