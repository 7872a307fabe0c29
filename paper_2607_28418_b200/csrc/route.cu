// wide_route: router scores and per-token group selection (Section 3.1, Eq. 4; fixed-budget
// top-k reading of Appendix A).  The decision is taken on fp64 sums of exact products so that
// it does not depend on summation order.
#include "internal.h"
#include "ptx.cuh"

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
// Scores come from the tensor cores in fp32 (exact products, fp32 accumulation), as `nsplit`
// partial slabs over K that are summed here in fp32; inside a slab the score GEMM spreads its
// k-steps over `a` accumulators that it adds up at the end.  Their error is bounded by
//   eps_t = kAccumErr * chain * ||x_t|| * max_g ||w_g||,   chain = D / (nsplit * a) + a + nsplit
// (a per-element accumulation error along each accumulator's chain plus the two short sums, times
// the Cauchy-Schwarz bound on the sum of absolute products).  A group whose fp32 score is further
// than 2*eps_t from the selection boundary keeps its fp32 decision; the few groups inside that
// band get their score recomputed exactly in fp64, and the band is re-ranked on those exact
// values.  The result equals the fp64 decision of the slow path provided the accumulator loses at
// most 2^-23 of the running sum per step: the tensor core's accumulation order and rounding are
// not specified (it may truncate where an FMA chain rounds to nearest, 2^-24), so the bound takes
// the truncation figure; the measured error is two orders of magnitude below it.
constexpr float kAccumErr = 1.1920929e-7f;  // 2^-23 per accumulated element

constexpr int kSelTokens = 2;  // tokens per CTA in select_band_kernel (two warps each)
constexpr int kBatch = 8;      // 16-byte loads in flight per lane and operand
constexpr int kMaxSlabs = 8;   // K-split partial score slabs summed by select_band_kernel
constexpr int kBandMax = 16;   // band members re-scored per token between two block barriers

// Exact x_t . w_g in fp64 by one warp, both rows streamed from L2 (bf16 products are exact in
// fp64).  Four independent accumulators keep the dependent chain of fp64 FMAs short.  The result
// is valid in every lane.
__device__ __forceinline__ double warp_dot_f64(const __nv_bfloat16* __restrict__ xrow, const __nv_bfloat16* __restrict__ wrow,
                                               int nch, int lane) {
    const uint4* xv = reinterpret_cast<const uint4*>(xrow);
    const uint4* wv = reinterpret_cast<const uint4*>(wrow);
    double acc[4] = {0.0, 0.0, 0.0, 0.0};
    for (int base = 0; base < nch; base += 32 * kBatch) {
        uint4 a[kBatch], b[kBatch];
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
            const int i = base + lane + 32 * j;
            a[j] = i < nch ? __ldg(xv + i) : make_uint4(0u, 0u, 0u, 0u);
            b[j] = i < nch ? __ldg(wv + i) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
            const __nv_bfloat162* ah = reinterpret_cast<const __nv_bfloat162*>(&a[j]);
            const __nv_bfloat162* bh = reinterpret_cast<const __nv_bfloat162*>(&b[j]);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 fa = __bfloat1622float2(ah[e]), fb = __bfloat1622float2(bh[e]);
                acc[e] = fma(static_cast<double>(fa.x), static_cast<double>(fb.x), acc[e]);
                acc[e] = fma(static_cast<double>(fa.y), static_cast<double>(fb.y), acc[e]);
            }
        }
    }
    double r = (acc[0] + acc[1]) + (acc[2] + acc[3]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) r += __shfl_xor_sync(0xffffffffu, r, o);
    return r;
}

// The same for two weight rows at once: x is read once and the two chains of fp64 multiply-adds (the
// slow part: this GPU issues about two of them per clock and SM) run side by side.
__device__ __forceinline__ void warp_dot_f64_x2(const __nv_bfloat16* __restrict__ xrow, const __nv_bfloat16* __restrict__ wrow0,
                                                const __nv_bfloat16* __restrict__ wrow1, int nch, int lane, double& r0, double& r1) {
    constexpr int kB = 4;
    const uint4* xv = reinterpret_cast<const uint4*>(xrow);
    const uint4* wv0 = reinterpret_cast<const uint4*>(wrow0);
    const uint4* wv1 = reinterpret_cast<const uint4*>(wrow1);
    double a0[4] = {0.0, 0.0, 0.0, 0.0}, a1[4] = {0.0, 0.0, 0.0, 0.0};
    for (int base = 0; base < nch; base += 32 * kB) {
        uint4 a[kB], b0[kB], b1[kB];
#pragma unroll
        for (int j = 0; j < kB; ++j) {
            const int i = base + lane + 32 * j;
            a[j] = i < nch ? __ldg(xv + i) : make_uint4(0u, 0u, 0u, 0u);
            b0[j] = i < nch ? __ldg(wv0 + i) : make_uint4(0u, 0u, 0u, 0u);
            b1[j] = i < nch ? __ldg(wv1 + i) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int j = 0; j < kB; ++j) {
            const __nv_bfloat162* ah = reinterpret_cast<const __nv_bfloat162*>(&a[j]);
            const __nv_bfloat162* bh0 = reinterpret_cast<const __nv_bfloat162*>(&b0[j]);
            const __nv_bfloat162* bh1 = reinterpret_cast<const __nv_bfloat162*>(&b1[j]);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 fa = __bfloat1622float2(ah[e]), f0 = __bfloat1622float2(bh0[e]), f1 = __bfloat1622float2(bh1[e]);
                const double xa = static_cast<double>(fa.x), xb = static_cast<double>(fa.y);
                a0[e] = fma(xa, static_cast<double>(f0.x), a0[e]);
                a0[e] = fma(xb, static_cast<double>(f0.y), a0[e]);
                a1[e] = fma(xa, static_cast<double>(f1.x), a1[e]);
                a1[e] = fma(xb, static_cast<double>(f1.y), a1[e]);
            }
        }
    }
    r0 = (a0[0] + a0[1]) + (a0[2] + a0[3]);
    r1 = (a1[0] + a1[1]) + (a1[2] + a1[3]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        r0 += __shfl_xor_sync(0xffffffffu, r0, o);
        r1 += __shfl_xor_sync(0xffffffffu, r1, o);
    }
}

// Two warps per token, two tokens per CTA.  What bounds this kernel is the length of one warp's
// chain of dependent instructions and load round trips, not throughput, so the two independent
// halves of the work run side by side: the SELECT warp sums the score slabs and finds the kt-th
// largest, the NORM warp reads the x row for ||x_t||.  Lane l of the select warp holds the groups
// g = 32*j + l, j < KPL, which is also the layout of the packed mask words.  Scores map to
// unsigned keys that order like the floats; the kt-th largest key is found by a 16-step search on
// its bits, two at a time, with warp votes (no quadratic rank count), ties at that key go to the lower
// group index.  Band members (rare) are re-scored by all four warps of the CTA.
template <int KPL>
__global__ void __launch_bounds__(64 * kSelTokens, 8)   // every CTA of a 2048-token batch resident at once
select_band_kernel(const float* __restrict__ scores, int nsplit, int ld, const __nv_bfloat16* __restrict__ x,
                   const __nv_bfloat16* __restrict__ w, const float* __restrict__ wnorm, int T, int NG, int D, int k,
                   const int32_t* __restrict__ k_per_token, uint32_t* __restrict__ mask_bits,
                   float* __restrict__ scores_out, int chain) {
    __shared__ float s_xsq[kSelTokens];
    __shared__ int s_nb[kSelTokens];
    __shared__ int s_band[kSelTokens][kBandMax];
    __shared__ double s_ex[kSelTokens][kBandMax];
    wptx::grid_dep_wait();     // the score slabs come from the kernel before (see launch_select_band)
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int tt = warp >> 1;                       // token slot in the CTA
    const bool select_warp = (warp & 1) == 0;
    const int t = blockIdx.x * kSelTokens + tt;
    const bool live = t < T;                        // warp-uniform
    const int nch = D / 8;
    const int words = (NG + 31) >> 5;
    const size_t slab = static_cast<size_t>(T) * ld;
    const uint32_t lt_mask = (1u << lane) - 1u;
    const int kt = live ? min(max(k_per_token ? k_per_token[t] : k, 0), NG) : 0;
    const bool boundary = kt > 0 && kt < NG;

    float sv[KPL];
    uint32_t key[KPL];   // 0 for slots past NG, >= 1 for real groups
    bool sel[KPL], in_band[KPL];
    float wmax = 0.f, v_k = 0.f, v_k1 = 0.f;
#pragma unroll
    for (int j = 0; j < KPL; ++j) { sv[j] = 0.f; key[j] = 0u; sel[j] = false; in_band[j] = false; }

    if (!select_warp) {
        // ------------------------------------------------------------ NORM warp: ||x_t||^2
        float q[4] = {0.f, 0.f, 0.f, 0.f};
        if (boundary) {
            const uint4* xv = reinterpret_cast<const uint4*>(x + static_cast<size_t>(t) * D);
            for (int base = 0; base < nch; base += 32 * kBatch) {
                uint4 a[kBatch];
#pragma unroll
                for (int j = 0; j < kBatch; ++j) {
                    const int i = base + lane + 32 * j;
                    a[j] = i < nch ? __ldg(xv + i) : make_uint4(0u, 0u, 0u, 0u);
                }
#pragma unroll
                for (int j = 0; j < kBatch; ++j) {
                    const __nv_bfloat162* ah = reinterpret_cast<const __nv_bfloat162*>(&a[j]);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 f = __bfloat1622float2(ah[e]);
                        q[e] = fmaf(f.x, f.x, fmaf(f.y, f.y, q[e]));
                    }
                }
            }
        }
        float xsq = (q[0] + q[1]) + (q[2] + q[3]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) xsq += __shfl_xor_sync(0xffffffffu, xsq, o);
        if (lane == 0) s_xsq[tt] = xsq;
    } else if (live) {
        // ------------------------------------------------------------ SELECT warp
        // scores: every slab load of the warp is issued before the first sum
        float part[KPL][kMaxSlabs];
        float wn[KPL];
#pragma unroll
        for (int j = 0; j < KPL; ++j) {
            const int g = 32 * j + lane;
            const float* sp = scores + static_cast<size_t>(t) * ld + g;
#pragma unroll
            for (int ks = 0; ks < kMaxSlabs; ++ks) part[j][ks] = (g < NG && ks < nsplit) ? __ldg(sp + ks * slab) : 0.f;
            wn[j] = g < NG ? __ldg(wnorm + g) : 0.f;
        }
#pragma unroll
        for (int j = 0; j < KPL; ++j) {
            const int g = 32 * j + lane;
            float v = 0.f;
#pragma unroll
            for (int ks = 0; ks < kMaxSlabs; ++ks) v += part[j][ks];
            v += 0.0f;  // -0 -> +0
            sv[j] = v;
            const uint32_t u = __float_as_uint(v);
            const uint32_t ord = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
            key[j] = g < NG ? max(ord, 1u) : 0u;
            wmax = fmaxf(wmax, wn[j]);
            sel[j] = kt == NG && g < NG;
            if (scores_out && g < NG) scores_out[static_cast<size_t>(t) * NG + g] = v;
        }
        if (boundary) {
            wmax = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(wmax)));  // norms are >= 0
            // kt-th largest key, two bits per step: the three candidates of a step are counted side by side,
            // so the chain of dependent steps is half as long as a bit-by-bit search's
            uint32_t key_k = 0u;
#pragma unroll 4
            for (int bit = 30; bit >= 0; bit -= 2) {
                const uint32_t c1 = key_k | (1u << bit), c2 = key_k | (2u << bit), c3 = key_k | (3u << bit);
                int n1 = 0, n2 = 0, n3 = 0;
#pragma unroll
                for (int j = 0; j < KPL; ++j) {
                    n1 += __popc(__ballot_sync(0xffffffffu, key[j] >= c1));
                    n2 += __popc(__ballot_sync(0xffffffffu, key[j] >= c2));
                    n3 += __popc(__ballot_sync(0xffffffffu, key[j] >= c3));
                }
                key_k = n3 >= kt ? c3 : (n2 >= kt ? c2 : (n1 >= kt ? c1 : key_k));
            }
            int n_gt = 0;
#pragma unroll
            for (int j = 0; j < KPL; ++j) n_gt += __popc(__ballot_sync(0xffffffffu, key[j] > key_k));
            const int need = kt - n_gt;   // how many of the groups tied at key_k are taken (>= 1)
            int n_tie = 0;
            uint32_t below = 0u;          // largest key under key_k
#pragma unroll
            for (int j = 0; j < KPL; ++j) {
                const bool tie = key[j] == key_k;
                const uint32_t b = __ballot_sync(0xffffffffu, tie);
                sel[j] = key[j] > key_k || (tie && n_tie + __popc(b & lt_mask) < need);
                n_tie += __popc(b);
                if (key[j] < key_k) below = max(below, key[j]);
            }
            below = __reduce_max_sync(0xffffffffu, below);
            // kt-th and (kt+1)-th largest scores, back from their keys; the latter is the tied
            // value itself when more groups tie than are taken
            v_k = __uint_as_float((key_k & 0x80000000u) ? (key_k & 0x7fffffffu) : ~key_k);
            v_k1 = n_tie > need ? v_k : __uint_as_float((below & 0x80000000u) ? (below & 0x7fffffffu) : ~below);
        }
    }
    __syncthreads();   // ||x_t||^2 is there

    // band half-width 2 * eps_t (a little slack for the fp32 evaluation of the bound itself)
    int nb = 0, m_hi = 0;
    if (select_warp && boundary) {
        const float steps = static_cast<float>(chain);
        const float tau = 2.f * kAccumErr * steps * sqrtf(s_xsq[tt]) * 1.0001f * wmax;
#pragma unroll
        for (int j = 0; j < KPL; ++j) {
            const bool valid = key[j] != 0u;
            in_band[j] = valid && (sel[j] ? (sv[j] - v_k1 <= tau) : (v_k - sv[j] <= tau));
            const uint32_t b = __ballot_sync(0xffffffffu, in_band[j]);
            if (in_band[j]) {
                const int slot = nb + __popc(b & lt_mask);
                if (slot < kBandMax) s_band[tt][slot] = 32 * j + lane;
            }
            nb += __popc(b);
            m_hi += __popc(__ballot_sync(0xffffffffu, in_band[j] && sel[j]));
        }
    }
    if (select_warp && lane == 0) s_nb[tt] = nb;
    __syncthreads();   // band lists are there

    // Exact re-scoring.  The common case (at most kBandMax members per token) is spread over all
    // warps of the CTA; a longer band is re-scored by its own select warp alone.
    int total = 0;
#pragma unroll
    for (int i = 0; i < kSelTokens; ++i) total += min(s_nb[i], kBandMax);
    if (total > 0) {
        for (int item = warp; item < total; item += 2 * kSelTokens) {
            int tok = 0, i = item;
            while (i >= min(s_nb[tok], kBandMax)) { i -= min(s_nb[tok], kBandMax); ++tok; }
            const int t2 = blockIdx.x * kSelTokens + tok;
            const double e = warp_dot_f64(x + static_cast<size_t>(t2) * D, w + static_cast<size_t>(s_band[tok][i]) * D, nch, lane);
            if (lane == 0) s_ex[tok][i] = e;
        }
    }
    __syncthreads();   // exact scores are there

    if (select_warp && nb > 0) {   // then the band holds at least the two groups on either side of the boundary
        double ex[KPL];
        int seen = 0;
#pragma unroll
        for (int j = 0; j < KPL; ++j) {
            ex[j] = 0.0;
            uint32_t bits = __ballot_sync(0xffffffffu, in_band[j]);
            const int first = seen;
            seen += __popc(bits);
            if (nb <= kBandMax) {
                if (in_band[j]) ex[j] = s_ex[tt][first + __popc(bits & lt_mask)];
            } else {
                while (bits) {
                    const int l = __ffs(bits) - 1;
                    bits &= bits - 1;
                    const double e = warp_dot_f64(x + static_cast<size_t>(t) * D, w + static_cast<size_t>(32 * j + l) * D, nch, lane);
                    if (lane == l) ex[j] = e;
                }
            }
        }
        // band members are re-ranked among themselves on the exact scores
        int beats[KPL];
#pragma unroll
        for (int j = 0; j < KPL; ++j) beats[j] = 0;
#pragma unroll
        for (int j = 0; j < KPL; ++j) {
            uint32_t bits = __ballot_sync(0xffffffffu, in_band[j]);
            while (bits) {
                const int l = __ffs(bits) - 1;
                bits &= bits - 1;
                const double u = __shfl_sync(0xffffffffu, ex[j], l);
                const int h = 32 * j + l;
#pragma unroll
                for (int jj = 0; jj < KPL; ++jj) beats[jj] += (u > ex[jj]) || (u == ex[jj] && h < 32 * jj + lane);
            }
        }
#pragma unroll
        for (int j = 0; j < KPL; ++j)
            if (in_band[j]) sel[j] = beats[j] < m_hi;
    }
    if (select_warp && live) {
#pragma unroll
        for (int j = 0; j < KPL; ++j) {
            const uint32_t word = __ballot_sync(0xffffffffu, sel[j]);
            if (lane == 0 && j < words) mask_bits[static_cast<size_t>(t) * words + j] = word;
        }
    }
}

template <int KPL>
void launch_select_band(cudaStream_t s, int T, const float* sc32, int ksplit, int ld, const __nv_bfloat16* x,
                        const __nv_bfloat16* w, const float* wn, int NG, int D, int k, const int32_t* k_per_token,
                        uint32_t* mask_bits, float* scores, int chain, bool dependent) {
    // behind the score GEMM of the same call: as its programmatic dependent the launch overlaps that kernel's tail
    // (the kernel waits before it touches memory); the ordinary way while per-kernel timing brackets every launch
    if (dependent)
        wide_launch_dependent(select_band_kernel<KPL>, dim3((T + kSelTokens - 1) / kSelTokens), dim3(64 * kSelTokens), 0, s, sc32,
                              ksplit, ld, x, w, wn, T, NG, D, k, k_per_token, mask_bits, scores, chain);
    else
        select_band_kernel<KPL><<<(T + kSelTokens - 1) / kSelTokens, 64 * kSelTokens, 0, s>>>(
            sc32, ksplit, ld, x, w, wn, T, NG, D, k, k_per_token, mask_bits, scores, chain);
}

// ---------------------------------------------------------------------------- small batches (decode), top-k
// One launch for at most kRsMaxTokens tokens.  A CTA takes eight tokens, eight groups and one of KS
// slices of the hidden dimension: the tokens' slices of x sit in shared memory, a warp streams its
// slice of one row of the router weight once (one round trip) and forms fp32 partial scores against all
// eight tokens on the CUDA cores (a lane accumulates every 32nd 16-byte piece, the lanes' sums are added
// by shuffles), with its part of ||w_g||^2 and ||x_t||^2 on the side.  Partial scores and norms go to
// the scratch; the CTA that arrives last for a tile of tokens (a ticket per tile, put back to zero by
// that CTA) selects: one warp per token adds the KS partials in a fixed order and then runs the same
// bitwise search for the k-th largest score, the same band of half-width 2 * eps_t around the boundary
// and the same exact fp64 re-scoring of the band's members as select_band_kernel, here with
//   eps_t = 1.01 * 2^-24 * (D / (32 KS) + 5 + KS) * ||x_t|| * max_g ||w_g||:
// every score is the end of a chain of at most D / (32 KS) fused multiply-adds in a lane, five shuffle
// additions and KS - 1 additions of the partials, each an IEEE operation rounded to nearest (relative
// error 2^-24, unlike the tensor core's unspecified accumulator), so its error is at most
// gamma_n * sum |x_i w_i| with n the chain length, and the sum is at most ||x|| ||w|| (Cauchy-Schwarz);
// the factor 1.01 covers the second-order terms of gamma_n.  The norms of the weight rows are the same for every
// tile of tokens: every tile writes them, with the same bits, to the same place.
constexpr int kRsTokens = 8;
constexpr int kRsGroups = 8;
constexpr int kRsMaxTokens = 64;

// scratch of the one-launch router, in floats: partial scores [KS][T][NG], partial ||w||^2 [KS][NG],
// partial ||x||^2 [T][KS]
__host__ __device__ inline size_t route_small_floats(int T, int NG, int KS) {
    return static_cast<size_t>(KS) * (static_cast<size_t>(T) * NG + NG + T);
}

template <int KPL>
__global__ void __launch_bounds__(32 * kRsGroups)
route_small_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ w, int T, int NG, int D, int k,
                   const int32_t* __restrict__ k_per_token, uint32_t* __restrict__ mask_bits, float* __restrict__ scores_out,
                   float* __restrict__ scratch, int KS, int ppq, unsigned* __restrict__ tickets) {
    extern __shared__ uint4 rs_smem[];   // x slices of the tile's tokens, bf16 [kRsTokens][ppq pieces]
    __shared__ int s_last;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nch = D / 8;
    const int chunk = blockIdx.x / KS, kq = blockIdx.x - chunk * KS;
    const int q_lo = min(nch, kq * ppq), q_hi = min(nch, q_lo + ppq);   // this slice's pieces of a row
    const int t0 = blockIdx.y * kRsTokens;
    const int nt = min(kRsTokens, T - t0);
    float* slab = scratch;                                          // [KS][T][NG]
    float* wsq_part = scratch + static_cast<size_t>(KS) * T * NG;   // [KS][NG]
    float* xsq_part = wsq_part + static_cast<size_t>(KS) * NG;      // [T][KS]
    const uint4* x4 = reinterpret_cast<const uint4*>(x);
    for (int tt = warp; tt < kRsTokens; tt += kRsGroups) {
        for (int p = lane; p < ppq; p += 32)
            rs_smem[tt * ppq + p] = (tt < nt && q_lo + p < q_hi) ? __ldg(x4 + static_cast<size_t>(t0 + tt) * nch + q_lo + p)
                                                                 : make_uint4(0u, 0u, 0u, 0u);
    }
    __syncthreads();

    // ---- partial scores of this warp's group against the tile's tokens
    const int g = chunk * kRsGroups + warp;
    if (g < NG) {
        const uint4* w4 = reinterpret_cast<const uint4*>(w + static_cast<size_t>(g) * D) + q_lo;
        float acc[kRsTokens];
#pragma unroll
        for (int tt = 0; tt < kRsTokens; ++tt) acc[tt] = 0.f;
        float wsq = 0.f;
        for (int base = 0; base < q_hi - q_lo; base += 32 * kBatch) {
            uint4 wv[kBatch];
#pragma unroll
            for (int j = 0; j < kBatch; ++j) {
                const int i = base + lane + 32 * j;
                wv[j] = i < q_hi - q_lo ? __ldg(w4 + i) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int j = 0; j < kBatch; ++j) {
                const int i = base + lane + 32 * j;
                if (i < q_hi - q_lo) {
                    const uint32_t ww[4] = {wv[j].x, wv[j].y, wv[j].z, wv[j].w};
                    float wf[8];
#pragma unroll
                    for (int p = 0; p < 4; ++p) {
                        wf[2 * p] = __uint_as_float(ww[p] << 16);
                        wf[2 * p + 1] = __uint_as_float(ww[p] & 0xffff0000u);
                        wsq = fmaf(wf[2 * p], wf[2 * p], fmaf(wf[2 * p + 1], wf[2 * p + 1], wsq));
                    }
#pragma unroll
                    for (int tt = 0; tt < kRsTokens; ++tt) {
                        if (tt < nt) {
                            const uint4 xv = rs_smem[tt * ppq + i];
                            const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
                            for (int p = 0; p < 4; ++p) {
                                acc[tt] = fmaf(wf[2 * p], __uint_as_float(xw[p] << 16), acc[tt]);
                                acc[tt] = fmaf(wf[2 * p + 1], __uint_as_float(xw[p] & 0xffff0000u), acc[tt]);
                            }
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) wsq += __shfl_xor_sync(0xffffffffu, wsq, o);
#pragma unroll
        for (int tt = 0; tt < kRsTokens; ++tt) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc[tt] += __shfl_xor_sync(0xffffffffu, acc[tt], o);
            if (lane == tt && tt < nt) slab[(static_cast<size_t>(kq) * T + t0 + tt) * NG + g] = acc[tt];
        }
        if (lane == 0) wsq_part[kq * NG + g] = wsq;   // the same bits from every tile of tokens
    }
    if (chunk == 0 && warp < nt) {
        // this slice's part of ||x_t||^2, token t0 + warp
        float xsq = 0.f;
        for (int p = lane; p < ppq; p += 32) {
            const uint4 xv = rs_smem[warp * ppq + p];
            const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float a = __uint_as_float(xw[q] << 16), b = __uint_as_float(xw[q] & 0xffff0000u);
                xsq = fmaf(a, a, fmaf(b, b, xsq));
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) xsq += __shfl_xor_sync(0xffffffffu, xsq, o);
        if (lane == 0) xsq_part[(t0 + warp) * KS + kq] = xsq;
    }

    // ---- the CTA that completes the tile's scores selects
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const unsigned old = atomicAdd(tickets + blockIdx.y, 1u);
        s_last = old + 1u == gridDim.x ? 1 : 0;
        if (s_last) tickets[blockIdx.y] = 0u;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    const int t = t0 + warp;
    if (warp >= nt) return;
    const int words = (NG + 31) >> 5;
    const uint32_t lt_mask = (1u << lane) - 1u;
    const int kt = min(max(k_per_token ? k_per_token[t] : k, 0), NG);
    const bool boundary = kt > 0 && kt < NG;
    // (the partials are read with loops of fixed length, so that all loads are on their way before the first sum)
    float xsq = 0.f;
    {
        float part[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) part[q] = q < KS ? __ldcg(xsq_part + t * KS + q) : 0.f;
#pragma unroll
        for (int q = 0; q < 4; ++q) xsq += part[q];
    }

    float sv[KPL];
    uint32_t key[KPL];   // 0 for slots past NG, >= 1 for real groups
    bool sel[KPL], in_band[KPL];
    float wmax = 0.f, v_k = 0.f, v_k1 = 0.f;
    float sp[KPL][4], wp[KPL][4];
#pragma unroll
    for (int j = 0; j < KPL; ++j) {
        const int gg = 32 * j + lane;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const bool live = gg < NG && q < KS;
            sp[j][q] = live ? __ldcg(slab + (static_cast<size_t>(q) * T + t) * NG + gg) : 0.f;
            wp[j][q] = live ? __ldcg(wsq_part + q * NG + gg) : 0.f;
        }
    }
#pragma unroll
    for (int j = 0; j < KPL; ++j) {
        const int gg = 32 * j + lane;
        float v = 0.f, wn = 0.f;
#pragma unroll
        for (int q = 0; q < 4; ++q) {   // slices beyond KS add an exact zero
            v += sp[j][q];
            wn += wp[j][q];
        }
        v += 0.0f;  // -0 -> +0
        sv[j] = v;
        const uint32_t u = __float_as_uint(v);
        const uint32_t ord = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
        key[j] = gg < NG ? max(ord, 1u) : 0u;
        wmax = fmaxf(wmax, wn);
        sel[j] = kt == NG && gg < NG;
        in_band[j] = false;
        if (scores_out && gg < NG) scores_out[static_cast<size_t>(t) * NG + gg] = v;
    }
    int nb = 0, m_hi = 0;
    if (boundary) {
        wmax = sqrtf(__uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(wmax)))) * 1.0001f;  // norms are >= 0
        // kt-th largest key, two bits per step: the three candidates of a step are counted side by side, so
        // the chain of dependent steps is half as long as a bit-by-bit search's
        uint32_t key_k = 0u;
#pragma unroll 4
        for (int bit = 30; bit >= 0; bit -= 2) {
            const uint32_t c1 = key_k | (1u << bit), c2 = key_k | (2u << bit), c3 = key_k | (3u << bit);
            int n1 = 0, n2 = 0, n3 = 0;
#pragma unroll
            for (int j = 0; j < KPL; ++j) {
                n1 += __popc(__ballot_sync(0xffffffffu, key[j] >= c1));
                n2 += __popc(__ballot_sync(0xffffffffu, key[j] >= c2));
                n3 += __popc(__ballot_sync(0xffffffffu, key[j] >= c3));
            }
            key_k = n3 >= kt ? c3 : (n2 >= kt ? c2 : (n1 >= kt ? c1 : key_k));
        }
        int n_gt = 0;
#pragma unroll
        for (int j = 0; j < KPL; ++j) n_gt += __popc(__ballot_sync(0xffffffffu, key[j] > key_k));
        const int need = kt - n_gt;   // how many of the groups tied at key_k are taken (>= 1)
        int n_tie = 0;
        uint32_t below = 0u;          // largest key under key_k
#pragma unroll
        for (int j = 0; j < KPL; ++j) {
            const bool tie = key[j] == key_k;
            const uint32_t b = __ballot_sync(0xffffffffu, tie);
            sel[j] = key[j] > key_k || (tie && n_tie + __popc(b & lt_mask) < need);
            n_tie += __popc(b);
            if (key[j] < key_k) below = max(below, key[j]);
        }
        below = __reduce_max_sync(0xffffffffu, below);
        v_k = __uint_as_float((key_k & 0x80000000u) ? (key_k & 0x7fffffffu) : ~key_k);
        v_k1 = n_tie > need ? v_k : __uint_as_float((below & 0x80000000u) ? (below & 0x7fffffffu) : ~below);
        // band half-width 2 * eps_t (a little slack for the fp32 evaluation of the bound itself)
        // ppq / 4 >= D / (32 KS) multiply-adds per lane; 1.001: the bound itself is evaluated in fp32 from
        // norms that were summed in fp32
        const float tau = 2.f * 1.01f * 5.9604645e-8f * static_cast<float>(ppq / 4 + 5 + KS) * sqrtf(xsq) * 1.001f * wmax;
#pragma unroll
        for (int j = 0; j < KPL; ++j) {
            const bool valid = key[j] != 0u;
            in_band[j] = valid && (sel[j] ? (sv[j] - v_k1 <= tau) : (v_k - sv[j] <= tau));
            nb += __popc(__ballot_sync(0xffffffffu, in_band[j]));
            m_hi += __popc(__ballot_sync(0xffffffffu, in_band[j] && sel[j]));
        }
    }
    if (nb > 0) {   // then the band holds at least the two groups on either side of the boundary
        // exact scores of the band's members, two at a time (the same value whichever way a member is paired:
        // each dot product has its own accumulators and the same order of operations)
        double ex[KPL];
#pragma unroll
        for (int j = 0; j < KPL; ++j) ex[j] = 0.0;
        const __nv_bfloat16* xrow = x + static_cast<size_t>(t) * D;
        int pend = -1;   // a member waiting for a partner
#pragma unroll
        for (int j = 0; j < KPL; ++j) {
            uint32_t bits = __ballot_sync(0xffffffffu, in_band[j]);
            while (bits) {
                const int h = 32 * j + __ffs(bits) - 1;
                bits &= bits - 1;
                if (pend < 0) {
                    pend = h;
                    continue;
                }
                double e0, e1;
                warp_dot_f64_x2(xrow, w + static_cast<size_t>(pend) * D, w + static_cast<size_t>(h) * D, nch, lane, e0, e1);
#pragma unroll
                for (int jj = 0; jj < KPL; ++jj) {
                    if (32 * jj + lane == pend) ex[jj] = e0;
                    if (32 * jj + lane == h) ex[jj] = e1;
                }
                pend = -1;
            }
        }
        if (pend >= 0) {
            const double e = warp_dot_f64(xrow, w + static_cast<size_t>(pend) * D, nch, lane);
#pragma unroll
            for (int jj = 0; jj < KPL; ++jj)
                if (32 * jj + lane == pend) ex[jj] = e;
        }
        // band members are re-ranked among themselves on the exact scores
        int beats[KPL];
#pragma unroll
        for (int j = 0; j < KPL; ++j) beats[j] = 0;
#pragma unroll
        for (int j = 0; j < KPL; ++j) {
            uint32_t bits = __ballot_sync(0xffffffffu, in_band[j]);
            while (bits) {
                const int l = __ffs(bits) - 1;
                bits &= bits - 1;
                const double u = __shfl_sync(0xffffffffu, ex[j], l);
                const int h = 32 * j + l;
#pragma unroll
                for (int jj = 0; jj < KPL; ++jj) beats[jj] += (u > ex[jj]) || (u == ex[jj] && h < 32 * jj + lane);
            }
        }
#pragma unroll
        for (int j = 0; j < KPL; ++j)
            if (in_band[j]) sel[j] = beats[j] < m_hi;
    }
#pragma unroll
    for (int j = 0; j < KPL; ++j) {
        const uint32_t word = __ballot_sync(0xffffffffu, sel[j]);
        if (lane == 0 && j < words) mask_bits[static_cast<size_t>(t) * words + j] = word;
    }
}

template <int KPL>
int launch_route_small(cudaStream_t s, int T, const __nv_bfloat16* x, const __nv_bfloat16* w, int NG, int D, int k,
                       const int32_t* k_per_token, uint32_t* mask_bits, float* scores, float* scratch, int KS,
                       unsigned* tickets) {
    const int ppq = ((D / 8 + KS - 1) / KS + 31) / 32 * 32;   // 16-byte pieces of a row per slice
    const int smem = kRsTokens * ppq * 16;
    if (cudaFuncSetAttribute(route_small_kernel<KPL>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
        return WIDE_ERR_CUDA;
    route_small_kernel<KPL><<<dim3((NG + kRsGroups - 1) / kRsGroups * KS, (T + kRsTokens - 1) / kRsTokens), 32 * kRsGroups, smem, s>>>(
        x, w, T, NG, D, k, k_per_token, mask_bits, scores, scratch, KS, ppq, tickets);
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}

// ---------------------------------------------------------------------------- fast pair-argmax path (bf16)
// Eq. 4 with the bottleneck product on the tensor cores: u = x W1 comes from the same K-split
// score GEMM as the top-k form (W1 transposed once per call, its rank <= 32 columns are the
// "groups"), with the same rigorous bound on its error.  The logits l = u W2 are then formed in
// fp32 per token and a pair is decided when its margin |l0 - l1| exceeds everything the errors of
// u and of the fp32 product can add up to.  A pair that is too close to call (about one in 140
// with Gaussian weights) is marked and decided by a second kernel from
//     l0 - l1 = x . d_g,   d_g = W1 (W2[:, 2g] - W2[:, 2g+1])   (d_g in fp64, once per call),
// one fp64 dot product of length D per marked pair.  fp64 FMAs are scarce on this part (a few per
// clock and SM), which is why they are kept for the marked pairs.  If even that dot product is
// within 2^-36 of zero relative to ||x|| ||d_g|| (an exact tie, in practice), the token is redone the
// long way, u = x W1 and l = u W2 in fp64, which is the definition.
constexpr int kPairMaxRank = 32;

__global__ void __launch_bounds__(256)
transpose_w1_kernel(const __nv_bfloat16* __restrict__ w1, int D, int rank, int NG, __nv_bfloat16* __restrict__ w1t,
                    float* __restrict__ dn2) {
    for (int g = blockIdx.x * blockDim.x + threadIdx.x; g < NG; g += gridDim.x * blockDim.x) dn2[g] = 0.f;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < static_cast<long long>(D) * rank;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int c = static_cast<int>(i / D), d = static_cast<int>(i % D);
        w1t[i] = w1[static_cast<size_t>(d) * rank + c];
    }
}

// d64[g][i] = sum_c W1[i][c] (W2[c][2g] - W2[c][2g+1]) in fp64; dn2[g] += sum_i d^2 (fp32, rounded up).
// Block = 128 rows i x 32 groups.
__global__ void __launch_bounds__(128)
pair_delta_kernel(const __nv_bfloat16* __restrict__ w1, const __nv_bfloat16* __restrict__ w2, int D, int rank, int NG,
                  double* __restrict__ d64, float* __restrict__ dn2, const __nv_bfloat16* __restrict__ gamma = nullptr) {
    __shared__ double delta[kPairMaxRank][32];
    __shared__ float sq[32];
    const int tid = threadIdx.x, g0 = blockIdx.y * 32, i = blockIdx.x * 128 + tid;
    for (int e = tid; e < rank * 32; e += 128) {
        const int c = e / 32, g = g0 + e % 32;
        delta[c][e % 32] = g < NG ? static_cast<double>(__bfloat162float(w2[static_cast<size_t>(c) * 2 * NG + 2 * g])) -
                                        static_cast<double>(__bfloat162float(w2[static_cast<size_t>(c) * 2 * NG + 2 * g + 1]))
                                  : 0.0;
    }
    if (tid < 32) sq[tid] = 0.f;
    __syncthreads();
    double w[kPairMaxRank];
    const double gi = (gamma && i < D) ? static_cast<double>(__bfloat162float(gamma[i])) : 1.0;   // row i of diag(gamma) W1
#pragma unroll
    for (int c = 0; c < kPairMaxRank; ++c)
        w[c] = (c < rank && i < D) ? gi * static_cast<double>(__bfloat162float(w1[static_cast<size_t>(i) * rank + c])) : 0.0;
    for (int gg = 0; gg < 32 && g0 + gg < NG; ++gg) {
        double a = 0.0;
#pragma unroll
        for (int c = 0; c < kPairMaxRank; ++c)
            if (c < rank) a = fma(w[c], delta[c][gg], a);
        if (i < D) d64[static_cast<size_t>(g0 + gg) * D + i] = a;
        float q = static_cast<float>(a);
        q = q * q * 1.0001f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
        if ((tid & 31) == 0) atomicAdd(&sq[gg], q);
    }
    __syncthreads();
    if (tid < 32 && g0 + tid < NG) atomicAdd(dn2 + g0 + tid, sq[tid]);
}

// One warp per token.  Lane c holds u_c (c < rank); lane l decides the groups l, l + 32, ...
__global__ void __launch_bounds__(128)
pair_band_kernel(const float* __restrict__ u_slabs, int nsplit, int ld, const __nv_bfloat16* __restrict__ x,
                 const __nv_bfloat16* __restrict__ w2, const float* __restrict__ wnorm, int T, int NG, int D, int rank,
                 uint32_t* __restrict__ mask_bits, float* __restrict__ scores_out, uint32_t* __restrict__ close_bits,
                 int chain, int split = 0, float norm_eps = -1.f) {
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * 4 + (threadIdx.x >> 5);
    if (t >= T) return;
    const int words = (NG + 31) >> 5;
    const size_t slab = static_cast<size_t>(T) * ld;
    // split: the bottleneck weights were given as a bf16 pair (hi in columns [0, rank), lo behind them)
    float u = 0.f;
    if (lane < rank)
        for (int ks = 0; ks < nsplit; ++ks) {
            u += __ldg(u_slabs + ks * slab + static_cast<size_t>(t) * ld + lane);
            if (split) u += __ldg(u_slabs + ks * slab + static_cast<size_t>(t) * ld + rank + lane);
        }
    // ||x_t||
    float xsq = 0.f;
    const uint4* xv = reinterpret_cast<const uint4*>(x + static_cast<size_t>(t) * D);
    for (int i = lane; i < D / 8; i += 32) {
        const uint4 a = __ldg(xv + i);
        const __nv_bfloat162* ah = reinterpret_cast<const __nv_bfloat162*>(&a);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(ah[e]);
            xsq = fmaf(f.x, f.x, fmaf(f.y, f.y, xsq));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) xsq += __shfl_xor_sync(0xffffffffu, xsq, o);
    // error bound of u_c (see the top-k form), then of the fp32 product below
    const float steps = static_cast<float>(chain);
    float eu = lane < rank ? kAccumErr * steps * sqrtf(xsq) * 1.0001f * __ldg(wnorm + lane) : 0.f;
    if (split && lane < rank)   // the lo product's accumulation error, the hi + lo sum, and what the pair leaves out (2^-18 |w|)
        eu += sqrtf(xsq) * 1.0001f * (kAccumErr * steps * __ldg(wnorm + rank + lane) + 7.6293945e-6f * __ldg(wnorm + lane)) +
              kAccumErr * fabsf(u);
    const float au = fabsf(u);
    // the logits of the normalised input differ from these by the positive factor 1 / rms(x_t)
    const float out_scale = norm_eps >= 0.f ? rsqrtf(xsq / static_cast<float>(D) + norm_eps) : 1.f;
    if (lane == 0) close_bits[static_cast<size_t>(t) * 32 + 31] = __float_as_uint(sqrtf(xsq) * 1.0001f);
    for (int j = 0; j < words; ++j) {
        const int g = 32 * j + lane;
        float l0 = 0.f, l1 = 0.f, band = 0.f, mag = 0.f;
        for (int c = 0; c < rank; ++c) {
            const float uc = __shfl_sync(0xffffffffu, u, c), ec = __shfl_sync(0xffffffffu, eu, c);
            const float ac = __shfl_sync(0xffffffffu, au, c);
            if (g < NG) {
                const float a0 = __bfloat162float(w2[static_cast<size_t>(c) * 2 * NG + 2 * g]);
                const float a1 = __bfloat162float(w2[static_cast<size_t>(c) * 2 * NG + 2 * g + 1]);
                l0 = fmaf(uc, a0, l0);
                l1 = fmaf(uc, a1, l1);
                const float aa = fabsf(a0) + fabsf(a1);
                band = fmaf(ec, aa, band);
                mag = fmaf(ac, aa, mag);
            }
        }
        // fp32 rounding of the two sums and of their difference: (rank + 2) * 2^-24 * sum |u||a|
        band = (band + static_cast<float>(rank + 2) * kAccumErr * mag) * 1.001f;
        const bool sel = g < NG && l0 >= l1;
        const bool close = g < NG && fabsf(l0 - l1) <= band;
        const unsigned word = __ballot_sync(0xffffffffu, sel), cword = __ballot_sync(0xffffffffu, close);
        if (lane == 0) {
            mask_bits[static_cast<size_t>(t) * words + j] = word;
            close_bits[static_cast<size_t>(t) * 32 + j] = cword;
        }
        if (scores_out && g < NG) {
            scores_out[static_cast<size_t>(t) * 2 * NG + 2 * g] = l0 * out_scale;
            scores_out[static_cast<size_t>(t) * 2 * NG + 2 * g + 1] = l1 * out_scale;
        }
    }
}

// The marked pairs, exactly.  One block per token (most have nothing marked and leave at once).
__global__ void __launch_bounds__(128)
pair_exact_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ w1,
                  const __nv_bfloat16* __restrict__ w2, const double* __restrict__ d64, const float* __restrict__ dn2,
                  int T, int D, int rank, int NG, const uint32_t* __restrict__ close_bits,
                  uint32_t* __restrict__ mask_bits, float* __restrict__ scores_out,
                  const __nv_bfloat16* __restrict__ gamma = nullptr, float norm_eps = -1.f) {
    __shared__ double s_part[4];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int words = (NG + 31) >> 5;
    for (int t = blockIdx.x; t < T; t += gridDim.x) {
        const uint32_t cw = close_bits[static_cast<size_t>(t) * 32 + lane];   // words [0, W) marks, word 31 ||x||
        if (!__any_sync(0xffffffffu, lane < words && cw != 0u)) continue;      // the same in all four warps
        const __nv_bfloat16* xr = x + static_cast<size_t>(t) * D;
        const float xnorm = __uint_as_float(__shfl_sync(0xffffffffu, cw, 31));
        const float out_scale = norm_eps >= 0.f ? rsqrtf(xnorm * xnorm / static_cast<float>(D) + norm_eps) : 1.f;
        bool long_way = false;
        for (int j = 0; j < words; ++j) {
            uint32_t bits = __shfl_sync(0xffffffffu, cw, j);
            uint32_t word = mask_bits[static_cast<size_t>(t) * words + j];
            while (bits) {
                const int b = __ffs(bits) - 1;
                bits &= bits - 1;
                const int g = 32 * j + b;
                const double* dr = d64 + static_cast<size_t>(g) * D;
                // eight consecutive elements per thread and step: one 16-byte load of x, four of d_g
                double acc[8] = {0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0};
#pragma unroll 4
                for (int i = threadIdx.x * 8; i < D; i += 1024) {
                    const uint4 xa = *reinterpret_cast<const uint4*>(xr + i);
                    const __nv_bfloat162* xh = reinterpret_cast<const __nv_bfloat162*>(&xa);
                    const double2* dv = reinterpret_cast<const double2*>(dr + i);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 f = __bfloat1622float2(xh[e]);
                        const double2 d = dv[e];
                        acc[2 * e] = fma(static_cast<double>(f.x), d.x, acc[2 * e]);
                        acc[2 * e + 1] = fma(static_cast<double>(f.y), d.y, acc[2 * e + 1]);
                    }
                }
                double m = ((acc[0] + acc[1]) + (acc[2] + acc[3])) + ((acc[4] + acc[5]) + (acc[6] + acc[7]));
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) m += __shfl_xor_sync(0xffffffffu, m, o);
                if (lane == 0) s_part[warp] = m;
                __syncthreads();
                m = (s_part[0] + s_part[1]) + (s_part[2] + s_part[3]);
                __syncthreads();
                if (fabs(m) <= 1.4551915e-11 * static_cast<double>(xnorm * sqrtf(dn2[g]) * 1.001f)) long_way = true;   // 2^-36
                word = m >= 0.0 ? (word | (1u << b)) : (word & ~(1u << b));
                if (scores_out && threadIdx.x == 0) {
                    // keep the pair's mean, set its difference to the exact one
                    float* sp = scores_out + static_cast<size_t>(t) * 2 * NG + 2 * g;
                    const float mid = 0.5f * (sp[0] + sp[1]);
                    sp[0] = mid + 0.5f * static_cast<float>(m) * out_scale;
                    sp[1] = mid - 0.5f * static_cast<float>(m) * out_scale;
                }
            }
            if (threadIdx.x == 0) mask_bits[static_cast<size_t>(t) * words + j] = word;
        }
        if (long_way && warp == 0) {
            // the definition: u = x W1, l = u W2, all in fp64
            double uu = 0.0;   // lane c ends up with u_c
            for (int c = 0; c < rank; ++c) {
                double a = 0.0;
                for (int i = lane; i < D; i += 32) {
                    double xi = static_cast<double>(__bfloat162float(xr[i]));
                    if (gamma) xi *= static_cast<double>(__bfloat162float(gamma[i]));   // exact: 16 significant bits
                    a = fma(xi, static_cast<double>(__bfloat162float(w1[static_cast<size_t>(i) * rank + c])), a);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
                if (lane == c) uu = a;
            }
            for (int j = 0; j < words; ++j) {
                const int g = 32 * j + lane;
                double l0 = 0.0, l1 = 0.0;
                for (int c = 0; c < rank; ++c) {
                    const double uc = __shfl_sync(0xffffffffu, uu, c);
                    if (g < NG) {
                        l0 = fma(uc, static_cast<double>(__bfloat162float(w2[static_cast<size_t>(c) * 2 * NG + 2 * g])), l0);
                        l1 = fma(uc, static_cast<double>(__bfloat162float(w2[static_cast<size_t>(c) * 2 * NG + 2 * g + 1])), l1);
                    }
                }
                const unsigned word = __ballot_sync(0xffffffffu, g < NG && l0 >= l1);
                if (lane == 0) mask_bits[static_cast<size_t>(t) * words + j] = word;
                if (scores_out && g < NG) {
                    scores_out[static_cast<size_t>(t) * 2 * NG + 2 * g] = static_cast<float>(l0) * out_scale;
                    scores_out[static_cast<size_t>(t) * 2 * NG + 2 * g + 1] = static_cast<float>(l1) * out_scale;
                }
            }
        }
    }
}

// Prepared form of the bottleneck weights for wide_route_pair_norm: row c of w1t is column c of
// diag(gamma) W1 rounded to bf16 (hi), row rank + c what that rounding left over, again in bf16 (lo).
// gamma[i] * W1[i][c] has 16 significant bits, so it is exact in fp32 and hi + lo misses it by at
// most 2^-18 of its size.
__global__ void __launch_bounds__(256)
pair_prepare_w1_kernel(const __nv_bfloat16* __restrict__ w1, const __nv_bfloat16* __restrict__ gamma, int D, int rank, int NG,
                       __nv_bfloat16* __restrict__ w1t, float* __restrict__ dn2) {
    for (int g = blockIdx.x * blockDim.x + threadIdx.x; g < NG; g += gridDim.x * blockDim.x) dn2[g] = 0.f;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < static_cast<long long>(D) * rank;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int c = static_cast<int>(i / D), d = static_cast<int>(i % D);
        const float p = __bfloat162float(w1[static_cast<size_t>(d) * rank + c]) * (gamma ? __bfloat162float(gamma[d]) : 1.f);
        const __nv_bfloat16 hi = __float2bfloat16_rn(p);
        w1t[i] = hi;
        w1t[static_cast<size_t>(rank) * D + i] = __float2bfloat16_rn(p - __bfloat162float(hi));
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

// ---- Eq. 4 on the RMSNorm of the hidden state, with the weight-only work done once (prepare)
namespace {
struct PairPrepared {
    __nv_bfloat16* w1t;   // [2 rank, D]
    double* d64;          // [NG, D]
    float* dn2;           // [NG]
};
PairPrepared carve_prepared(void* base, int D, int rank, int NG) {
    char* b = static_cast<char*>(base);
    PairPrepared p;
    p.w1t = reinterpret_cast<__nv_bfloat16*>(b);
    b += wide_align_up(static_cast<size_t>(2) * rank * D * 2, 256);
    p.d64 = reinterpret_cast<double*>(b);
    b += wide_align_up(static_cast<size_t>(NG) * D * sizeof(double), 256);
    p.dn2 = reinterpret_cast<float*>(b);
    return p;
}
}  // namespace

size_t wide_route_pair_prepared_size(int D, int rank, int NG) {
    return wide_align_up(static_cast<size_t>(2) * rank * D * 2, 256) + wide_align_up(static_cast<size_t>(NG) * D * sizeof(double), 256) +
           wide_align_up(static_cast<size_t>(NG) * sizeof(float), 256);
}

bool wide_route_pair_norm_supported(int D, int rank, int NG) {
    return D % 64 == 0 && D <= 16384 && rank <= kPairMaxRank && rank % 8 == 0 && NG <= 192;
}

int wide_launch_route_pair_prepare(wide_ctx* ctx, cudaStream_t s, const void* w1, const void* w2, const void* gamma, int D,
                                   int rank, int NG, void* prepared) {
    const PairPrepared p = carve_prepared(prepared, D, rank, NG);
    const __nv_bfloat16* w1b = static_cast<const __nv_bfloat16*>(w1);
    const __nv_bfloat16* gb = static_cast<const __nv_bfloat16*>(gamma);
    {
        WideLaunch l(ctx, s, "route_pair_prepare_w1");
        pair_prepare_w1_kernel<<<64, 256, 0, s>>>(w1b, gb, D, rank, NG, p.w1t, p.dn2);
    }
    WideLaunch l(ctx, s, "route_pair_delta");
    pair_delta_kernel<<<dim3((D + 127) / 128, (NG + 31) / 32), 128, 0, s>>>(w1b, static_cast<const __nv_bfloat16*>(w2), D, rank,
                                                                             NG, p.d64, p.dn2, gb);
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}

size_t wide_route_pair_norm_workspace(int T, int rank) {
    const int ld = (2 * rank + 31) / 32 * 32;
    return wide_align_up(static_cast<size_t>(T) * ld * sizeof(float) * kMaxSlabs, 256) + wide_align_up(static_cast<size_t>(T) * 128, 256) + 1024;
}

int wide_launch_route_pair_norm(wide_ctx* ctx, cudaStream_t s, const void* x, int T, int D, const void* w1, const void* w2,
                                int rank, int NG, const void* gamma, float eps, void* prepared, uint32_t* mask_bits,
                                float* scores, void* ws) {
    if (T == 0) return WIDE_OK;
    const PairPrepared p = carve_prepared(prepared, D, rank, NG);
    const int ld = (2 * rank + 31) / 32 * 32;
    char* wsb = static_cast<char*>(ws);
    float* slabs = reinterpret_cast<float*>(wsb);
    const size_t off1 = wide_align_up(static_cast<size_t>(T) * ld * sizeof(float) * kMaxSlabs, 256);
    uint32_t* close_bits = reinterpret_cast<uint32_t*>(wsb + off1);
    float* wn = reinterpret_cast<float*>(wsb + off1 + wide_align_up(static_cast<size_t>(T) * 128, 256));
    const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(x);
    const __nv_bfloat16* w2b = static_cast<const __nv_bfloat16*>(w2);
    int ksplit = 1, chain = D;
    const int rc = wide_launch_scores_tc(ctx, s, x, p.w1t, T, 2 * rank, ld, D, slabs, wn, kMaxSlabs, &ksplit, &chain);
    if (rc != WIDE_OK) return rc;
    {
        WideLaunch l(ctx, s, "route_pair_band");
        pair_band_kernel<<<(T + 3) / 4, 128, 0, s>>>(slabs, ksplit, ld, xb, w2b, wn, T, NG, D, rank, mask_bits, scores, close_bits,
                                                      chain, 1, eps);
    }
    WideLaunch l(ctx, s, "route_pair_exact");
    const int grid = T < 16 * ctx->sm_count ? T : 16 * ctx->sm_count;
    pair_exact_kernel<<<grid, 128, 0, s>>>(xb, static_cast<const __nv_bfloat16*>(w1), w2b, p.d64, p.dn2, T, D, rank, NG,
                                           close_bits, mask_bits, scores, static_cast<const __nv_bfloat16*>(gamma), eps);
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}

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
        // decode batches: scores and selection in one launch on the CUDA cores, the hidden dimension cut into as
        // many slices (4, 2 or 1) as the scratch holds partial scores for
        int KS = 4;
        while (KS > 1 && route_small_floats(T, NG, KS) * sizeof(float) > wide_route_workspace(T, NG, rank) - 1024) KS >>= 1;
        if (T <= kRsMaxTokens && !(flags & WIDE_FLAG_FORCE_PREFILL) &&
            route_small_floats(T, NG, KS) * sizeof(float) <= wide_route_workspace(T, NG, rank) - 1024 &&
            kRsTokens * ((D / 8 + KS - 1) / KS + 31) * 16 <= 200 * 1024) {
            WideLaunch l(ctx, s, "route_small");
            const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(x);
            const __nv_bfloat16* wb = static_cast<const __nv_bfloat16*>(w_router);
            switch ((NG + 31) / 32) {
#define WIDE_RS_CASE(n) \
    case n: return launch_route_small<n>(s, T, xb, wb, NG, D, k, k_per_token, mask_bits, scores, sc32, KS, ctx->d_tickets + 2040);
                WIDE_RS_CASE(1) WIDE_RS_CASE(2) WIDE_RS_CASE(3) WIDE_RS_CASE(4)
                WIDE_RS_CASE(5) WIDE_RS_CASE(6) WIDE_RS_CASE(7) WIDE_RS_CASE(8)
#undef WIDE_RS_CASE
                default: return WIDE_ERR_UNSUPPORTED_SHAPE;
            }
        }
        float* wn = reinterpret_cast<float*>(static_cast<char*>(ws) + wide_route_workspace(T, NG, rank) - 1024);
        // as many K-split slabs as the first part of the workspace holds (at most 8)
        const size_t part0 = wide_route_workspace(T, NG, rank) - 1024;
        int max_split = static_cast<int>(part0 / (static_cast<size_t>(T) * ld * sizeof(float)));
        if (max_split > kMaxSlabs) max_split = kMaxSlabs;
        if (max_split < 1) max_split = 1;
        int ksplit = 1, chain = D;
        const int rc = wide_launch_scores_tc(ctx, s, x, w_router, T, NG, ld, D, sc32, wn, max_split, &ksplit, &chain);
        if (rc != WIDE_OK) return rc;
        WideLaunch l(ctx, s, "route_select_band");
        const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(x);
        const __nv_bfloat16* wb = static_cast<const __nv_bfloat16*>(w_router);
        switch ((NG + 31) / 32) {   // mask words per token = groups held per lane
#define WIDE_SEL_CASE(n) \
    case n: launch_select_band<n>(s, T, sc32, ksplit, ld, xb, wb, wn, NG, D, k, k_per_token, mask_bits, scores, chain, !ctx->prof); break;
            WIDE_SEL_CASE(1) WIDE_SEL_CASE(2) WIDE_SEL_CASE(3) WIDE_SEL_CASE(4)
            WIDE_SEL_CASE(5) WIDE_SEL_CASE(6) WIDE_SEL_CASE(7) WIDE_SEL_CASE(8)
#undef WIDE_SEL_CASE
            default: return WIDE_ERR_UNSUPPORTED_SHAPE;
        }
        return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
    }
    if (mode == WIDE_ROUTE_PAIR_ARGMAX && dtype == WIDE_BF16 && D % 64 == 0 && D <= 16384 && ctx->encode_tiled &&
        !(flags & WIDE_FLAG_SIMT) && rank <= kPairMaxRank && rank % 8 == 0 && NG <= 192 &&
        static_cast<size_t>(T) * rank * sizeof(double) >= static_cast<size_t>(rank) * D * 2 &&
        static_cast<size_t>(T) * 2048 >= static_cast<size_t>(NG) * D * sizeof(double)) {
        // workspace: [0] u slabs (fp32 [ks][T, 32]) | [1] W1^T (bf16 [rank, D]) | [2] marked pairs (bits [T, W])
        //            | [3] d_g (fp64 [NG, D]) | tail: column norms of W1 (256 floats at most) and ||d_g||^2
        const size_t off1 = wide_align_up(static_cast<size_t>(T) * 2 * NG * sizeof(double), 256);
        const size_t off2 = off1 + wide_align_up(static_cast<size_t>(T) * rank * sizeof(double), 256);
        const size_t off3 = off2 + wide_align_up(static_cast<size_t>(T) * 128, 256);
        const size_t total = wide_route_workspace(T, NG, rank);
        char* wsb = static_cast<char*>(ws);
        float* slabs = static_cast<float*>(ws);
        __nv_bfloat16* w1t = reinterpret_cast<__nv_bfloat16*>(wsb + off1);
        uint32_t* close_bits = reinterpret_cast<uint32_t*>(wsb + off2);
        double* d64 = reinterpret_cast<double*>(wsb + off3);
        float* wn = reinterpret_cast<float*>(wsb + total - 1024);      // 32 floats used
        float* dn2 = wn + 64;                                           // NG <= 192 floats behind them
        const int ld = 32;
        int max_split = static_cast<int>(off1 / (static_cast<size_t>(T) * ld * sizeof(float)));
        if (max_split > kMaxSlabs) max_split = kMaxSlabs;
        if (max_split < 1) max_split = 1;
        const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(x);
        const __nv_bfloat16* w1b = static_cast<const __nv_bfloat16*>(w_router);
        const __nv_bfloat16* w2b = static_cast<const __nv_bfloat16*>(w2);
        {
            WideLaunch l(ctx, s, "route_pair_transpose");
            transpose_w1_kernel<<<64, 256, 0, s>>>(w1b, D, rank, NG, w1t, dn2);
        }
        {
            WideLaunch l(ctx, s, "route_pair_delta");
            pair_delta_kernel<<<dim3((D + 127) / 128, (NG + 31) / 32), 128, 0, s>>>(w1b, w2b, D, rank, NG, d64, dn2);
        }
        int ksplit = 1, chain = D;
        const int rc = wide_launch_scores_tc(ctx, s, x, w1t, T, rank, ld, D, slabs, wn, max_split, &ksplit, &chain);
        if (rc != WIDE_OK) return rc;
        {
            WideLaunch l(ctx, s, "route_pair_band");
            pair_band_kernel<<<(T + 3) / 4, 128, 0, s>>>(slabs, ksplit, ld, xb, w2b, wn, T, NG, D, rank, mask_bits, scores,
                                                          close_bits, chain);
        }
        WideLaunch l(ctx, s, "route_pair_exact");
        const int grid = T < 16 * ctx->sm_count ? T : 16 * ctx->sm_count;
        pair_exact_kernel<<<grid, 128, 0, s>>>(xb, w1b, w2b, d64, dn2, T, D, rank, NG, close_bits, mask_bits, scores);
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
