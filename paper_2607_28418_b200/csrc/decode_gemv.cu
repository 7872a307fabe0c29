// Decode path of wide_ffn / wide_oproj for a very small batch: matrix-vector products on the CUDA
// cores (the GEMV dispatch the paper's Appendix B names for tiny M).
//
// With a handful of tokens a weight element is used by a handful of multiply-adds, so the tensor
// cores have nothing to add: the work is reading each needed weight byte once, and a kernel of
// plain 16-byte loads has no tile pipeline to fill and drain, no accumulators in L2 and no tickets.
// As in the tensor-core decode kernel the reorder is bypassed: every CTA forms the union U of the
// groups some token selected, and only the rows / columns of groups in U are read.
//
//   pass 1 (FFN)  one warp per hidden channel c of a group in U: the rows W_gate[c, :] and W_up[c, :]
//                 are streamed once (a lane takes every 32nd 16-byte piece), x_t sits in shared memory
//                 as fp32, the lanes' partial sums are added by shuffles and
//                 h[t, c] = M[t, g] ? silu(gate) * up : 0 goes to scratch as bf16.  The channels of U
//                 Most of U's channels are dealt out in equal contiguous shares, one per CTA (whole
//                 rounds of 16, one channel per warp); the rest is a pool that the warps draw from
//                 one channel at a time through a counter, so that SMs the memory system serves a
//                 little slower than others do not hold everybody up at the barrier.
//   grid barrier  (cooperative launch; bounded wait).  A first line of W_down per lane is on its way
//                 into L2 when a CTA arrives; more would only queue ahead of the barrier's own traffic.
//   pass 2        one warp per output row n: the pieces of W_down[n, :] (or W_o[n, :]) that belong to
//                 groups in U are streamed once, h (or the masked attention output) sits in shared
//                 memory as bf16, compacted in the order of U; the sums are written straight to y.
//                 No atomics, no zero-initialisation, no second kernel.
//   O-projection  pass 2 alone, no barrier.
#include <cuda.h>

#include "internal.h"
#include "ptx.cuh"

namespace {

using namespace wptx;

constexpr int kThreadsV = 512;
constexpr int kWarpsV = kThreadsV / 32;
constexpr int kBatch1 = 4;   // 16-byte pieces per lane, row and request batch in pass 1 (two rows, two batches in flight)
constexpr int kBatch2 = 8;   // the same in pass 2 (one row)

struct GemvArgs {
    int is_ffn;
    int B, D, inner, G, NG, words;
    const uint32_t* mask_bits;
    const __nv_bfloat16* act;   // FFN: x [B, D]; O-projection: attention output [B, inner]
    const __nv_bfloat16* wg;
    const __nv_bfloat16* wu;
    const __nv_bfloat16* wd;    // W_down [D, inner] or W_o [D, inner]
    __nv_bfloat16* h;           // scratch [B, inner]
    void* y;
    int out_bf16;
    unsigned* bar;              // grid barrier words of the context: arrivals, departures; [2] the channel pool's counter
    int* status;
    unsigned long long wait_ns;
};

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }
__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Two fp32 multiply-adds in one instruction: d = a * b + c on both halves of 64-bit register pairs.
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t pack2f(float lo, float hi) {
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
    return d;
}
__device__ __forceinline__ float sum2f(uint64_t v) {
    float lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
    return lo + hi;
}
// the two bf16 of a 32-bit word as a pair of floats (a bf16 is the upper half of the float)
__device__ __forceinline__ uint64_t bf2_to_f2(uint32_t w) {
    return pack2f(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}

// Every CTA of the co-resident grid meets here once per launch: the same two self-resetting words and
// the same protocol as the tensor-core decode kernel (arrivals counted with a fire-and-forget red
// after a fence, departures counted off the critical path, the last one to leave zeroes both).
__device__ bool gemv_grid_barrier(unsigned* bar, unsigned long long wait_ns, int* status) {
    __shared__ int s_passed;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        asm volatile("red.global.add.u32 [%0], 1;" ::"l"(bar) : "memory");
        bool passed = true;
        const uint64_t start = globaltimer_ns();
        while (ld_acquire(bar) < gridDim.x) {
            if (globaltimer_ns() - start > wait_ns) {
                atomicExch(status, WIDE_ERR_TIMEOUT);
                passed = false;
                break;
            }
        }
        s_passed = passed;
    }
    __syncthreads();
    const bool passed = s_passed != 0;
    if (threadIdx.x == kThreadsV - 1 && passed && atomicAdd(bar + 1, 1u) + 1u == gridDim.x) {
        bar[0] = 0u;
        bar[1] = 0u;
        bar[2] = 0u;   // pass 1 is over for everybody: the pool's counter goes back to zero as well
    }
    return passed;
}

// Pieces [i_lo, i_hi) of the rows pg and pu (16 bytes = 8 weights each; a lane takes every 32nd)
// against the NB token vectors in shared memory: xs4 holds, per token, the first four floats of every
// piece and then the last four of every piece, so that the lanes of a warp read neighbouring 16 bytes.
// Returns this lane's partial sums.
template <int NB>
__device__ __forceinline__ void gate_up_dot(const uint4* __restrict__ pg, const uint4* __restrict__ pu, int i_lo, int i_hi,
                                            const float4* __restrict__ xs4, int nch, int lane, float (&ag)[NB], float (&au)[NB]) {
    uint64_t g2[NB], u2[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) g2[b] = u2[b] = 0ull;
    uint4 cg[kBatch1], cu[kBatch1], ng[kBatch1], nu[kBatch1];
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
    for (int j = 0; j < kBatch1; ++j) {
        const int i = i_lo + lane + 32 * j;
        cg[j] = i < i_hi ? ld_stream(pg + i) : zero;
        cu[j] = i < i_hi ? ld_stream(pu + i) : zero;
    }
#pragma unroll 1
    for (int base = i_lo; base < i_hi; base += 32 * kBatch1) {
        const int nbase = base + 32 * kBatch1;
        if (nbase < i_hi) {
#pragma unroll
            for (int j = 0; j < kBatch1; ++j) {
                const int i = nbase + lane + 32 * j;
                ng[j] = i < i_hi ? ld_stream(pg + i) : zero;
                nu[j] = i < i_hi ? ld_stream(pu + i) : zero;
            }
        }
#pragma unroll
        for (int j = 0; j < kBatch1; ++j) {
            const int i = base + lane + 32 * j;
            if (i < i_hi) {
                const uint64_t gw[4] = {bf2_to_f2(cg[j].x), bf2_to_f2(cg[j].y), bf2_to_f2(cg[j].z), bf2_to_f2(cg[j].w)};
                const uint64_t uw[4] = {bf2_to_f2(cu[j].x), bf2_to_f2(cu[j].y), bf2_to_f2(cu[j].z), bf2_to_f2(cu[j].w)};
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    const float4 x0 = xs4[b * 2 * nch + i], x1 = xs4[(b * 2 + 1) * nch + i];
                    const uint64_t xv[4] = {pack2f(x0.x, x0.y), pack2f(x0.z, x0.w), pack2f(x1.x, x1.y), pack2f(x1.z, x1.w)};
#pragma unroll
                    for (int p = 0; p < 4; ++p) {
                        g2[b] = fma2(gw[p], xv[p], g2[b]);
                        u2[b] = fma2(uw[p], xv[p], u2[b]);
                    }
                }
            }
        }
#pragma unroll
        for (int j = 0; j < kBatch1; ++j) { cg[j] = ng[j]; cu[j] = nu[j]; }
    }
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        ag[b] = sum2f(g2[b]);
        au[b] = sum2f(u2[b]);
    }
}

template <int NB>
__global__ void __launch_bounds__(kThreadsV, 1) decode_gemv_kernel(const GemvArgs a) {
    extern __shared__ uint4 smem4[];
    __shared__ int s_union[WIDE_MAX_GROUPS];
    __shared__ unsigned char s_tok[WIDE_MAX_GROUPS];   // which of the tokens selected the union's slot
    __shared__ int s_nunion;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // x as fp32 in shared memory (FFN): per token the first four floats of every 8-element piece, then the
    // last four of every piece.  Nothing here depends on the masks, so it runs beside the union below.
    if (a.is_ffn) {
        const int nch = a.D / 8;
        float4* xs4w = reinterpret_cast<float4*>(smem4);
        const uint4* x4 = reinterpret_cast<const uint4*>(a.act);
        for (int b = 0; b < NB; ++b) {
            for (int i = tid; i < nch; i += kThreadsV) {
                const uint4 v = b < a.B ? __ldg(x4 + static_cast<size_t>(b) * nch + i) : make_uint4(0u, 0u, 0u, 0u);
                xs4w[b * 2 * nch + i] = make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u),
                                                    __uint_as_float(v.y << 16), __uint_as_float(v.y & 0xffff0000u));
                xs4w[(b * 2 + 1) * nch + i] = make_float4(__uint_as_float(v.z << 16), __uint_as_float(v.z & 0xffff0000u),
                                                          __uint_as_float(v.w << 16), __uint_as_float(v.w & 0xffff0000u));
            }
        }
    }
    if (warp == 0) {
        // A wait that expired in an earlier decode kernel leaves the barrier words dirty until wide_status
        // resets them: with the status word set, this call does nothing at all (one thread reads the word,
        // so the whole CTA takes the same way).
        const int status_now = lane == 0 ? __ldcg(a.status) : WIDE_OK;
        // union of the batch's masks, ascending, with the tokens that selected each slot
        int pos = 0;
        for (int w = 0; w < a.words; ++w) {
            uint32_t mw[NB];
            uint32_t u = 0;
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                mw[b] = b < a.B ? a.mask_bits[static_cast<size_t>(b) * a.words + w] : 0u;
                u |= mw[b];
            }
            const int g = w * 32 + lane;
            const bool in = g < a.NG && ((u >> lane) & 1u);
            const unsigned vote = __ballot_sync(0xffffffffu, in);
            if (in) {
                const int slot = pos + __popc(vote & ((1u << lane) - 1u));
                unsigned tok = 0;
#pragma unroll
                for (int b = 0; b < NB; ++b) tok |= ((mw[b] >> lane) & 1u) << b;
                s_union[slot] = g;
                s_tok[slot] = static_cast<unsigned char>(tok);
            }
            pos += __popc(vote);
        }
        if (lane == 0) s_nunion = status_now != WIDE_OK ? -1 : pos;
    }
    __syncthreads();
    const int n_union = s_nunion;
    if (n_union < 0) return;

    if (n_union == 0) {
        // nothing is active: the output is exactly zero
        const long long n = static_cast<long long>(a.B) * a.D;
        for (long long i = static_cast<long long>(blockIdx.x) * kThreadsV + tid; i < n; i += static_cast<long long>(gridDim.x) * kThreadsV) {
            if (a.out_bf16) static_cast<__nv_bfloat16*>(a.y)[i] = __float2bfloat16_rn(0.f);
            else static_cast<float*>(a.y)[i] = 0.f;
        }
        return;
    }

    const int cpg = a.G / 8;                 // 16-byte pieces per group and row of W_down (a power of two)
    const int cpg_shift = __ffs(cpg) - 1;
    const int nq = n_union * cpg;            // pieces of a W_down row that belong to the union
    const int row4 = a.inner / 8;            // pieces of a whole row of W_down (and of h)
    // shared memory: [pass 1: x as fp32, NB x D] / [pass 2: h as bf16, NB x nq pieces], then the piece table
    float* xs = reinterpret_cast<float*>(smem4);
    uint4* hs4 = smem4;
    const int region4 = max(a.is_ffn ? NB * a.D / 4 : 0, NB * row4);
    int* s_off = reinterpret_cast<int*>(smem4 + region4);     // piece q of the union -> piece of the row
    for (int q = tid; q < nq; q += kThreadsV) s_off[q] = (s_union[q >> cpg_shift] << cpg_shift) + (q & (cpg - 1));

    // rows of pass 2 dealt to this CTA
    const int n_lo = static_cast<int>(static_cast<long long>(blockIdx.x) * a.D / gridDim.x);
    const int n_hi = static_cast<int>(static_cast<long long>(blockIdx.x + 1) * a.D / gridDim.x);
    const uint4* wd4 = reinterpret_cast<const uint4*>(a.wd);

    if (a.is_ffn) {
        // ------------------------------------------------------------------ pass 1
        const int nch = a.D / 8;
        const long long total = static_cast<long long>(n_union) * a.G;
        auto channel_of = [&](int e, int& slot) {
            slot = e / a.G;
            return s_union[slot] * a.G + (e - slot * a.G);
        };
        const float4* xs4 = reinterpret_cast<const float4*>(xs);
        auto channel = [&](int e) {
            int slot;
            const int c = channel_of(e, slot);
            float ag[NB], au[NB];
            gate_up_dot<NB>(reinterpret_cast<const uint4*>(a.wg + static_cast<size_t>(c) * a.D),
                            reinterpret_cast<const uint4*>(a.wu + static_cast<size_t>(c) * a.D), 0, nch, xs4, nch, lane, ag, au);
#pragma unroll
            for (int b = 0; b < NB; ++b) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    ag[b] += __shfl_xor_sync(0xffffffffu, ag[b], o);
                    au[b] += __shfl_xor_sync(0xffffffffu, au[b], o);
                }
            }
            if (lane == 0) {
                const unsigned tok = s_tok[slot];
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    if (b < a.B) {
                        const float hval = ((tok >> b) & 1u) ? ag[b] / (1.f + __expf(-ag[b])) * au[b] : 0.f;
                        a.h[static_cast<size_t>(b) * a.inner + c] = __float2bfloat16_rn(hval);
                    }
                }
            }
        };
        // fixed shares: whole rounds of one channel per warp, about 27/32 of the work
        const int fixed = static_cast<int>(total * 27 / 32 / gridDim.x) / kWarpsV * kWarpsV;
        const int e_lo = static_cast<int>(blockIdx.x) * fixed;
        unsigned ticket = 0;
        for (int e = e_lo + warp; e < e_lo + fixed; e += kWarpsV) {
            if (e + kWarpsV >= e_lo + fixed && lane == 0) ticket = atomicAdd(a.bar + 2, 1u);   // asked for one channel ahead
            channel(e);
        }
        if (fixed == 0 && lane == 0) ticket = atomicAdd(a.bar + 2, 1u);
        // the pool
        const int pool_lo = static_cast<int>(gridDim.x) * fixed;
        while (true) {
            const int e = pool_lo + static_cast<int>(__shfl_sync(0xffffffffu, ticket, 0));
            if (e >= total) break;
            if (lane == 0) ticket = atomicAdd(a.bar + 2, 1u);
            channel(e);
        }
    }

    // ---------------------------------------------------------------------- pass 2
    __syncthreads();   // the piece table is complete (and pass 1 is done with x)
    // the first 4 KB of every warp's first row are asked for before the barrier (128-byte lines; a group's
    // piece of a row is G * 2 bytes, a multiple of 128)
    if (n_lo + warp < n_hi && lane * 8 < nq) prefetch_l2(wd4 + static_cast<size_t>(n_lo + warp) * row4 + s_off[lane * 8]);
    if (a.is_ffn) {
        if (!gemv_grid_barrier(a.bar, a.wait_ns, a.status)) return;
    }
    // h (bf16) of the union's channels, compacted in the union's order
    {
        const uint4* src4 = reinterpret_cast<const uint4*>(a.is_ffn ? a.h : a.act);
        const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
        for (int b = 0; b < NB; ++b) {
            if (b >= a.B) {
                for (int q = tid; q < nq; q += kThreadsV) hs4[b * nq + q] = zero4;
                continue;
            }
            const uint4* srow = src4 + static_cast<size_t>(b) * row4;
            for (int q0 = tid; q0 < nq; q0 += 4 * kThreadsV) {
                uint4 v[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int q = q0 + j * kThreadsV;
                    v[j] = zero4;
                    if (q < nq) {
                        if (a.is_ffn) v[j] = __ldcg(srow + s_off[q]);   // written by other CTAs of this launch
                        else if ((s_tok[q >> cpg_shift] >> b) & 1u) v[j] = __ldg(srow + s_off[q]);
                    }
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int q = q0 + j * kThreadsV;
                    if (q < nq) hs4[b * nq + q] = v[j];
                }
            }
        }
    }
    __syncthreads();
    uint4 cur[kBatch2], nxt[kBatch2];
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
    int n = n_lo + warp;
    if (n < n_hi) {
        const uint4* row = wd4 + static_cast<size_t>(n) * row4;
#pragma unroll
        for (int j = 0; j < kBatch2; ++j) {
            const int q = lane + 32 * j;
            cur[j] = q < nq ? ld_stream(row + s_off[q]) : zero;
        }
    }
    for (; n < n_hi; n += kWarpsV) {
        const uint4* row = wd4 + static_cast<size_t>(n) * row4;
        uint64_t acc2[NB];
#pragma unroll
        for (int b = 0; b < NB; ++b) acc2[b] = 0ull;
#pragma unroll 1
        for (int base = 0; base < nq; base += 32 * kBatch2) {
            const int nbase = base + 32 * kBatch2;
            if (nbase < nq) {
#pragma unroll
                for (int j = 0; j < kBatch2; ++j) {
                    const int q = nbase + lane + 32 * j;
                    nxt[j] = q < nq ? ld_stream(row + s_off[q]) : zero;
                }
            } else if (n + kWarpsV < n_hi) {
                // the next row's first pieces
                const uint4* nrow = row + static_cast<size_t>(kWarpsV) * row4;
#pragma unroll
                for (int j = 0; j < kBatch2; ++j) {
                    const int q = lane + 32 * j;
                    nxt[j] = q < nq ? ld_stream(nrow + s_off[q]) : zero;
                }
            }
#pragma unroll
            for (int j = 0; j < kBatch2; ++j) {
                const int q = base + lane + 32 * j;
                if (q < nq) {
                    const uint64_t ww[4] = {bf2_to_f2(cur[j].x), bf2_to_f2(cur[j].y), bf2_to_f2(cur[j].z), bf2_to_f2(cur[j].w)};
#pragma unroll
                    for (int b = 0; b < NB; ++b) {
                        const uint4 hv = hs4[b * nq + q];
                        acc2[b] = fma2(ww[0], bf2_to_f2(hv.x), acc2[b]);
                        acc2[b] = fma2(ww[1], bf2_to_f2(hv.y), acc2[b]);
                        acc2[b] = fma2(ww[2], bf2_to_f2(hv.z), acc2[b]);
                        acc2[b] = fma2(ww[3], bf2_to_f2(hv.w), acc2[b]);
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < kBatch2; ++j) cur[j] = nxt[j];
        }
        float acc[NB];
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            acc[b] = sum2f(acc2[b]);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc[b] += __shfl_xor_sync(0xffffffffu, acc[b], o);
        }
        if (lane == 0) {
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                if (b < a.B) {
                    if (a.out_bf16) static_cast<__nv_bfloat16*>(a.y)[static_cast<size_t>(b) * a.D + n] = __float2bfloat16_rn(acc[b]);
                    else static_cast<float*>(a.y)[static_cast<size_t>(b) * a.D + n] = acc[b];
                }
            }
        }
    }
}

size_t gemv_smem_bytes(bool is_ffn, int nb, int D, int inner) {
    const size_t xs = is_ffn ? 4 * static_cast<size_t>(D) : 0, hs = 2 * static_cast<size_t>(inner);
    return static_cast<size_t>(nb) * (xs > hs ? xs : hs) + static_cast<size_t>(inner / 8) * 4;
}

template <int NB>
int launch_gemv(wide_ctx* ctx, cudaStream_t s, const GemvArgs& a, size_t smem) {
    WIDE_CUDA_CHECK(cudaFuncSetAttribute(decode_gemv_kernel<NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    GemvArgs args = a;
    void* params[] = {&args};
    WideLaunch l(ctx, s, a.is_ffn ? "decode_ffn_gemv" : "decode_oproj_gemv");
    if (a.is_ffn) {
        // cooperative: the grid barrier needs every CTA resident (one per SM)
        WIDE_CUDA_CHECK(cudaLaunchCooperativeKernel(reinterpret_cast<void*>(decode_gemv_kernel<NB>), dim3(ctx->sm_count),
                                                    dim3(kThreadsV), params, smem, s));
    } else {
        decode_gemv_kernel<NB><<<ctx->sm_count, kThreadsV, smem, s>>>(args);
        if (cudaGetLastError() != cudaSuccess) return WIDE_ERR_CUDA;
    }
    return WIDE_OK;
}

int padded_tokens(int T) { return T == 1 ? 1 : 2; }

}  // namespace

bool wide_decode_gemv_fits(bool is_ffn, int T, int D, int inner, int G) {
    if (T < 1 || T > WIDE_DECODE_GEMV_MAX_TOKENS) return false;
    if (D % 8 != 0 || G < 64 || (G & (G - 1)) != 0 || inner % G != 0 || inner / G > WIDE_MAX_GROUPS) return false;
    return gemv_smem_bytes(is_ffn, padded_tokens(T), D, inner) <= 220u * 1024u;
}

int wide_launch_decode_gemv(wide_ctx* ctx, cudaStream_t s, bool is_ffn, const void* act, const void* wg, const void* wu,
                            const void* wd, int T, int D, int inner, int G, const uint32_t* mask_bits, void* y,
                            int out_dtype, void* ws) {
    if (T == 0) return WIDE_OK;
    GemvArgs a{};
    a.is_ffn = is_ffn ? 1 : 0;
    a.B = T;
    a.D = D;
    a.inner = inner;
    a.G = G;
    a.NG = inner / G;
    a.words = (a.NG + 31) / 32;
    a.mask_bits = mask_bits;
    a.act = static_cast<const __nv_bfloat16*>(act);
    a.wg = static_cast<const __nv_bfloat16*>(wg);
    a.wu = static_cast<const __nv_bfloat16*>(wu);
    a.wd = static_cast<const __nv_bfloat16*>(wd);
    a.h = static_cast<__nv_bfloat16*>(ws);
    a.y = y;
    a.out_bf16 = out_dtype == WIDE_BF16 ? 1 : 0;
    a.bar = reinterpret_cast<unsigned*>(ctx->d_status) + 4;
    a.status = ctx->d_status;
    a.wait_ns = ctx->wait_ns;
    const int nb = padded_tokens(T);
    const size_t smem = gemv_smem_bytes(is_ffn, nb, D, inner);
    if (nb == 1) return launch_gemv<1>(ctx, s, a, smem);
    return launch_gemv<2>(ctx, s, a, smem);
}
