// Decode form of the head-group-masked attention (Algorithm 4, last paragraph: for a handful of
// query tokens the mask reordering is bypassed, routing is checked at the block level, and the
// online softmax runs split over the keys).  The work is reading K and V once, so it runs on the
// CUDA cores and is measured against HBM bandwidth.
//
// A CTA owns one KV head and one slice of the keys, and serves every query row that reads this
// KV head: R = tokens_q * (n_q_heads / n_kv_heads) rows (R <= 8).  If none of those rows is active
// under the head-group mask the CTA exits at once and the head's K and V are never read -- that is
// where the masked layer saves its bytes.  Within a CTA each warp takes chunks of 32 keys:
//   scores   lane = key: the lane holds its key row in registers and dots it with the R query
//            rows (shared memory, pre-multiplied by scale * log2 e);
//   softmax  per row across the warp (running maximum, sum), probabilities parked in shared memory;
//   PV       lane = 4 (or 2) output dimensions: the warp reads each V row coalesced.
// The four warps' partial (m, l, O) are merged in shared memory and written to a scratch slab; a
// second small kernel merges the key slices, normalises, and writes zeros for inactive pairs.
#include <math_constants.h>

#include "internal.h"

namespace {

constexpr int kMaxRows = 8;      // query rows per KV head served by one CTA
constexpr int kDecWarps = 4;
constexpr int kMaxSplits = 32;

__device__ __forceinline__ float exp2_fast(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int HD, int RT>   // RT: compile-time bound of the rows served (1, 2, 4 or 8)
__global__ void __launch_bounds__(32 * kDecWarps)
attn_decode_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                   const __nv_bfloat16* __restrict__ v, const uint32_t* __restrict__ mask_bits, int words, int Tq,
                   int Tk, int Hq, int Hkv, int hpg, int causal, float scale_log2e, int keys_per_split,
                   float* __restrict__ part) {
    constexpr int kDL = HD / 32;                  // output dimensions per lane
    constexpr int kVec = HD / 8;                  // 16-byte pieces of a key row
    __shared__ float qs[RT][HD];
    __shared__ float ps[kDecWarps][RT][32];
    __shared__ float wm[kDecWarps][RT], wl[kDecWarps][RT];
    __shared__ float wo[kDecWarps][RT][HD];
    __shared__ int s_any;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int split = blockIdx.x, hkv = blockIdx.y;
    const int rep = Hq / Hkv;
    const int R = Tq * rep;
    const int delta = Tk - Tq;
    const size_t ldq = static_cast<size_t>(Hq) * HD, ldk = static_cast<size_t>(Hkv) * HD;

    // block-level routing check: does any row served here execute its head group?
    if (tid == 0) s_any = 0;
    __syncthreads();
    if (tid < R) {
        const int t = tid / rep, h = hkv * rep + tid % rep;
        if (wide_mask_bit(mask_bits, words, t, h / hpg)) s_any = 1;
    }
    __syncthreads();
    if (!s_any) return;

    for (int i = tid; i < R * HD; i += 32 * kDecWarps) {
        const int r = i / HD, d = i % HD;
        const int t = r / rep, h = hkv * rep + r % rep;
        qs[r][d] = __bfloat162float(q[t * ldq + static_cast<size_t>(h) * HD + d]) * scale_log2e;
    }
    __syncthreads();

    const int j0 = split * keys_per_split, j1 = min(Tk, j0 + keys_per_split);
    float m[RT], l[RT], o[RT][kDL];
#pragma unroll
    for (int r = 0; r < RT; ++r) {
        m[r] = -CUDART_INF_F;
        l[r] = 0.f;
#pragma unroll
        for (int d = 0; d < kDL; ++d) o[r][d] = 0.f;
    }

    for (int c0 = j0 + warp * 32; c0 < j1; c0 += 32 * kDecWarps) {
        const int j = c0 + lane;
        const bool valid = j < j1;
        // scores: this lane's key row against every query row
        uint4 kr[kVec];
        const uint4* kp = reinterpret_cast<const uint4*>(k + static_cast<size_t>(valid ? j : j1 - 1) * ldk + static_cast<size_t>(hkv) * HD);
#pragma unroll
        for (int i = 0; i < kVec; ++i) kr[i] = __ldg(kp + i);
        // with few query rows there are registers to spare: the chunk's V rows are requested now,
        // together with the key rows, so that a chunk costs one load latency instead of two
        constexpr bool kEarlyV = RT <= 2;
        uint2 vr[kEarlyV ? 32 : 1];
        const int nk = min(32, j1 - c0);
        if (kEarlyV) {
#pragma unroll
            for (int u = 0; u < 32; ++u) {
                const __nv_bfloat16* vp = v + static_cast<size_t>(c0 + min(u, nk - 1)) * ldk + static_cast<size_t>(hkv) * HD + lane * kDL;
                if (kDL == 4) vr[u] = __ldg(reinterpret_cast<const uint2*>(vp));
                else vr[u] = make_uint2(__ldg(reinterpret_cast<const uint32_t*>(vp)), 0u);
            }
        }
        float s[RT];
#pragma unroll
        for (int r = 0; r < RT; ++r) {
            s[r] = -CUDART_INF_F;
            if (r < R) {
                float a = 0.f;
#pragma unroll
                for (int i = 0; i < kVec; ++i) {
                    const __nv_bfloat162* kh = reinterpret_cast<const __nv_bfloat162*>(&kr[i]);
                    const float4 qa = *reinterpret_cast<const float4*>(&qs[r][8 * i]);
                    const float4 qb = *reinterpret_cast<const float4*>(&qs[r][8 * i + 4]);
                    const float2 k0 = __bfloat1622float2(kh[0]), k1 = __bfloat1622float2(kh[1]);
                    const float2 k2 = __bfloat1622float2(kh[2]), k3 = __bfloat1622float2(kh[3]);
                    a = fmaf(qa.x, k0.x, a); a = fmaf(qa.y, k0.y, a); a = fmaf(qa.z, k1.x, a); a = fmaf(qa.w, k1.y, a);
                    a = fmaf(qb.x, k2.x, a); a = fmaf(qb.y, k2.y, a); a = fmaf(qb.z, k3.x, a); a = fmaf(qb.w, k3.y, a);
                }
                const int lim = causal ? (r / rep) + delta : Tk - 1;   // last key this row may see
                if (valid && j <= lim) s[r] = a;
            }
        }
        // online softmax per row across the 32 keys of the chunk
#pragma unroll
        for (int r = 0; r < RT; ++r) {
            if (r < R) {
                float mx = s[r];
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
                const float m_new = fmaxf(m[r], mx);
                const float m_use = m_new == -CUDART_INF_F ? 0.f : m_new;
                const float p = exp2_fast(s[r] - m_use);
                const float alpha = exp2_fast(m[r] - m_use);
                float sum = p;
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
                l[r] = fmaf(l[r], alpha, sum);
                m[r] = m_new;
#pragma unroll
                for (int d = 0; d < kDL; ++d) o[r][d] *= alpha;
                ps[warp][r][lane] = p;
            }
        }
        __syncwarp();
        // PV: the warp reads each V row of the chunk once, lane = kDL output dimensions.  The rows
        // are fetched in batches of kVB loads per lane before any is used (this phase is bound by
        // load latency, not by instructions).
        constexpr int kVB = 8;
        if (kEarlyV) {
#pragma unroll
            for (int u = 0; u < 32; ++u) {
                if (u < nk) {
                    float vv[4];
                    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&vr[u].x));
                    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&vr[u].y));
                    vv[0] = a.x; vv[1] = a.y; vv[2] = b.x; vv[3] = b.y;
#pragma unroll
                    for (int r = 0; r < RT; ++r) {
                        if (r < R) {
                            const float p = ps[warp][r][u];
#pragma unroll
                            for (int d = 0; d < kDL; ++d) o[r][d] = fmaf(p, vv[d], o[r][d]);
                        }
                    }
                }
            }
        }
        for (int k0 = kEarlyV ? nk : 0; k0 < nk; k0 += kVB) {
            uint2 raw[kVB];
#pragma unroll
            for (int u = 0; u < kVB; ++u) {
                const int kk = min(k0 + u, nk - 1);
                const __nv_bfloat16* vp = v + static_cast<size_t>(c0 + kk) * ldk + static_cast<size_t>(hkv) * HD + lane * kDL;
                if (kDL == 4) raw[u] = __ldg(reinterpret_cast<const uint2*>(vp));
                else raw[u] = make_uint2(__ldg(reinterpret_cast<const uint32_t*>(vp)), 0u);
            }
#pragma unroll
            for (int u = 0; u < kVB; ++u) {
                if (k0 + u < nk) {
                    float vv[4];
                    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw[u].x));
                    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw[u].y));
                    vv[0] = a.x; vv[1] = a.y; vv[2] = b.x; vv[3] = b.y;
#pragma unroll
                    for (int r = 0; r < RT; ++r) {
                        if (r < R) {
                            const float p = ps[warp][r][k0 + u];
#pragma unroll
                            for (int d = 0; d < kDL; ++d) o[r][d] = fmaf(p, vv[d], o[r][d]);
                        }
                    }
                }
            }
        }
        __syncwarp();
    }

    // merge the four warps, write this key slice's partial result
#pragma unroll
    for (int r = 0; r < RT; ++r) {
        if (r < R) {
            if (lane == 0) { wm[warp][r] = m[r]; wl[warp][r] = l[r]; }
#pragma unroll
            for (int d = 0; d < kDL; ++d) wo[warp][r][lane * kDL + d] = o[r][d];
        }
    }
    __syncthreads();
    float* dst = part + (static_cast<size_t>(split) * Hkv + hkv) * R * (HD + 2);
    for (int i = tid; i < R * HD; i += 32 * kDecWarps) {
        const int r = i / HD, d = i % HD;
        float mm = -CUDART_INF_F;
#pragma unroll
        for (int w = 0; w < kDecWarps; ++w) mm = fmaxf(mm, wm[w][r]);
        const float m_use = mm == -CUDART_INF_F ? 0.f : mm;
        float acc = 0.f, ll = 0.f;
#pragma unroll
        for (int w = 0; w < kDecWarps; ++w) {
            const float a = exp2_fast(wm[w][r] - m_use);
            acc = fmaf(wo[w][r][d], a, acc);
            ll = fmaf(wl[w][r], a, ll);
        }
        dst[r * (HD + 2) + 2 + d] = acc;
        if (d == 0) {
            dst[r * (HD + 2)] = mm;
            dst[r * (HD + 2) + 1] = ll;
        }
    }
}

// One CTA per (token, query head): merge the key slices, normalise, write bf16; zeros for an
// inactive (token, group) pair or a query that saw no key.
template <int HD>
__global__ void __launch_bounds__(HD)
attn_decode_merge_kernel(const float* __restrict__ part, const uint32_t* __restrict__ mask_bits, int words, int Tq,
                         int Hq, int Hkv, int hpg, int n_splits, __nv_bfloat16* __restrict__ o) {
    const int t = blockIdx.x / Hq, h = blockIdx.x % Hq, d = threadIdx.x;
    const int rep = Hq / Hkv, R = Tq * rep;
    const int hkv = h / rep, r = t * rep + h % rep;
    float out = 0.f;
    if (wide_mask_bit(mask_bits, words, t, h / hpg)) {
        float mm = -CUDART_INF_F;
        for (int s = 0; s < n_splits; ++s) mm = fmaxf(mm, part[((static_cast<size_t>(s) * Hkv + hkv) * R + r) * (HD + 2)]);
        const float m_use = mm == -CUDART_INF_F ? 0.f : mm;
        float acc = 0.f, ll = 0.f;
        for (int s = 0; s < n_splits; ++s) {
            const float* p = part + ((static_cast<size_t>(s) * Hkv + hkv) * R + r) * (HD + 2);
            const float a = exp2_fast(p[0] - m_use);
            acc = fmaf(p[2 + d], a, acc);
            ll = fmaf(p[1], a, ll);
        }
        out = ll > 0.f ? acc / ll : 0.f;
    }
    o[(static_cast<size_t>(t) * Hq + h) * HD + d] = __float2bfloat16_rn(out);
}

template <int HD>
int launch_attn_decode(wide_ctx* ctx, cudaStream_t s, const void* q, const void* k, const void* v,
                       const uint32_t* mask_bits, int Tq, int Tk, int Hq, int Hkv, int hpg, int causal, float scale,
                       void* o) {
    const int rep = Hq / Hkv, R = Tq * rep;
    const int words = (Hq / hpg + 31) / 32;
    // enough key slices for about eight resident CTAs per SM (the kernel hides its load latency by
    // occupancy), at least 128 keys each, and the scratch slab must hold them
    int n_splits = (8 * ctx->sm_count + Hkv - 1) / Hkv;
    if (n_splits > (Tk + 127) / 128) n_splits = (Tk + 127) / 128;
    if (n_splits > kMaxSplits) n_splits = kMaxSplits;
    const size_t per_split = static_cast<size_t>(Hkv) * R * (HD + 2) * sizeof(float);
    while (n_splits > 1 && n_splits * per_split > ctx->attn_part_bytes) --n_splits;
    if (n_splits < 1 || per_split > ctx->attn_part_bytes) return WIDE_ERR_UNSUPPORTED_SHAPE;
    const int kps = ((Tk + n_splits - 1) / n_splits + 31) / 32 * 32;
    n_splits = (Tk + kps - 1) / kps;
    {
        WideLaunch l(ctx, s, "attn_decode");
        const dim3 grid(n_splits, Hkv);
        const __nv_bfloat16 *qb = static_cast<const __nv_bfloat16*>(q), *kb = static_cast<const __nv_bfloat16*>(k),
                            *vb = static_cast<const __nv_bfloat16*>(v);
        const float sl = scale * 1.4426950408889634f;
#define WIDE_DEC_CASE(rt) \
    attn_decode_kernel<HD, rt><<<grid, 32 * kDecWarps, 0, s>>>(qb, kb, vb, mask_bits, words, Tq, Tk, Hq, Hkv, hpg, causal, sl, \
                                                              kps, ctx->attn_part)
        if (R <= 1) WIDE_DEC_CASE(1);
        else if (R <= 2) WIDE_DEC_CASE(2);
        else if (R <= 4) WIDE_DEC_CASE(4);
        else WIDE_DEC_CASE(8);
#undef WIDE_DEC_CASE
    }
    if (cudaGetLastError() != cudaSuccess) return WIDE_ERR_CUDA;
    WideLaunch l(ctx, s, "attn_decode_merge");
    attn_decode_merge_kernel<HD><<<Tq * Hq, HD, 0, s>>>(ctx->attn_part, mask_bits, words, Tq, Hq, Hkv, hpg, n_splits,
                                                         static_cast<__nv_bfloat16*>(o));
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}

}  // namespace

bool wide_attn_decode_fits(int Tq, int Hq, int Hkv) { return Tq * (Hq / Hkv) <= kMaxRows; }

int wide_launch_attn_decode(wide_ctx* ctx, cudaStream_t s, const void* q, const void* k, const void* v,
                            const uint32_t* mask_bits, int Tq, int Tk, int Hq, int Hkv, int head_dim, int hpg,
                            int causal, float scale, void* o) {
    if (head_dim == 128) return launch_attn_decode<128>(ctx, s, q, k, v, mask_bits, Tq, Tk, Hq, Hkv, hpg, causal, scale, o);
    if (head_dim == 64) return launch_attn_decode<64>(ctx, s, q, k, v, mask_bits, Tq, Tk, Hq, Hkv, hpg, causal, scale, o);
    return WIDE_ERR_UNSUPPORTED_SHAPE;
}
