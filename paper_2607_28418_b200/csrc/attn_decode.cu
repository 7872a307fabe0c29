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
#include <cuda.h>
#include <math_constants.h>

#include "internal.h"
#include "ptx.cuh"

namespace {

constexpr int kMaxRows = 8;      // query rows per KV head served by one CTA
constexpr int kDecWarps = 4;
constexpr int kMaxSplits = 128;

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

// ------------------------------------------------------------------------------------------------
// The same computation with K and V brought in by TMA through a ring in shared memory, so that the
// bytes in flight do not depend on what the warps' registers hold: a producer thread keeps four
// stages of 32 keys (K tile + V tile, 2 x 32 x HD x 2 bytes) requested, one per consumer warp.  Warp
// w takes the tiles w, w + 4, ... and they always land in stage w, so each barrier has one waiter
// that sees every one of its phases (a warp that skipped a phase of a barrier could not tell the
// phase it waits for from the one before).  Three such CTAs fit an SM.  Every CTA first lists the KV heads that any row reads (the routing check),
// then the CTAs are dealt out evenly over those heads only: n_splits = gridDim.x / n_active key
// slices per head, so that a layer with half of its heads switched off uses every SM on the other
// half.  CTA c serves head c / n_splits, slice c % n_splits; block 0 leaves n_splits in hdr[0] for
// the merge kernel.  Scores are computed with lane = key from shared memory: lane l reads the
// 16-byte pieces of its key row in the order (i + l) mod (HD / 8), which keeps the eight lanes of
// a quarter warp on different banks; the query rows are stored as two float4 tables to match.
constexpr int kRingKeys = 32;
constexpr int kRingConsumers = 4;
constexpr int kRingStages = kRingConsumers;   // stage = consumer warp
constexpr int kRingThreads = 32 * (kRingConsumers + 1);

template <int HD, int RT>
__global__ void __launch_bounds__(kRingThreads, 3)
attn_decode_ring_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                        const __nv_bfloat16* __restrict__ q, const uint32_t* __restrict__ mask_bits, int words, int Tq,
                        int Tk, int Hq, int Hkv, int hpg, int causal, float scale_log2e, int max_splits,
                        float* __restrict__ part, int* __restrict__ hdr, int* status, unsigned long long wait_ns) {
    using namespace wptx;
    constexpr int kDL = HD / 32;                  // output dimensions per lane
    constexpr int kVec = HD / 8;                  // 16-byte pieces of a key row
    constexpr int kTileBytes = kRingKeys * HD * 2;
    extern __shared__ uint8_t smem_raw[];
    __shared__ float4 qa[RT][kVec], qb[RT][kVec];
    __shared__ float ps[kRingConsumers][RT][32];
    __shared__ float wm[kRingConsumers][RT], wl[kRingConsumers][RT];
    __shared__ uint8_t s_heads[256];
    __shared__ int s_nact;
    __shared__ int s_abort;
    __shared__ int s_issued;
    __shared__ __align__(8) uint64_t s_bars[2 * kRingStages];
    uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~static_cast<uintptr_t>(127));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rep = Hq / Hkv;
    const int R = Tq * rep;
    const int delta = Tk - Tq;
    const size_t ldq = static_cast<size_t>(Hq) * HD;
    const uint32_t full = smem_u32(s_bars), empty = smem_u32(s_bars + kRingStages);

    if (tid == 0) {
        for (int st = 0; st < kRingStages; ++st) {
            mbar_init(full + 8 * st, 1);
            mbar_init(empty + 8 * st, 1);
        }
        s_abort = 0;
        s_issued = 0;
        fence_barrier_init();
        prefetch_tmap(&tmK);
        prefetch_tmap(&tmV);
    }
    if (warp == 0) {
        // the KV heads that some row reads, ascending
        int pos = 0;
        for (int h0 = 0; h0 < Hkv; h0 += 32) {
            const int hkv = h0 + lane;
            bool any = false;
            if (hkv < Hkv)
                for (int r = 0; r < R; ++r) any = any || wide_mask_bit(mask_bits, words, r / rep, (hkv * rep + r % rep) / hpg);
            const unsigned vote = __ballot_sync(0xffffffffu, any);
            if (any) s_heads[pos + __popc(vote & ((1u << lane) - 1u))] = static_cast<uint8_t>(hkv);
            pos += __popc(vote);
        }
        if (lane == 0) s_nact = pos;
    }
    __syncthreads();
    const int n_act = s_nact;
    if (n_act == 0) {
        if (blockIdx.x == 0 && tid == 0) hdr[0] = 1;
        return;
    }
    int n_splits = min(min(static_cast<int>(gridDim.x) / n_act, (Tk + kRingKeys - 1) / kRingKeys), max_splits);
    if (n_splits < 1) n_splits = 1;
    const int kps = ((Tk + n_splits - 1) / n_splits + kRingKeys - 1) / kRingKeys * kRingKeys;
    n_splits = (Tk + kps - 1) / kps;          // no empty slice
    if (blockIdx.x == 0 && tid == 0) hdr[0] = n_splits;
    // with fewer CTAs than active heads (a host-side sizing error) the surplus heads would be lost
    if (static_cast<int>(gridDim.x) < n_act) {
        if (blockIdx.x == 0 && tid == 0) atomicExch(status, WIDE_ERR_UNSUPPORTED_SHAPE);
        return;
    }
    if (static_cast<int>(blockIdx.x) >= n_act * n_splits) return;
    const int hkv = s_heads[blockIdx.x / n_splits], split = blockIdx.x % n_splits;
    const int j0 = split * kps, j1 = min(Tk, j0 + kps);
    const int ntiles = (j1 - j0 + kRingKeys - 1) / kRingKeys;

    for (int i = tid; i < R * kVec; i += kRingThreads) {
        const int r = i / kVec, c = i % kVec;
        const int t = r / rep, h = hkv * rep + r % rep;
        const __nv_bfloat16* qp = q + t * ldq + static_cast<size_t>(h) * HD + 8 * c;
        qa[r][c] = make_float4(__bfloat162float(qp[0]) * scale_log2e, __bfloat162float(qp[1]) * scale_log2e,
                               __bfloat162float(qp[2]) * scale_log2e, __bfloat162float(qp[3]) * scale_log2e);
        qb[r][c] = make_float4(__bfloat162float(qp[4]) * scale_log2e, __bfloat162float(qp[5]) * scale_log2e,
                               __bfloat162float(qp[6]) * scale_log2e, __bfloat162float(qp[7]) * scale_log2e);
    }
    __syncthreads();

    float m[RT], l[RT], o[RT][kDL];
#pragma unroll
    for (int r = 0; r < RT; ++r) {
        m[r] = -CUDART_INF_F;
        l[r] = 0.f;
#pragma unroll
        for (int d = 0; d < kDL; ++d) o[r][d] = 0.f;
    }

    if (warp == kRingConsumers) {
        if (lane == 0) {
            const uint64_t stream_policy = l2_policy_evict_first();   // K and V are read once
            for (int t = 0; t < ntiles; ++t) {
                const int st = t % kRingStages;
                const uint32_t ph = (t / kRingStages) & 1;
                if (!mbar_wait(empty + 8 * st, ph ^ 1u, wait_ns, &s_abort)) break;
                mbar_arrive_expect_tx(full + 8 * st, 2 * kTileBytes);
                const uint32_t dst = smem_u32(ring + st * 2 * kTileBytes);
                tma_load_2d_hint(dst, &tmK, hkv * HD, j0 + t * kRingKeys, full + 8 * st, stream_policy);
                tma_load_2d_hint(dst + kTileBytes, &tmV, hkv * HD, j0 + t * kRingKeys, full + 8 * st, stream_policy);
                s_issued = t + 1;
            }
        }
    } else {
        for (int t = warp; t < ntiles; t += kRingConsumers) {
            const int st = t % kRingStages;
            const uint32_t ph = (t / kRingStages) & 1;
            if (!mbar_wait_warp(full + 8 * st, ph, wait_ns, &s_abort)) break;
            const uint8_t* kt = ring + st * 2 * kTileBytes;
            const uint8_t* vt = kt + kTileBytes;
            {
                const int c0 = j0 + t * kRingKeys;
                const int j = c0 + lane;
                const bool valid = j < j1;
                const uint8_t* krow = kt + lane * (HD * 2);
                float a[RT];
#pragma unroll
                for (int r = 0; r < RT; ++r) a[r] = 0.f;
#pragma unroll
                for (int i = 0; i < kVec; ++i) {
                    const int c = (i + lane) & (kVec - 1);
                    const uint4 kk = *reinterpret_cast<const uint4*>(krow + c * 16);
                    const __nv_bfloat162* kh = reinterpret_cast<const __nv_bfloat162*>(&kk);
                    const float2 k0 = __bfloat1622float2(kh[0]), k1 = __bfloat1622float2(kh[1]);
                    const float2 k2 = __bfloat1622float2(kh[2]), k3 = __bfloat1622float2(kh[3]);
#pragma unroll
                    for (int r = 0; r < RT; ++r) {
                        if (r < R) {
                            const float4 x0 = qa[r][c], x1 = qb[r][c];
                            a[r] = fmaf(x0.x, k0.x, a[r]); a[r] = fmaf(x0.y, k0.y, a[r]);
                            a[r] = fmaf(x0.z, k1.x, a[r]); a[r] = fmaf(x0.w, k1.y, a[r]);
                            a[r] = fmaf(x1.x, k2.x, a[r]); a[r] = fmaf(x1.y, k2.y, a[r]);
                            a[r] = fmaf(x1.z, k3.x, a[r]); a[r] = fmaf(x1.w, k3.y, a[r]);
                        }
                    }
                }
#pragma unroll
                for (int r = 0; r < RT; ++r) {
                    if (r < R) {
                        const int lim = causal ? (r / rep) + delta : Tk - 1;   // last key this row may see
                        const float sc = (valid && j <= lim) ? a[r] : -CUDART_INF_F;
                        float mx = sc;
#pragma unroll
                        for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
                        const float m_new = fmaxf(m[r], mx);
                        const float m_use = m_new == -CUDART_INF_F ? 0.f : m_new;
                        const float p = exp2_fast(sc - m_use);
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
                const int nk = min(32, j1 - c0);
                const uint8_t* vrow = vt + lane * (kDL * 2);
#pragma unroll 8
                for (int u = 0; u < nk; ++u) {
                    float vv[4];
                    if (kDL == 4) {
                        const uint2 raw = *reinterpret_cast<const uint2*>(vrow + u * (HD * 2));
                        const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
                        const float2 y = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
                        vv[0] = x.x; vv[1] = x.y; vv[2] = y.x; vv[3] = y.y;
                    } else {
                        const uint32_t raw = *reinterpret_cast<const uint32_t*>(vrow + u * (HD * 2));
                        const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw));
                        vv[0] = x.x; vv[1] = x.y; vv[2] = 0.f; vv[3] = 0.f;
                    }
#pragma unroll
                    for (int r = 0; r < RT; ++r) {
                        if (r < R) {
                            const float p = ps[warp][r][u];
#pragma unroll
                            for (int d = 0; d < kDL; ++d) o[r][d] = fmaf(p, vv[d], o[r][d]);
                        }
                    }
                }
                __syncwarp();
            }
            if (lane == 0) mbar_arrive(empty + 8 * st);
        }
    }
    __syncthreads();   // every tile that was requested has been consumed (or the wait ran out): the ring is free
    if (s_abort) {
        if (tid == 0) {
            atomicExch(status, WIDE_ERR_TIMEOUT);
            // copies that were requested may still be on their way into this CTA's shared memory:
            // give them one more bounded wait before the CTA ends
            volatile int never = 0;
            for (int t = max(0, s_issued - kRingStages); t < s_issued; ++t)
                mbar_wait(full + 8 * (t % kRingStages), (t / kRingStages) & 1, wait_ns, &never);
        }
        return;
    }

    // merge the four warps (their partial O goes through the ring's memory), write this slice's partial
    float* wo = reinterpret_cast<float*>(ring);   // [kRingConsumers][RT][HD]
    if (warp < kRingConsumers) {
#pragma unroll
        for (int r = 0; r < RT; ++r) {
            if (r < R) {
                if (lane == 0) { wm[warp][r] = m[r]; wl[warp][r] = l[r]; }
#pragma unroll
                for (int d = 0; d < kDL; ++d) wo[(warp * RT + r) * HD + lane * kDL + d] = o[r][d];
            }
        }
    }
    __syncthreads();
    float* dst = part + (static_cast<size_t>(split) * Hkv + hkv) * R * (HD + 2);
    for (int i = tid; i < R * HD; i += kRingThreads) {
        const int r = i / HD, d = i % HD;
        float mm = -CUDART_INF_F;
#pragma unroll
        for (int w = 0; w < kRingConsumers; ++w) mm = fmaxf(mm, wm[w][r]);
        const float m_use = mm == -CUDART_INF_F ? 0.f : mm;
        float acc = 0.f, ll = 0.f;
#pragma unroll
        for (int w = 0; w < kRingConsumers; ++w) {
            const float al = exp2_fast(wm[w][r] - m_use);
            acc = fmaf(wo[(w * RT + r) * HD + d], al, acc);
            ll = fmaf(wl[w][r], al, ll);
        }
        dst[r * (HD + 2) + 2 + d] = acc;
        if (d == 0) {
            dst[r * (HD + 2)] = mm;
            dst[r * (HD + 2) + 1] = ll;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// The ring kernel for more than one query row per KV head (grouped-query attention, or a few new
// tokens at once).  With R rows every key costs 2 * R * HD multiply-adds, which the CUDA cores cannot
// issue at the rate HBM delivers the keys; the rows are therefore padded to the 16 rows of a
// warp-level tensor-core instruction (mma.sync m16n8k16, bf16 in, fp32 out -- with at most eight real
// rows there is no shape here for the 64-row tcgen05 instructions).  Same CTA layout as above: one
// producer thread, four consumer warps, a stage of 32 keys per warp.  K and V tiles are laid down by
// TMA in the 128-byte swizzle, [64-column half][32 keys][128 B], so that ldmatrix reads them without
// bank conflicts: K as it lies (the B operand of S = Q K^T), V transposed on the way in (the B operand
// of O += P V).  The score fragments are turned into the probabilities' A fragments in registers.
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// d (16x8, fp32) += a (16x16, bf16, row-major) * b (16x8, bf16, column-major); rows 8..15 of a are zero
// here, so the two accumulators of those rows (x2, x3) stay zero and are shared by all tiles.
__device__ __forceinline__ void mma_16816(float& d0, float& d1, float& x2, float& x3, uint32_t a0, uint32_t a2, uint32_t b0,
                                          uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d0), "+f"(d1), "+f"(x2), "+f"(x3)
                 : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}

template <int HD>
__global__ void __launch_bounds__(kRingThreads, 2)
attn_decode_ring_mma_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                            const __nv_bfloat16* __restrict__ q, const uint32_t* __restrict__ mask_bits, int words, int Tq,
                            int Tk, int Hq, int Hkv, int hpg, int causal, float scale_log2e, int max_splits,
                            float* __restrict__ part, int* __restrict__ hdr, int* status, unsigned long long wait_ns) {
    using namespace wptx;
    constexpr int kHalves = HD / 64;               // 64-column halves of a K or V tile
    constexpr int kHalfBytes = kRingKeys * 128;    // 32 keys x 128 B
    constexpr int kTileBytes = kHalves * kHalfBytes;
    constexpr int kKS = HD / 16;                   // k-steps of S = Q K^T
    constexpr int kNT = HD / 8;                    // 8-column tiles of O
    extern __shared__ uint8_t smem_raw[];
    __shared__ float wm[kRingConsumers][8], wl[kRingConsumers][8];
    __shared__ uint8_t s_heads[256];
    __shared__ int s_nact;
    __shared__ int s_abort;
    __shared__ int s_issued;
    __shared__ __align__(8) uint64_t s_bars[2 * kRingStages];
    uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rep = Hq / Hkv;
    const int R = Tq * rep;                        // <= 8
    const int delta = Tk - Tq;
    const size_t ldq = static_cast<size_t>(Hq) * HD;
    const uint32_t full = smem_u32(s_bars), empty = smem_u32(s_bars + kRingStages);

    if (tid == 0) {
        for (int st = 0; st < kRingStages; ++st) {
            mbar_init(full + 8 * st, 1);
            mbar_init(empty + 8 * st, 1);
        }
        s_abort = 0;
        s_issued = 0;
        fence_barrier_init();
        prefetch_tmap(&tmK);
        prefetch_tmap(&tmV);
    }
    if (warp == 0) {
        int pos = 0;   // the KV heads that some row reads, ascending
        for (int h0 = 0; h0 < Hkv; h0 += 32) {
            const int hkv = h0 + lane;
            bool any = false;
            if (hkv < Hkv)
                for (int r = 0; r < R; ++r) any = any || wide_mask_bit(mask_bits, words, r / rep, (hkv * rep + r % rep) / hpg);
            const unsigned vote = __ballot_sync(0xffffffffu, any);
            if (any) s_heads[pos + __popc(vote & ((1u << lane) - 1u))] = static_cast<uint8_t>(hkv);
            pos += __popc(vote);
        }
        if (lane == 0) s_nact = pos;
    }
    __syncthreads();
    const int n_act = s_nact;
    if (n_act == 0) {
        if (blockIdx.x == 0 && tid == 0) hdr[0] = 1;
        return;
    }
    int n_splits = min(min(static_cast<int>(gridDim.x) / n_act, (Tk + kRingKeys - 1) / kRingKeys), max_splits);
    if (n_splits < 1) n_splits = 1;
    const int kps = ((Tk + n_splits - 1) / n_splits + kRingKeys - 1) / kRingKeys * kRingKeys;
    n_splits = (Tk + kps - 1) / kps;          // no empty slice
    if (blockIdx.x == 0 && tid == 0) hdr[0] = n_splits;
    if (static_cast<int>(gridDim.x) < n_act) {
        if (blockIdx.x == 0 && tid == 0) atomicExch(status, WIDE_ERR_UNSUPPORTED_SHAPE);
        return;
    }
    if (static_cast<int>(blockIdx.x) >= n_act * n_splits) return;
    const int hkv = s_heads[blockIdx.x / n_splits], split = blockIdx.x % n_splits;
    const int j0 = split * kps, j1 = min(Tk, j0 + kps);
    const int ntiles = (j1 - j0 + kRingKeys - 1) / kRingKeys;

    // this thread's query row (fragment row lane / 4) and its A fragments: a0 = columns 16 ks + 2 (lane % 4) + {0, 1},
    // a2 = the same + 8
    const int qr = lane >> 2, qc = (lane & 3) * 2;
    const bool row_ok = qr < R;
    uint32_t qa0[kKS], qa2[kKS];
    {
        const int t = row_ok ? qr / rep : 0, h = hkv * rep + (row_ok ? qr % rep : 0);
        const __nv_bfloat16* qp = q + t * ldq + static_cast<size_t>(h) * HD + qc;
#pragma unroll
        for (int ks = 0; ks < kKS; ++ks) {
            qa0[ks] = row_ok ? *reinterpret_cast<const uint32_t*>(qp + 16 * ks) : 0u;
            qa2[ks] = row_ok ? *reinterpret_cast<const uint32_t*>(qp + 16 * ks + 8) : 0u;
        }
    }
    const int lim = causal ? (row_ok ? qr / rep : 0) + delta : Tk - 1;   // last key this row may see
    float m = -CUDART_INF_F, l = 0.f, x2 = 0.f, x3 = 0.f;
    float o[kNT][2];
#pragma unroll
    for (int nt = 0; nt < kNT; ++nt) { o[nt][0] = 0.f; o[nt][1] = 0.f; }

    if (warp == kRingConsumers) {
        if (lane == 0) {
            const uint64_t stream_policy = l2_policy_evict_first();   // K and V are read once
            for (int t = 0; t < ntiles; ++t) {
                const int st = t % kRingStages;
                const uint32_t ph = (t / kRingStages) & 1;
                if (!mbar_wait(empty + 8 * st, ph ^ 1u, wait_ns, &s_abort)) break;
                mbar_arrive_expect_tx(full + 8 * st, 2 * kTileBytes);
                const uint32_t dst = smem_u32(ring + st * 2 * kTileBytes);
#pragma unroll
                for (int hb = 0; hb < kHalves; ++hb) {
                    tma_load_2d_hint(dst + hb * kHalfBytes, &tmK, hkv * HD + 64 * hb, j0 + t * kRingKeys, full + 8 * st, stream_policy);
                    tma_load_2d_hint(dst + kTileBytes + hb * kHalfBytes, &tmV, hkv * HD + 64 * hb, j0 + t * kRingKeys, full + 8 * st,
                                     stream_policy);
                }
                s_issued = t + 1;
            }
        }
    } else {
        // ldmatrix row addresses of this lane: matrix lane / 8 of an x4 load, row lane % 8
        const int lrow = lane & 7, lmat = lane >> 3;
        for (int t = warp; t < ntiles; t += kRingConsumers) {
            const int st = t % kRingStages;
            const uint32_t ph = (t / kRingStages) & 1;
            if (!mbar_wait_warp(full + 8 * st, ph, wait_ns, &s_abort)) break;
            const uint32_t kt = smem_u32(ring + st * 2 * kTileBytes), vt = kt + kTileBytes;
            const int c0 = j0 + t * kRingKeys;
            // S = Q K^T: four 8-key tiles, kKS k-steps.  One x4 load = (k-step ks, columns +0 / +8) and (ks + 1, +0 / +8)
            float sc[4][2];
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                sc[nt][0] = 0.f; sc[nt][1] = 0.f;
                const int krow = 8 * nt + lrow;
#pragma unroll
                for (int ks = 0; ks < kKS; ks += 2) {
                    const int h0 = 16 * (ks + (lmat >> 1)) + 8 * (lmat & 1);           // first column of this lane's matrix
                    const uint32_t addr = kt + (h0 >> 6) * kHalfBytes + krow * 128 + ((((h0 & 63) >> 3) ^ (krow & 7)) << 4);
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4(addr, b0, b1, b2, b3);
                    mma_16816(sc[nt][0], sc[nt][1], x2, x3, qa0[ks], qa2[ks], b0, b1);
                    mma_16816(sc[nt][0], sc[nt][1], x2, x3, qa0[ks + 1], qa2[ks + 1], b2, b3);
                }
            }
            // online softmax of this thread's row over the tile's 32 keys (the row is spread over 4 lanes)
            float mx = -CUDART_INF_F;
#pragma unroll
            for (int nt = 0; nt < 4; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int j = c0 + 8 * nt + qc + e;
                    sc[nt][e] = (j < j1 && j <= lim) ? sc[nt][e] * scale_log2e : -CUDART_INF_F;
                    mx = fmaxf(mx, sc[nt][e]);
                }
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m, mx);
            const float m_use = m_new == -CUDART_INF_F ? 0.f : m_new;
            const float alpha = exp2_fast(m - m_use);
            float sum = 0.f;
            uint32_t pa[4];
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                const float p0 = exp2_fast(sc[nt][0] - m_use), p1 = exp2_fast(sc[nt][1] - m_use);
                sum += p0 + p1;
                const __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
                pa[nt] = *reinterpret_cast<const uint32_t*>(&pk);
            }
            sum += __shfl_xor_sync(0xffffffffu, sum, 1);
            sum += __shfl_xor_sync(0xffffffffu, sum, 2);
            l = fmaf(l, alpha, sum);
            m = m_new;
#pragma unroll
            for (int nt = 0; nt < kNT; ++nt) { o[nt][0] *= alpha; o[nt][1] *= alpha; }
            // O += P V: two k-steps of 16 keys; one transposed x4 load = (column tile nt, keys +0 / +8) and (nt + 1, ...)
#pragma unroll
            for (int kk = 0; kk < 2; ++kk) {
                const int vrow = 16 * kk + 8 * (lmat & 1) + lrow;
#pragma unroll
                for (int nt = 0; nt < kNT; nt += 2) {
                    const int ch = nt + (lmat >> 1);                                   // 8-column chunk of the head dimension
                    const uint32_t addr = vt + (ch >> 3) * kHalfBytes + vrow * 128 + (((ch & 7) ^ (vrow & 7)) << 4);
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4_trans(addr, b0, b1, b2, b3);
                    mma_16816(o[nt][0], o[nt][1], x2, x3, pa[2 * kk], pa[2 * kk + 1], b0, b1);
                    mma_16816(o[nt + 1][0], o[nt + 1][1], x2, x3, pa[2 * kk], pa[2 * kk + 1], b2, b3);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty + 8 * st);
        }
    }
    __syncthreads();   // every tile that was requested has been consumed (or the wait ran out): the ring is free
    if (s_abort) {
        if (tid == 0) {
            atomicExch(status, WIDE_ERR_TIMEOUT);
            volatile int never = 0;
            for (int t = max(0, s_issued - kRingStages); t < s_issued; ++t)
                mbar_wait(full + 8 * (t % kRingStages), (t / kRingStages) & 1, wait_ns, &never);
        }
        return;
    }

    // merge the four warps (their partial O goes through the ring's memory), write this slice's partial
    float* wo = reinterpret_cast<float*>(ring);   // [kRingConsumers][8][HD]
    if (warp < kRingConsumers && row_ok) {
        if ((lane & 3) == 0) { wm[warp][qr] = m; wl[warp][qr] = l; }
#pragma unroll
        for (int nt = 0; nt < kNT; ++nt) {
            wo[(warp * 8 + qr) * HD + 8 * nt + qc] = o[nt][0];
            wo[(warp * 8 + qr) * HD + 8 * nt + qc + 1] = o[nt][1];
        }
    }
    __syncthreads();
    float* dst = part + (static_cast<size_t>(split) * Hkv + hkv) * R * (HD + 2);
    for (int i = tid; i < R * HD; i += kRingThreads) {
        const int r = i / HD, d = i % HD;
        float mm = -CUDART_INF_F;
#pragma unroll
        for (int w = 0; w < kRingConsumers; ++w) mm = fmaxf(mm, wm[w][r]);
        const float m_use = mm == -CUDART_INF_F ? 0.f : mm;
        float acc = 0.f, ll = 0.f;
#pragma unroll
        for (int w = 0; w < kRingConsumers; ++w) {
            const float al = exp2_fast(wm[w][r] - m_use);
            acc = fmaf(wo[(w * 8 + r) * HD + d], al, acc);
            ll = fmaf(wl[w][r], al, ll);
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
__global__ void __launch_bounds__(4 * HD)
attn_decode_merge_kernel(const float* __restrict__ part, const uint32_t* __restrict__ mask_bits, int words, int Tq,
                         int Hq, int Hkv, int hpg, int n_splits_host, const int* __restrict__ hdr,
                         __nv_bfloat16* __restrict__ o) {
    // 4 * HD threads: thread (quarter qt, dimension d) takes the slices qt, qt + 4, ...; all of its loads
    // (at most kMaxSplits / 4) are requested before anything is used, so the kernel costs about one
    // load latency whatever the number of slices.
    constexpr int kPer = kMaxSplits / 4;
    const int n_splits = hdr ? *hdr : n_splits_host;
    const int t = blockIdx.x / Hq, h = blockIdx.x % Hq;
    const int qt = threadIdx.x / HD, d = threadIdx.x % HD;
    const int rep = Hq / Hkv, R = Tq * rep;
    const int hkv = h / rep, r = t * rep + h % rep;
    __shared__ float s_m[kMaxSplits], s_w[kMaxSplits];
    __shared__ float s_acc[4][HD], s_ll[4];
    const bool on = wide_mask_bit(mask_bits, words, t, h / hpg);   // the same for the whole CTA
    if (on) {
        const size_t stride = static_cast<size_t>(Hkv) * R * (HD + 2);
        const float* p0 = part + (static_cast<size_t>(hkv) * R + r) * (HD + 2);
        for (int sp = threadIdx.x; sp < n_splits; sp += 4 * HD) {
            s_m[sp] = __ldcg(p0 + sp * stride);
            s_w[sp] = __ldcg(p0 + sp * stride + 1);
        }
        float vals[kPer];
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            const int sp = qt + 4 * i;
            vals[i] = sp < n_splits ? __ldcg(p0 + sp * stride + 2 + d) : 0.f;
        }
        __syncthreads();
        float mm = -CUDART_INF_F;
        for (int sp = 0; sp < n_splits; ++sp) mm = fmaxf(mm, s_m[sp]);
        const float m_use = mm == -CUDART_INF_F ? 0.f : mm;
        float acc = 0.f, ll = 0.f;
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            const int sp = qt + 4 * i;
            if (sp < n_splits) {
                const float a = exp2_fast(s_m[sp] - m_use);
                acc = fmaf(vals[i], a, acc);
                ll = fmaf(s_w[sp], a, ll);
            }
        }
        s_acc[qt][d] = acc;
        if (d == 0) s_ll[qt] = ll;
        __syncthreads();
    }
    if (qt == 0) {
        float out = 0.f;
        if (on) {
            const float acc = (s_acc[0][d] + s_acc[1][d]) + (s_acc[2][d] + s_acc[3][d]);
            const float ll = (s_ll[0] + s_ll[1]) + (s_ll[2] + s_ll[3]);
            out = ll > 0.f ? acc / ll : 0.f;
        }
        o[(static_cast<size_t>(t) * Hq + h) * HD + d] = __float2bfloat16_rn(out);
    }
}

template <int HD>
int launch_attn_decode(wide_ctx* ctx, cudaStream_t s, const void* q, const void* k, const void* v,
                       const uint32_t* mask_bits, int Tq, int Tk, int Hq, int Hkv, int hpg, int causal, float scale,
                       void* o) {
    const int rep = Hq / Hkv, R = Tq * rep;
    const int words = (Hq / hpg + 31) / 32;
    // enough key slices for about seven CTAs per SM over all KV heads (the kernel hides its load
    // latency by occupancy; more and shorter slices cost more in set-up and merging than they gain
    // in balance: 30 slices per head took 83 + 19 us at 32 768 keys, 26 take 77 + 11, 45 take 95 + 13),
    // at least 128 keys each, and the scratch slab must hold them
    int n_splits = (7 * ctx->sm_count + Hkv - 1) / Hkv;
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
    attn_decode_merge_kernel<HD><<<Tq * Hq, 4 * HD, 0, s>>>(ctx->attn_part, mask_bits, words, Tq, Hq, Hkv, hpg, n_splits,
                                                         nullptr, static_cast<__nv_bfloat16*>(o));
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// K or V cache [rows, cols] bf16 as a 2-D tensor; a box is 64 rows of one head's HD columns, laid
// down row by row (no swizzle).
bool make_kv_tmap(const wide_ctx* ctx, CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, int hd) {
    if (!ctx->encode_tiled) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(hd), static_cast<cuuint32_t>(kRingKeys)};
    const cuuint32_t estr[2] = {1, 1};
    return reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
               map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int HD>
int launch_attn_decode_ring(wide_ctx* ctx, cudaStream_t s, const void* q, const void* k, const void* v,
                            const uint32_t* mask_bits, int Tq, int Tk, int Hq, int Hkv, int hpg, int causal, float scale,
                            void* o) {
    const int rep = Hq / Hkv, R = Tq * rep;
    const int words = (Hq / hpg + 31) / 32;
    if (Hkv > 256) return WIDE_ERR_UNSUPPORTED_SHAPE;
    CUtensorMap tmK, tmV;
    if (!make_kv_tmap(ctx, &tmK, k, static_cast<uint64_t>(Tk), static_cast<uint64_t>(Hkv) * HD, HD) ||
        !make_kv_tmap(ctx, &tmV, v, static_cast<uint64_t>(Tk), static_cast<uint64_t>(Hkv) * HD, HD))
        return WIDE_ERR_CUDA;
    // the last 256 bytes of the scratch slab hold the slice count the kernel settles on
    const size_t per_split = static_cast<size_t>(Hkv) * R * (HD + 2) * sizeof(float);
    const size_t slab = ctx->attn_part_bytes - 256;
    int max_splits = static_cast<int>(slab / per_split);
    if (max_splits > kMaxSplits) max_splits = kMaxSplits;
    if (max_splits < 1) return WIDE_ERR_UNSUPPORTED_SHAPE;
    int* hdr = reinterpret_cast<int*>(reinterpret_cast<char*>(ctx->attn_part) + slab);
    int grid = 0;   // as many CTAs as are resident at once (set per instantiation below); never fewer than KV heads
    if (R >= 2) {
        // several query rows per KV head: the tensor-core form (tiles in the 128-byte swizzle)
        CUtensorMap smK, smV;
        if (!wide_make_tmap_bf16(ctx, &smK, k, static_cast<uint64_t>(Tk), static_cast<uint64_t>(Hkv) * HD, kRingKeys) ||
            !wide_make_tmap_bf16(ctx, &smV, v, static_cast<uint64_t>(Tk), static_cast<uint64_t>(Hkv) * HD, kRingKeys))
            return WIDE_ERR_CUDA;
        constexpr int kSmemM = kRingStages * 2 * kRingKeys * HD * 2 + 1024;
        WIDE_CUDA_CHECK(cudaFuncSetAttribute(attn_decode_ring_mma_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kSmemM));
        int per_sm = 0;
        WIDE_CUDA_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, attn_decode_ring_mma_kernel<HD>, kRingThreads,
                                                                      kSmemM));
        grid = (per_sm > 0 ? per_sm : 1) * ctx->sm_count;
        if (grid < Hkv) grid = Hkv;
        {
            WideLaunch l(ctx, s, "attn_decode");
            attn_decode_ring_mma_kernel<HD><<<grid, kRingThreads, kSmemM, s>>>(
                smK, smV, static_cast<const __nv_bfloat16*>(q), mask_bits, words, Tq, Tk, Hq, Hkv, hpg, causal,
                scale * 1.4426950408889634f, max_splits, ctx->attn_part, hdr, ctx->d_status, ctx->wait_ns);
        }
        if (cudaGetLastError() != cudaSuccess) return WIDE_ERR_CUDA;
        WideLaunch l(ctx, s, "attn_decode_merge");
        attn_decode_merge_kernel<HD><<<Tq * Hq, 4 * HD, 0, s>>>(ctx->attn_part, mask_bits, words, Tq, Hq, Hkv, hpg, 0, hdr,
                                                             static_cast<__nv_bfloat16*>(o));
        return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
    }
    constexpr int kSmem = kRingStages * 2 * kRingKeys * HD * 2 + 128;
    const __nv_bfloat16* qb = static_cast<const __nv_bfloat16*>(q);
    const float sl = scale * 1.4426950408889634f;
    {
        WideLaunch l(ctx, s, "attn_decode");
#define WIDE_RING_CASE(rt)                                                                                              \
    do {                                                                                                                \
        WIDE_CUDA_CHECK(cudaFuncSetAttribute(attn_decode_ring_kernel<HD, rt>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                             kSmem));                                                                   \
        int per_sm = 0;                                                                                                 \
        WIDE_CUDA_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, attn_decode_ring_kernel<HD, rt>,          \
                                                                      kRingThreads, kSmem));                            \
        grid = (per_sm > 0 ? per_sm : 1) * ctx->sm_count;                                                               \
        if (grid < Hkv) grid = Hkv;                                                                                     \
        attn_decode_ring_kernel<HD, rt><<<grid, kRingThreads, kSmem, s>>>(tmK, tmV, qb, mask_bits, words, Tq, Tk, Hq, Hkv, \
                                                                         hpg, causal, sl, max_splits, ctx->attn_part, hdr, \
                                                                         ctx->d_status, ctx->wait_ns);                  \
    } while (0)
        if (R <= 1) WIDE_RING_CASE(1);
        else if (R <= 2) WIDE_RING_CASE(2);
        else if (R <= 4) WIDE_RING_CASE(4);
        else WIDE_RING_CASE(8);
#undef WIDE_RING_CASE
    }
    if (cudaGetLastError() != cudaSuccess) return WIDE_ERR_CUDA;
    WideLaunch l(ctx, s, "attn_decode_merge");
    attn_decode_merge_kernel<HD><<<Tq * Hq, 4 * HD, 0, s>>>(ctx->attn_part, mask_bits, words, Tq, Hq, Hkv, hpg, 0, hdr,
                                                         static_cast<__nv_bfloat16*>(o));
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}

}  // namespace

bool wide_attn_decode_fits(int Tq, int Hq, int Hkv) { return Tq * (Hq / Hkv) <= kMaxRows; }

int wide_launch_attn_decode(wide_ctx* ctx, cudaStream_t s, const void* q, const void* k, const void* v,
                            const uint32_t* mask_bits, int Tq, int Tk, int Hq, int Hkv, int head_dim, int hpg,
                            int causal, float scale, void* o, unsigned flags) {
    // K and V through a TMA ring unless the caller asks for the plain-load kernel; the caches' rows
    // must then start on 16-byte boundaries, which head sizes 64 and 128 give
    const bool ring = ctx->encode_tiled && !(flags & WIDE_FLAG_SIMT) && (reinterpret_cast<uintptr_t>(k) & 15) == 0 &&
                      (reinterpret_cast<uintptr_t>(v) & 15) == 0;
    if (head_dim == 128)
        return ring ? launch_attn_decode_ring<128>(ctx, s, q, k, v, mask_bits, Tq, Tk, Hq, Hkv, hpg, causal, scale, o)
                    : launch_attn_decode<128>(ctx, s, q, k, v, mask_bits, Tq, Tk, Hq, Hkv, hpg, causal, scale, o);
    if (head_dim == 64)
        return ring ? launch_attn_decode_ring<64>(ctx, s, q, k, v, mask_bits, Tq, Tk, Hq, Hkv, hpg, causal, scale, o)
                    : launch_attn_decode<64>(ctx, s, q, k, v, mask_bits, Tq, Tk, Hq, Hkv, hpg, causal, scale, o);
    return WIDE_ERR_UNSUPPORTED_SHAPE;
}
