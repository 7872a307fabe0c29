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
            if (!mbar_wait(full + 8 * st, ph, wait_ns, &s_abort)) break;
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

// One CTA per (token, query head): merge the key slices, normalise, write bf16; zeros for an
// inactive (token, group) pair or a query that saw no key.
template <int HD>
__global__ void __launch_bounds__(HD)
attn_decode_merge_kernel(const float* __restrict__ part, const uint32_t* __restrict__ mask_bits, int words, int Tq,
                         int Hq, int Hkv, int hpg, int n_splits_host, const int* __restrict__ hdr,
                         __nv_bfloat16* __restrict__ o) {
    const int n_splits = hdr ? *hdr : n_splits_host;
    const int t = blockIdx.x / Hq, h = blockIdx.x % Hq, d = threadIdx.x;
    const int rep = Hq / Hkv, R = Tq * rep;
    const int hkv = h / rep, r = t * rep + h % rep;
    __shared__ float s_m[kMaxSplits], s_w[kMaxSplits];
    float out = 0.f;
    if (wide_mask_bit(mask_bits, words, t, h / hpg)) {   // the same for the whole CTA
        const size_t stride = static_cast<size_t>(Hkv) * R * (HD + 2);
        const float* p0 = part + (static_cast<size_t>(hkv) * R + r) * (HD + 2);
        // the slices' (m, l) first, all at once, so that the sums below wait for one load latency
        for (int s = d; s < n_splits; s += HD) {
            s_m[s] = __ldcg(p0 + s * stride);
            s_w[s] = __ldcg(p0 + s * stride + 1);
        }
        __syncthreads();
        float mm = -CUDART_INF_F;
        for (int s = 0; s < n_splits; ++s) mm = fmaxf(mm, s_m[s]);
        const float m_use = mm == -CUDART_INF_F ? 0.f : mm;
        float acc = 0.f, ll = 0.f;
#pragma unroll 16
        for (int s = 0; s < n_splits; ++s) {
            const float a = exp2_fast(s_m[s] - m_use);
            acc = fmaf(__ldcg(p0 + s * stride + 2 + d), a, acc);
            ll = fmaf(s_w[s], a, ll);
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
    attn_decode_merge_kernel<HD><<<Tq * Hq, HD, 0, s>>>(ctx->attn_part, mask_bits, words, Tq, Hq, Hkv, hpg, n_splits,
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
    attn_decode_merge_kernel<HD><<<Tq * Hq, HD, 0, s>>>(ctx->attn_part, mask_bits, words, Tq, Hq, Hkv, hpg, 0, hdr,
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
