// Head-group-masked FlashAttention prefill on tcgen05 (Algorithm 4): query-tile admission through
// the reordered mask, gathered Q rows, dense K/V tiles streamed by TMA, online softmax, scatter
// epilogue.
//
// One CTA owns one (query head h, tile m of 128 rows of the head's routing group g in that group's
// sorted order).  Tiles past the group's active count exit at once (block-level predicate); the
// rows of a tile are gathered through perm[g] (row-level predicate: rows past the count are
// computed on a clamped copy and dropped in the epilogue).  Per key tile t of 128 keys:
//     S  = Q K_t^T                (UMMA, fp32 in TMEM, two buffers)
//     P  = exp2(S*c - m), row statistics m, l   (softmax warps: one thread per row, S read twice from
//                                  TMEM so that a row never has to live in registers)
//     O += P V_t                  (UMMA accumulating in TMEM; P goes through shared memory as a bf16
//                                  K-major operand, V_t is used as loaded, as an MN-major operand)
// O stays in TMEM for the whole key loop.  A row's reference maximum m is only raised when the
// running maximum has grown by more than 2^8 since it was set (P then stays below 2^8, harmless in
// bf16 / fp32); raising it rescales that warp's rows of O in TMEM (load, multiply, store), which
// after the first tiles is rare, so the softmax warps carry no accumulator registers at all.
// A softmax group hands its S buffer back as soon as the row is in registers, and the UMMA warp
// then issues the group's next scores (tile t+2) BEFORE the PV of tile t, so a group never waits
// for its scores and the tensor core works while the softmax warps are busy.  The two kinds of
// UMMA have an issuing thread each (a single thread's waits, fences and commits for both took
// longer per tile than the tensor core needs), and K and V have a producer warp each: their
// rings drain at different points of the loop.  The softmax is the slower side (one exponential per
// score), so two groups of four warps share the rows: group 0 takes the even key tiles, group 1
// the odd ones, each with its own (m, l, O) per row and its own S / P / O buffers; the two
// partial results are merged once at the end (the split-key form of the online softmax).  Causal attention shortens the key range to the largest
// active query position of the tile (+ delta = T_k - T_q); only tiles that straddle a row's limit
// evaluate element-wise predicates.
//
// Outputs of inactive (token, group) pairs are exact zeros, written by the CTAs of the tiles that hold no
// (or not only) active rows before they do anything else.
// Every mbarrier wait is bounded.
#include <cuda.h>
#include <math_constants.h>

#include "internal.h"
#include "ptx.cuh"

namespace {

using namespace wptx;

constexpr int kQ = 128;        // query rows per tile (UMMA M)
constexpr int kKV = 128;       // keys per tile
constexpr int kBK = 64;        // bf16 elements per 128-byte swizzle row
constexpr int kBlk = 16384;    // bytes of one [128 rows x 64 elements] swizzled block
constexpr int kThreads = 384;  // K producer, QK issuer, 2 groups of 4 softmax warps, V producer, PV issuer

// Shared-memory descriptor of an MN-major operand in the 128-byte swizzle: the tile is stored as
// loaded by TMA, rows = K index (128 bytes = 64 elements of the MN dimension each).  Blocks of 64
// MN elements are `lbo` bytes apart, groups of 8 K rows 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_sw128_mn(uint32_t smem_addr, uint32_t lbo) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>(lbo >> 4) << 16;
    d |= static_cast<uint64_t>(1024 >> 4) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(2) << 61;
    return d;
}

__host__ __device__ constexpr uint32_t idesc_bf16(int m, int n, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) |
           (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(m >> 4) << 24);
}

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int HD>
constexpr int attn_smem_bytes() {
    // Q, 2 K stages, 2 V stages, 2 P buffers, barriers, alignment slack
    return (HD / kBK) * kBlk + 4 * (HD / kBK) * kBlk + 2 * (kKV / kBK) * kBlk + 256 + 1024;
}

// q [T_q, H_q*HD], o likewise; K/V come through the tensor maps ([T_k, H_kv*HD], box 64 x 128).
template <int HD>
__global__ void __launch_bounds__(kThreads, 1)
attn_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
            const __nv_bfloat16* __restrict__ q, const int32_t* __restrict__ perm, const int32_t* __restrict__ counts,
            int Tq, int Tk, int Hq, int Hkv, int hpg, int causal, float scale_log2e,
            __nv_bfloat16* __restrict__ o, int* __restrict__ status, unsigned long long wait_ns) {
    constexpr int kKB = HD / kBK;          // 64-wide blocks along the head dimension
    constexpr int kQBytes = kKB * kBlk;
    constexpr int kKVBytes = kKB * kBlk;   // one K (or V) tile
    constexpr int kPBytes = (kKV / kBK) * kBlk;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const size_t ldq = static_cast<size_t>(Hq) * HD;

    // heavy (late, long key range) tiles first
    const int n_mt = (Tq + kQ - 1) / kQ;
    const int m = n_mt - 1 - static_cast<int>(blockIdx.x) / Hq;
    const int h = static_cast<int>(blockIdx.x) % Hq;
    const int g = h / hpg;
    const int hkv = h / (Hq / Hkv);
    const int c = counts[g];
    const int32_t* rows = perm + static_cast<size_t>(g) * Tq + m * kQ;
    // Block-level predicate: sorted positions >= counts[g] are the tokens that skip this head group, and
    // their outputs are exact zeros.  A tile with no active row only writes those zeros (such tiles
    // come first in the launch order and are gone at once); the tile that holds the boundary writes them
    // for its inactive tail before it starts.
    const int n_valid = max(0, min(kQ, c - m * kQ));
    {
        const int n_rows = min(kQ, Tq - m * kQ);
        constexpr int kPieces = HD / 8;
        for (int i = n_valid * kPieces + tid; i < n_rows * kPieces; i += kThreads) {
            const int row = rows[i / kPieces];
            reinterpret_cast<uint4*>(o + row * ldq + static_cast<size_t>(h) * HD)[i % kPieces] = make_uint4(0u, 0u, 0u, 0u);
        }
    }
    if (n_valid == 0) return;
    const int delta = Tk - Tq;
    // key range: up to the largest active query position of the tile
    int j_max = Tk;
    if (causal) j_max = min(Tk, delta + 1 + rows[n_valid - 1]);
    const int NT = j_max > 0 ? (j_max + kKV - 1) / kKV : 0;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* q_s = base;
    uint8_t* k_s = q_s + kQBytes;             // 2 stages
    uint8_t* v_s = k_s + 2 * kKVBytes;        // 2 stages
    uint8_t* p_s = v_s + 2 * kKVBytes;        // 2 buffers
    uint64_t* bars = reinterpret_cast<uint64_t*>(p_s + 2 * kPBytes);
    const uint32_t k_full = smem_u32(bars), k_empty = smem_u32(bars + 2), v_full = smem_u32(bars + 4),
                   v_empty = smem_u32(bars + 6), s_full = smem_u32(bars + 8), s_free = smem_u32(bars + 10),
                   p_ready = smem_u32(bars + 12), pv_full = smem_u32(bars + 14), pv_free = smem_u32(bars + 16),
                   q_ready = smem_u32(bars + 18);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 19);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(k_full + 8 * i, 1);
            mbar_init(k_empty + 8 * i, 1);
            mbar_init(v_full + 8 * i, 1);
            mbar_init(v_empty + 8 * i, 1);
            mbar_init(s_full + 8 * i, 1);
            mbar_init(s_free + 8 * i, 128);
            mbar_init(p_ready + 8 * i, 128);
            mbar_init(pv_full + 8 * i, 1);
        }
        mbar_init(q_ready, 256);
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmK);
        prefetch_tmap(&tmV);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0 || warp == 10) {
        // ------------------------------------------------------------------ TMA producers: K (warp 0), V (warp 10)
        if (lane == 0) {
            const bool is_k = warp == 0;
            const uint32_t full = is_k ? k_full : v_full, empty = is_k ? k_empty : v_empty;
            uint8_t* ring = is_k ? k_s : v_s;
            const CUtensorMap* tm = is_k ? &tmK : &tmV;
            bool ok = true;
            for (int t = 0; t < NT; ++t) {
                const int s = t & 1;
                const uint32_t ph = (t >> 1) & 1;
                if (!mbar_wait(empty + 8 * s, ph ^ 1u, wait_ns, abort_flag)) { ok = false; break; }
                mbar_arrive_expect_tx(full + 8 * s, kKVBytes);
                for (int kb = 0; kb < kKB; ++kb)
                    tma_load_2d(smem_u32(ring + s * kKVBytes + kb * kBlk), tm, hkv * HD + kb * kBK, t * kKV, full + 8 * s);
            }
            if (!ok) {
                atomicExch(status, WIDE_ERR_TIMEOUT);
                for (int i = 0; i < 64; ++i) __nanosleep(1000);   // let copies in flight land
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ UMMA issuer: S = Q K^T
        if (lane == 0) {
            constexpr uint32_t idesc_qk = idesc_bf16(kQ, kKV, false);
            bool ok = NT == 0 || mbar_wait(q_ready, 0, wait_ns, abort_flag);
            fence_proxy_async_smem();  // the Q rows were written through the generic proxy (cp.async)
            uint64_t qdesc[kKB];
#pragma unroll
            for (int kb = 0; kb < kKB; ++kb) qdesc[kb] = umma_desc_sw128(smem_u32(q_s + kb * kBlk));
            auto issue_qk = [&](int t) -> bool {
                const int s = t & 1;
                if (!mbar_wait(k_full + 8 * s, (t >> 1) & 1, wait_ns, abort_flag)) return false;
                tc_fence_after_sync();
                const uint64_t kdesc = umma_desc_sw128(smem_u32(k_s + s * kKVBytes));
#pragma unroll
                for (int k16 = 0; k16 < HD / 16; ++k16)
                    umma_bf16(tmem_base + s * kKV, qdesc[k16 / 4] + 2 * (k16 % 4),
                              kdesc + (k16 / 4) * (kBlk >> 4) + 2 * (k16 % 4), idesc_qk, k16 > 0 ? 1u : 0u);
                umma_commit(k_empty + 8 * s);
                umma_commit(s_full + 8 * s);
                return true;
            };
            if (ok && NT > 0) ok = issue_qk(0);
            if (ok && NT > 1) ok = issue_qk(1);
            // the group of tile t has its scores in registers: its next scores can be computed now
            for (int t = 0; t + 2 < NT && ok; ++t) {
                if (!mbar_wait(s_free + 8 * (t & 1), (t >> 1) & 1, wait_ns, abort_flag)) { ok = false; break; }
                ok = issue_qk(t + 2);
            }
            if (!ok) atomicExch(status, WIDE_ERR_TIMEOUT);
        }
    } else if (warp == 11) {
        // ------------------------------------------------------------------ UMMA issuer: O += P V
        if (lane == 0) {
            constexpr uint32_t idesc_pv = idesc_bf16(kQ, HD, true);
            bool ok = true;
            for (int t = 0; t < NT; ++t) {
                const int s = t & 1;
                const uint32_t ph = (t >> 1) & 1;
                if (!mbar_wait(v_full + 8 * s, ph, wait_ns, abort_flag)) { ok = false; break; }
                if (!mbar_wait(p_ready + 8 * s, ph, wait_ns, abort_flag)) { ok = false; break; }
                fence_proxy_async_smem();   // P was written through the generic proxy
                tc_fence_after_sync();
                const uint64_t pdesc = umma_desc_sw128(smem_u32(p_s + s * kPBytes));
                const uint64_t vdesc = umma_desc_sw128_mn(smem_u32(v_s + s * kKVBytes), kBlk);
#pragma unroll
                for (int k16 = 0; k16 < kKV / 16; ++k16)
                    umma_bf16(tmem_base + 256 + s * HD, pdesc + (k16 / 4) * (kBlk >> 4) + 2 * (k16 % 4),
                              vdesc + k16 * (2048 >> 4), idesc_pv, (t >= 2 || k16 > 0) ? 1u : 0u);
                umma_commit(v_empty + 8 * s);
                umma_commit(pv_full + 8 * s);
            }
            if (!ok) atomicExch(status, WIDE_ERR_TIMEOUT);
        }
    } else {
        // ------------------------------------------------------------------ softmax warps (2..9)
        const int st = tid - 64;                     // 0..255
        const int grp = (warp - 2) >> 2;             // 0: even key tiles, 1: odd key tiles
        const int quarter = warp & 3;                // TMEM lane quarter this warp may read
        const int r = quarter * 32 + lane;           // row of the tile owned by this thread
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        bool ok = true;

        // Q prologue: 16-byte chunks, 8 consecutive threads copy one 128-byte row of a block
        if (NT > 0) {
            const int chunk = st & 7;
#pragma unroll
            for (int i = 0; i < kQ / 32; ++i) {
                const int row = (st >> 3) + 32 * i;
                const int src_row = rows[min(row, n_valid - 1)];
                const uint8_t* src = reinterpret_cast<const uint8_t*>(q + src_row * ldq + static_cast<size_t>(h) * HD) + 16 * chunk;
#pragma unroll
                for (int kb = 0; kb < kKB; ++kb)
                    cp_async_16(smem_u32(q_s + kb * kBlk) + static_cast<uint32_t>(row) * 128u +
                                    ((static_cast<uint32_t>(chunk) ^ static_cast<uint32_t>(row & 7)) << 4),
                                src + kb * 128);
            }
            cp_async_mbar_arrive_noinc(q_ready);
        }

        const int pos = rows[min(r, n_valid - 1)];
        const int lim = causal ? min(pos + delta, Tk - 1) : Tk - 1;   // last visible key of this row
        float mref = -CUDART_INF_F, lrow = 0.f;      // reference maximum (log2 units, scaled), row sum
        const int b = grp;                           // this group's S / P / O buffer
        const uint32_t o_addr = lane_addr + 256 + b * HD;
        constexpr float kRaise = 8.f;                // raise the reference only for a growth above 2^8

        int last = -1;
        for (int t = grp; t < NT; t += 2) {
            const uint32_t ph = (t >> 1) & 1;
            if (!mbar_wait_warp(s_full + 8 * b, ph, wait_ns, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const int j0 = t * kKV;
            const bool edge = j0 + kKV - 1 > lim;     // this row needs element-wise predicates here
            // The whole score row comes into registers with one TMEM round trip (the latency of a
            // tcgen05.ld is what a chunked loop would pay per chunk), and S is handed back to the
            // UMMA warp before any arithmetic: the next scores of this group are computed meanwhile.
            uint32_t v[kKV];
#pragma unroll
            for (int c0 = 0; c0 < kKV; c0 += 32) tmem_ld_32x32(lane_addr + b * kKV + c0, reinterpret_cast<uint32_t(&)[32]>(v[c0]));
            tmem_ld_wait();
            tc_fence_before_sync();
            mbar_arrive(s_free + 8 * b);
            // row maximum of the raw scores (the scale is positive)
            float mx4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
            if (!edge) {
#pragma unroll
                for (int i = 0; i < kKV; ++i) mx4[i & 3] = fmaxf(mx4[i & 3], __uint_as_float(v[i]));
            } else {
#pragma unroll
                for (int i = 0; i < kKV; ++i) {
                    if (j0 + i > lim) v[i] = 0xff800000u;   // -inf: exp2 gives an exact zero below
                    mx4[i & 3] = fmaxf(mx4[i & 3], __uint_as_float(v[i]));
                }
            }
            const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * scale_log2e;
            // the previous PV of this group has to be complete before P is overwritten or O rescaled
            if (last >= 0 && !mbar_wait_warp(pv_full + 8 * b, (last >> 1) & 1, wait_ns, abort_flag)) { ok = false; break; }
            float alpha = 1.f;
            const bool raise = mx > mref + kRaise || (mref == -CUDART_INF_F && mx > mref);
            if (raise) {
                alpha = fast_exp2(mref - mx);        // 0 when this is the first key the row sees
                mref = mx;
            }
            if (last >= 0 && __any_sync(0xffffffffu, raise)) {
                tc_fence_after_sync();
#pragma unroll 1
                for (int c0 = 0; c0 < HD; c0 += 16) {
                    uint32_t w[16];
                    tmem_ld_32x16(o_addr + c0, w);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 16; ++i) w[i] = __float_as_uint(__uint_as_float(w[i]) * alpha);
                    tmem_st_32x16(o_addr + c0, w);
                }
                tmem_st_wait();
            }
            const float m_use = mref == -CUDART_INF_F ? 0.f : mref;     // a row that has seen no key yet
            // P = exp2(S*c - m) as bf16 into the operand layout, row sum
            float rs4[4] = {0.f, 0.f, 0.f, 0.f};
            uint8_t* prow = p_s + b * kPBytes + r * 128;
            // sixteen scores at a time, each step over all sixteen before the next (arguments, then
            // exponentials, then sums and packing): the steps of one score depend on each other, so
            // score-by-score code runs at the sum of the instruction latencies
#pragma unroll
            for (int c0 = 0; c0 < kKV; c0 += 16) {
                float x[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) x[i] = fmaf(__uint_as_float(v[c0 + i]), scale_log2e, -m_use);
#pragma unroll
                for (int i = 0; i < 16; ++i) x[i] = fast_exp2(x[i]);
#pragma unroll
                for (int i = 0; i < 16; i += 4) {
                    rs4[0] += x[i];
                    rs4[1] += x[i + 1];
                    rs4[2] += x[i + 2];
                    rs4[3] += x[i + 3];
                }
                uint32_t pk[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) pk[i] = pack2(x[2 * i], x[2 * i + 1]);
                *reinterpret_cast<uint4*>(prow + (c0 / kBK) * kBlk + ((((c0 % kBK) / 8) ^ (r & 7)) << 4)) =
                    make_uint4(pk[0], pk[1], pk[2], pk[3]);
                *reinterpret_cast<uint4*>(prow + (c0 / kBK) * kBlk + (((((c0 + 8) % kBK) / 8) ^ (r & 7)) << 4)) =
                    make_uint4(pk[4], pk[5], pk[6], pk[7]);
            }
            lrow = fmaf(lrow, alpha, (rs4[0] + rs4[1]) + (rs4[2] + rs4[3]));
            tc_fence_before_sync();
            fence_proxy_async_smem();
            mbar_arrive(p_ready + 8 * b);
            last = t;
        }
        if (ok && last >= 0) ok = mbar_wait_warp(pv_full + 8 * b, (last >> 1) & 1, wait_ns, abort_flag);
        tc_fence_after_sync();
        if (NT > 0) cp_async_wait_all();
        const float mrow = mref;

        // Merge the two groups' partial results.  By now every S = Q K^T has completed (the PV of a
        // tile is issued after the S of the next one and UMMAs complete in order), so the K stages
        // are free: group 1 parks (m, l, O) there, column-major so that a warp writes 128 bytes.
        float* xo = reinterpret_cast<float*>(k_s);                  // [HD][128]
        float* xml = reinterpret_cast<float*>(q_s);                 // [2][128]
        const bool two = NT > 1;   // with a single key tile group 1 has nothing (and S may still be running)
        if (grp == 1 && two) {
#pragma unroll 1
            for (int c0 = 0; c0 < HD; c0 += 32) {
                uint32_t v[32];
                tmem_ld_32x32(o_addr + c0, v);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) xo[(c0 + i) * kQ + r] = __uint_as_float(v[i]);
            }
            xml[r] = mrow;
            xml[kQ + r] = lrow;
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (grp == 0) {
            const float m1 = two ? xml[r] : -CUDART_INF_F, l1 = two ? xml[kQ + r] : 0.f;
            const float m_all = fmaxf(mrow, m1);
            const float m_use = m_all == -CUDART_INF_F ? 0.f : m_all;
            const float a0 = fast_exp2(mrow - m_use), a1 = fast_exp2(m1 - m_use);
            const float l_all = lrow * a0 + l1 * a1;
            const float inv = l_all > 0.f ? 1.f / l_all : 0.f;
            // epilogue: normalise and scatter the active rows (O of group 0 comes straight from TMEM)
            uint4* dst = reinterpret_cast<uint4*>(o + pos * ldq + static_cast<size_t>(h) * HD);
#pragma unroll 1
            for (int c0 = 0; c0 < HD; c0 += 32) {
                uint32_t v[32];
                if (last >= 0) {
                    tmem_ld_32x32(o_addr + c0, v);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = 0u;
                }
                if (ok && r < n_valid) {
#pragma unroll
                    for (int v8 = 0; v8 < 4; ++v8) {
                        float f[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            f[e] = (__uint_as_float(v[8 * v8 + e]) * a0 + (two ? xo[(c0 + 8 * v8 + e) * kQ + r] : 0.f) * a1) * inv;
                        dst[c0 / 8 + v8] = make_uint4(pack2(f[0], f[1]), pack2(f[2], f[3]), pack2(f[4], f[5]), pack2(f[6], f[7]));
                    }
                }
            }
        }
        if (!ok && lane == 0) atomicExch(status, WIDE_ERR_TIMEOUT);
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

template <int HD>
int launch_attn(wide_ctx* ctx, cudaStream_t s, const void* q, const void* k, const void* v, int Tq, int Tk, int Hq,
                int Hkv, int hpg, const int32_t* perm, const int32_t* counts, int causal, float scale, void* o) {
    CUtensorMap tmK, tmV;
    if (!wide_make_tmap_bf16(ctx, &tmK, k, Tk, static_cast<uint64_t>(Hkv) * HD, kKV) ||
        !wide_make_tmap_bf16(ctx, &tmV, v, Tk, static_cast<uint64_t>(Hkv) * HD, kKV))
        return WIDE_ERR_CUDA;
    constexpr int smem = attn_smem_bytes<HD>();
    WIDE_CUDA_CHECK(cudaFuncSetAttribute(attn_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    const int n_main = ((Tq + kQ - 1) / kQ) * Hq;
    WideLaunch l(ctx, s, "attn_prefill");
    attn_kernel<HD><<<n_main, kThreads, smem, s>>>(
        tmK, tmV, static_cast<const __nv_bfloat16*>(q), perm, counts, Tq, Tk, Hq, Hkv, hpg, causal,
        scale * 1.4426950408889634f, static_cast<__nv_bfloat16*>(o), ctx->d_status, ctx->wait_ns);
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}

}  // namespace

int wide_launch_attn_prefill_tc(wide_ctx* ctx, cudaStream_t s, const void* q, const void* k, const void* v, int Tq,
                                int Tk, int Hq, int Hkv, int head_dim, int hpg, const int32_t* perm,
                                const int32_t* counts, int causal, float scale, void* o) {
    if (head_dim == 128) return launch_attn<128>(ctx, s, q, k, v, Tq, Tk, Hq, Hkv, hpg, perm, counts, causal, scale, o);
    if (head_dim == 64) return launch_attn<64>(ctx, s, q, k, v, Tq, Tk, Hq, Hkv, hpg, perm, counts, causal, scale, o);
    return WIDE_ERR_UNSUPPORTED_SHAPE;
}
