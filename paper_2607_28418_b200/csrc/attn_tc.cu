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
//     PV = P V_t                  (UMMA; P goes through shared memory as a bf16 K-major operand,
//                                  V_t is used as loaded, as an MN-major operand; two TMEM buffers)
//     O  = O * alpha + PV         (softmax warps, O in registers)
// The UMMA warp issues S of tile t+1 before PV of tile t, so the tensor core works on the next
// scores while the softmax warps are busy.  Causal attention shortens the key range to the largest
// active query position of the tile (+ delta = T_k - T_q); only tiles that straddle a row's limit
// evaluate element-wise predicates.
//
// Outputs of inactive (token, group) pairs are zeroed by a few extra CTAs of the same grid.
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
constexpr int kThreads = 192;  // TMA warp, UMMA warp, 4 softmax warps

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
            int Tq, int Tk, int Hq, int Hkv, int hpg, int causal, float scale_log2e, int n_main,
            __nv_bfloat16* __restrict__ o, int* __restrict__ status, unsigned long long wait_ns) {
    constexpr int kKB = HD / kBK;          // 64-wide blocks along the head dimension
    constexpr int kQBytes = kKB * kBlk;
    constexpr int kKVBytes = kKB * kBlk;   // one K (or V) tile
    constexpr int kPBytes = (kKV / kBK) * kBlk;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int NG = Hq / hpg;
    const size_t ldq = static_cast<size_t>(Hq) * HD;

    if (static_cast<int>(blockIdx.x) >= n_main) {
        // ------------------------------------------------ zero the outputs of inactive pairs
        const int nz = gridDim.x - n_main, zi = blockIdx.x - n_main;
        const int ppr = hpg * HD / 8;  // 16-byte pieces per (row, group)
        for (int g = 0; g < NG; ++g) {
            const int c = counts[g];
            const long long total = static_cast<long long>(Tq - c) * ppr;
            for (long long i = static_cast<long long>(zi) * kThreads + tid; i < total; i += static_cast<long long>(nz) * kThreads) {
                const int j = c + static_cast<int>(i / ppr), piece = static_cast<int>(i % ppr);
                const int row = perm[static_cast<size_t>(g) * Tq + j];
                reinterpret_cast<uint4*>(o + row * ldq + static_cast<size_t>(g) * hpg * HD)[piece] = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        return;
    }

    // heavy (late, long key range) tiles first
    const int n_mt = (Tq + kQ - 1) / kQ;
    const int m = n_mt - 1 - static_cast<int>(blockIdx.x) / Hq;
    const int h = static_cast<int>(blockIdx.x) % Hq;
    const int g = h / hpg;
    const int hkv = h / (Hq / Hkv);
    const int c = counts[g];
    if (m * kQ >= c) return;   // block-level predicate: no active row in this tile
    const int n_valid = min(kQ, c - m * kQ);
    const int delta = Tk - Tq;
    const int32_t* rows = perm + static_cast<size_t>(g) * Tq + m * kQ;
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
            mbar_init(pv_free + 8 * i, 128);
        }
        mbar_init(q_ready, 128);
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

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (K, V)
        if (lane == 0) {
            bool ok = true;
            for (int t = 0; t < NT && ok; ++t) {
                const int s = t & 1;
                const uint32_t ph = (t >> 1) & 1;
                if (!mbar_wait(k_empty + 8 * s, ph ^ 1u, wait_ns, abort_flag)) { ok = false; break; }
                mbar_arrive_expect_tx(k_full + 8 * s, kKVBytes);
                for (int kb = 0; kb < kKB; ++kb)
                    tma_load_2d(smem_u32(k_s + s * kKVBytes + kb * kBlk), &tmK, hkv * HD + kb * kBK, t * kKV, k_full + 8 * s);
                if (!mbar_wait(v_empty + 8 * s, ph ^ 1u, wait_ns, abort_flag)) { ok = false; break; }
                mbar_arrive_expect_tx(v_full + 8 * s, kKVBytes);
                for (int kb = 0; kb < kKB; ++kb)
                    tma_load_2d(smem_u32(v_s + s * kKVBytes + kb * kBlk), &tmV, hkv * HD + kb * kBK, t * kKV, v_full + 8 * s);
            }
            if (!ok) {
                atomicExch(status, WIDE_ERR_TIMEOUT);
                for (int i = 0; i < 64; ++i) __nanosleep(1000);   // let copies in flight land
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ UMMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_qk = idesc_bf16(kQ, kKV, false);
            constexpr uint32_t idesc_pv = idesc_bf16(kQ, HD, true);
            bool ok = NT == 0 || mbar_wait(q_ready, 0, wait_ns, abort_flag);
            fence_proxy_async_smem();  // Q rows and P tiles are written through the generic proxy
            auto issue_qk = [&](int t) -> bool {
                const int s = t & 1;
                const uint32_t ph = (t >> 1) & 1;
                if (!mbar_wait(k_full + 8 * s, ph, wait_ns, abort_flag)) return false;
                if (!mbar_wait(s_free + 8 * s, ph ^ 1u, wait_ns, abort_flag)) return false;
                tc_fence_after_sync();
#pragma unroll
                for (int k16 = 0; k16 < HD / 16; ++k16) {
                    const uint64_t adesc = umma_desc_sw128(smem_u32(q_s + (k16 / 4) * kBlk)) + 2 * (k16 % 4);
                    const uint64_t bdesc = umma_desc_sw128(smem_u32(k_s + s * kKVBytes + (k16 / 4) * kBlk)) + 2 * (k16 % 4);
                    umma_bf16(tmem_base + s * kKV, adesc, bdesc, idesc_qk, k16 > 0 ? 1u : 0u);
                }
                umma_commit(k_empty + 8 * s);
                umma_commit(s_full + 8 * s);
                return true;
            };
            if (ok && NT > 0) ok = issue_qk(0);
            for (int t = 0; t < NT && ok; ++t) {
                if (t + 1 < NT && !issue_qk(t + 1)) { ok = false; break; }
                const int s = t & 1;
                const uint32_t ph = (t >> 1) & 1;
                if (!mbar_wait(v_full + 8 * s, ph, wait_ns, abort_flag)) { ok = false; break; }
                if (!mbar_wait(p_ready + 8 * s, ph, wait_ns, abort_flag)) { ok = false; break; }
                if (!mbar_wait(pv_free + 8 * s, ph ^ 1u, wait_ns, abort_flag)) { ok = false; break; }
                fence_proxy_async_smem();
                tc_fence_after_sync();
#pragma unroll
                for (int k16 = 0; k16 < kKV / 16; ++k16) {
                    const uint64_t adesc = umma_desc_sw128(smem_u32(p_s + s * kPBytes + (k16 / 4) * kBlk)) + 2 * (k16 % 4);
                    const uint64_t bdesc = umma_desc_sw128_mn(smem_u32(v_s + s * kKVBytes + k16 * 2048), kBlk);
                    umma_bf16(tmem_base + 256 + s * HD, adesc, bdesc, idesc_pv, k16 > 0 ? 1u : 0u);
                }
                umma_commit(v_empty + 8 * s);
                umma_commit(pv_full + 8 * s);
            }
            if (!ok) atomicExch(status, WIDE_ERR_TIMEOUT);
        }
    } else {
        // ------------------------------------------------------------------ softmax warps (2..5)
        const int st = tid - 64;                     // 0..127
        const int quarter = warp & 3;                // TMEM lane quarter this warp may read
        const int r = quarter * 32 + lane;           // row of the tile owned by this thread
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        bool ok = true;

        // Q prologue: 16-byte chunks, 8 consecutive threads copy one 128-byte row of a block
        if (NT > 0) {
            const int chunk = st & 7;
#pragma unroll
            for (int i = 0; i < kQ / 16; ++i) {
                const int row = (st >> 3) + 16 * i;
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
        float mrow = -CUDART_INF_F, lrow = 0.f, alpha_pending = 1.f;
        float acc[HD];
#pragma unroll
        for (int i = 0; i < HD; ++i) acc[i] = 0.f;

        auto accumulate = [&](int u, float alpha) -> bool {
            const int b = u & 1;
            const uint32_t ph = (u >> 1) & 1;
            if (!mbar_wait(pv_full + 8 * b, ph, wait_ns, abort_flag)) return false;
            tc_fence_after_sync();
#pragma unroll
            for (int c0 = 0; c0 < HD; c0 += 32) {
                uint32_t v[32];
                tmem_ld_32x32(lane_addr + 256 + b * HD + c0, v);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) acc[c0 + i] = fmaf(acc[c0 + i], alpha, __uint_as_float(v[i]));
            }
            tc_fence_before_sync();
            mbar_arrive(pv_free + 8 * b);
            return true;
        };

        for (int t = 0; t < NT; ++t) {
            const int b = t & 1;
            const uint32_t ph = (t >> 1) & 1;
            if (!mbar_wait(s_full + 8 * b, ph, wait_ns, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const int j0 = t * kKV;
            const bool edge = j0 + kKV - 1 > lim;     // this row needs element-wise predicates here
            // pass 1: row maximum
            float mx = -CUDART_INF_F;
#pragma unroll 1
            for (int c0 = 0; c0 < kKV; c0 += 32) {
                uint32_t v[32];
                tmem_ld_32x32(lane_addr + b * kKV + c0, v);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const float sv = __uint_as_float(v[i]) * scale_log2e;
                    mx = fmaxf(mx, (!edge || j0 + c0 + i <= lim) ? sv : -CUDART_INF_F);
                }
            }
            const float m_new = fmaxf(mrow, mx);
            const float m_use = m_new == -CUDART_INF_F ? 0.f : m_new;   // a row that has seen no key yet
            const float alpha = fast_exp2(mrow - m_use);
            // pass 2: P = exp2(S*c - m) as bf16 into the operand layout, row sum
            float rs = 0.f;
            uint8_t* prow = p_s + b * kPBytes + r * 128;
#pragma unroll 1
            for (int c0 = 0; c0 < kKV; c0 += 32) {
                uint32_t v[32];
                tmem_ld_32x32(lane_addr + b * kKV + c0, v);
                tmem_ld_wait();
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    float p0 = fast_exp2(fmaf(__uint_as_float(v[i]), scale_log2e, -m_use));
                    float p1 = fast_exp2(fmaf(__uint_as_float(v[i + 1]), scale_log2e, -m_use));
                    if (edge) {
                        if (j0 + c0 + i > lim) p0 = 0.f;
                        if (j0 + c0 + i + 1 > lim) p1 = 0.f;
                    }
                    rs += p0 + p1;
                    pk[i >> 1] = pack2(p0, p1);
                }
                uint8_t* blk = prow + (c0 / kBK) * kBlk;
                const int ch0 = (c0 % kBK) / 8;
#pragma unroll
                for (int v4 = 0; v4 < 4; ++v4)
                    *reinterpret_cast<uint4*>(blk + (((ch0 + v4) ^ (r & 7)) << 4)) =
                        make_uint4(pk[4 * v4], pk[4 * v4 + 1], pk[4 * v4 + 2], pk[4 * v4 + 3]);
            }
            lrow = fmaf(lrow, alpha, rs);
            mrow = m_new;
            tc_fence_before_sync();
            mbar_arrive(s_free + 8 * b);
            fence_proxy_async_smem();
            mbar_arrive(p_ready + 8 * b);
            // O of the previous tile while the tensor core works on this one
            if (t > 0 && !accumulate(t - 1, alpha_pending)) { ok = false; break; }
            alpha_pending = alpha;
        }
        if (ok && NT > 0) ok = accumulate(NT - 1, alpha_pending);
        if (NT > 0) cp_async_wait_all();

        // epilogue: normalise and scatter the active rows
        if (ok && r < n_valid) {
            const float inv = lrow > 0.f ? 1.f / lrow : 0.f;
            uint4* dst = reinterpret_cast<uint4*>(o + pos * ldq + static_cast<size_t>(h) * HD);
#pragma unroll
            for (int v8 = 0; v8 < HD / 8; ++v8)
                dst[v8] = make_uint4(pack2(acc[8 * v8] * inv, acc[8 * v8 + 1] * inv), pack2(acc[8 * v8 + 2] * inv, acc[8 * v8 + 3] * inv),
                                     pack2(acc[8 * v8 + 4] * inv, acc[8 * v8 + 5] * inv), pack2(acc[8 * v8 + 6] * inv, acc[8 * v8 + 7] * inv));
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
    const int n_zero = ctx->sm_count / 4 > 0 ? ctx->sm_count / 4 : 1;
    WideLaunch l(ctx, s, "attn_prefill");
    attn_kernel<HD><<<n_main + n_zero, kThreads, smem, s>>>(
        tmK, tmV, static_cast<const __nv_bfloat16*>(q), perm, counts, Tq, Tk, Hq, Hkv, hpg, causal,
        scale * 1.4426950408889634f, n_main, static_cast<__nv_bfloat16*>(o), ctx->d_status, ctx->wait_ns);
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
