// GEMM-K in its per-group form (Eq. 10, Algorithm 3): the K-axis product of wide_oproj and of the
// down projection of wide_ffn, driven by the reordered mask instead of by token tiles.
//
//   item (g, m, n)   rows   = sorted positions [128 m, 128 (m+1)) of group g's active prefix (perm)
//                    K      = the group's own channels [gG, (g+1)G) only
//                    output = columns [256 n, 256 (n+1))
//   partial[128, 256] = A[rows, gG:(g+1)G] * B[256 n : 256 (n+1), gG:(g+1)G]^T          (tcgen05, TMEM)
//   Y[perm[g][j], 256 n ...] += partial[j - 128 m, :]   for j < counts[g]                (scatter-reduce)
//
// Only active (tile, group) blocks are touched, so the FLOPs are the algorithmic ones (rows padded to
// 128); the price is the reduction of T*k*N partial sums into Y, which runs at the L2's reduction rate
// (measured on this part: 5.5-6.0 TB/s for red.global.add.v4 that covers whole 128-byte lines, half
// of that when every lane of a warp instruction hits a line of its own).  The epilogue therefore
// transposes each accumulator chunk through shared memory so that 8 lanes reduce one row's 128
// bytes, and the accumulator is double-buffered in TMEM so the reduction of item i overlaps the MMAs
// of item i+1.  The A rows are gathered through the permutation with cp.async straight into the
// 128-byte swizzle (as the gate/up kernel does); B comes by TMA.
//
// Reduction type: fp32 (red.global.add.v4.f32 into an fp32 Y) or bf16 (red.global.add.noftz.v4.bf16x2
// straight into a bf16 Y: half the reduction bytes; the partial sums of one output element, one per
// active group of its token, are then added in bf16).
//
// Which K-axis kernel runs is decided ON THE DEVICE, without a host read-back: every kernel of the
// pair evaluates wide_kaxis_group_chosen() on `counts` when it starts, and the one that is not chosen
// returns at once.
#include <cuda.h>

#include "internal.h"
#include "ptx.cuh"

namespace {

using namespace wptx;

// bf16 sums: 4 stages, 8 epilogue warps.  fp32 sums move twice the bytes per item through a chain of
// dependent steps (TMEM load, staging, reduction), which made the epilogue the longer leg of the TMEM
// double buffer (tensor pipe 24 % active); that variant trades a ring stage for four more epilogue warps.
template <bool kBf16Red> struct KCfg {
    static constexpr int kStages = kBf16Red ? 4 : 3;
    static constexpr int kEpiWarps = kBf16Red ? 8 : 12;
    static constexpr int kThreads = 32 * (6 + kEpiWarps);   // TMA, MMA, 4 gather warps, epilogue warps
    static constexpr int kStaging = kEpiWarps * 4096;       // 32 rows x 128 B per epilogue warp
};
constexpr int kBM = 128;
constexpr int kBK = 64;
constexpr int kBN = 256;
constexpr int kABytes = kBM * kBK * 2;          // 16 KB
constexpr int kBBytes = kBN * kBK * 2;          // 32 KB
constexpr int kStageBytes = kABytes + kBBytes;  // 48 KB
constexpr int kAccCols = 256;
template <bool kBf16Red> constexpr int smem_k() {
    return KCfg<kBf16Red>::kStages * kStageBytes + KCfg<kBf16Red>::kStaging + (2 * KCfg<kBf16Red>::kStages + 4) * 8 + 16 + 1024;
}

__device__ __forceinline__ void red_add_v4_f32(void* p, uint4 v) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(__uint_as_float(v.x)),
                 "f"(__uint_as_float(v.y)), "f"(__uint_as_float(v.z)), "f"(__uint_as_float(v.w))
                 : "memory");
}
__device__ __forceinline__ void red_add_v4_bf16x2(void* p, uint4 v) {
    asm volatile("red.global.add.noftz.v4.bf16x2 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Items of this launch: group g contributes nt_g * n_n of them (nt_g = row tiles of its active
// prefix), numbered group-major; inside a group the column block runs fastest, so the CTAs that work
// side by side share their A rows.
struct ItemMap {
    const int* off;   // [NG + 1] prefix of nt_g
    int NG, n_n;
    __device__ int total() const { return off[NG] * n_n; }
    __device__ void locate(int item, int& g, int& m, int& n) const {
        const int tile = item / n_n;
        n = item - tile * n_n;
        int lo = 0, hi = NG;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (off[mid] <= tile) lo = mid; else hi = mid;
        }
        g = lo;
        m = tile - off[lo];
    }
};

template <bool kBf16Red>
__global__ void __launch_bounds__(KCfg<kBf16Red>::kThreads, 1)
gemmk_group_kernel(const __grid_constant__ CUtensorMap tmB, const __nv_bfloat16* __restrict__ A, int lda,
                   const int32_t* __restrict__ perm, const int32_t* __restrict__ counts,
                   const int32_t* __restrict__ a_row_of_token, int NG, int T, int N, int G, void* __restrict__ Y,
                   int thr_q, int* __restrict__ status, unsigned long long wait_ns) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ int s_off[WIDE_MAX_GROUPS + 1];
    constexpr int kStagesK = KCfg<kBf16Red>::kStages;
    constexpr int kEpiWarps = KCfg<kBf16Red>::kEpiWarps;
    constexpr int kStagingBytes = KCfg<kBf16Red>::kStaging;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (!wide_kaxis_group_chosen(counts, NG, T, thr_q)) return;   // the owner-computes kernel runs instead

    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* staging = base + kStagesK * kStageBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(staging + kStagingBytes);
    const uint32_t full = smem_u32(bars), empty = smem_u32(bars + kStagesK);
    const uint32_t tfull = smem_u32(bars + 2 * kStagesK), tempty = smem_u32(bars + 2 * kStagesK + 2);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStagesK + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    if (tid == 0) {
        for (int s = 0; s < kStagesK; ++s) {
            mbar_init(full + 8 * s, 1 + 128);   // TMA producer + one arrival per gather thread
            mbar_init(empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull + 8 * b, 1);
            mbar_init(tempty + 8 * b, kEpiWarps);
        }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmB);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), 2 * kAccCols);
        tmem_relinquish();
    }
    if (warp == 2) {
        // prefix sums of the row tiles per group
        int run = 0;
        for (int b0 = 0; b0 < NG; b0 += 32) {
            const int g = b0 + lane;
            const int v = g < NG ? (counts[g] + kBM - 1) / kBM : 0;
            int p = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int u = __shfl_up_sync(0xffffffffu, p, o);
                if (lane >= o) p += u;
            }
            if (g < NG) s_off[g] = run + p - v;
            run += __shfl_sync(0xffffffffu, p, 31);
        }
        if (lane == 0) s_off[NG] = run;
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const ItemMap items{s_off, NG, (N + kBN - 1) / kBN};
    const int n_items = items.total();
    const int ksub = G / kBK;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (B tiles)
        if (lane == 0) {
            int it = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                int g, m, n;
                items.locate(item, g, m, n);
                for (int kk = 0; kk < ksub; ++kk, ++it) {
                    const int s = it % kStagesK;
                    const uint32_t ph = (it / kStagesK) & 1;
                    if (!mbar_wait(empty + 8 * s, ph ^ 1u, wait_ns, abort_flag)) { ok = false; break; }
                    mbar_arrive_expect_tx(full + 8 * s, kBBytes);
                    tma_load_2d(smem_u32(base + s * kStageBytes) + kABytes, &tmB, g * G + kk * kBK, n * kBN, full + 8 * s);
                }
            }
            if (!ok) {
                atomicExch(status, WIDE_ERR_TIMEOUT);
                for (int i = 0; i < 64; ++i) __nanosleep(1000);   // let copies in flight land
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ UMMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(kBM, kBN);
            int it = 0, tc = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++tc) {
                const int buf = tc & 1;
                if (!mbar_wait(tempty + 8 * buf, ((tc >> 1) & 1) ^ 1u, wait_ns, abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * kAccCols;
                for (int kk = 0; kk < ksub; ++kk, ++it) {
                    const int s = it % kStagesK;
                    const uint32_t ph = (it / kStagesK) & 1;
                    if (!mbar_wait(full + 8 * s, ph, wait_ns, abort_flag)) { ok = false; break; }
                    fence_proxy_async_smem();   // the A rows were written through the generic proxy (cp.async)
                    tc_fence_after_sync();
                    const uint32_t a_addr = smem_u32(base + s * kStageBytes);
                    const uint64_t adesc = umma_desc_sw128(a_addr);
                    const uint64_t bdesc = umma_desc_sw128(a_addr + kABytes);
#pragma unroll
                    for (int k4 = 0; k4 < kBK / 16; ++k4)
                        umma_bf16(d_tmem, adesc + 2 * k4, bdesc + 2 * k4, idesc, (kk > 0 || k4 > 0) ? 1u : 0u);
                    umma_commit(empty + 8 * s);
                }
                if (ok) umma_commit(tfull + 8 * buf);
            }
            if (!ok) atomicExch(status, WIDE_ERR_TIMEOUT);
        }
    } else if (warp < 6) {
        // ------------------------------------------------------------------ A gather (warps 2..5)
        // 8 consecutive lanes copy the 8 16-byte chunks of one row; instruction i of gather warp w
        // copies tile rows 16 i + 4 w + lane / 8.  Rows past the group's count are real tokens of the
        // permutation's inactive tail (their results are dropped), so nothing is clamped but T.
        // An item has only G / 64 k-steps, so the row addresses of the NEXT item are fetched while the
        // current one is copied: the dependent loads (permutation, row map) would otherwise stall the
        // gather for a memory round trip at every item boundary, which the 4-stage ring cannot hide.
        const int chunk = lane & 7;
        const int row0 = (warp - 2) * 4 + (lane >> 3);
        auto row_sources = [&](int item, const uint8_t* (&src)[8]) {
            int g, m, n;
            items.locate(item, g, m, n);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                int j = m * kBM + row0 + 16 * i;
                if (j >= T) j = T - 1;
                int tok = perm[static_cast<size_t>(g) * T + j];
                if (a_row_of_token) tok = a_row_of_token[tok];
                src[i] = reinterpret_cast<const uint8_t*>(A + static_cast<size_t>(tok) * lda + g * G) + 16 * chunk;
            }
        };
        int it = 0;
        bool ok = true;
        const uint8_t* src[8];
        const uint8_t* nxt[8];
        if (static_cast<int>(blockIdx.x) < n_items) row_sources(blockIdx.x, src);
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
            const int next_item = item + gridDim.x;
            if (next_item < n_items) row_sources(next_item, nxt);
            for (int kk = 0; kk < ksub; ++kk, ++it) {
                const int s = it % kStagesK;
                const uint32_t ph = (it / kStagesK) & 1;
                if (!mbar_wait_warp(empty + 8 * s, ph ^ 1u, wait_ns, abort_flag)) { ok = false; break; }
                const uint32_t a_dst = smem_u32(base + s * kStageBytes);
                const size_t koff = static_cast<size_t>(kk) * (kBK * 2);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = row0 + 16 * i;
                    cp_async_16(a_dst + static_cast<uint32_t>(r) * 128u +
                                    ((static_cast<uint32_t>(chunk) ^ static_cast<uint32_t>(r & 7)) << 4),
                                src[i] + koff);
                }
                cp_async_mbar_arrive_noinc(full + 8 * s);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) src[i] = nxt[i];
        }
        cp_async_wait_all();
        if (!ok && lane == 0) atomicExch(status, WIDE_ERR_TIMEOUT);
    } else {
        // ------------------------------------------------------------------ epilogue (warps 6 ..)
        // Warps w, w + 4 (, w + 8) share a TMEM lane quarter and split the accumulator's columns.
        // Thread = accumulator row (TMEM lane).  A chunk is 128 bytes of an output row (32 fp32 or
        // 64 bf16 columns): the thread writes its row's chunk into the warp's staging tile (16-byte
        // pieces, piece v of row r in slot v ^ (r & 7)), then the warp reads it back 4 rows x 8
        // pieces at a time and reduces whole 128-byte lines into Y.
        const int q = warp & 3;
        const int part = (warp - 6) >> 2;
        // column range of this warp: halves of 128, or thirds of 96 / 96 / 64
        const int col_lo = kEpiWarps == 8 ? part * 128 : part * 96;
        const int col_hi = kEpiWarps == 8 ? col_lo + 128 : (part == 2 ? kBN : col_lo + 96);
        uint4* stage = reinterpret_cast<uint4*>(staging + (warp - 6) * 4096);
        constexpr int kEsz = kBf16Red ? 2 : 4;
        constexpr int kChunkCols = 128 / kEsz;
        int tc = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++tc) {
            int g, m, n;
            items.locate(item, g, m, n);
            const int j = m * kBM + q * 32 + lane;
            const int tok = j < counts[g] ? perm[static_cast<size_t>(g) * T + j] : -1;
            const int buf = tc & 1;
            if (!mbar_wait_warp(tfull + 8 * buf, (tc >> 1) & 1, wait_ns, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + buf * kAccCols;
#pragma unroll 1
            for (int c0 = col_lo; c0 < col_hi; c0 += kChunkCols) {
                uint32_t r[32];
                tmem_ld_32x32(taddr + c0, r);
                if constexpr (kBf16Red) {
                    uint32_t r2[32];
                    tmem_ld_32x32(taddr + c0 + 32, r2);
                    tmem_ld_wait();
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        stage[lane * 8 + (v ^ (lane & 7))] =
                            make_uint4(pack_bf16(__uint_as_float(r[8 * v]), __uint_as_float(r[8 * v + 1])),
                                       pack_bf16(__uint_as_float(r[8 * v + 2]), __uint_as_float(r[8 * v + 3])),
                                       pack_bf16(__uint_as_float(r[8 * v + 4]), __uint_as_float(r[8 * v + 5])),
                                       pack_bf16(__uint_as_float(r[8 * v + 6]), __uint_as_float(r[8 * v + 7])));
                        stage[lane * 8 + ((v + 4) ^ (lane & 7))] =
                            make_uint4(pack_bf16(__uint_as_float(r2[8 * v]), __uint_as_float(r2[8 * v + 1])),
                                       pack_bf16(__uint_as_float(r2[8 * v + 2]), __uint_as_float(r2[8 * v + 3])),
                                       pack_bf16(__uint_as_float(r2[8 * v + 4]), __uint_as_float(r2[8 * v + 5])),
                                       pack_bf16(__uint_as_float(r2[8 * v + 6]), __uint_as_float(r2[8 * v + 7])));
                    }
                } else {
                    tmem_ld_wait();
#pragma unroll
                    for (int v = 0; v < 8; ++v)
                        stage[lane * 8 + (v ^ (lane & 7))] = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                }
                if (c0 + kChunkCols >= col_hi) {
                    // the accumulator has been read out: hand it back before the last reductions
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tempty + 8 * buf);
                } else {
                    __syncwarp();
                }
                const int col = n * kBN + c0;          // first column of the chunk
                const int piece = lane & 7;
                const bool col_ok = col + (piece + 1) * (16 / kEsz) <= N;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int rr = 4 * i + (lane >> 3);
                    const int tr = __shfl_sync(0xffffffffu, tok, rr);
                    const uint4 val = stage[rr * 8 + (piece ^ (rr & 7))];
                    if (tr >= 0 && col_ok) {
                        uint8_t* dst = static_cast<uint8_t*>(Y) + (static_cast<size_t>(tr) * N + col) * kEsz + piece * 16;
                        if constexpr (kBf16Red) red_add_v4_bf16x2(dst, val);
                        else red_add_v4_f32(dst, val);
                    }
                }
                __syncwarp();
            }
        }
        if (!ok && lane == 0) atomicExch(status, WIDE_ERR_TIMEOUT);
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 2 * kAccCols);
    }
}

// Before the K-axis kernels: when the per-group kernel is chosen, clear the reduction target;
// otherwise (and when `a` is given) write the masked copy of the input the owner-computes kernel
// reads:  out[rank(t), c] = M[t, c/G] ? a[t, c] : 0.
__global__ void __launch_bounds__(256)
kaxis_prep_kernel(const int32_t* __restrict__ counts, int NG, int T, int thr_q, uint4* __restrict__ zero_ptr,
                  long long zero_vecs, const uint4* __restrict__ a, const uint32_t* __restrict__ mask_bits,
                  const int32_t* __restrict__ token_rank, int words, int K, int G, uint4* __restrict__ out) {
    const long long tid = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
    const long long nthreads = static_cast<long long>(gridDim.x) * blockDim.x;
    if (counts != nullptr && wide_kaxis_group_chosen(counts, NG, T, thr_q)) {
        for (long long i = tid; i < zero_vecs; i += nthreads) zero_ptr[i] = make_uint4(0u, 0u, 0u, 0u);
        return;
    }
    if (a == nullptr) return;
    const int vec_per_row = K / 8, vec_per_group = G / 8;
    const long long total = static_cast<long long>(T) * vec_per_row;
    for (long long i = tid; i < total; i += nthreads) {
        const int t = static_cast<int>(i / vec_per_row);
        const int g = static_cast<int>(i % vec_per_row) / vec_per_group;
        const long long o = token_rank ? static_cast<long long>(token_rank[t]) * vec_per_row + (i % vec_per_row) : i;
        out[o] = wide_mask_bit(mask_bits, words, t, g) ? a[i] : make_uint4(0u, 0u, 0u, 0u);
    }
}

// fp32 sums -> bf16 output, only when the per-group kernel ran.
__global__ void __launch_bounds__(256)
kaxis_convert_kernel(const int32_t* __restrict__ counts, int NG, int T, int thr_q, const float4* __restrict__ acc,
                     uint2* __restrict__ y, long long n_vec) {
    if (!wide_kaxis_group_chosen(counts, NG, T, thr_q)) return;
    const long long nthreads = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < n_vec; i += nthreads) {
        const float4 v = acc[i];
        y[i] = make_uint2(pack_bf16(v.x, v.y), pack_bf16(v.z, v.w));
    }
}

}  // namespace

int wide_launch_kaxis_prep(wide_ctx* ctx, cudaStream_t s, const int32_t* counts, int NG, int T, int thr_q, void* zero_ptr,
                           size_t zero_bytes, const void* a, const uint32_t* mask_bits, const int32_t* token_rank, int K,
                           int G, void* a_masked) {
    const long long work_a = a ? static_cast<long long>(T) * (K / 8) : 0;
    const long long work = work_a > static_cast<long long>(zero_bytes / 16) ? work_a : static_cast<long long>(zero_bytes / 16);
    if (work == 0) return WIDE_OK;
    long long blocks = (work + 255) / 256;
    if (blocks > ctx->sm_count * 8) blocks = ctx->sm_count * 8;
    const int words = (K / (G > 0 ? G : 1) + 31) / 32;
    WideLaunch l(ctx, s, counts ? "kaxis_prep" : "prefill_mask_rows");
    kaxis_prep_kernel<<<static_cast<int>(blocks), 256, 0, s>>>(counts, NG, T, thr_q, static_cast<uint4*>(zero_ptr),
                                                               static_cast<long long>(zero_bytes / 16),
                                                               static_cast<const uint4*>(a), mask_bits, token_rank, words, K, G,
                                                               static_cast<uint4*>(a_masked));
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}

int wide_launch_gemmk_group_tc(wide_ctx* ctx, cudaStream_t s, const void* A, int lda, const void* B, int T, int N, int K,
                               int G, const int32_t* perm, const int32_t* counts, const int32_t* a_row_of_token, void* Y,
                               bool bf16_red, int thr_q, const char* name) {
    if (T == 0) return WIDE_OK;
    CUtensorMap tmB;
    if (!wide_make_tmap_bf16(ctx, &tmB, B, N, K, kBN)) return WIDE_ERR_CUDA;
    const int NG = K / G;
    WideLaunch l(ctx, s, name);
    if (bf16_red) {
        WIDE_CUDA_CHECK(cudaFuncSetAttribute(gemmk_group_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_k<true>()));
        gemmk_group_kernel<true><<<ctx->sm_count, KCfg<true>::kThreads, smem_k<true>(), s>>>(
            tmB, static_cast<const __nv_bfloat16*>(A), lda, perm, counts, a_row_of_token, NG, T, N, G, Y, thr_q,
            ctx->d_status, ctx->wait_ns);
    } else {
        WIDE_CUDA_CHECK(cudaFuncSetAttribute(gemmk_group_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_k<false>()));
        gemmk_group_kernel<false><<<ctx->sm_count, KCfg<false>::kThreads, smem_k<false>(), s>>>(
            tmB, static_cast<const __nv_bfloat16*>(A), lda, perm, counts, a_row_of_token, NG, T, N, G, Y, thr_q,
            ctx->d_status, ctx->wait_ns);
    }
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}

int wide_launch_kaxis_convert(wide_ctx* ctx, cudaStream_t s, const int32_t* counts, int NG, int T, int thr_q,
                              const float* acc, void* y_bf16, size_t n_elems) {
    const long long n_vec = static_cast<long long>(n_elems / 4);
    if (n_vec == 0) return WIDE_OK;
    long long blocks = (n_vec + 255) / 256;
    if (blocks > ctx->sm_count * 8) blocks = ctx->sm_count * 8;
    WideLaunch l(ctx, s, "kaxis_convert");
    kaxis_convert_kernel<<<static_cast<int>(blocks), 256, 0, s>>>(counts, NG, T, thr_q, reinterpret_cast<const float4*>(acc),
                                                                  static_cast<uint2*>(y_bf16), n_vec);
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}
