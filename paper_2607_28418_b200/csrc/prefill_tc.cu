// Prefill path of wide_ffn / wide_oproj / wide_qproj (and the score GEMM of wide_route) on the
// 5th-generation tensor cores (tcgen05 + TMEM), operands staged by TMA (weights, hidden
// activation) or gathered with cp.async (token rows selected through the reorder permutation).
//
//   gateup_kernel   Algorithm 2 (GEMM-MN, N-axis): a work item is one or two consecutive 128-row
//                   tiles of a group's sorted active rows times one block of the group's channels.
//                   A = gathered rows of X, B = the group's rows of W_gate and W_up side by side
//                   (one UMMA of N = 2*BN), fp32 accumulators in TMEM, epilogue silu(gate)*up ->
//                   bf16, scattered through the permutation straight into the token-major hidden
//                   activation H (rows past the group's count are dropped); the same warps zero
//                   the group's inactive rows of H.  With kLinear the same kernel is the routed
//                   linear layer of wide_qproj (one weight, plain store).
//   down_kernel     Eq. 10 (K-axis) in owner-computes form: a CTA owns a 128-token x BN output tile
//                   and walks the K-groups, skipping every group that no token of the tile selected
//                   (block-level predicate on the mask of the tile's tokens); inactive (token,
//                   group) pairs inside an active block are exact zeros of H.  No atomics,
//                   deterministic, output written once.  Also the K-split score GEMM of the router.
//   down256_kernel  the same product with 256-token tiles and column tiles of even widths.
//
// All are persistent (at most one CTA per SM) and warp-specialised: TMA producer, UMMA issuer,
// (gather warps,) epilogue warps over a shared-memory ring; down_kernel double-buffers its TMEM
// accumulator, the 256-row items of the other two fill TMEM.  Every mbarrier wait is bounded.
#include <cuda.h>

#include "internal.h"
#include "ptx.cuh"

namespace {

using namespace wptx;

constexpr int kStages = 4;
constexpr int kBM = 128;              // rows per tile (UMMA M)
constexpr int kBK = 64;               // bf16 elements per k-step = one 128-byte swizzle row
constexpr int kABytes = kBM * kBK * 2;  // 16 KB
constexpr int kAccCols = 256;         // TMEM columns per accumulator buffer
constexpr int kMaskWords = WIDE_MAX_GROUPS / 32;

struct SmemLayout {
    uint8_t* stage_base;
    uint32_t full, empty, tfull, tempty;  // shared-space addresses of barrier arrays
    uint32_t* tmem_slot;
    volatile int* abort_flag;
};

template <int kBBytes>
__device__ __forceinline__ SmemLayout carve_smem(uint8_t* raw) {
    SmemLayout L;
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~static_cast<uintptr_t>(1023));
    L.stage_base = base;
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + kStages * (kABytes + kBBytes));
    L.full = smem_u32(bars);
    L.empty = smem_u32(bars + kStages);
    L.tfull = smem_u32(bars + 2 * kStages);
    L.tempty = smem_u32(bars + 2 * kStages + 2);
    L.tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 4);
    L.abort_flag = reinterpret_cast<volatile int*>(L.tmem_slot + 1);
    return L;
}

template <int kBBytes>
constexpr int smem_bytes() {
    return kStages * (kABytes + kBBytes) + (2 * kStages + 4) * 8 + 16 + 1024;
}

// OR of the mask words of tokens [t0, t0 + 128) computed by one warp; every lane gets the result.
// `order` (may be null = identity) maps a row position to its token.
__device__ __forceinline__ void tile_mask_or(const uint32_t* __restrict__ mask_bits, const int32_t* __restrict__ order,
                                             int words, int T, int t0, int lane, uint32_t (&act)[kMaskWords]) {
#pragma unroll
    for (int w = 0; w < kMaskWords; ++w) act[w] = 0u;
    if (mask_bits == nullptr) {
#pragma unroll
        for (int w = 0; w < kMaskWords; ++w) act[w] = 0xffffffffu;
        return;
    }
    for (int i = lane; i < kBM; i += 32) {
        const int p = t0 + i;
        if (p < T) {
            const int t = order ? order[p] : p;
#pragma unroll
            for (int w = 0; w < kMaskWords; ++w)
                if (w < words) act[w] |= mask_bits[static_cast<size_t>(t) * words + w];
        }
    }
#pragma unroll
    for (int w = 0; w < kMaskWords; ++w) act[w] = __reduce_or_sync(0xffffffffu, act[w]);
}

__device__ __forceinline__ void report_timeout(int* status) { atomicExch(status, WIDE_ERR_TIMEOUT); }

// Give copies that are still in flight time to land before the CTA gives up its shared memory.
__device__ __forceinline__ void abort_grace() {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Output of the down / output projection when the groups are sharded over GPUs (tensor parallelism
// over the pruned dimension): this rank's tile is a PART of y (Eq. 10 summed over this rank's groups
// only), and the sum over ranks is a reduce-scatter over token rows.  Fused here: instead of storing
// its part and handing it to a collective, the epilogue adds every row straight into the fp32 shard
// of the rank that owns the row, with red.global.add over peer memory (plain peer accesses through
// NVLink issued by the epilogue threads; no bulk or tensor copy touches another GPU's memory).  base[r] = rank r's shard [rows_per_rank, N] fp32, zero before any
// rank starts and complete once every rank's kernel has finished (the caller's two barriers).
// world == 0: ordinary output.
struct PeerOut {
    float* base[8];
    int world;
    int rows_per_rank;
};

__device__ __forceinline__ void red_add_f32x4(float* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(__uint_as_float(a)), "f"(__uint_as_float(b)),
                 "f"(__uint_as_float(c)), "f"(__uint_as_float(d))
                 : "memory");
}

// ======================================================================================= down
// Y[T, N] = A[T, K] * B[N, K]^T with K split into groups of G; group g is skipped for a token tile
// when no token of the tile has bit g set (mask_bits == nullptr: nothing is skipped).
template <int BN>
__global__ void __launch_bounds__(192, 1)
down_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const uint32_t* __restrict__ mask_bits, const int32_t* __restrict__ order, int words, int T, int N, int K,
            int G, void* __restrict__ Y,
            int out_bf16, int ksplit, const __nv_bfloat16* __restrict__ aux_w, int aux_rows,
            float* __restrict__ aux_norm, const int32_t* __restrict__ sel_counts, int sel_thr, int acc_split,
            const PeerOut peer, int* __restrict__ status, unsigned long long wait_ns) {
    constexpr int kBBytes = BN * kBK * 2;
    constexpr int kStageBytes = kABytes + kBBytes;
    extern __shared__ uint8_t smem_raw[];
    grid_dep_launch();   // as the score GEMM of the router: the selection kernel behind it may be scheduled as CTAs leave
    if (wide_kaxis_group_chosen(sel_counts, K / G, T, sel_thr)) return;   // the per-group kernel runs instead
    SmemLayout L = carve_smem<kBBytes>(smem_raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(L.full + 8 * s, 1);
            mbar_init(L.empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(L.tfull + 8 * b, 1);
            mbar_init(L.tempty + 8 * b, 4);
        }
        *L.abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(L.tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *L.tmem_slot;

    // ksplit > 1: the K-groups (exactly ksplit of them) are spread over separate CTAs and each
    // writes its partial product into its own [T, N] slab of Y; nothing is masked in that mode.
    const int n_m = (T + kBM - 1) / kBM, n_n = (N + BN - 1) / BN;
    const int n_mn = n_m * n_n;
    const int n_tiles = n_mn * ksplit;
    const int NG = K / G, ksub = G / kBK;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        int it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
            const int mn = tile % n_mn, only = ksplit > 1 ? tile / n_mn : -1;
            const int m = mn % n_m, n = mn / n_m;
            uint32_t act[kMaskWords];
            tile_mask_or(mask_bits, order, words, T, m * kBM, lane, act);
            if (lane == 0) {
                for (int g = 0; g < NG && ok; ++g) {
                    if (!((act[g >> 5] >> (g & 31)) & 1u) || (only >= 0 && g != only)) continue;
                    for (int kk = 0; kk < ksub; ++kk, ++it) {
                        const int s = it % kStages;
                        const uint32_t ph = (it / kStages) & 1;
                        if (!mbar_wait(L.empty + 8 * s, ph ^ 1u, wait_ns, L.abort_flag)) { ok = false; break; }
                        mbar_arrive_expect_tx(L.full + 8 * s, kStageBytes);
                        const uint32_t a_dst = smem_u32(L.stage_base + s * kStageBytes);
                        const int kcol = g * G + kk * kBK;
                        tma_load_2d(a_dst, &tmA, kcol, m * kBM, L.full + 8 * s);
                        tma_load_2d(a_dst + kABytes, &tmB, kcol, n * BN, L.full + 8 * s);
                    }
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        }
        if (!ok && lane == 0) { report_timeout(status); abort_grace(); }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ UMMA issuer
        constexpr uint32_t idesc = umma_idesc_bf16(kBM, BN);
        int it = 0, tc = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++tc) {
            const int mn = tile % n_mn, only = ksplit > 1 ? tile / n_mn : -1;
            const int m = mn % n_m;
            uint32_t act[kMaskWords];
            tile_mask_or(mask_bits, order, words, T, m * kBM, lane, act);
            if (lane == 0) {
                const int buf = tc & 1;
                const uint32_t tph = (tc >> 1) & 1;
                if (!mbar_wait(L.tempty + 8 * buf, tph ^ 1u, wait_ns, L.abort_flag)) ok = false;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * kAccCols;
                uint32_t accumulate = 0;
                int steps_done = 0;
                for (int g = 0; g < NG && ok; ++g) {
                    if (!((act[g >> 5] >> (g & 31)) & 1u) || (only >= 0 && g != only)) continue;
                    for (int kk = 0; kk < ksub; ++kk, ++it, ++steps_done) {
                        const int s = it % kStages;
                        const uint32_t ph = (it / kStages) & 1;
                        if (!mbar_wait(L.full + 8 * s, ph, wait_ns, L.abort_flag)) { ok = false; break; }
                        tc_fence_after_sync();
                        const uint32_t a_addr = smem_u32(L.stage_base + s * kStageBytes);
                        const uint64_t adesc = umma_desc_sw128(a_addr);
                        const uint64_t bdesc = umma_desc_sw128(a_addr + kABytes);
                        if (acc_split > 1) {
                            // score mode: the k-steps go round-robin to acc_split accumulators (one tile
                            // per CTA, so they may take the whole tensor memory), which shortens every
                            // fp32 accumulation chain by that factor; the epilogue adds them up
                            const uint32_t d_acc = tmem_base + (steps_done % acc_split) * BN;
#pragma unroll
                            for (int k4 = 0; k4 < kBK / 16; ++k4)
                                umma_bf16(d_acc, adesc + 2 * k4, bdesc + 2 * k4, idesc, (steps_done >= acc_split || k4 > 0) ? 1u : 0u);
                            accumulate = 1;
                            umma_commit(L.empty + 8 * s);
                            continue;
                        }
#pragma unroll
                        for (int k4 = 0; k4 < kBK / 16; ++k4) {
                            umma_bf16(d_tmem, adesc + 2 * k4, bdesc + 2 * k4, idesc, accumulate);
                            accumulate = 1;
                        }
                        umma_commit(L.empty + 8 * s);
                    }
                }
                if (ok) {
                    if (accumulate) umma_commit(L.tfull + 8 * buf);
                    else mbar_arrive(L.tfull + 8 * buf);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        }
        if (!ok && lane == 0) report_timeout(status);
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int q = warp & 3;  // TMEM lane quarter this warp may read
        int tc = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++tc) {
            const int mn = tile % n_mn, slab = ksplit > 1 ? tile / n_mn : 0;
            const int m = mn % n_m, n = mn / n_m;
            uint32_t act[kMaskWords];
            tile_mask_or(mask_bits, order, words, T, m * kBM, lane, act);
            bool any = false;
            for (int g = 0; g < NG; ++g) any = any || ((act[g >> 5] >> (g & 31)) & 1u);
            const int buf = tc & 1;
            const uint32_t tph = (tc >> 1) & 1;
            if (!mbar_wait_warp(L.tfull + 8 * buf, tph, wait_ns, L.abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const int pos = m * kBM + q * 32 + lane;              // row position of the tile
            const int row = (order && pos < T) ? order[pos] : pos;  // token that owns this output row
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + buf * kAccCols;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t r[32];
                if (any) {
                    tmem_ld_32x32(taddr + c0, r);
                    tmem_ld_wait();
                    for (int a = 1; a < acc_split; ++a) {
                        uint32_t r2[32];
                        tmem_ld_32x32(taddr + a * BN + c0, r2);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) + __uint_as_float(r2[i]));
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = 0u;
                }
                const int col = n * BN + c0;
                if (peer.world > 0) {
                    // this rank's part of the row, added into the shard of the rank that owns the row
                    if (any && row < T && col + 32 <= N) {
                        float* dst = peer.base[row / peer.rows_per_rank] +
                                     static_cast<size_t>(row % peer.rows_per_rank) * N + col;
#pragma unroll
                        for (int v = 0; v < 8; ++v) red_add_f32x4(dst + 4 * v, r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                    }
                } else if (row < T && col + 32 <= N) {
                    if (out_bf16) {
                        uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(Y) + static_cast<size_t>(row) * N + col);
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            uint4 o;
                            o.x = pack_bf16(__uint_as_float(r[8 * v + 0]), __uint_as_float(r[8 * v + 1]));
                            o.y = pack_bf16(__uint_as_float(r[8 * v + 2]), __uint_as_float(r[8 * v + 3]));
                            o.z = pack_bf16(__uint_as_float(r[8 * v + 4]), __uint_as_float(r[8 * v + 5]));
                            o.w = pack_bf16(__uint_as_float(r[8 * v + 6]), __uint_as_float(r[8 * v + 7]));
                            dst[v] = o;
                        }
                    } else {
                        uint4* dst = reinterpret_cast<uint4*>(static_cast<float*>(Y) + static_cast<size_t>(slab) * T * N +
                                                              static_cast<size_t>(row) * N + col);
#pragma unroll
                        for (int v = 0; v < 8; ++v) dst[v] = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(L.tempty + 8 * buf);
        }
        if (!ok && lane == 0) report_timeout(status);
    }

    // Spare CTAs (blockIdx.x >= n_tiles) carry a side job: the Euclidean norm of every row of
    // aux_w, slightly rounded up, one warp per row (the router's error bound needs it).
    if (aux_norm != nullptr && static_cast<int>(blockIdx.x) >= n_tiles) {
        const int first = (static_cast<int>(blockIdx.x) - n_tiles) * 6;
        const int r = first + warp;
        if (r < aux_rows) {
            const uint4* rowp = reinterpret_cast<const uint4*>(aux_w + static_cast<size_t>(r) * K);
            float acc = 0.f;
            for (int i = lane; i < K / 8; i += 32) {
                const uint4 v = rowp[i];
                const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 f = __bfloat1622float2(h[e]);
                    acc = fmaf(f.x, f.x, fmaf(f.y, f.y, acc));
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            if (lane == 0) aux_norm[r] = sqrtf(acc) * 1.0001f;
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

// ======================================================================================= down, 256-row tiles
// Same product as down_kernel, but a CTA owns a 256-token x 256-output tile: two M=128 UMMAs per
// 16-wide k-slice share one B tile in shared memory, so a k-step moves 64 KB for twice the FLOPs
// (1.5x fewer bytes per FLOP than the 128 x 256 tile) and the 3-stage ring covers 1.5x more
// latency.  The two accumulators fill all 512 TMEM columns, so the epilogue of a tile does not
// overlap the next tile's MMAs (a few percent); with one or two tiles per CTA that is cheap.
// The N extent is cut into n_n column tiles whose widths are multiples of 16 and differ by at
// most 16 (the host picks n_n so that the tiles fill the SMs evenly: 18 tiles of 224/240 columns
// instead of 16 of 256 put 144 CTAs to work at T=2048, N=4096 where 128 would leave 20 SMs idle).
constexpr int kStages2 = 3;
constexpr int kA2Bytes = 2 * kABytes;            // 256 rows x 128 B
constexpr int kB2Bytes = 256 * kBK * 2;          // 256 rows x 128 B
constexpr int kStage2Bytes = kA2Bytes + kB2Bytes;
constexpr int kSmem2 = kStages2 * kStage2Bytes + (2 * kStages2 + 2) * 8 + 16 + 1024;

__global__ void __launch_bounds__(192, 1)
down256_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const uint32_t* __restrict__ mask_bits, const int32_t* __restrict__ order, int words, int T, int N,
               int K, int G, void* __restrict__ Y,
               int out_bf16, int n_n, int box_n, unsigned* __restrict__ queue, const int32_t* __restrict__ sel_counts,
               int sel_thr, const PeerOut peer, int* __restrict__ status, unsigned long long wait_ns) {
    extern __shared__ uint8_t smem_raw[];
    if (wide_kaxis_group_chosen(sel_counts, K / G, T, sel_thr)) return;   // the per-group kernel runs instead
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + kStages2 * kStage2Bytes);
    const uint32_t full = smem_u32(bars), empty = smem_u32(bars + kStages2);
    const uint32_t tfull = smem_u32(bars + 2 * kStages2), tempty = smem_u32(bars + 2 * kStages2 + 1);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages2 + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    // Tiles are handed out by a global counter (tiles of a clustered mask differ in how many
    // groups they skip, so a fixed assignment leaves SMs idle).  The producer warp fetches the next
    // tile index and passes it to the UMMA warp and the four epilogue warps through a two-slot
    // ring in shared memory: sq_full[slot] <- producer, sq_empty[slot] <- the five readers.
    __shared__ int sq_tile[2];
    __shared__ uint64_t sq_bars[4];
    const uint32_t sq_full = smem_u32(sq_bars), sq_empty = smem_u32(sq_bars + 2);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < kStages2; ++s) {
            mbar_init(full + 8 * s, 1);
            mbar_init(empty + 8 * s, 1);
        }
        mbar_init(tfull, 1);
        mbar_init(tempty, 4);
        for (int i = 0; i < 2; ++i) {
            mbar_init(sq_full + 8 * i, 1);
            mbar_init(sq_empty + 8 * i, 5);
        }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // When this kernel is launched as a programmatic dependent of the gate / up kernel (launch_down_auto), it may
    // run up to here, and on through its tile masks (mask and token order are older than the gate / up kernel, which
    // is launched the ordinary way), while that kernel's last CTAs finish; grid_dep_wait() stands before the first load
    // of H and before the first store to Y.

    const int n_m = (T + 255) / 256;
    const int n_tiles = n_m * n_n;
    const int NG = K / G, ksub = G / kBK;
    // column tile n covers [col0(n), col0(n) + width(n)): sixteenths of N dealt as evenly as possible
    const int q16 = (N + 15) / 16, q_base = q16 / n_n, q_rem = q16 % n_n;
    auto col0 = [&](int n) { return 16 * (n * q_base + min(n, q_rem)); };
    auto width = [&](int n) { return 16 * (q_base + (n < q_rem ? 1 : 0)); };
    const uint32_t stage_tx = kA2Bytes + static_cast<uint32_t>(box_n) * (kBK * 2);   // TMA always moves whole boxes
    // a reader warp takes the tc-th tile of this CTA from the ring (-1: no more tiles, -2: gave up)
    auto next_tile = [&](int tc) -> int {
        const int slot = tc & 1;
        int tile = -2;
        if (lane == 0) {
            if (mbar_wait(sq_full + 8 * slot, (tc >> 1) & 1, wait_ns, abort_flag)) {
                tile = sq_tile[slot];
                mbar_arrive(sq_empty + 8 * slot);
            }
        }
        return __shfl_sync(0xffffffffu, tile, 0);
    };

    // OR of the mask words of the tile's 256 tokens
    auto tile_mask = [&](int m, uint32_t (&act)[kMaskWords]) {
        uint32_t hi[kMaskWords];
        tile_mask_or(mask_bits, order, words, T, m * 256, lane, act);
        tile_mask_or(mask_bits, order, words, T, m * 256 + 128, lane, hi);
#pragma unroll
        for (int w = 0; w < kMaskWords; ++w) act[w] |= hi[w];
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        int it = 0;
        bool ok = true;
        for (int tc = 0; ok; ++tc) {
            // fetch the next tile and publish it (the first one is this CTA's own index)
            int tile = -1;
            if (lane == 0) {
                const int slot = tc & 1;
                if (!mbar_wait(sq_empty + 8 * slot, ((tc >> 1) & 1) ^ 1u, wait_ns, abort_flag)) {
                    ok = false;
                } else {
                    const unsigned got = tc == 0 ? blockIdx.x : gridDim.x + atomicAdd(queue, 1u);
                    tile = got < static_cast<unsigned>(n_tiles) ? static_cast<int>(got) : -1;
                    sq_tile[slot] = tile;
                    mbar_arrive(sq_full + 8 * slot);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            tile = __shfl_sync(0xffffffffu, tile, 0);
            if (!ok || tile < 0) break;
            const int m = tile % n_m, n = tile / n_m;
            uint32_t act[kMaskWords];
            tile_mask(m, act);
            if (lane == 0) {
                if (tc == 0) grid_dep_wait();     // H comes from the kernel before
                for (int g = 0; g < NG && ok; ++g) {
                    if (!((act[g >> 5] >> (g & 31)) & 1u)) continue;
                    for (int kk = 0; kk < ksub; ++kk, ++it) {
                        const int s = it % kStages2;
                        const uint32_t ph = (it / kStages2) & 1;
                        if (!mbar_wait(empty + 8 * s, ph ^ 1u, wait_ns, abort_flag)) { ok = false; break; }
                        mbar_arrive_expect_tx(full + 8 * s, stage_tx);
                        const uint32_t a_dst = smem_u32(base + s * kStage2Bytes);
                        const int kcol = g * G + kk * kBK;
                        tma_load_2d(a_dst, &tmA, kcol, m * 256, full + 8 * s);
                        tma_load_2d(a_dst + kA2Bytes, &tmB, kcol, col0(n), full + 8 * s);
                    }
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        }
        if (lane == 0) {
            // the CTA that finishes last puts the counters back to zero for the next launch
            if (ok && atomicAdd(queue + 1, 1u) + 1u == gridDim.x) {
                queue[0] = 0u;
                queue[1] = 0u;
            }
            if (!ok) { report_timeout(status); abort_grace(); }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ UMMA issuer
        int it = 0;
        bool ok = true;
        for (int tc = 0; ok; ++tc) {
            const int tile = next_tile(tc);
            if (tile < 0) { ok = tile == -1; break; }
            const int m = tile % n_m;
            const uint32_t idesc = umma_idesc_bf16(kBM, width(tile / n_m));
            uint32_t act[kMaskWords];
            tile_mask(m, act);
            if (lane == 0) {
                if (!mbar_wait(tempty, (tc & 1) ^ 1u, wait_ns, abort_flag)) ok = false;
                tc_fence_after_sync();
                uint32_t accumulate = 0;
                for (int g = 0; g < NG && ok; ++g) {
                    if (!((act[g >> 5] >> (g & 31)) & 1u)) continue;
                    for (int kk = 0; kk < ksub; ++kk, ++it) {
                        const int s = it % kStages2;
                        const uint32_t ph = (it / kStages2) & 1;
                        if (!mbar_wait(full + 8 * s, ph, wait_ns, abort_flag)) { ok = false; break; }
                        tc_fence_after_sync();
                        const uint32_t a_addr = smem_u32(base + s * kStage2Bytes);
                        const uint64_t adesc0 = umma_desc_sw128(a_addr);
                        const uint64_t adesc1 = umma_desc_sw128(a_addr + kABytes);
                        const uint64_t bdesc = umma_desc_sw128(a_addr + kA2Bytes);
#pragma unroll
                        for (int k4 = 0; k4 < kBK / 16; ++k4) {
                            umma_bf16(tmem_base, adesc0 + 2 * k4, bdesc + 2 * k4, idesc, accumulate);
                            umma_bf16(tmem_base + 256, adesc1 + 2 * k4, bdesc + 2 * k4, idesc, accumulate);
                            accumulate = 1;
                        }
                        umma_commit(empty + 8 * s);
                    }
                }
                if (ok) {
                    if (accumulate) umma_commit(tfull);
                    else mbar_arrive(tfull);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        }
        if (!ok && lane == 0) report_timeout(status);
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int q = warp & 3;
        bool ok = true;
        for (int tc = 0; ok; ++tc) {
            const int tile = next_tile(tc);
            if (tile < 0) { ok = tile == -1; break; }
            const int m = tile % n_m, n = tile / n_m;
            uint32_t act[kMaskWords];
            tile_mask(m, act);
            bool any = false;
            for (int g = 0; g < NG; ++g) any = any || ((act[g >> 5] >> (g & 31)) & 1u);
            if (!mbar_wait_warp(tfull, tc & 1, wait_ns, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            if (tc == 0) grid_dep_wait();         // nothing is stored before the kernel before has completed (a tile without
                                                  // an active group gets here without a load behind it)
#pragma unroll 1
            for (int half = 0; half < 2; ++half) {
                const int pos = m * 256 + half * 128 + q * 32 + lane;
                const int row = (order && pos < T) ? order[pos] : pos;   // token that owns this output row
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + half * 256;
                const int wn = width(n), cbase = col0(n);
#pragma unroll 1
                for (int c0 = 0; c0 < wn; c0 += 32) {
                    // widths are multiples of 16: the last chunk of a tile may hold 16 columns
                    const bool whole = c0 + 32 <= wn;
                    uint32_t r[32];
                    if (any) {
                        if (whole) {
                            tmem_ld_32x32(taddr + c0, r);
                            tmem_ld_wait();
                        } else {
                            uint32_t r16[16];
                            tmem_ld_32x16(taddr + c0, r16);
                            tmem_ld_wait();
#pragma unroll
                            for (int i = 0; i < 16; ++i) { r[i] = r16[i]; r[16 + i] = 0u; }
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = 0u;
                    }
                    const int col = cbase + c0;
                    const int ncol = whole ? 32 : 16;
                    if (peer.world > 0) {
                        if (any && row < T && col + ncol <= N) {
                            float* dst = peer.base[row / peer.rows_per_rank] +
                                         static_cast<size_t>(row % peer.rows_per_rank) * N + col;
#pragma unroll
                            for (int v = 0; v < 8; ++v)
                                if (4 * v < ncol) red_add_f32x4(dst + 4 * v, r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                        }
                    } else if (row < T && col + ncol <= N) {
                        if (out_bf16) {
                            uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(Y) + static_cast<size_t>(row) * N + col);
#pragma unroll
                            for (int v = 0; v < 4; ++v) {
                                uint4 o;
                                o.x = pack_bf16(__uint_as_float(r[8 * v + 0]), __uint_as_float(r[8 * v + 1]));
                                o.y = pack_bf16(__uint_as_float(r[8 * v + 2]), __uint_as_float(r[8 * v + 3]));
                                o.z = pack_bf16(__uint_as_float(r[8 * v + 4]), __uint_as_float(r[8 * v + 5]));
                                o.w = pack_bf16(__uint_as_float(r[8 * v + 6]), __uint_as_float(r[8 * v + 7]));
                                if (8 * v < ncol) dst[v] = o;
                            }
                        } else {
                            uint4* dst = reinterpret_cast<uint4*>(static_cast<float*>(Y) + static_cast<size_t>(row) * N + col);
#pragma unroll
                            for (int v = 0; v < 8; ++v)
                                if (4 * v < ncol) dst[v] = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                        }
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty);
        }
        if (!ok && lane == 0) report_timeout(status);
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

// ======================================================================================= gate/up
// Items.  A group g with c_g active tokens has nt_g = ceil(c_g / 128) row tiles in its sorted
// order.  Two consecutive tiles of the same (group, channel sub-block) form a DOUBLE item: 256
// gathered rows, two M=128 UMMAs per 16-wide k-slice sharing the weight tile in shared memory
// (1.5x fewer bytes per FLOP, the ring covers 1.5x more latency).  Doubles are dealt round-robin
// for as many full rounds as there are.  What is left of them is either cut back into 128-row SINGLE
// items and dealt together with the odd last tiles, so that every CTA ends within one single item of
// the others, or (when many doubles are left: a single costs about 0.7 of a double, two of them 1.4)
// run as one more, partial round of doubles with the odd tiles dealt from the idle CTAs on; whichever
// ends earlier by that cost model.  Every CTA derives the same schedule from `counts` alone (prefix
// sums in shared memory).
// The two accumulators of a double fill TMEM, so an item's epilogue does not overlap the next
// item's MMAs; it is kept short instead (8 epilogue warps, fast SiLU).
struct GuItem {
    int gs;     // group * nsub + sub-block
    int m;      // first 128-row tile
    int rows;   // 128 or 256
};

struct GuSched {
    const int* dbl_off;   // [n_gs + 1] prefix of doubles per (group, sub)
    const int* sgl_off;   // [n_gs + 1] prefix of odd last tiles
    int n_gs, nD, nS, grid, rfull, remD, nS2, pos;
    bool tail_doubles;    // the doubles left after the full rounds run as doubles
    __device__ GuSched(const int* d, const int* sg, int n) : dbl_off(d), sgl_off(sg), n_gs(n), grid(gridDim.x), pos(0) {
        nD = d[n];
        nS = sg[n];
        rfull = nD / grid;
        remD = nD - rfull * grid;
        nS2 = 2 * remD + nS;
        // end of the tail in tenths of a double item's time, a single item counted as 7
        const int cost_cut = 7 * ((nS2 + grid - 1) / grid);
        const int idle = grid - remD;
        const int cost_keep = max(7 * ((nS + grid - 1) / grid), 10 + 7 * (nS > idle ? (nS - idle + grid - 1) / grid : 0));
        tail_doubles = remD > 0 && cost_keep < cost_cut;
    }
    __device__ int find(const int* off, int idx) const {  // largest i with off[i] <= idx
        int lo = 0, hi = n_gs;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (off[mid] <= idx) lo = mid; else hi = mid;
        }
        return lo;
    }
    __device__ bool next(GuItem& it) {
        const int b = blockIdx.x;
        if (pos < rfull) {
            const int di = pos * grid + b;
            it.gs = find(dbl_off, di);
            it.m = 2 * (di - dbl_off[it.gs]);
            it.rows = 256;
            ++pos;
            return true;
        }
        if (tail_doubles) {
            // one partial round of doubles on CTAs 0 .. remD-1, the odd tiles dealt round-robin from CTA remD on
            const bool has_double = b < remD;
            if (pos == rfull && has_double) {
                const int di = rfull * grid + b;
                it.gs = find(dbl_off, di);
                it.m = 2 * (di - dbl_off[it.gs]);
                it.rows = 256;
                ++pos;
                return true;
            }
            const int q = pos - rfull - (has_double ? 1 : 0);         // singles this CTA has taken
            const int si = q * grid + (b - remD + grid) % grid;
            if (si >= nS) return false;
            it.gs = find(sgl_off, si);
            it.m = 2 * (dbl_off[it.gs + 1] - dbl_off[it.gs]);            // the odd tile follows the group's doubles
            it.rows = 128;
            ++pos;
            return true;
        }
        const int idx = (pos - rfull) * grid + b;
        if (idx >= nS2) return false;
        if (idx < 2 * remD) {
            const int di = rfull * grid + (idx >> 1);
            it.gs = find(dbl_off, di);
            it.m = 2 * (di - dbl_off[it.gs]) + (idx & 1);
        } else {
            const int si = idx - 2 * remD;
            it.gs = find(sgl_off, si);
            it.m = 2 * (dbl_off[it.gs + 1] - dbl_off[it.gs]);   // the odd tile follows the group's doubles
        }
        it.rows = 128;
        ++pos;
        return true;
    }
};

// silu(g) * u with one special-function instruction: silu(g) = h + h * tanh(h), h = g / 2
// (tanh.approx is good to about 2^-11, below the bf16 rounding of the result).
__device__ __forceinline__ float silu_mul_fast(float g, float u) {
    const float h = 0.5f * g;
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(h));
    return fmaf(h, t, h) * u;
}

constexpr int kGuThreads = 448;  // TMA, MMA, 4 gather warps, 8 epilogue warps

// kLinear = false: gate/up + SwiGLU, an item covers BN channels (B = BN rows of W_gate stacked on
// BN rows of W_up).  kLinear = true: the same GEMM-MN for ONE weight and no activation (the
// routed Q projection): an item covers 2*BN output channels (B = 2*BN consecutive rows of W).
template <int BN, bool kLinear>  // UMMA N = 2*BN
__global__ void __launch_bounds__(kGuThreads, 1)
gateup_kernel(const __grid_constant__ CUtensorMap tmG, const __grid_constant__ CUtensorMap tmU,
              const __nv_bfloat16* __restrict__ X, const int32_t* __restrict__ perm,
              const int32_t* __restrict__ counts, const int32_t* __restrict__ token_rank, int NG, int T, int D, int Dff,
              int G, __nv_bfloat16* __restrict__ H, int* __restrict__ status, unsigned long long wait_ns) {
    constexpr int kStagesG = BN == 128 ? 3 : 4;
    constexpr int kAB = 2 * kABytes;              // 256 rows x 128 B
    constexpr int kBBytes = 2 * BN * kBK * 2;
    constexpr int kStageBytes = kAB + kBBytes;
    constexpr int kMaxGs = WIDE_MAX_GROUPS * 4;  // (group, sub-block) pairs: G <= 512, BN >= 128 there
    extern __shared__ uint8_t smem_raw[];
    __shared__ int s_dbl[kMaxGs + 1];
    __shared__ int s_sgl[kMaxGs + 1];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + kStagesG * kStageBytes);
    const uint32_t full = smem_u32(bars), empty = smem_u32(bars + kStagesG);
    const uint32_t tfull = smem_u32(bars + 2 * kStagesG), tempty = smem_u32(bars + 2 * kStagesG + 1);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStagesG + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr int kItemCh = kLinear ? 2 * BN : BN;   // output channels of one item
    const int nsub = G / kItemCh;
    const int n_gs = NG * nsub;

    if (tid == 0) {
        for (int s = 0; s < kStagesG; ++s) {
            mbar_init(full + 8 * s, 1 + 128);  // TMA producer + one arrival per gather thread
            mbar_init(empty + 8 * s, 1);
        }
        mbar_init(tfull, 1);
        mbar_init(tempty, 8);
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmG);
        prefetch_tmap(&tmU);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    grid_dep_launch();   // the down projection behind this kernel may set itself up on SMs that this kernel has left
    if (warp == 2) {
        // prefix sums of doubles and odd tiles per (group, sub-block)
        int dsum = 0, ssum = 0;
        for (int base_i = 0; base_i < n_gs; base_i += 32) {
            const int i = base_i + lane;
            int dv = 0, sv = 0;
            if (i < n_gs) {
                const int nt = (counts[i / nsub] + kBM - 1) / kBM;
                dv = nt >> 1;
                sv = nt & 1;
            }
            int dp = dv, sp = sv;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int a = __shfl_up_sync(0xffffffffu, dp, o), c = __shfl_up_sync(0xffffffffu, sp, o);
                if (lane >= o) { dp += a; sp += c; }
            }
            if (i < n_gs) {
                s_dbl[i] = dsum + dp - dv;
                s_sgl[i] = ssum + sp - sv;
            }
            dsum += __shfl_sync(0xffffffffu, dp, 31);
            ssum += __shfl_sync(0xffffffffu, sp, 31);
        }
        if (lane == 0) {
            s_dbl[n_gs] = dsum;
            s_sgl[n_gs] = ssum;
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const int nk = D / kBK;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (weights)
        if (lane == 0) {
            int it = 0;
            bool ok = true;
            GuSched sched(s_dbl, s_sgl, n_gs);
            GuItem w;
            // A group's weight tile is read by the few CTAs that run the group's items side by side and
            // is dead afterwards: it should leave L2 before x (which every item gathers from) and H.
            const uint64_t wpol = l2_policy_evict_first();
            while (ok && sched.next(w)) {
                const int crow = (w.gs / nsub) * G + (w.gs % nsub) * kItemCh;
                for (int k = 0; k < nk; ++k, ++it) {
                    const int s = it % kStagesG;
                    const uint32_t ph = (it / kStagesG) & 1;
                    if (!mbar_wait(empty + 8 * s, ph ^ 1u, wait_ns, abort_flag)) { ok = false; break; }
                    mbar_arrive_expect_tx(full + 8 * s, kBBytes);
                    const uint32_t b_dst = smem_u32(base + s * kStageBytes) + kAB;
                    tma_load_2d_hint(b_dst, &tmG, k * kBK, crow, full + 8 * s, wpol);
                    tma_load_2d_hint(b_dst + BN * kBK * 2, &tmU, k * kBK, kLinear ? crow + BN : crow, full + 8 * s, wpol);
                }
            }
            if (!ok) { report_timeout(status); abort_grace(); }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ UMMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(kBM, 2 * BN);
            int it = 0, tc = 0;
            bool ok = true;
            GuSched sched(s_dbl, s_sgl, n_gs);
            GuItem w;
            while (ok && sched.next(w)) {
                if (!mbar_wait(tempty, (tc & 1) ^ 1u, wait_ns, abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                for (int k = 0; k < nk; ++k, ++it) {
                    const int s = it % kStagesG;
                    const uint32_t ph = (it / kStagesG) & 1;
                    if (!mbar_wait(full + 8 * s, ph, wait_ns, abort_flag)) { ok = false; break; }
                    fence_proxy_async_smem();  // the A rows were written through the generic proxy (cp.async)
                    tc_fence_after_sync();
                    const uint32_t a_addr = smem_u32(base + s * kStageBytes);
                    const uint64_t adesc0 = umma_desc_sw128(a_addr);
                    const uint64_t adesc1 = umma_desc_sw128(a_addr + kABytes);
                    const uint64_t bdesc = umma_desc_sw128(a_addr + kAB);
#pragma unroll
                    for (int k4 = 0; k4 < kBK / 16; ++k4) {
                        const uint32_t accumulate = (k > 0 || k4 > 0) ? 1u : 0u;
                        umma_bf16(tmem_base, adesc0 + 2 * k4, bdesc + 2 * k4, idesc, accumulate);
                        if (w.rows == 256) umma_bf16(tmem_base + 256, adesc1 + 2 * k4, bdesc + 2 * k4, idesc, accumulate);
                    }
                    umma_commit(empty + 8 * s);
                }
                if (ok) umma_commit(tfull);
                ++tc;
            }
            if (!ok) report_timeout(status);
        }
    } else if (warp < 6) {
        // ------------------------------------------------------------------ A gather (warps 2..5)
        // 16-byte cp.async copies land in the 128-byte-swizzle pattern; the stage's mbarrier counts
        // one arrival per thread when that thread's copies have landed, so the gather runs as far
        // ahead as the ring allows.  Coalesced mapping: 8 consecutive lanes copy the 8 chunks of
        // one row, one warp instruction covers 4 whole rows; instruction i of gather warp w copies
        // tile rows 16*i + 4*w + lane/8  (i < 8 for a 128-row item, i < 16 for a 256-row item).
        const int chunk = lane & 7;
        const int row0 = (warp - 2) * 4 + (lane >> 3);
        int it = 0;
        bool ok = true;
        GuSched sched(s_dbl, s_sgl, n_gs);
        GuItem w;
        while (ok && sched.next(w)) {
            const int g = w.gs / nsub;
            const int ni = w.rows / 16;
            const uint8_t* src[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                int j = w.m * kBM + row0 + 16 * i;
                if (j >= T) j = T - 1;
                const int tok = i < ni ? perm[static_cast<size_t>(g) * T + j] : 0;
                src[i] = reinterpret_cast<const uint8_t*>(X + static_cast<size_t>(tok) * D) + 16 * chunk;
            }
            for (int k = 0; k < nk; ++k, ++it) {
                const int s = it % kStagesG;
                const uint32_t ph = (it / kStagesG) & 1;
                if (!mbar_wait_warp(empty + 8 * s, ph ^ 1u, wait_ns, abort_flag)) { ok = false; break; }
                const uint32_t a_dst = smem_u32(base + s * kStageBytes);
                const size_t koff = static_cast<size_t>(k) * (kBK * 2);
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    if (i < ni) {
                        const int r = row0 + 16 * i;
                        cp_async_16(a_dst + static_cast<uint32_t>(r) * 128u +
                                        ((static_cast<uint32_t>(chunk) ^ static_cast<uint32_t>(r & 7)) << 4),
                                    src[i] + koff);
                    }
                }
                cp_async_mbar_arrive_noinc(full + 8 * s);
            }
        }
        cp_async_wait_all();
        if (!ok && lane == 0) report_timeout(status);
    } else {
        // ------------------------------------------------------------------ epilogue (warps 6..13)
        // warp pair (w, w+4) shares a TMEM lane quarter and splits the item's channels in two
        const int q = warp & 3;
        const int ew = warp - 6;
        const int chalf = ew >> 2;
        const int e = ew * 32 + lane;  // 0..255
        constexpr int kCh = BN / 2;    // channels per epilogue warp
        uint4* ep_stage = reinterpret_cast<uint4*>(base + kStagesG * kStageBytes + 128) + ew * 128;  // 2 KB per warp
        int tc = 0;
        bool ok = true;
        if constexpr (kLinear) {
            // the output is a result, not scratch: a group nobody selected has no item that would
            // zero its columns, so the CTAs share those rows here
            for (int g0 = 0; g0 < NG; ++g0) {
                if (counts[g0] != 0) continue;
                const int ppr = G / 8;   // 16-byte pieces per row
                for (long long i = static_cast<long long>(blockIdx.x) * 256 + e; i < static_cast<long long>(T) * ppr;
                     i += static_cast<long long>(gridDim.x) * 256)
                    reinterpret_cast<uint4*>(H + (i / ppr) * Dff + g0 * G)[i % ppr] = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        GuSched sched(s_dbl, s_sgl, n_gs);
        GuItem w;
        while (ok && sched.next(w)) {
            const int g = w.gs / nsub, sub = w.gs % nsub;
            const int c = counts[g];
            {
                // While the MMAs of this item run: zero this item's share of the group's INACTIVE
                // rows of H (sorted positions [c, T) split evenly over the group's row tiles), so
                // that the down projection reads exact zeros for every inactive (token, group) pair
                // of a group that is active anywhere.  Groups nobody selected are never read.
                // kLpr consecutive lanes write one row's piece, so a warp store touches whole
                // lines (scattered 16-byte stores would keep the L1 busy and starve the gather).
                constexpr int kLpr = kItemCh / 8;     // lanes per row: one 16-byte store each
                constexpr int kRows = 256 / kLpr;     // rows per sweep of the 8 warps
                const int nt = (c + kBM - 1) / kBM;
                const int per = (T - c + nt - 1) / nt;
                const int zr = e / kLpr, zp = e % kLpr;
                for (int mm = w.m; mm < w.m + w.rows / kBM; ++mm) {
                    const int j0 = c + mm * per;
                    const int j1 = min(T, j0 + per);
                    for (int jj = j0 + zr; jj < j1; jj += kRows) {
                        int tz = perm[static_cast<size_t>(g) * T + jj];
                        if (token_rank) tz = token_rank[tz];   // H rows are kept in clustered token order
                        reinterpret_cast<uint4*>(H + static_cast<size_t>(tz) * Dff + g * G + sub * kItemCh)[zp] =
                            make_uint4(0u, 0u, 0u, 0u);
                    }
                }
            }
            // the H rows of this item's tokens, fetched before the accumulators are ready
            int tokh[2];
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int j = (w.m + half) * kBM + q * 32 + lane;
                int tok = (half < w.rows / kBM && j < c) ? perm[static_cast<size_t>(g) * T + j] : -1;
                if (tok >= 0 && token_rank) tok = token_rank[tok];   // H rows are kept in clustered token order
                tokh[half] = tok;
            }
            if (!mbar_wait_warp(tfull, tc & 1, wait_ns, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            for (int half = 0; half < w.rows / kBM; ++half) {
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + half * 256 + chalf * kCh;
#pragma unroll 1
                for (int c0 = 0; c0 < kCh; c0 += 32) {
                    uint32_t gr[32], ur[32];
                    tmem_ld_32x32(taddr + c0, gr);
                    tmem_ld_32x32(taddr + BN + c0, ur);
                    tmem_ld_wait();
                    // lane = row here; transpose through shared memory so that 4 lanes write one
                    // row's 64 bytes (a warp store then touches 8 rows instead of 32)
                    // one pass (SwiGLU) or two (linear: the "gate" and the "up" columns are two
                    // separate blocks of output channels, BN apart)
#pragma unroll
                    for (int pass = 0; pass < (kLinear ? 2 : 1); ++pass) {
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            uint32_t o[4];
#pragma unroll
                            for (int x4 = 0; x4 < 4; ++x4) {
                                const int i = 8 * v + 2 * x4;
                                if constexpr (kLinear) {
                                    const uint32_t (&src)[32] = pass == 0 ? gr : ur;
                                    o[x4] = pack_bf16(__uint_as_float(src[i]), __uint_as_float(src[i + 1]));
                                } else {
                                    o[x4] = pack_bf16(silu_mul_fast(__uint_as_float(gr[i]), __uint_as_float(ur[i])),
                                                      silu_mul_fast(__uint_as_float(gr[i + 1]), __uint_as_float(ur[i + 1])));
                                }
                            }
                            // piece v of row `lane` sits in slot v ^ ((lane >> 1) & 3): no bank conflicts
                            // on the way in (8 rows, one piece) nor on the way out (2 rows, 4 pieces)
                            ep_stage[lane * 4 + (v ^ ((lane >> 1) & 3))] = make_uint4(o[0], o[1], o[2], o[3]);
                        }
                        __syncwarp();
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int r = 8 * i + (lane >> 2), pc = lane & 3;
                            const int tr = __shfl_sync(0xffffffffu, tokh[half], r);
                            const uint4 val = ep_stage[r * 4 + (pc ^ ((r >> 1) & 3))];
                            if (tr >= 0)
                                *reinterpret_cast<uint4*>(H + static_cast<size_t>(tr) * Dff + g * G + sub * kItemCh + pass * BN +
                                                          chalf * kCh + c0 + pc * 8) = val;
                        }
                        __syncwarp();
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty);
            ++tc;
        }
        if (!ok && lane == 0) report_timeout(status);
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

// --------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 2-D bf16 row-major [rows, cols] tensor, box = [box_rows, 64 columns], 128-byte swizzle.
bool make_tmap_bf16(const wide_ctx* ctx, CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols,
                    uint32_t box_rows) {
    if (!ctx->encode_tiled) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(kBK), box_rows};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
        map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

template <int BN>
int launch_down(wide_ctx* ctx, cudaStream_t s, const void* A, const void* B, const uint32_t* mask_bits, int T,
                int N, int K, int G, void* Y, int out_dtype, int b_rows = -1, const char* name = "prefill_down",
                int ksplit = 1, float* aux_norm = nullptr, const int32_t* order = nullptr,
                const int32_t* sel_counts = nullptr, int sel_thr = WIDE_KAXIS_NEVER, int acc_split = 1,
                const PeerOut* peer = nullptr) {
    CUtensorMap tmA, tmB;
    if (b_rows < 0) b_rows = N;  // rows of B that exist; rows up to N beyond them read as zero
    if (!make_tmap_bf16(ctx, &tmA, A, T, K, kBM) || !make_tmap_bf16(ctx, &tmB, B, b_rows, K, BN)) return WIDE_ERR_CUDA;
    constexpr int smem = smem_bytes<BN * kBK * 2>();
    WIDE_CUDA_CHECK(cudaFuncSetAttribute(down_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    const int n_tiles = ((T + kBM - 1) / kBM) * ((N + BN - 1) / BN) * ksplit;
    int grid = n_tiles < ctx->sm_count ? n_tiles : ctx->sm_count;
    if (aux_norm) grid = n_tiles + (b_rows + 5) / 6;  // spare CTAs for the row norms of B
    const int words = (K / G + 31) / 32;
    WideLaunch l(ctx, s, name);
    down_kernel<BN><<<grid, 192, smem, s>>>(tmA, tmB, mask_bits, order, words, T, N, K, G, Y, out_dtype == WIDE_BF16 ? 1 : 0,
                                            ksplit, static_cast<const __nv_bfloat16*>(B), b_rows, aux_norm, sel_counts, sel_thr,
                                            acc_split, peer ? *peer : PeerOut{}, ctx->d_status, ctx->wait_ns);
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}

// Column tiling of the 256-row kernel: the number of column tiles n_n (widths = sixteenths of N
// dealt evenly, at most 256) that minimises waves x width, with a mild penalty for narrow tiles
// (a narrower B tile is reused by fewer FLOPs).  Returns the cost in units of a 256-wide tile.
double pick_down256_tiling(int sm, int T, int N, int* n_n_out, int* wmax_out) {
    const int n_m = (T + 255) / 256, q16 = (N + 15) / 16;
    const int nn0 = (N + 255) / 256;
    double best = 1e30;
    for (int nn = nn0; nn <= nn0 + nn0 / 2 + 1 && nn <= q16; ++nn) {
        const int wmax = 16 * ((q16 + nn - 1) / nn);
        if (wmax > 256 || wmax < 160) continue;
        const int waves = (n_m * nn + sm - 1) / sm;
        const double cost = waves * (wmax / 256.0) * (1.0 + 0.5 * (256 - wmax) / 256.0);
        if (cost < best - 1e-9) { best = cost; *n_n_out = nn; *wmax_out = wmax; }
    }
    return best;
}

// Picks the tile height for the down / output projection: 256-row tiles move fewer bytes per FLOP
// (about 0.8 of the time per row), 128-row tiles quantise better over the SMs.
int launch_down_auto(wide_ctx* ctx, cudaStream_t s, const void* A, const void* B, const uint32_t* mask_bits, int T,
                     int N, int K, int G, void* Y, int out_dtype, const int32_t* order,
                     const int32_t* sel_counts = nullptr, int sel_thr = WIDE_KAXIS_NEVER, const PeerOut* peer = nullptr,
                     bool after_gateup = false) {
    const int sm = ctx->sm_count;
    const int t128 = ((T + 127) / 128) * ((N + 255) / 256);
    int n_n = (N + 255) / 256, wmax = 256;
    const double cost128 = static_cast<double>((t128 + sm - 1) / sm);
    const double cost256 = pick_down256_tiling(sm, T, N, &n_n, &wmax) * 2.0 * 0.8;
    if (cost128 <= cost256)
        return launch_down<256>(ctx, s, A, B, mask_bits, T, N, K, G, Y, out_dtype, -1, "prefill_down", 1, nullptr, order,
                                sel_counts, sel_thr, 1, peer);
    CUtensorMap tmA, tmB;
    if (!make_tmap_bf16(ctx, &tmA, A, T, K, 256) || !make_tmap_bf16(ctx, &tmB, B, N, K, wmax)) return WIDE_ERR_CUDA;
    WIDE_CUDA_CHECK(cudaFuncSetAttribute(down256_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem2));
    const int t256 = ((T + 255) / 256) * n_n;
    const int grid = t256 < sm ? t256 : sm;
    const int words = (K / G + 31) / 32;
    WideLaunch l(ctx, s, "prefill_down");
    if (after_gateup && !sel_counts && !ctx->prof) {   // (per-kernel timing brackets every launch with events: ordinary launches then)
        // The kernel before this one in the stream is the gate / up kernel of the same call, which lets its dependents
        // start as its CTAs leave: this kernel sets itself up and forms its tile masks (from the mask and the token
        // order, both older than the gate / up kernel) meanwhile, and waits before it loads H or stores anything.
        // Only then: after any other kernel the early reads could see that kernel's unfinished writes.
        WIDE_CUDA_CHECK(wide_launch_dependent(down256_kernel, dim3(grid), dim3(192), kSmem2, s, tmA, tmB, mask_bits, order, words, T,
                                              N, K, G, Y, out_dtype == WIDE_BF16 ? 1 : 0, n_n, wmax,
                                              reinterpret_cast<unsigned*>(ctx->d_status) + 8, sel_counts, sel_thr,
                                              peer ? *peer : PeerOut{}, ctx->d_status, ctx->wait_ns));
        return WIDE_OK;
    }
    down256_kernel<<<grid, 192, kSmem2, s>>>(tmA, tmB, mask_bits, order, words, T, N, K, G, Y, out_dtype == WIDE_BF16 ? 1 : 0,
                                             n_n, wmax, reinterpret_cast<unsigned*>(ctx->d_status) + 8, sel_counts, sel_thr,
                                             peer ? *peer : PeerOut{}, ctx->d_status, ctx->wait_ns);
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}

template <int BN, bool kLinear>
int launch_gateup(wide_ctx* ctx, cudaStream_t s, const void* x, const void* wg, const void* wu, int T, int D,
                  int Dff, int G, const int32_t* perm, const int32_t* counts, const int32_t* token_rank, void* h) {
    CUtensorMap tmG, tmU;
    if (!make_tmap_bf16(ctx, &tmG, wg, Dff, D, BN) || !make_tmap_bf16(ctx, &tmU, wu, Dff, D, BN)) return WIDE_ERR_CUDA;
    constexpr int stages = BN == 128 ? 3 : 4;
    constexpr int smem = stages * (2 * kABytes + 2 * BN * kBK * 2) + 128 + 8 * 2048 + 1024;  // ring, barriers, epilogue staging
    WIDE_CUDA_CHECK(cudaFuncSetAttribute(gateup_kernel<BN, kLinear>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    WideLaunch l(ctx, s, kLinear ? "prefill_linear_mn" : "prefill_gateup");
    gateup_kernel<BN, kLinear><<<ctx->sm_count, kGuThreads, smem, s>>>(
        tmG, tmU, static_cast<const __nv_bfloat16*>(x), perm, counts, token_rank, Dff / G, T, D, Dff, G,
        static_cast<__nv_bfloat16*>(h), ctx->d_status, ctx->wait_ns);
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}

// Which K-axis kernel a prefill call uses.  Measured on the 13B output projection and on the 8B down
// projection (T = 4096): the per-group kernel (Algorithm 3) costs c * p of the owner-computes kernel's
// time, p = padded active fraction, with c = 1.35 (G = 512, bf16 sums), 2.1 (256, bf16), 3.7 (128, bf16),
// 2.0 (512, fp32 sums incl. clearing and converting the scratch), 3.1 (256, fp32), 5.5 (128, fp32):
// c = 0.6 + beta / G with beta = 380 for bf16 sums and 640 for fp32 sums fits all six.  The first term is
// the tensor work (128 x 256 tiles move more operand bytes per FLOP than the owner kernel's 256 x 256),
// the second the T*k*N partial sums that go through the L2's reduction units.  The per-group kernel is
// taken when c * p <= 0.9.  Group sizes below 256 take part in the device-side choice only when the
// caller opts into bf16 sums; otherwise the choice would add two empty launches to every call that
// stays with the owner-computes kernel.
struct KaxisPlan {
    int thr_q;       // threshold of wide_kaxis_group_chosen
    bool bf16_red;   // reduce straight into the bf16 output
    bool use_acc;    // reduce in fp32 into scratch, then convert
};

KaxisPlan plan_kaxis(int G, int NG, int out_dtype, bool have_perm, unsigned flags) {
    KaxisPlan p;
    // bf16 sums by default only where a token has few partial sums (at most 16 groups): measured
    // max error 7.7e-3 of max|y| with 5 of 10 groups against 2.9e-3 for the owner-computes kernel
    // (whose only rounding is the bf16 output); 1.0e-2 with 14 of 56 groups and 1.7e-2 with 28 of 112,
    // too close to the 2e-2 bar to be anything but the caller's explicit choice.
    p.bf16_red = out_dtype == WIDE_BF16 && ((flags & WIDE_FLAG_REDUCE_BF16) || NG <= 16);
    p.use_acc = out_dtype == WIDE_BF16 && !p.bf16_red;
    if (!have_perm || (flags & WIDE_FLAG_KAXIS_OWNER)) {
        p.thr_q = WIDE_KAXIS_NEVER;
    } else if (flags & WIDE_FLAG_KAXIS_GROUP) {
        p.thr_q = WIDE_KAXIS_ALWAYS;
    } else if (G >= 256 || (G >= 128 && (flags & WIDE_FLAG_REDUCE_BF16))) {
        const double c = 0.6 + (p.bf16_red ? 380.0 : 640.0) / G;
        p.thr_q = static_cast<int>(1024.0 * 0.9 / c);
    } else {
        p.thr_q = WIDE_KAXIS_NEVER;
    }
    return p;
}

// The K-axis product y = A (.)_G M  B^T shared by the down projection and the output projection.
//   a_rows      [T, K] rows the per-group kernel gathers (row a_row_of_token[t] holds token t)
//   a_owner     [T, K] operand of the owner-computes kernel: zeros for inactive pairs, rows in
//               `order`; when a_unmasked is given it is written here first (masking pass)
int launch_kaxis(wide_ctx* ctx, cudaStream_t s, const KaxisPlan& plan, const void* a_rows, const int32_t* a_row_of_token,
                 const void* a_unmasked, void* a_owner, const void* B, int T, int N, int K, int G,
                 const uint32_t* mask_bits, const int32_t* perm, const int32_t* counts, const int32_t* order,
                 const int32_t* rank, void* y, int out_dtype, void* acc, const char* group_name, bool after_gateup = false) {
    const int NG = K / G;
    int rc;
    if (plan.thr_q == WIDE_KAXIS_NEVER) {
        if (a_unmasked) {
            rc = wide_launch_kaxis_prep(ctx, s, nullptr, NG, T, plan.thr_q, nullptr, 0, a_unmasked, mask_bits, rank, K, G, a_owner);
            if (rc != WIDE_OK) return rc;
        }
        return launch_down_auto(ctx, s, a_owner, B, mask_bits, T, N, K, G, y, out_dtype, order, nullptr, WIDE_KAXIS_NEVER, nullptr,
                                after_gateup && !a_unmasked);
    }
    void* target = plan.use_acc ? acc : y;
    const size_t target_bytes = static_cast<size_t>(T) * N * (plan.bf16_red ? 2 : 4);
    const bool always = plan.thr_q >= WIDE_KAXIS_ALWAYS;
    rc = wide_launch_kaxis_prep(ctx, s, counts, NG, T, plan.thr_q, target, target_bytes, always ? nullptr : a_unmasked,
                                mask_bits, rank, K, G, a_owner);
    if (rc != WIDE_OK) return rc;
    rc = wide_launch_gemmk_group_tc(ctx, s, a_rows, K, B, T, N, K, G, perm, counts, a_row_of_token, target, plan.bf16_red,
                                    plan.thr_q, group_name);
    if (rc != WIDE_OK) return rc;
    if (!always) {
        rc = launch_down_auto(ctx, s, a_owner, B, mask_bits, T, N, K, G, y, out_dtype, order, counts, plan.thr_q);
        if (rc != WIDE_OK) return rc;
    }
    if (plan.use_acc) return wide_launch_kaxis_convert(ctx, s, counts, NG, T, plan.thr_q, static_cast<const float*>(acc), y,
                                                       static_cast<size_t>(T) * N);
    return WIDE_OK;
}

}  // namespace

bool wide_make_tmap_bf16(const wide_ctx* ctx, CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols,
                         uint32_t box_rows) {
    return make_tmap_bf16(ctx, map, base, rows, cols, box_rows);
}

int wide_launch_ffn_prefill_tc(wide_ctx* ctx, cudaStream_t s, const void* x, const void* wg, const void* wu,
                               const void* wd, int T, int D, int Dff, int G, const uint32_t* mask_bits,
                               const int32_t* perm, const int32_t* counts, const int32_t* token_order,
                               const int32_t* token_rank, void* y, int out_dtype, void* h, void* acc, unsigned flags) {
    if (T == 0) return WIDE_OK;
    // H [T, Dff] is kept in clustered token order when token_order / token_rank are given (row
    // token_rank[t] holds token t), else in token order.  Inactive (token, group) pairs of H must
    // read as zero in the owner-computes down projection: the gate/up kernel's epilogue warps write
    // those zeros.  The per-group down projection gathers active rows only.
    int rc = (G == 64) ? launch_gateup<64, false>(ctx, s, x, wg, wu, T, D, Dff, G, perm, counts, token_rank, h)
                       : launch_gateup<128, false>(ctx, s, x, wg, wu, T, D, Dff, G, perm, counts, token_rank, h);
    if (rc != WIDE_OK) return rc;
    const KaxisPlan plan = plan_kaxis(G, Dff / G, out_dtype, true, flags);
    return launch_kaxis(ctx, s, plan, h, token_rank, nullptr, h, wd, T, D, Dff, G, mask_bits, perm, counts, token_order,
                        token_rank, y, out_dtype, acc, "prefill_down_group", true);
}

// Group-sharded FFN part with the reduce-scatter fused into the down projection's epilogue (see
// PeerOut): gate/up on this rank's groups, then the owner-computes down kernel adding its tiles into
// the shards of the ranks that own the rows.
int wide_launch_ffn_prefill_tp(wide_ctx* ctx, cudaStream_t s, const void* x, const void* wg, const void* wu,
                               const void* wd, int T, int D, int Dff, int G, const uint32_t* mask_bits,
                               const int32_t* perm, const int32_t* counts, const int32_t* token_order,
                               const int32_t* token_rank, float* const* shards, int world, int rows_per_rank, void* h) {
    if (T == 0) return WIDE_OK;
    PeerOut peer{};
    peer.world = world;
    peer.rows_per_rank = rows_per_rank;
    for (int r = 0; r < world; ++r) peer.base[r] = shards[r];
    int rc = (G == 64) ? launch_gateup<64, false>(ctx, s, x, wg, wu, T, D, Dff, G, perm, counts, token_rank, h)
                       : launch_gateup<128, false>(ctx, s, x, wg, wu, T, D, Dff, G, perm, counts, token_rank, h);
    if (rc != WIDE_OK) return rc;
    return launch_down_auto(ctx, s, h, wd, mask_bits, T, D, Dff, G, nullptr, WIDE_F32, token_order, nullptr, WIDE_KAXIS_NEVER,
                            &peer);
}

// y[t, gG:(g+1)G] = x_t W[gG:(g+1)G, :]^T for active (t, g), exact zeros elsewhere (Algorithm 2 with a
// plain store epilogue).  G = 128 runs items of 128 channels, G >= 256 items of 256.
int wide_launch_linear_mn_tc(wide_ctx* ctx, cudaStream_t s, const void* x, const void* w, int T, int D, int Nout,
                             int G, const int32_t* perm, const int32_t* counts, void* y) {
    if (T == 0) return WIDE_OK;
    return (G == 128) ? launch_gateup<64, true>(ctx, s, x, w, w, T, D, Nout, G, perm, counts, nullptr, y)
                      : launch_gateup<128, true>(ctx, s, x, w, w, T, D, Nout, G, perm, counts, nullptr, y);
}

int wide_launch_oproj_prefill_tc(wide_ctx* ctx, cudaStream_t s, const void* a, const void* wo, int T, int D,
                                 int K, int G, const uint32_t* mask_bits, const int32_t* perm, const int32_t* counts,
                                 const int32_t* token_order, const int32_t* token_rank, void* y, int out_dtype,
                                 void* a_masked, void* acc, unsigned flags) {
    if (T == 0) return WIDE_OK;
    const KaxisPlan plan = plan_kaxis(G, K / G, out_dtype, perm != nullptr && counts != nullptr, flags);
    // The per-group kernel gathers active rows of the input as it stands.  The owner-computes kernel
    // needs zeros for the inactive pairs: an input that already has them is its operand as it
    // stands (tokens in their own order), any other input goes through the masking pass first (and
    // lands in clustered token order when one is given).
    if (flags & WIDE_FLAG_INPUT_MASKED)
        return launch_kaxis(ctx, s, plan, a, nullptr, nullptr, const_cast<void*>(a), wo, T, D, K, G, mask_bits, perm, counts,
                            nullptr, nullptr, y, out_dtype, acc, "prefill_oproj_group");
    return launch_kaxis(ctx, s, plan, a, nullptr, a, a_masked, wo, T, D, K, G, mask_bits, perm, counts, token_order,
                        token_rank, y, out_dtype, acc, "prefill_oproj_group");
}

// scores (fp32) = x[T, D] * w_router[NG, D]^T on the tensor cores, K split `ksplit` ways: slab ks
// [T, ld] holds the partial sum over columns [ks*D/ksplit, (ks+1)*D/ksplit); ld = NG rounded up to
// 32, columns >= NG are zeros (weight rows past NG are zero-filled by the TMA).  The same launch
// writes ||w_g|| (rounded up) to wnorm[0..NG).  Returns the ksplit it used through *ksplit_out.
int wide_launch_scores_tc(wide_ctx* ctx, cudaStream_t s, const void* x, const void* w_router, int T, int NG,
                          int ld, int D, float* scores, float* wnorm, int max_split, int* ksplit_out, int* chain_out) {
    const int n_m = (T + kBM - 1) / kBM;
    int ksplit = 1;
    // more CTAs while each keeps >= 8 k-steps, the slabs fit, and everything is co-resident
    while (ksplit * 2 <= max_split && D % (ksplit * 2 * kBK) == 0 && D / (ksplit * 2 * kBK) >= 8 &&
           n_m * ksplit * 2 + (NG + 5) / 6 <= ctx->sm_count)
        ksplit *= 2;
    *ksplit_out = ksplit;
    // Every CTA has one tile here (the grid is the tile count plus the norm CTAs), so the k-steps of
    // a slab can be spread over several accumulators: up to 4 of 128 columns or 2 of 256.
    const int ksteps = D / ksplit / kBK;
    int acc = ld <= 128 ? 4 : 2;
    while (acc > 1 && ksteps < 2 * acc) acc >>= 1;
    *chain_out = (D / ksplit + acc - 1) / acc + acc + ksplit;
    if (T == 0) return WIDE_OK;
    if (ld <= 128)
        return launch_down<128>(ctx, s, x, w_router, nullptr, T, ld, D, D / ksplit, scores, WIDE_F32, NG,
                                "route_scores_tc", ksplit, wnorm, nullptr, nullptr, WIDE_KAXIS_NEVER, acc);
    return launch_down<256>(ctx, s, x, w_router, nullptr, T, ld, D, D / ksplit, scores, WIDE_F32, NG,
                            "route_scores_tc", ksplit, wnorm, nullptr, nullptr, WIDE_KAXIS_NEVER, acc);
}
