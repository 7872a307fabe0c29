// Head-group-masked FlashAttention prefill on tcgen05 (Algorithm 4): query-tile admission through
// the reordered mask, gathered Q rows, dense K/V tiles streamed by TMA, online softmax, scatter
// epilogue.
//
// A work item is one (query head h, tile m of 128 rows of the head's routing group g in that group's
// sorted order).  Tiles past the group's active count are no items at all (block-level predicate);
// the rows of a tile are gathered through perm[g] (row-level predicate: rows past the count are
// computed on a clamped copy and dropped in the epilogue).  Per key tile t of 128 keys:
//     S  = Q K_t^T                (UMMA, fp32 in TMEM, two buffers)
//     P  = exp2(S*c - m), row statistics m, l   (softmax warps: one thread per row)
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
// rings drain at different points of the loop.  Two groups of four softmax warps share the key
// tiles: group 0 takes the even ones, group 1 the odd ones, each with its own (m, l, O) per row
// and its own S / P / O buffers; the two partial results are merged at the end of the item (the
// split-key form of the online softmax), each group finishing half of the output columns from
// both accumulators.  Causal attention shortens the key range to the largest active query
// position of the tile (+ delta = T_k - T_q); only tiles that straddle a row's limit evaluate
// element-wise predicates.
//
// The grid is one CTA per SM, and a CTA works through items until the list is empty: every ring,
// barrier phase and tensor-memory buffer carries over from one item to the next.  Items are drawn
// with an atomic add from a list ordered heavy (late rows, long key range) first, one item ahead,
// by the V producer, which passes them to the other roles through a two-slot queue in shared
// memory.  The K producer's warp gathers the next item's Q rows as soon as the last QK^T of the
// current item has read Q, so the next item's first scores are computed under the current
// item's last key tiles and merge: what an item costs beyond its key tiles is the merge alone.
// (With one CTA per item, the prologue, the pipeline fill and the merge of every item ran with
// the tensor core idle: 27 % of the kernel.)
//
// Outputs of inactive (token, group) pairs are exact zeros, written by the softmax warps of all
// CTAs before their first item.  Every mbarrier wait is bounded, and nothing else blocks: the
// softmax groups meet through mbarriers, not named barriers, so an expired wait anywhere lets
// every role run to the kernel's end.
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

__device__ __forceinline__ void st_global_v8(void* p, const uint32_t (&v)[8]) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(v[0]), "r"(v[1]), "r"(v[2]),
                 "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
                 : "memory");
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

constexpr int kBarBytes = 512;   // mbarriers, the tensor-memory slot, the abort flag, two work-item slots
constexpr int kXmlBytes = 2 * 2 * kQ * 4;   // (m, l) of both softmax groups for the merge

template <int HD>
constexpr int attn_smem_bytes() {
    // Q, 2 K stages, 2 V stages, 2 P buffers, barriers, (m, l) exchange, alignment slack
    return (HD / kBK) * kBlk + 4 * (HD / kBK) * kBlk + 2 * (kKV / kBK) * kBlk + kBarBytes + kXmlBytes + 512;
}

// q [T_q, H_q*HD], o likewise; K/V come through the tensor maps ([T_k, H_kv*HD], box 64 x 128).
// sched[0]: the next work item (heavy tiles first), sched[1]: CTAs that have finished; both are zero
// between launches (the last CTA to finish puts them back).
template <int HD>
__global__ void __launch_bounds__(kThreads, 1)
attn_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
            const __nv_bfloat16* __restrict__ q, const int32_t* __restrict__ perm, const int32_t* __restrict__ counts,
            int Tq, int Tk, int Hq, int Hkv, int hpg, int causal, float scale_log2e,
            __nv_bfloat16* __restrict__ o, int* __restrict__ status, int* __restrict__ sched, int smem_bytes,
            unsigned long long wait_ns) {
    constexpr int kKB = HD / kBK;          // 64-wide blocks along the head dimension
    constexpr int kQBytes = kKB * kBlk;
    constexpr int kKVBytes = kKB * kBlk;   // one K (or V) tile
    constexpr int kPBytes = (kKV / kBK) * kBlk;
    constexpr int kHalf = HD / 2;          // output columns each softmax group finishes in the merge
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const size_t ldq = static_cast<size_t>(Hq) * HD;
    const int n_mt = (Tq + kQ - 1) / kQ;
    const int delta = Tk - Tq;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* q_s = base;
    uint8_t* k_s = q_s + kQBytes;             // 2 stages
    uint8_t* v_s = k_s + 2 * kKVBytes;        // 2 stages
    uint8_t* p_s = v_s + 2 * kKVBytes;        // 2 buffers
    uint64_t* bars = reinterpret_cast<uint64_t*>(p_s + 2 * kPBytes);
    float* xml = reinterpret_cast<float*>(p_s + 2 * kPBytes + kBarBytes);   // [group][m | l][row]
    if (xml + 4 * kQ > reinterpret_cast<float*>(smem_raw + smem_bytes)) {   // the window starts less aligned than assumed
        if (tid == 0) atomicExch(status, WIDE_ERR_CUDA);
        return;
    }
    const uint32_t k_full = smem_u32(bars), k_empty = smem_u32(bars + 2), v_full = smem_u32(bars + 4),
                   v_empty = smem_u32(bars + 6), s_full = smem_u32(bars + 8), s_free = smem_u32(bars + 10),
                   p_ready = smem_u32(bars + 12), pv_full = smem_u32(bars + 14), q_ready = smem_u32(bars + 16),
                   q_free = smem_u32(bars + 17), x_ready = smem_u32(bars + 18), x_done = smem_u32(bars + 20),
                   item_full = smem_u32(bars + 22), item_empty = smem_u32(bars + 24);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 26);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int4* item_slot = reinterpret_cast<volatile int4*>(bars + 28);   // two slots: (m, h, n_valid, NT); m < 0: no more work

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
            mbar_init(x_ready + 8 * i, 128);
            mbar_init(x_done + 8 * i, 128);
            mbar_init(item_full + 8 * i, 1);
            mbar_init(item_empty + 8 * i, 11);   // K, QK, PV threads and the eight softmax warps
        }
        mbar_init(q_ready, 32);
        mbar_init(q_free, 1);
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

    // A reader's view of the work queue: item number il sits in slot il & 1.
    auto read_item = [&](int il, int4& it) -> bool {          // one thread
        const int sl = il & 1;
        if (!mbar_wait(item_full + 8 * sl, (il >> 1) & 1, wait_ns, abort_flag)) return false;
        it.x = item_slot[sl].x, it.y = item_slot[sl].y, it.z = item_slot[sl].z, it.w = item_slot[sl].w;
        mbar_arrive(item_empty + 8 * sl);
        return true;
    };
    auto read_item_warp = [&](int il, int4& it) -> bool {     // a whole warp, one arrival
        const int sl = il & 1;
        if (!mbar_wait_warp(item_full + 8 * sl, (il >> 1) & 1, wait_ns, abort_flag)) return false;
        it.x = item_slot[sl].x, it.y = item_slot[sl].y, it.z = item_slot[sl].z, it.w = item_slot[sl].w;
        __syncwarp();
        if (lane == 0) mbar_arrive(item_empty + 8 * sl);
        return true;
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ Q gather (32 lanes) and K producer (lane 0)
        bool ok = true;
        int n_k = 0;
        for (int il = 0; ok; ++il) {
            int4 it;
            ok = read_item_warp(il, it);
            if (!ok || it.x < 0) break;
            const int m = it.x, h = it.y, n_valid = it.z, NT = it.w;
            // the last S = Q K^T of the previous item has read Q
            if (il > 0 && !mbar_wait_warp(q_free, (il - 1) & 1, wait_ns, abort_flag)) { ok = false; break; }
            const int32_t* rows = perm + static_cast<size_t>(h / hpg) * Tq + m * kQ;
            const int chunk = lane & 7;     // 16-byte chunks: 8 consecutive lanes copy one 128-byte row of a block
#pragma unroll 8
            for (int i = 0; i < kQ / 4; ++i) {
                const int row = (lane >> 3) + 4 * i;
                const int src_row = rows[min(row, n_valid - 1)];
                const uint8_t* src = reinterpret_cast<const uint8_t*>(q + src_row * ldq + static_cast<size_t>(h) * HD) + 16 * chunk;
#pragma unroll
                for (int kb = 0; kb < kKB; ++kb)
                    cp_async_16(smem_u32(q_s + kb * kBlk) + static_cast<uint32_t>(row) * 128u +
                                    ((static_cast<uint32_t>(chunk) ^ static_cast<uint32_t>(row & 7)) << 4),
                                src + kb * 128);
            }
            cp_async_mbar_arrive_noinc(q_ready);
            if (lane == 0) {
                const int hkv = h / (Hq / Hkv);
                for (int t = 0; t < NT; ++t, ++n_k) {
                    const int s = n_k & 1;
                    if (!mbar_wait(k_empty + 8 * s, ((n_k >> 1) & 1) ^ 1u, wait_ns, abort_flag)) { ok = false; break; }
                    mbar_arrive_expect_tx(k_full + 8 * s, kKVBytes);
                    for (int kb = 0; kb < kKB; ++kb)
                        tma_load_2d(smem_u32(k_s + s * kKVBytes + kb * kBlk), &tmK, hkv * HD + kb * kBK, t * kKV, k_full + 8 * s);
                }
            }
            ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
        }
        cp_async_wait_all();
        if (!ok && lane == 0) {
            atomicExch(status, WIDE_ERR_TIMEOUT);
            for (int i = 0; i < 64; ++i) __nanosleep(1000);   // let copies in flight land
        }
    } else if (warp == 10) {
        // ------------------------------------------------------------------ V producer, and the work queue's writer
        int m_top = 0;     // query tiles that hold an active row of some group
        for (int g = lane; g < Hq / hpg; g += 32) m_top = max(m_top, (min(counts[g], Tq) + kQ - 1) / kQ);
        m_top = __reduce_max_sync(0xffffffffu, m_top);
        if (lane == 0) {
            // The work list: query tiles from the last one that holds an active row of any group down
            // to tile 0 (heavy tiles, i.e. late rows with a long key range, first), every head of a
            // tile in turn.  A draw is one atomic add; tiles without an active row of the head's group
            // are skipped.
            const int n_list = m_top * Hq;
            auto resolve = [&](int it) -> int4 {
                while (true) {
                    if (it >= n_list) return make_int4(-1, 0, 0, 0);
                    const int m = m_top - 1 - it / Hq, h = it % Hq, g = h / hpg;
                    // Block-level predicate: sorted positions >= counts[g] are the tokens that skip this head group
                    const int n_valid = max(0, min(kQ, counts[g] - m * kQ));
                    if (n_valid > 0) {
                        // key range: up to the largest active query position of the tile
                        int j_max = Tk;
                        if (causal) j_max = min(Tk, delta + 1 + perm[static_cast<size_t>(g) * Tq + m * kQ + n_valid - 1]);
                        return make_int4(m, h, n_valid, j_max > 0 ? (j_max + kKV - 1) / kKV : 0);
                    }
                    it = atomicAdd(sched, 1);
                }
            };
            auto post = [&](int n, const int4& it) {
                const int sl = n & 1;
                item_slot[sl].x = it.x, item_slot[sl].y = it.y, item_slot[sl].z = it.z, item_slot[sl].w = it.w;
                mbar_arrive(item_full + 8 * sl);
            };
            bool ok = true;
            int n_v = 0;
            int4 cur = resolve(atomicAdd(sched, 1));
            post(0, cur);
            for (int il = 0; ok && cur.x >= 0; ++il) {
                const int hkv = cur.y / (Hq / Hkv), NT = cur.w;
                // The next item is drawn late (the list stays shared out by who is free, not by who asked
                // first) but a few key tiles before the K producer wants it: Q of the next item is
                // gathered and its first scores are computed under the merge of this one.
                const int t_draw = max(NT - 4, 0);
                int4 nxt = make_int4(-1, 0, 0, 0);
                auto draw_and_post = [&]() -> bool {
                    nxt = resolve(atomicAdd(sched, 1));
                    // item il + 1 goes into the slot of item il - 1, which every reader left long ago
                    if (il >= 1 && !mbar_wait(item_empty + 8 * ((il + 1) & 1), ((il - 1) >> 1) & 1, wait_ns, abort_flag)) return false;
                    post(il + 1, nxt);
                    return true;
                };
                if (NT == 0) ok = draw_and_post();
                for (int t = 0; t < NT && ok; ++t, ++n_v) {
                    if (t == t_draw && !draw_and_post()) { ok = false; break; }
                    const int s = n_v & 1;
                    if (!mbar_wait(v_empty + 8 * s, ((n_v >> 1) & 1) ^ 1u, wait_ns, abort_flag)) { ok = false; break; }
                    mbar_arrive_expect_tx(v_full + 8 * s, kKVBytes);
                    for (int kb = 0; kb < kKB; ++kb)
                        tma_load_2d(smem_u32(v_s + s * kKVBytes + kb * kBlk), &tmV, hkv * HD + kb * kBK, t * kKV, v_full + 8 * s);
                }
                if (!ok) break;
                cur = nxt;
            }
            if (!ok) {
                atomicExch(status, WIDE_ERR_TIMEOUT);
                for (int i = 0; i < 64; ++i) __nanosleep(1000);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ UMMA issuer: S = Q K^T
        if (lane == 0) {
            constexpr uint32_t idesc_qk = idesc_bf16(kQ, kKV, false);
            uint64_t qdesc[kKB];
#pragma unroll
            for (int kb = 0; kb < kKB; ++kb) qdesc[kb] = umma_desc_sw128(smem_u32(q_s + kb * kBlk));
            bool ok = true;
            int n_k = 0, c0 = 0, c1 = 0;   // K tiles consumed; scores written into S[0], S[1] so far
            for (int il = 0; ok; ++il) {
                int4 it;
                ok = read_item(il, it);
                if (!ok || it.x < 0) break;
                const int NT = it.w;
                if (!mbar_wait(q_ready, il & 1, wait_ns, abort_flag)) { ok = false; break; }
                fence_proxy_async_smem();  // the Q rows were written through the generic proxy (cp.async)
                // The group of tile t hands S back as soon as its scores are in registers, so the scores of
                // tile t+2 are computed while that group is busy and ahead of the PV of tile t.
                for (int t = 0; t < NT; ++t, ++n_k) {
                    const int b = t & 1, cb = b ? c1 : c0;
                    if (cb > 0 && !mbar_wait(s_free + 8 * b, (cb - 1) & 1, wait_ns, abort_flag)) { ok = false; break; }
                    const int s = n_k & 1;
                    if (!mbar_wait(k_full + 8 * s, (n_k >> 1) & 1, wait_ns, abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint64_t kdesc = umma_desc_sw128(smem_u32(k_s + s * kKVBytes));
#pragma unroll
                    for (int k16 = 0; k16 < HD / 16; ++k16)
                        umma_bf16(tmem_base + b * kKV, qdesc[k16 / 4] + 2 * (k16 % 4),
                                  kdesc + (k16 / 4) * (kBlk >> 4) + 2 * (k16 % 4), idesc_qk, k16 > 0 ? 1u : 0u);
                    umma_commit(k_empty + 8 * s);
                    umma_commit(s_full + 8 * b);
                    if (b) ++c1; else ++c0;
                }
                if (ok) umma_commit(q_free);   // Q may be overwritten once these have completed
            }
            if (!ok) atomicExch(status, WIDE_ERR_TIMEOUT);
        }
    } else if (warp == 11) {
        // ------------------------------------------------------------------ UMMA issuer: O += P V
        if (lane == 0) {
            constexpr uint32_t idesc_pv = idesc_bf16(kQ, HD, true);
            bool ok = true;
            int n_v = 0, c0 = 0, c1 = 0;
            for (int il = 0; ok; ++il) {
                int4 it;
                ok = read_item(il, it);
                if (!ok || it.x < 0) break;
                const int NT = it.w;
                for (int t = 0; t < NT; ++t, ++n_v) {
                    const int b = t & 1, cb = b ? c1 : c0, s = n_v & 1;
                    if (!mbar_wait(v_full + 8 * s, (n_v >> 1) & 1, wait_ns, abort_flag)) { ok = false; break; }
                    // P of the group's first tile is written after the group has read the previous item's O
                    // out of tensor memory, so this wait also says that O[b] may be overwritten
                    if (!mbar_wait(p_ready + 8 * b, cb & 1, wait_ns, abort_flag)) { ok = false; break; }
                    fence_proxy_async_smem();   // P was written through the generic proxy
                    tc_fence_after_sync();
                    const uint64_t pdesc = umma_desc_sw128(smem_u32(p_s + b * kPBytes));
                    const uint64_t vdesc = umma_desc_sw128_mn(smem_u32(v_s + s * kKVBytes), kBlk);
#pragma unroll
                    for (int k16 = 0; k16 < kKV / 16; ++k16)
                        umma_bf16(tmem_base + 256 + b * HD, pdesc + (k16 / 4) * (kBlk >> 4) + 2 * (k16 % 4),
                                  vdesc + k16 * (2048 >> 4), idesc_pv, (t >= 2 || k16 > 0) ? 1u : 0u);
                    umma_commit(v_empty + 8 * s);
                    umma_commit(pv_full + 8 * b);
                    if (b) ++c1; else ++c0;
                }
            }
            if (!ok) atomicExch(status, WIDE_ERR_TIMEOUT);
        }
    } else {
        // ------------------------------------------------------------------ softmax warps (2..9)
        const int st = tid - 64;                     // 0..255
        const int b = (warp - 2) >> 2;               // group: 0 takes the even key tiles, 1 the odd ones; also its S / P / O buffer
        const int quarter = warp & 3;                // TMEM lane quarter this warp may read
        const int r = quarter * 32 + lane;           // row of the tile owned by this thread
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        const uint32_t o_addr = lane_addr + 256 + b * HD;
        constexpr float kRaise = 8.f;                // raise the reference only for a growth above 2^8
        const bool o_32 = (reinterpret_cast<uintptr_t>(o) & 31) == 0;   // rows of o start on 32-byte boundaries
        bool ok = true;

        // Outputs of (token, group) pairs that skip the group: exact zeros, shared out over all CTAs.
        // A group's heads are adjacent columns of o, its skipped tokens the tail of its sorted order.
        {
            // a warp per row, rows dealt round-robin over all softmax warps of the grid
            const int pieces = hpg * HD / 8;
            const int n_warps = static_cast<int>(gridDim.x) * 8;
            const int my_warp = static_cast<int>(blockIdx.x) * 8 + (st >> 5);
            for (int g = 0; g < Hq / hpg; ++g) {
                const int c = min(counts[g], Tq);
                const int32_t* rows_g = perm + static_cast<size_t>(g) * Tq + c;
                const int n = Tq - c;
                for (int i0 = my_warp; i0 < n; i0 += 4 * n_warps) {
                    int row[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) row[u] = i0 + u * n_warps < n ? rows_g[i0 + u * n_warps] : -1;
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (row[u] >= 0) {
                            uint4* dst = reinterpret_cast<uint4*>(o + row[u] * ldq + static_cast<size_t>(g) * hpg * HD);
                            for (int pc = lane; pc < pieces; pc += 32) dst[pc] = make_uint4(0u, 0u, 0u, 0u);
                        }
                }
            }
        }

        int cnt = 0;                                 // key tiles this group has taken so far
        for (int il = 0; ok; ++il) {
            int4 cur;
            if (!read_item_warp(il, cur)) { ok = false; break; }
            if (cur.x < 0) break;
            const int h = cur.y, n_valid = cur.z, NT = cur.w;
            const int pos = perm[static_cast<size_t>(h / hpg) * Tq + cur.x * kQ + min(r, n_valid - 1)];
            const int n_mine = (NT - b + 1) >> 1;
            const int lim = causal ? min(pos + delta, Tk - 1) : Tk - 1;   // last visible key of this row
            float mref = -CUDART_INF_F, lrow = 0.f;      // reference maximum (log2 units, scaled), row sum

            for (int j = 0; j < n_mine && ok; ++j, ++cnt) {
                const int t = b + 2 * j;
                if (!mbar_wait_warp(s_full + 8 * b, cnt & 1, wait_ns, abort_flag)) { ok = false; break; }
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
                if (j > 0) {
                    if (!mbar_wait_warp(pv_full + 8 * b, (cnt - 1) & 1, wait_ns, abort_flag)) { ok = false; break; }
                } else if (il > 0) {
                    // the other group reads O[b] in the previous item's merge: P (hence the next PV into O[b]) waits for it
                    if (!mbar_wait_warp(x_done + 8 * b, (il - 1) & 1, wait_ns, abort_flag)) { ok = false; break; }
                }
                float alpha = 1.f;
                const bool raise = mx > mref + kRaise || (mref == -CUDART_INF_F && mx > mref);
                if (raise) {
                    alpha = fast_exp2(mref - mx);        // 0 when this is the first key the row sees
                    mref = mx;
                }
                if (j > 0 && __any_sync(0xffffffffu, raise)) {
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
            }

            // Merge of the two groups' partial results (the split-key form of the online softmax).  Both
            // accumulators hold row r in tensor-memory lane r, so a thread reads its row of either one:
            // each group finishes half of the output columns from O[0] and O[1] directly, and only
            // (m, l) go through shared memory.
            const bool mine = n_mine > 0, theirs = (NT + b) >> 1 > 0;   // the other group takes (NT - (1 - b) + 1) / 2 tiles
            if (ok) {
                if (mine) ok = mbar_wait_warp(pv_full + 8 * b, (cnt - 1) & 1, wait_ns, abort_flag);
                else if (il > 0) ok = mbar_wait_warp(x_done + 8 * b, (il - 1) & 1, wait_ns, abort_flag);
            }
            xml[(2 * b) * kQ + r] = mref;
            xml[(2 * b + 1) * kQ + r] = lrow;
            mbar_arrive(x_ready + 8 * b);     // this group's O is final, its (m, l) are written
            if (ok) ok = mbar_wait_warp(x_ready + 8 * (1 - b), il & 1, wait_ns, abort_flag);
            tc_fence_after_sync();
            {
                const int keep_c = b == 0 ? 0 : kHalf;
                const float m1 = xml[(2 * (1 - b)) * kQ + r], l1 = xml[(2 * (1 - b) + 1) * kQ + r];
                const float m_all = fmaxf(mref, m1);
                const float m_use = m_all == -CUDART_INF_F ? 0.f : m_all;
                const float a0 = fast_exp2(mref - m_use), a1 = fast_exp2(m1 - m_use);
                const float l_all = lrow * a0 + l1 * a1;
                const float inv = l_all > 0.f ? 1.f / l_all : 0.f;
                const float f0 = a0 * inv, f1 = a1 * inv;
                // normalise and scatter the active rows
                __nv_bfloat16* dst = o + pos * ldq + static_cast<size_t>(h) * HD + keep_c;
#pragma unroll 1
                for (int c0 = 0; c0 < kHalf; c0 += 32) {
                    uint32_t w0[32], w1[32];
                    tmem_ld_32x32(o_addr + keep_c + c0, w0);
                    tmem_ld_32x32(lane_addr + 256 + (1 - b) * HD + keep_c + c0, w1);
                    tmem_ld_wait();
                    // a group without a key tile in this item: its accumulator is stale (any bits), not zero
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        w0[i] = mine ? w0[i] : 0u;
                        w1[i] = theirs ? w1[i] : 0u;
                    }
                    if (ok && r < n_valid) {
#pragma unroll
                        for (int c1 = 0; c1 < 32; c1 += 16) {
                            uint32_t pk[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                pk[e] = pack2(__uint_as_float(w0[c1 + 2 * e]) * f0 + __uint_as_float(w1[c1 + 2 * e]) * f1,
                                              __uint_as_float(w0[c1 + 2 * e + 1]) * f0 + __uint_as_float(w1[c1 + 2 * e + 1]) * f1);
                            if (o_32) {
                                st_global_v8(dst + c0 + c1, pk);       // a whole 32-byte sector per store
                            } else {
                                reinterpret_cast<uint4*>(dst + c0 + c1)[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                                reinterpret_cast<uint4*>(dst + c0 + c1)[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                            }
                        }
                    }
                }
            }
            tc_fence_before_sync();
            mbar_arrive(x_done + 8 * (1 - b));   // the other group's accumulator and (m, l) are its own again
        }
        if (!ok && lane == 0) atomicExch(status, WIDE_ERR_TIMEOUT);
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
    if (tid == 0) {
        // every CTA has drawn its last item by now: the last one to get here zeroes the queue for the next launch
        __threadfence();
        if (atomicAdd(sched + 1, 1) == static_cast<int>(gridDim.x) - 1) {
            sched[0] = 0;
            sched[1] = 0;
            __threadfence();
        }
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
    const int grid = n_main < ctx->sm_count ? n_main : ctx->sm_count;
    WideLaunch l(ctx, s, "attn_prefill");
    attn_kernel<HD><<<grid, kThreads, smem, s>>>(
        tmK, tmV, static_cast<const __nv_bfloat16*>(q), perm, counts, Tq, Tk, Hq, Hkv, hpg, causal,
        scale * 1.4426950408889634f, static_cast<__nv_bfloat16*>(o), ctx->d_status, ctx->d_status + 10, smem, ctx->wait_ns);
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
