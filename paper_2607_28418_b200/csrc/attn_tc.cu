// Head-group-masked FlashAttention prefill on tcgen05 (Algorithm 4): query-tile admission through
// the reordered mask, gathered Q rows, dense K/V tiles streamed by TMA, online softmax, scatter
// epilogue.
//
// A work item is one (query head h, tile m of 128 rows of the head's routing group g in that group's
// sorted order).  Tiles past the group's active count are no items at all (block-level predicate);
// the rows of a tile are gathered through perm[g] (row-level predicate: rows past the count are
// computed on a clamped copy and dropped in the epilogue).  Per key tile t of 128 keys:
//     S  = Q K_t^T                (UMMA, both operands in shared memory, fp32 in TMEM)
//     P  = exp2(S*c - m), row statistics m, l   (softmax warps)
//     O += P V_t                  (UMMA with P read from TENSOR MEMORY as the A operand, V_t used as
//                                  TMA loaded it, as an MN-major B operand; fp32 in TMEM)
// Two groups of four softmax warps share every key tile: group 0 takes its keys 0..63, group 1 its
// keys 64..127, a thread per (row, half).  Each group keeps its own (m, l) per row and its own
// accumulator: the PV of a tile is eight UMMAs, four into O[0] from the first 64 keys and four into
// O[1] from the others, so no group ever needs the other's row maximum (the split-key form of the
// online softmax, split inside the tile), and the two partial results are merged once at the end of
// the item, each group finishing half of the output columns from both accumulators (row r is
// tensor-memory lane r in either).  A thread's half row of scores comes into registers with one
// TMEM round trip and S is handed back at once, so the scores of tile t+1 are computed while the
// groups work on tile t; P goes back to tensor memory as 32 columns of bf16 pairs per group (two
// buffers, so the PV of tile t runs under the softmax of tile t+1).  P never touches shared
// memory: what the tensor core reads from it per key tile is Q, K and V (96 KB instead of 128 KB) and
// nothing is written to it but the TMA loads.  A row's reference maximum m is only raised when the
// running maximum has grown by more than 2^8 since it was set (P then stays below 2^8, harmless in
// bf16 / fp32); raising it rescales that group's rows of O in TMEM (load, multiply, store), rare
// after the first tiles.  The two kinds of UMMA have an issuing thread each, K and V a producer
// each.  Causal attention shortens the key range to the largest active query position of the tile
// (+ delta = T_k - T_q); only half tiles that straddle a row's limit evaluate element-wise predicates.
// TMEM: S 128 columns, P 2 x 64, O 2 x head_dim.
//
// The grid is one CTA per SM, and a CTA works through items until the list is empty: every ring,
// barrier phase and tensor-memory buffer carries over from one item to the next.  A CTA's first
// item is its own number in the list (heavy items, i.e. late rows with a long key range, first);
// the others are drawn with an atomic add, a few key tiles before they are needed, by the V
// producer, which passes them to the other roles through a two-slot queue in shared memory.  The
// K producer's warp gathers the next item's Q rows as soon as the last QK^T of the current item has
// read Q, so the next item's first scores are computed under the current item's last key tiles
// and merge: what an item costs beyond its key tiles is the merge alone.  (With one CTA per item
// the prologue, the pipeline fill and the merge of every item ran with the tensor core idle: 27 %
// of the kernel.)  The first item's Q rows are gathered by the softmax warps, which have nothing
// else to do until its scores exist.
//
// Outputs of inactive (token, group) pairs are exact zeros, written by the softmax warps once their
// CTA has no item left, in blocks of 32 rows drawn from a second counter: the CTAs that finish
// first write most of them.  Every mbarrier wait is bounded, and nothing else blocks: the softmax
// groups meet through mbarriers, not named barriers, so an expired wait anywhere lets every role
// run to the kernel's end.  (Every mbarrier is initialised exactly once: a second mbarrier.init on
// a live barrier is undefined and, on this part, ends the launch with an error.)
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
constexpr int kSt = 2;         // K and V stages (three measured no faster); P lives in tensor memory, so shared memory holds Q and the two rings
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

// Packed fp32 pairs (two lanes of a 64-bit register): one instruction does two multiply-adds / adds,
// which halves the instruction count, and the code size, of the softmax arithmetic.
__device__ __forceinline__ uint64_t pack2f(float lo, float hi) {
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
    return d;
}
__device__ __forceinline__ void unpack2f(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// O += P V with P (the A operand) read from tensor memory: 16 keys of a row are 8 columns of packed bf16 pairs.
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tmem_st_32x32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
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
    // Q, kSt K stages, kSt V stages, barriers, (m, l) exchange, alignment slack
    return (HD / kBK) * kBlk + 2 * kSt * (HD / kBK) * kBlk + kBarBytes + kXmlBytes + 512;
}

// q [T_q, H_q*HD], o likewise; K/V come through the tensor maps ([T_k, H_kv*HD], box 64 x 128).
// sched[0]: the next work item (heavy tiles first, after the one every CTA starts with), sched[1]: CTAs that
// have finished, sched[2]: the next block of rows to zero; all zero between launches (the last CTA to
// finish puts them back).
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
    constexpr int kHalf = HD / 2;          // output columns each softmax group finishes in the merge
    constexpr int kHalfKV = kKV / 2;       // keys of a tile each softmax group takes
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const size_t ldq = static_cast<size_t>(Hq) * HD;
    const int delta = Tk - Tq;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* q_s = base;
    uint8_t* k_s = q_s + kQBytes;             // kSt stages
    uint8_t* v_s = k_s + kSt * kKVBytes;      // kSt stages
    uint64_t* bars = reinterpret_cast<uint64_t*>(v_s + kSt * kKVBytes);
    float* xml = reinterpret_cast<float*>(v_s + kSt * kKVBytes + kBarBytes);   // [group][m | l][row]
    if (xml + 4 * kQ > reinterpret_cast<float*>(smem_raw + smem_bytes)) {   // the window starts less aligned than assumed
        if (tid == 0) atomicExch(status, WIDE_ERR_CUDA);
        return;
    }
    const uint32_t k_full = smem_u32(bars), k_empty = smem_u32(bars + 3), v_full = smem_u32(bars + 6),
                   v_empty = smem_u32(bars + 9), s_full = smem_u32(bars + 12), s_free = smem_u32(bars + 13),
                   p_ready = smem_u32(bars + 14), pv_full = smem_u32(bars + 16), q_ready = smem_u32(bars + 18),
                   q_free = smem_u32(bars + 19), q_ready0 = smem_u32(bars + 20), x_ready = smem_u32(bars + 21),
                   x_done = smem_u32(bars + 23), item_full = smem_u32(bars + 25), item_empty = smem_u32(bars + 27);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 29);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int4* item_slot = reinterpret_cast<volatile int4*>(bars + 30);   // two slots: (m, h, n_valid, NT); m < 0: no more work

    if (tid == 0) {
        for (int i = 0; i < kSt; ++i) {
            mbar_init(k_full + 8 * i, 1);
            mbar_init(k_empty + 8 * i, 1);
            mbar_init(v_full + 8 * i, 1);
            mbar_init(v_empty + 8 * i, 1);
        }
        mbar_init(s_full, 1);
        mbar_init(s_free, 256);
        for (int i = 0; i < 2; ++i) {
            mbar_init(p_ready + 8 * i, 256);
            mbar_init(pv_full + 8 * i, 1);
            mbar_init(x_ready + 8 * i, 128);
            mbar_init(x_done + 8 * i, 128);
            mbar_init(item_full + 8 * i, 1);
            mbar_init(item_empty + 8 * i, 11);   // K, QK, PV threads and the eight softmax warps
        }
        mbar_init(q_ready, 32);
        mbar_init(q_ready0, 256);   // the first item's Q rows are gathered by the softmax warps, idle until its scores
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
            for (int i = 0; i < (il > 0 ? kQ / 4 : 0); ++i) {
                const int row = (lane >> 3) + 4 * i;
                const int src_row = rows[min(row, n_valid - 1)];
                const uint8_t* src = reinterpret_cast<const uint8_t*>(q + src_row * ldq + static_cast<size_t>(h) * HD) + 16 * chunk;
#pragma unroll
                for (int kb = 0; kb < kKB; ++kb)
                    cp_async_16(smem_u32(q_s + kb * kBlk) + static_cast<uint32_t>(row) * 128u +
                                    ((static_cast<uint32_t>(chunk) ^ static_cast<uint32_t>(row & 7)) << 4),
                                src + kb * 128);
            }
            if (il > 0) cp_async_mbar_arrive_noinc(q_ready);
            if (lane == 0) {
                const int hkv = h / (Hq / Hkv);
                for (int t = 0; t < NT; ++t, ++n_k) {
                    const int s = n_k % kSt;
                    if (!mbar_wait(k_empty + 8 * s, ((n_k / kSt) & 1) ^ 1u, wait_ns, abort_flag)) { ok = false; break; }
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
                    it = atomicAdd(sched, 1) + static_cast<int>(gridDim.x);
                }
            };
            auto post = [&](int n, const int4& it) {
                const int sl = n & 1;
                item_slot[sl].x = it.x, item_slot[sl].y = it.y, item_slot[sl].z = it.z, item_slot[sl].w = it.w;
                mbar_arrive(item_full + 8 * sl);
            };
            bool ok = true;
            int n_v = 0;
            // the first item of a CTA is its own number in the list: no draw, the counter counts from gridDim.x on
            int4 cur = resolve(static_cast<int>(blockIdx.x));
            post(0, cur);
            for (int il = 0; ok && cur.x >= 0; ++il) {
                const int hkv = cur.y / (Hq / Hkv), NT = cur.w;
                // The next item is drawn late (the list stays shared out by who is free, not by who asked
                // first) but a few key tiles before the K producer wants it: Q of the next item is
                // gathered and its first scores are computed under the merge of this one.
                const int t_draw = max(NT - 4, 0);
                int4 nxt = make_int4(-1, 0, 0, 0);
                auto draw_and_post = [&]() -> bool {
                    nxt = resolve(atomicAdd(sched, 1) + static_cast<int>(gridDim.x));
                    // item il + 1 goes into the slot of item il - 1, which every reader left long ago
                    if (il >= 1 && !mbar_wait(item_empty + 8 * ((il + 1) & 1), ((il - 1) >> 1) & 1, wait_ns, abort_flag)) return false;
                    post(il + 1, nxt);
                    return true;
                };
                if (NT == 0) ok = draw_and_post();
                for (int t = 0; t < NT && ok; ++t, ++n_v) {
                    if (t == t_draw && !draw_and_post()) { ok = false; break; }
                    const int s = n_v % kSt;
                    if (!mbar_wait(v_empty + 8 * s, ((n_v / kSt) & 1) ^ 1u, wait_ns, abort_flag)) { ok = false; break; }
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
            int n_k = 0;   // key tiles so far, over all items: K stage n_k % kSt
            for (int il = 0; ok; ++il) {
                int4 it;
                ok = read_item(il, it);
                if (!ok || it.x < 0) break;
                const int NT = it.w;
                if (!(il == 0 ? mbar_wait(q_ready0, 0, wait_ns, abort_flag) : mbar_wait(q_ready, (il - 1) & 1, wait_ns, abort_flag))) { ok = false; break; }
                fence_proxy_async_smem();  // the Q rows were written through the generic proxy (cp.async)
                // The softmax warps hand S back as soon as the scores are in registers, so the scores of
                // tile t+1 are computed while they work on tile t.
                for (int t = 0; t < NT; ++t, ++n_k) {
                    const int s = n_k % kSt;
                    // one S buffer: the softmax warps have the previous tile's scores in registers
                    if (n_k >= 1 && !mbar_wait(s_free, (n_k - 1) & 1, wait_ns, abort_flag)) { ok = false; break; }
                    if (!mbar_wait(k_full + 8 * s, (n_k / kSt) & 1, wait_ns, abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint64_t kdesc = umma_desc_sw128(smem_u32(k_s + s * kKVBytes));
#pragma unroll
                    for (int k16 = 0; k16 < HD / 16; ++k16)
                        umma_bf16(tmem_base, qdesc[k16 / 4] + 2 * (k16 % 4),
                                  kdesc + (k16 / 4) * (kBlk >> 4) + 2 * (k16 % 4), idesc_qk, k16 > 0 ? 1u : 0u);
                    umma_commit(k_empty + 8 * s);
                    umma_commit(s_full);
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
            int n_v = 0;   // key tiles so far, over all items: V stage n_v % kSt, P buffer n_v & 1
            for (int il = 0; ok; ++il) {
                int4 it;
                ok = read_item(il, it);
                if (!ok || it.x < 0) break;
                const int NT = it.w;
                for (int t = 0; t < NT; ++t, ++n_v) {
                    const int s = n_v % kSt, pb = n_v & 1;
                    if (!mbar_wait(v_full + 8 * s, (n_v / kSt) & 1, wait_ns, abort_flag)) { ok = false; break; }
                    // P of an item's first tile is written after every softmax thread has read the previous
                    // item's O out of tensor memory, so this wait also says that O may be overwritten
                    if (!mbar_wait(p_ready + 8 * pb, (n_v >> 1) & 1, wait_ns, abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint64_t vdesc = umma_desc_sw128_mn(smem_u32(v_s + s * kKVBytes), kBlk);
                    // keys 0..63 of the tile go to O[0], keys 64..127 to O[1] (the softmax group of each half
                    // keeps its own reference maximum)
#pragma unroll
                    for (int k16 = 0; k16 < kKV / 16; ++k16)
                        umma_bf16_ts(tmem_base + 256 + (k16 / 4) * HD, tmem_base + kKV + pb * (kKV / 2) + k16 * 8,
                                     vdesc + k16 * (2048 >> 4), idesc_pv, (t > 0 || (k16 % 4) > 0) ? 1u : 0u);
                    umma_commit(v_empty + 8 * s);
                    umma_commit(pv_full + 8 * pb);
                }
            }
            if (!ok) atomicExch(status, WIDE_ERR_TIMEOUT);
        }
    } else {
        // ------------------------------------------------------------------ softmax warps (2..9)
        const int st = tid - 64;                     // 0..255
        const int b = (warp - 2) >> 2;               // group: 0 takes keys 0..63 of every tile, 1 keys 64..127; also its accumulator O[b]
        const int quarter = warp & 3;                // TMEM lane quarter this warp may read
        const int r = quarter * 32 + lane;           // row of the tile owned by this thread
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        const uint32_t o_addr = lane_addr + 256 + b * HD;
        constexpr float kRaise = 8.f;                // raise the reference only for a growth above 2^8
        const bool o_32 = (reinterpret_cast<uintptr_t>(o) & 31) == 0;   // rows of o start on 32-byte boundaries
        bool ok = true;

        int cnt = 0;                                 // key tiles so far, over all items
        for (int il = 0; ok; ++il) {
            int4 cur;
            if (!read_item_warp(il, cur)) { ok = false; break; }
            if (cur.x < 0) break;
            const int h = cur.y, n_valid = cur.z, NT = cur.w;
            if (il == 0) {
                // Q rows of the CTA's first item: 16-byte chunks, 8 consecutive threads copy one 128-byte row of a block
                const int32_t* rows = perm + static_cast<size_t>(h / hpg) * Tq + cur.x * kQ;
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
                cp_async_mbar_arrive_noinc(q_ready0);
            }
            const int pos = perm[static_cast<size_t>(h / hpg) * Tq + cur.x * kQ + min(r, n_valid - 1)];
            const int lim = causal ? min(pos + delta, Tk - 1) : Tk - 1;   // last visible key of this row
            float mref = -CUDART_INF_F, lrow = 0.f;      // reference maximum (log2 units, scaled), row sum of this half

            for (int t = 0; t < NT && ok; ++t, ++cnt) {
                const int sb = cnt & 1;                   // P buffer of this tile
                if (!mbar_wait_warp(s_full, cnt & 1, wait_ns, abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                const int j0 = t * kKV + kHalfKV * b;     // first key of this thread's half of the tile
                const bool edge = j0 + kHalfKV - 1 > lim; // this row needs element-wise predicates here
                // The half row comes into registers with one TMEM round trip, and S is handed back to the
                // UMMA warp before any arithmetic: the next tile's scores are computed meanwhile.
                uint32_t v[kHalfKV];
#pragma unroll
                for (int c0 = 0; c0 < kHalfKV; c0 += 32)
                    tmem_ld_32x32(lane_addr + kHalfKV * b + c0, reinterpret_cast<uint32_t(&)[32]>(v[c0]));
                tmem_ld_wait();
                tc_fence_before_sync();
                mbar_arrive(s_free);
                // row maximum of the raw scores (the scale is positive)
                float mx4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
                if (edge) {
#pragma unroll
                    for (int i = 0; i < kHalfKV; ++i)
                        if (j0 + i > lim) v[i] = 0xff800000u;   // -inf: exp2 gives an exact zero below
                }
#pragma unroll
                for (int i = 0; i < kHalfKV; i += 8) {
                    mx4[0] = max3(mx4[0], __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
                    mx4[1] = max3(mx4[1], __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
                    mx4[2] = max3(mx4[2], __uint_as_float(v[i + 4]), __uint_as_float(v[i + 5]));
                    mx4[3] = max3(mx4[3], __uint_as_float(v[i + 6]), __uint_as_float(v[i + 7]));
                }
                const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * scale_log2e;
                // the PV that read this P buffer last (two tiles ago) has to be complete before P is overwritten
                if (cnt >= 2 && !mbar_wait_warp(pv_full + 8 * sb, ((cnt >> 1) - 1) & 1, wait_ns, abort_flag)) { ok = false; break; }
                float alpha = 1.f;
                const bool raise = mx > mref + kRaise || (mref == -CUDART_INF_F && mx > mref);
                if (raise) {
                    alpha = fast_exp2(mref - mx);        // 0 when this is the first key the row sees
                    mref = mx;
                }
                if (t > 0 && __any_sync(0xffffffffu, raise)) {
                    // O[b] holds this item's sums up to the previous tile, whose PV has to be complete
                    if (!mbar_wait_warp(pv_full + 8 * (sb ^ 1), ((cnt - 1) >> 1) & 1, wait_ns, abort_flag)) { ok = false; break; }
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
                // P = exp2(S*c - m) as bf16 into the operand layout (this half is one 64-key block), row sum
                uint64_t rs2[2] = {0ull, 0ull};              // four partial row sums, packed in pairs
                const uint64_t sc2 = pack2f(scale_log2e, scale_log2e), nm2 = pack2f(-m_use, -m_use);
                uint32_t pw[kHalfKV / 2];                    // this half row of P, bf16 pairs
                // sixteen scores at a time, each step over all sixteen before the next (arguments, then
                // exponentials, then sums and packing): the steps of one score depend on each other, so
                // score-by-score code runs at the sum of the instruction latencies
#pragma unroll
                for (int c0 = 0; c0 < kHalfKV; c0 += 16) {
                    float x[16];
#pragma unroll
                    for (int i = 0; i < 16; i += 2)
                        unpack2f(fma2(pack2f(__uint_as_float(v[c0 + i]), __uint_as_float(v[c0 + i + 1])), sc2, nm2), x[i], x[i + 1]);
#pragma unroll
                    for (int i = 0; i < 16; ++i) x[i] = fast_exp2(x[i]);
#pragma unroll
                    for (int i = 0; i < 16; i += 4) {
                        rs2[0] = add2(rs2[0], pack2f(x[i], x[i + 1]));
                        rs2[1] = add2(rs2[1], pack2f(x[i + 2], x[i + 3]));
                    }
#pragma unroll
                    for (int i = 0; i < 8; ++i) pw[c0 / 2 + i] = pack2(x[2 * i], x[2 * i + 1]);
                }
                // P goes to tensor memory (columns 128.. : two buffers of 64 columns, this group's 32 of them)
                tmem_st_32x32(lane_addr + kKV + sb * (kKV / 2) + (kHalfKV / 2) * b, pw);
                tmem_st_wait();
                float rs4[4];
                unpack2f(rs2[0], rs4[0], rs4[1]);
                unpack2f(rs2[1], rs4[2], rs4[3]);
                lrow = fmaf(lrow, alpha, (rs4[0] + rs4[1]) + (rs4[2] + rs4[3]));
                tc_fence_before_sync();
                mbar_arrive(p_ready + 8 * sb);
            }

            // Merge of the two groups' partial results (the split-key form of the online softmax).  Both
            // accumulators hold row r in tensor-memory lane r, so a thread reads its row of either one:
            // each group finishes half of the output columns from O[0] and O[1] directly, and only
            // (m, l) go through shared memory.
            const bool any = NT > 0;   // an item without a visible key: both accumulators are stale
            if (ok && NT > 0) ok = mbar_wait_warp(pv_full + 8 * ((cnt - 1) & 1), ((cnt - 1) >> 1) & 1, wait_ns, abort_flag);   // the last PV
            // the other group has read this group's (m, l) of the previous item
            if (ok && il > 0) ok = mbar_wait_warp(x_done + 8 * b, (il - 1) & 1, wait_ns, abort_flag);
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
                    // an item without a visible key issued no PV: the accumulators hold stale bits, not zeros
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        w0[i] = any ? w0[i] : 0u;
                        w1[i] = any ? w1[i] : 0u;
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
        cp_async_wait_all();
        // Outputs of (token, group) pairs that skip the group: exact zeros.  A group's heads are adjacent
        // columns of o, its skipped tokens the tail of its sorted order.  Blocks of 32 rows are drawn from a
        // second counter once a CTA has no item left, so the CTAs that run out of items first write most of them.
        if (ok) {
            const int n_groups = Hq / hpg, pieces = hpg * HD / 8;
            const int n_blocks = n_groups * ((Tq + 31) / 32);
            while (true) {
                int c = 0;
                if (lane == 0) c = atomicAdd(sched + 2, 1);
                c = __shfl_sync(0xffffffffu, c, 0);
                if (c >= n_blocks) break;
                const int g = c % n_groups, first = min(counts[g], Tq) + (c / n_groups) * 32;
                if (first >= Tq) continue;
                const int my_row = first + lane < Tq ? perm[static_cast<size_t>(g) * Tq + first + lane] : -1;
                for (int u = 0; u < 32; ++u) {
                    const int row = __shfl_sync(0xffffffffu, my_row, u);
                    if (row < 0) break;
                    uint4* dst = reinterpret_cast<uint4*>(o + row * ldq + static_cast<size_t>(g) * hpg * HD);
                    for (int pc = lane; pc < pieces; pc += 32) dst[pc] = make_uint4(0u, 0u, 0u, 0u);
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
    if (tid == 0) {
        // every CTA has drawn its last item by now: the last one to get here zeroes the queue for the next launch
        __threadfence();
        if (atomicAdd(sched + 1, 1) == static_cast<int>(gridDim.x) - 1) {
            sched[0] = 0;
            sched[1] = 0;
            sched[2] = 0;
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
