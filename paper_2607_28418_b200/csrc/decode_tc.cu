// Decode path (tokens <= 64) of wide_ffn / wide_oproj: memory-bound weight streaming in ONE
// persistent cooperative kernel (one CTA per SM).
//
// Reordering is bypassed (the paper does the same for T_q = 1 and dispatches GEMV-style kernels
// for tiny M); instead every CTA forms the union U of the groups selected by any token of the
// batch, and only the weight rows / columns of groups in U are read, each exactly once.
//
//   pass 1 (FFN)  W_gate / W_up rows of groups in U:  C^T[128 rows, NT tokens] += W_tile * X_tile^T
//                 (swap-AB: the weight tile is the 128-row UMMA operand, the padded batch is N).
//                 The k-steps of all row blocks form one long sequence that is cut into equal,
//                 contiguous shares, one per CTA, so every SM streams the same number of bytes and
//                 a row block is split between at most a few CTAs.  Weight tiles arrive by TMA
//                 through a ring of 8 to 10 stages (>= 128 KB in flight per SM), tcgen05 accumulates in
//                 TMEM, the epilogue adds each partial tile into an L2-resident fp32 accumulator
//                 with 16-byte red.add.  The CTA that adds the last partial of a 128-channel block
//                 (a ticket counter tells) turns it into h = M ? silu(gate) * up : 0 (bf16).
//       (O-proj)  instead: a_masked = M ? attn_out : 0
//   grid barrier  -- while waiting, each CTA has its first two W_down tiles on order (not the whole ring)
//   pass 2        W_down (or W_o): 128-row tiles x the columns of groups in U, same scheme; the CTA
//                 that adds the last partial of a row tile converts it to the output dtype.
//   Clearing the accumulators is nobody's critical path: the epilogue warps clear the output sums
//   at the start of pass 1 and the gate / up sums at the start of pass 2, a share per CTA.
//
// The fp32 accumulators, ticket counters and barrier words belong to the context; counters, barrier
// words and the gate / up sums are zero between calls.  One context must not run two decode calls concurrently.
#include <cuda.h>

#include "internal.h"
#include "ptx.cuh"

namespace {

using namespace wptx;

constexpr int kMaxStagesD = 16;            // ring depth is chosen per launch: as many stages as fit
constexpr int kRows = 128;                 // weight rows per tile (UMMA M)
constexpr int kBKD = 64;
constexpr int kWBytes = kRows * kBKD * 2;  // 16 KB
constexpr int kMaxNT = WIDE_DECODE_MAX_TOKENS;
constexpr int kActBytes = kMaxNT * kBKD * 2;  // 8 KB reserved per stage
constexpr int kRingBytesD = 8 * (kWBytes + kActBytes);  // 192 KB of shared memory for the ring
constexpr int kAccColsD = 64;              // TMEM columns per accumulator buffer
constexpr int kThreadsD = 192;

enum { MODE_GATEUP = 0, MODE_DOWN = 1 };

struct DecodeArgs {
    int is_ffn;
    int B, NT;
    int D, inner, G, NG, words;
    int rows_valid;        // gate/up weight rows fetched per TMA box: min(G, 128)
    int blocks_per_group;  // gate/up: max(1, G / 128)
    int gpb;               // gate/up: union groups per 128-row tile, max(1, 128 / G)
    int row_tiles;         // pass 2: ceil(D / 128)
    const uint32_t* mask_bits;
    const __nv_bfloat16* act_in;  // O-proj: attention output [B, inner]
    float* gate;           // [inner, NT] fp32 (token fastest), zero on entry; cleared again during pass 2
    float* up;
    float* yacc;           // [D, NT], cleared during pass 1 (or the masking phase)
    __nv_bfloat16* h;      // [64, inner] bf16 scratch (caller workspace)
    void* y;
    int out_bf16;
    unsigned* bar;         // grid barrier: arrivals, departures
    unsigned* tickets1;    // one per (union slot, 128-channel block)
    unsigned* tickets2;    // one per output row tile
    int* status;
    unsigned long long wait_ns;
};

struct Pipe {
    uint8_t* base;
    uint32_t full, empty, tfull, tempty;
    volatile int* abort_flag;
    uint32_t tmem_base;
    int n;   // k-steps issued / consumed so far (per role)
    int tc;  // accumulator tiles so far (per role)
    int nstages;       // ring depth
    int stage_bytes;   // 16 KB weight tile + NT x 128 B activation tile
};

// One contiguous piece of a CTA's share: `nsteps` k-steps of work block `blk` starting at step k0.
struct Segment { int blk, k0, nsteps; };

// Share of CTA `cta`: global k-steps [cta*L, min((cta+1)*L, total)), cut at block boundaries.
struct Share {
    int cur, end, spb;
    __device__ Share(int cta, int total, int L, int steps_per_block) : cur(cta * L), end(min((cta + 1) * L, total)), spb(steps_per_block) {
        if (cur > end) cur = end;
    }
    __device__ bool next(Segment& s) {
        if (cur >= end) return false;
        s.blk = cur / spb;
        s.k0 = cur - s.blk * spb;
        s.nsteps = min(spb - s.k0, end - cur);
        cur += s.nsteps;
        return true;
    }
};

// Number of CTAs whose share touches block `blk`.
__device__ __forceinline__ int pieces_of_block(int blk, int spb, int L) {
    const int first = blk * spb, last = first + spb - 1;
    return last / L - first / L + 1;
}

// Gate/up tiles: channel of tile row r of block `slot_blk` (= union slot * blocks_per_group + block,
// or, for groups narrower than a tile, the index of a pack of `gpb` consecutive union slots).
__device__ __forceinline__ int gateup_channel(const DecodeArgs& a, const int* s_union, int n_union, int slot_blk, int r,
                                              bool& valid) {
    if (a.gpb > 1) {
        const int slot = slot_blk * a.gpb + r / a.G;
        valid = slot < n_union;
        return valid ? s_union[slot] * a.G + r % a.G : 0;
    }
    const int ch = s_union[slot_blk / a.blocks_per_group] * a.G + (slot_blk % a.blocks_per_group) * kRows + r;
    valid = r < a.rows_valid && ch < a.inner;
    return ch;
}

__device__ __forceinline__ void red_add_v4(float* p, float a, float b, float c, float d) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ void epilogue_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
// The same barrier of the four epilogue warps, carrying an AND over a flag of every thread: a wait
// that one warp gave up must take all four out of the pass together, or the others would stand at
// the next barrier for good.
__device__ __forceinline__ bool epilogue_bar_and(bool flag) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.and.pred p, 1, 128, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out)
        : "r"(flag ? 1u : 0u)
        : "memory");
    return out != 0;
}

// All CTAs of the (co-resident) grid meet here; used once per launch.  bar[0] counts arrivals
// (a fire-and-forget red after a fence; thread 0 then polls with acquire loads), bar[1] departures:
// the CTA that leaves last puts both back to zero for the next launch, so the kernel can be replayed
// from a CUDA graph without host-side state.  Returns false if the wait expired.
__device__ bool grid_barrier(unsigned* bar, unsigned long long wait_ns, volatile int* abort_flag, int* status) {
    __shared__ int s_passed;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        // arrive without waiting for the counter's old value: one round trip less on the critical path
        asm volatile("red.global.add.u32 [%0], 1;" ::"l"(bar) : "memory");
        bool passed = true;
        if (!*abort_flag) {
            const uint64_t start = globaltimer_ns();
            while (ld_acquire_u32(bar) < gridDim.x) {
                if (globaltimer_ns() - start > wait_ns) {
                    *abort_flag = 1;
                    atomicExch(status, WIDE_ERR_TIMEOUT);
                    passed = false;
                    break;
                }
            }
        } else {
            passed = false;
        }
        s_passed = passed;
    }
    __syncthreads();
    // departures are counted off the critical path, by a thread that has nothing to do for a while
    if (threadIdx.x == kThreadsD - 1 && s_passed && atomicAdd(bar + 1, 1u) + 1u == gridDim.x) {
        bar[0] = 0u;
        bar[1] = 0u;
    }
    return *abort_flag == 0;
}

struct PassGeom {
    int n_blocks, spb, total, L;
};

__device__ __forceinline__ PassGeom geom_of(int mode, const DecodeArgs& a, int n_union) {
    PassGeom g;
    if (mode == MODE_GATEUP) {
        // block index = (slot * bpg + blk) * 2 + mat; groups narrower than a tile share one (gpb per tile)
        g.n_blocks = ((n_union + a.gpb - 1) / a.gpb) * a.blocks_per_group * 2;
        g.spb = a.D / kBKD;
    } else {
        g.n_blocks = a.row_tiles;
        g.spb = n_union * (a.G / kBKD);
    }
    g.total = g.n_blocks * g.spb;
    g.L = (g.total + gridDim.x - 1) / gridDim.x;
    if (g.L < 1) g.L = 1;
    return g;
}

// Producer side of one pass (single thread).  `pre` stages of this pass may already hold their
// weight tile (issued before the grid barrier); for those only the activation tile is loaded.
__device__ bool produce_pass(int mode, const DecodeArgs& a, const CUtensorMap* tmW0, const CUtensorMap* tmW1,
                             const CUtensorMap* tmAct, Pipe& P, const int* s_union, int n_union, int weights_only_steps,
                             int skip_weight_steps) {
    const PassGeom g = geom_of(mode, a, n_union);
    const int ksub = a.G / kBKD;
    const int rows_valid = mode == MODE_GATEUP ? a.rows_valid : kRows;
    const uint32_t act_tx = static_cast<uint32_t>(a.NT * kBKD * 2);
    const uint64_t stream_policy = l2_policy_evict_first();   // weight tiles are read once
    Share sh(blockIdx.x, g.total, g.L, g.spb);
    Segment sg;
    int step = 0;
    int n = P.n;
    while (sh.next(sg)) {
        int row0[2] = {0, 0}, nbox = 1, mat = 0;
        if (mode == MODE_GATEUP) {
            mat = sg.blk & 1;
            const int r = sg.blk >> 1;
            if (a.gpb > 1) {
                nbox = min(a.gpb, n_union - r * a.gpb);     // the last pack may be short
                for (int j = 0; j < nbox; ++j) row0[j] = s_union[r * a.gpb + j] * a.G;
            } else {
                row0[0] = s_union[r / a.blocks_per_group] * a.G + (r % a.blocks_per_group) * kRows;
            }
        } else {
            row0[0] = sg.blk * kRows;
        }
        const uint32_t stage_tx = static_cast<uint32_t>(nbox * rows_valid * kBKD * 2) + act_tx;
        const CUtensorMap* tw = mat ? tmW1 : tmW0;
        for (int i = 0; i < sg.nsteps; ++i, ++step, ++n) {
            if (weights_only_steps >= 0 && step >= weights_only_steps) return true;  // pre-issue done
            const int ks = sg.k0 + i;
            const int col = mode == MODE_GATEUP ? ks * kBKD : s_union[ks / ksub] * a.G + (ks % ksub) * kBKD;
            const int s = n % P.nstages;
            const uint32_t dst = smem_u32(P.base + s * P.stage_bytes);
            if (step >= skip_weight_steps) {
                const uint32_t ph = (n / P.nstages) & 1;
                if (!mbar_wait(P.empty + 8 * s, ph ^ 1u, a.wait_ns, P.abort_flag)) return false;
                mbar_arrive_expect_tx(P.full + 8 * s, stage_tx);
                for (int j = 0; j < nbox; ++j)
                    tma_load_2d_hint(dst + j * rows_valid * (kBKD * 2), tw, col, row0[j], P.full + 8 * s, stream_policy);
            }
            if (weights_only_steps < 0) tma_load_2d(dst + kWBytes, tmAct, col, 0, P.full + 8 * s);
        }
    }
    if (weights_only_steps < 0) P.n = n;
    return true;
}

__device__ bool mma_pass(int mode, const DecodeArgs& a, Pipe& P, int n_union) {
    const PassGeom g = geom_of(mode, a, n_union);
    const uint32_t idesc = umma_idesc_bf16(kRows, a.NT);
    Share sh(blockIdx.x, g.total, g.L, g.spb);
    Segment sg;
    while (sh.next(sg)) {
        const int buf = P.tc & 1;
        const uint32_t tph = (P.tc >> 1) & 1;
        if (!mbar_wait(P.tempty + 8 * buf, tph ^ 1u, a.wait_ns, P.abort_flag)) return false;
        tc_fence_after_sync();
        const uint32_t d_tmem = P.tmem_base + buf * kAccColsD;
        for (int i = 0; i < sg.nsteps; ++i, ++P.n) {
            const int s = P.n % P.nstages;
            const uint32_t ph = (P.n / P.nstages) & 1;
            if (!mbar_wait(P.full + 8 * s, ph, a.wait_ns, P.abort_flag)) return false;
            tc_fence_after_sync();
            const uint32_t w_addr = smem_u32(P.base + s * P.stage_bytes);
            const uint64_t adesc = umma_desc_sw128(w_addr);
            const uint64_t bdesc = umma_desc_sw128(w_addr + kWBytes);
#pragma unroll
            for (int k4 = 0; k4 < kBKD / 16; ++k4)
                umma_bf16(d_tmem, adesc + 2 * k4, bdesc + 2 * k4, idesc, (i > 0 || k4 > 0) ? 1u : 0u);
            umma_commit(P.empty + 8 * s);
        }
        umma_commit(P.tfull + 8 * buf);
        ++P.tc;
    }
    return true;
}

// Epilogue warps (4 warps, 128 threads; thread e = row e of the tile).
__device__ bool epilogue_pass(int mode, const DecodeArgs& a, Pipe& P, const int* s_union, int n_union, int* s_flag,
                              unsigned* s_tokmask) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q = warp & 3;
    const int e = (warp - 2) * 32 + lane;  // 0..127, unique per epilogue thread
    const PassGeom g = geom_of(mode, a, n_union);
    const int nb4 = (a.B + 3) / 4;  // 16-byte pieces of a row that hold real tokens
    {
        // The accumulators of the OTHER pass are idle now: put this CTA's share of them back to zero
        // (pass 1 clears the output sums that pass 2 will add to, pass 2 clears the gate / up sums for
        // the next call; the grid barrier between the passes orders both against their use).
        const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
        if (mode == MODE_GATEUP) {
            float4* p = reinterpret_cast<float4*>(a.yacc);
            const int n = a.D * (a.NT / 4);
            for (int i = blockIdx.x * 128 + e; i < n; i += gridDim.x * 128) p[i] = z;
        } else if (a.is_ffn) {
            float4* pg = reinterpret_cast<float4*>(a.gate);
            float4* pu = reinterpret_cast<float4*>(a.up);
            const int n = a.inner * (a.NT / 4);
            for (int i = blockIdx.x * 128 + e; i < n; i += gridDim.x * 128) { pg[i] = z; pu[i] = z; }
        }
    }
    {
        // Warm L2 with the accumulator rows this CTA will add to (they may have been evicted since
        // the previous call zeroed them), so the red.adds at the end of the pass hit L2.
        Share pre(blockIdx.x, g.total, g.L, g.spb);
        Segment ps;
        while (pre.next(ps)) {
            int prow;
            float* pbase;
            if (mode == MODE_GATEUP) {
                bool valid;
                prow = gateup_channel(a, s_union, n_union, ps.blk >> 1, e, valid);
                pbase = (ps.blk & 1) ? a.up : a.gate;
                if (!valid) continue;
            } else {
                prow = ps.blk * kRows + e;
                pbase = a.yacc;
                if (prow >= a.D) continue;
            }
            const char* p = reinterpret_cast<const char*>(pbase + static_cast<size_t>(prow) * a.NT);
            for (int off = 0; off < nb4 * 16; off += 128)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(p + off));
        }
    }
    Share sh(blockIdx.x, g.total, g.L, g.spb);
    Segment sg;
    while (sh.next(sg)) {
        int mat = 0, slot_blk = 0;
        const int rloc = q * 32 + lane;
        int row;
        bool live;
        if (mode == MODE_GATEUP) {
            mat = sg.blk & 1;
            slot_blk = sg.blk >> 1;
            row = gateup_channel(a, s_union, n_union, slot_blk, rloc, live);
        } else {
            row = sg.blk * kRows + rloc;
            live = row < a.D;
        }
        float* out = (mode == MODE_GATEUP ? (mat ? a.up : a.gate) : a.yacc) + static_cast<size_t>(row) * a.NT;
        const int buf = P.tc & 1;
        const uint32_t tph = (P.tc >> 1) & 1;
        const bool got = mbar_wait_warp(P.tfull + 8 * buf, tph, a.wait_ns, P.abort_flag);
        if (got) {
            tc_fence_after_sync();
            const uint32_t taddr = P.tmem_base + (static_cast<uint32_t>(q * 32) << 16) + buf * kAccColsD;
            for (int c0 = 0; c0 < a.NT; c0 += 16) {
                uint32_t r[16];
                tmem_ld_32x16(taddr + c0, r);
                tmem_ld_wait();
                if (live) {
#pragma unroll
                    for (int v = 0; v < 4; ++v)
                        if (c0 / 4 + v < nb4)
                            red_add_v4(out + c0 + 4 * v, __uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                       __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(P.tempty + 8 * buf);
            ++P.tc;
        }

        // ticket: has every piece of this block been added?
        __threadfence();
        if (!epilogue_bar_and(got)) return false;
        if (e == 0) {
            unsigned* tk;
            int expected;
            if (mode == MODE_GATEUP) {
                tk = a.tickets1 + slot_blk;
                expected = pieces_of_block(2 * slot_blk, g.spb, g.L) + pieces_of_block(2 * slot_blk + 1, g.spb, g.L);
            } else {
                tk = a.tickets2 + sg.blk;
                expected = pieces_of_block(sg.blk, g.spb, g.L);
            }
            const unsigned done = atomicAdd(tk, 1u) + 1u;
            const int last = done == static_cast<unsigned>(expected);
            if (last) *tk = 0u;
            *s_flag = last;
            __threadfence();
        }
        epilogue_bar_sync();
        if (*s_flag) {
            constexpr int kB4 = 8;  // 16-byte pieces per round: 2 * kB4 loads in flight per thread
            if (mode == MODE_GATEUP) {
                // h[b, ch] for the 128 (or G) channels of this block
                // which tokens execute which group of the tile: thread e looks at token e % 64 for
                // the group of the tile half e / 64 (one group per tile: both halves see the same)
                const int vslot = a.gpb > 1 ? slot_blk * a.gpb + (e >> 6) : slot_blk / a.blocks_per_group;
                const int vg = vslot < n_union ? s_union[vslot] : -1;
                const bool tb = vg >= 0 && (e & 63) < a.B && wide_mask_bit(a.mask_bits, a.words, e & 63, vg);
                const unsigned vote = __ballot_sync(0xffffffffu, tb);
                if (lane == 0) s_tokmask[e >> 5] = vote;
                epilogue_bar_sync();
                bool ch_valid;
                const int ch = gateup_channel(a, s_union, n_union, slot_blk, e, ch_valid);
                const int mh = a.gpb > 1 ? 2 * (e / a.G) : 0;   // the mask words of this thread's group
                const unsigned long long tokmask =
                    static_cast<unsigned long long>(s_tokmask[mh]) | (static_cast<unsigned long long>(s_tokmask[mh + 1]) << 32);
                if (ch_valid) {
                    const float4* gp = reinterpret_cast<const float4*>(a.gate + static_cast<size_t>(ch) * a.NT);
                    const float4* up = reinterpret_cast<const float4*>(a.up + static_cast<size_t>(ch) * a.NT);
                    __nv_bfloat16* hp = a.h + ch;                  // token b of this channel: hp[b * inner]
                    const unsigned long long tm = tokmask;
                    for (int b0 = 0; b0 < nb4; b0 += kB4) {
                        float4 gv[kB4], uv[kB4];
#pragma unroll
                        for (int j = 0; j < kB4; ++j) {
                            if (b0 + j < nb4) {
                                gv[j] = __ldcg(gp + b0 + j);
                                uv[j] = __ldcg(up + b0 + j);
                            }
                        }
#pragma unroll
                        for (int j = 0; j < kB4; ++j) {
                            if (b0 + j < nb4) {
                                // four tokens at a time, no branches: rows of h past the batch (up to
                                // the next multiple of four) are scratch and get zeros (their sums are zero)
                                const float e0 = __expf(-gv[j].x), e1 = __expf(-gv[j].y);
                                const float e2 = __expf(-gv[j].z), e3 = __expf(-gv[j].w);
                                const float r0 = __fdividef(gv[j].x, 1.f + e0) * uv[j].x;
                                const float r1 = __fdividef(gv[j].y, 1.f + e1) * uv[j].y;
                                const float r2 = __fdividef(gv[j].z, 1.f + e2) * uv[j].z;
                                const float r3 = __fdividef(gv[j].w, 1.f + e3) * uv[j].w;
                                const unsigned m4 = static_cast<unsigned>(tm >> (4 * (b0 + j))) & 15u;
                                __nv_bfloat16* hq = hp + static_cast<size_t>(4 * (b0 + j)) * a.inner;
                                hq[0] = __float2bfloat16_rn((m4 & 1u) ? r0 : 0.f);
                                hq[a.inner] = __float2bfloat16_rn((m4 & 2u) ? r1 : 0.f);
                                hq[2 * static_cast<size_t>(a.inner)] = __float2bfloat16_rn((m4 & 4u) ? r2 : 0.f);
                                hq[3 * static_cast<size_t>(a.inner)] = __float2bfloat16_rn((m4 & 8u) ? r3 : 0.f);
                            }
                        }
                    }
                }
            } else {
                const int orow = sg.blk * kRows + e;
                if (orow < a.D) {
                    float4* yp = reinterpret_cast<float4*>(a.yacc + static_cast<size_t>(orow) * a.NT);
                    for (int b0 = 0; b0 < nb4; b0 += kB4) {
                        float4 v[kB4];
#pragma unroll
                        for (int j = 0; j < kB4; ++j)
                            if (b0 + j < nb4) v[j] = __ldcg(yp + b0 + j);
#pragma unroll
                        for (int j = 0; j < kB4; ++j) {
                            if (b0 + j < nb4) {
                                const float vs[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    const int b = 4 * (b0 + j) + i;
                                    if (b < a.B) {
                                        const size_t o = static_cast<size_t>(b) * a.D + orow;
                                        if (a.out_bf16) static_cast<__nv_bfloat16*>(a.y)[o] = __float2bfloat16_rn(vs[i]);
                                        else static_cast<float*>(a.y)[o] = vs[i];
                                    }
                                }
                            }
                        }
                    }
                }
            }
        }
        epilogue_bar_sync();  // s_flag is rewritten by the next segment
    }
    return true;
}

__global__ void __launch_bounds__(kThreadsD, 1)
decode_fused_kernel(const __grid_constant__ CUtensorMap tmG, const __grid_constant__ CUtensorMap tmU,
                    const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmWd,
                    const __grid_constant__ CUtensorMap tmH, const DecodeArgs a) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ int s_union[WIDE_MAX_GROUPS];
    __shared__ int s_nunion;
    __shared__ int s_flag;
    __shared__ unsigned s_tokmask[4];
    // A wait that expired in an earlier kernel leaves the context's counters and sums dirty until
    // wide_status resets them: with the status word set, this call does nothing at all.
    if (*reinterpret_cast<volatile int*>(a.status) != WIDE_OK) return;
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + kRingBytesD);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kMaxStagesD + 4);
    Pipe P;
    P.base = base;
    P.full = smem_u32(bars);
    P.empty = smem_u32(bars + kMaxStagesD);
    P.tfull = smem_u32(bars + 2 * kMaxStagesD);
    P.tempty = smem_u32(bars + 2 * kMaxStagesD + 2);
    P.stage_bytes = kWBytes + a.NT * kBKD * 2;
    P.nstages = min(kMaxStagesD, kRingBytesD / P.stage_bytes);
    P.abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    P.n = 0;
    P.tc = 0;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < P.nstages; ++s) {
            mbar_init(P.full + 8 * s, 1);
            mbar_init(P.empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(P.tfull + 8 * b, 1);
            mbar_init(P.tempty + 8 * b, 4);
        }
        *P.abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmG);
        prefetch_tmap(&tmU);
        prefetch_tmap(&tmX);
        prefetch_tmap(&tmWd);
        prefetch_tmap(&tmH);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), 2 * kAccColsD);
        tmem_relinquish();
    }
    if (warp == 2) {
        // union of the batch's masks, ascending
        int pos = 0;
        for (int w = 0; w < a.words; ++w) {
            uint32_t u = 0;
            for (int t = lane; t < a.B; t += 32) u |= a.mask_bits[static_cast<size_t>(t) * a.words + w];
            u = __reduce_or_sync(0xffffffffu, u);
            const int g = w * 32 + lane;
            const bool in = g < a.NG && ((u >> lane) & 1u);
            const unsigned vote = __ballot_sync(0xffffffffu, in);
            if (in) s_union[pos + __popc(vote & ((1u << lane) - 1u))] = g;
            pos += __popc(vote);
        }
        if (lane == 0) s_nunion = pos;
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    P.tmem_base = *tmem_slot;
    const int n_union = s_nunion;
    const long long gtid = static_cast<long long>(blockIdx.x) * kThreadsD + tid;
    const long long gthreads = static_cast<long long>(gridDim.x) * kThreadsD;

    if (n_union == 0) {
        // nothing is active: the output is exactly zero and no accumulator was touched
        const long long n = static_cast<long long>(a.B) * a.D;
        for (long long i = gtid; i < n; i += gthreads) {
            if (a.out_bf16) static_cast<__nv_bfloat16*>(a.y)[i] = __float2bfloat16_rn(0.f);
            else static_cast<float*>(a.y)[i] = 0.f;
        }
    } else {
        bool ok = true;
        int pre = 0;  // stages of pass 2 whose weight tile was issued before the barrier
        // ---- pass 1
        if (a.is_ffn) {
            if (warp == 0) {
                if (lane == 0) {
                    ok = produce_pass(MODE_GATEUP, a, &tmG, &tmU, &tmX, P, s_union, n_union, -1, 0);
                    if (ok) {
                        // Ask for this CTA's first two W_down tiles while the others finish.  Only two:
                        // the CTAs that finish pass 1 last go through a chain of dependent L2 round
                        // trips (fence, ticket, sums, fence, barrier), and each of those takes about
                        // 3 us while every SM has a full ring of weight tiles on order, about 1 us
                        // when the memory system is quiet.
                        const PassGeom g2 = geom_of(MODE_DOWN, a, n_union);
                        const int mine = max(0, min((static_cast<int>(blockIdx.x) + 1) * g2.L, g2.total) -
                                                    min(static_cast<int>(blockIdx.x) * g2.L, g2.total));
                        pre = min(min(P.nstages, 2), mine);
                        ok = produce_pass(MODE_DOWN, a, &tmWd, &tmWd, &tmH, P, s_union, n_union, pre, 0);
                    }
                }
            } else if (warp == 1) {
                if (lane == 0) ok = mma_pass(MODE_GATEUP, a, P, n_union);
            } else {
                ok = epilogue_pass(MODE_GATEUP, a, P, s_union, n_union, &s_flag, s_tokmask);
            }
        } else {
            const int vec_per_row = a.inner / 8, vec_per_group = a.G / 8;
            const uint4* src = reinterpret_cast<const uint4*>(a.act_in);
            uint4* dst = reinterpret_cast<uint4*>(a.h);
            {
                float4* p = reinterpret_cast<float4*>(a.yacc);   // the output sums, cleared before pass 2 adds to them
                const long long n = static_cast<long long>(a.D) * (a.NT / 4);
                for (long long i = gtid; i < n; i += gthreads) p[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            for (long long i = gtid; i < static_cast<long long>(a.B) * vec_per_row; i += gthreads) {
                const int t = static_cast<int>(i / vec_per_row);
                const int g = static_cast<int>(i % vec_per_row) / vec_per_group;
                dst[i] = wide_mask_bit(a.mask_bits, a.words, t, g) ? src[i] : make_uint4(0u, 0u, 0u, 0u);
            }
        }
        if (!ok && lane == 0) atomicExch(a.status, WIDE_ERR_TIMEOUT);
        grid_barrier(a.bar, a.wait_ns, P.abort_flag, a.status);

        // ---- pass 2
        if (!*P.abort_flag) {
            if (warp == 0) {
                if (lane == 0) {
                    fence_proxy_async_all();  // h was written through the generic proxy by other CTAs
                    ok = produce_pass(MODE_DOWN, a, &tmWd, &tmWd, &tmH, P, s_union, n_union, -1, pre);
                    if (!ok) for (int i = 0; i < 64; ++i) __nanosleep(1000);
                }
            } else if (warp == 1) {
                if (lane == 0) ok = mma_pass(MODE_DOWN, a, P, n_union);
            } else {
                ok = epilogue_pass(MODE_DOWN, a, P, s_union, n_union, &s_flag, s_tokmask);
            }
            if (!ok && lane == 0) atomicExch(a.status, WIDE_ERR_TIMEOUT);
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(P.tmem_base, 2 * kAccColsD);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool make_tmap(const wide_ctx* ctx, CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    if (!ctx->encode_tiled) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(kBKD), box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
               map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kSmemD = kRingBytesD + (2 * kMaxStagesD + 4) * 8 + 16 + 1024;

int launch_decode(wide_ctx* ctx, cudaStream_t s, bool is_ffn, const void* x_or_a, const void* wg, const void* wu,
                  const void* wd, int B, int D, int inner, int G, const uint32_t* mask_bits, void* y, int out_dtype,
                  void* ws) {
    // The output sums sit at a fixed place (they are left as they are after a call and cleared at the
    // start of the next one, whatever its shape); the gate / up sums follow and are zero between calls.
    constexpr size_t kYaccFloats = static_cast<size_t>(kMaxNT) * 16384;
    if (D > 16384 || kYaccFloats + static_cast<size_t>(kMaxNT) * 2 * static_cast<size_t>(inner) > ctx->decode_acc_floats)
        return WIDE_ERR_UNSUPPORTED_SHAPE;
    DecodeArgs a{};
    a.is_ffn = is_ffn ? 1 : 0;
    a.B = B;
    a.NT = (B + 15) / 16 * 16;
    a.D = D;
    a.inner = inner;
    a.G = G;
    a.NG = inner / G;
    a.words = (a.NG + 31) / 32;
    a.rows_valid = G < kRows ? G : kRows;
    a.blocks_per_group = G / kRows > 0 ? G / kRows : 1;
    a.gpb = G < kRows ? kRows / G : 1;
    a.row_tiles = (D + kRows - 1) / kRows;
    a.mask_bits = mask_bits;
    a.act_in = static_cast<const __nv_bfloat16*>(x_or_a);
    a.yacc = ctx->decode_acc;
    a.gate = ctx->decode_acc + kYaccFloats;
    a.up = a.gate + static_cast<size_t>(kMaxNT) * inner;
    a.h = static_cast<__nv_bfloat16*>(ws);
    a.y = y;
    a.out_bf16 = out_dtype == WIDE_BF16 ? 1 : 0;
    a.bar = reinterpret_cast<unsigned*>(ctx->d_status) + 4;
    a.tickets1 = ctx->d_tickets;
    a.tickets2 = ctx->d_tickets + 1024;
    a.status = ctx->d_status;
    a.wait_ns = ctx->wait_ns;

    CUtensorMap tmG, tmU, tmX, tmWd, tmH;
    bool ok = make_tmap(ctx, &tmWd, wd, D, inner, kRows) && make_tmap(ctx, &tmH, a.h, B, inner, a.NT);
    if (is_ffn) {
        ok = ok && make_tmap(ctx, &tmG, wg, inner, D, a.rows_valid) && make_tmap(ctx, &tmU, wu, inner, D, a.rows_valid) &&
             make_tmap(ctx, &tmX, x_or_a, B, D, a.NT);
    } else {
        tmG = tmWd;
        tmU = tmWd;
        tmX = tmH;
    }
    if (!ok) return WIDE_ERR_CUDA;
    WIDE_CUDA_CHECK(cudaFuncSetAttribute(decode_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemD));
    void* params[] = {&tmG, &tmU, &tmX, &tmWd, &tmH, &a};
    WideLaunch l(ctx, s, is_ffn ? "decode_ffn_fused" : "decode_oproj_fused");
    // cooperative: the grid barrier needs every CTA resident (one per SM)
    WIDE_CUDA_CHECK(cudaLaunchCooperativeKernel(reinterpret_cast<void*>(decode_fused_kernel), dim3(ctx->sm_count),
                                                dim3(kThreadsD), params, kSmemD, s));
    return WIDE_OK;
}

}  // namespace

size_t wide_decode_workspace(int T, int D, int inner) {
    (void)T;
    (void)D;
    return wide_align_up(static_cast<size_t>(kMaxNT) * inner * 2, 256);  // h / masked activations, bf16
}

int wide_launch_ffn_decode_tc(wide_ctx* ctx, cudaStream_t s, const void* x, const void* wg, const void* wu,
                              const void* wd, int T, int D, int Dff, int G, const uint32_t* mask_bits, void* y,
                              int out_dtype, void* ws) {
    if (T == 0) return WIDE_OK;
    return launch_decode(ctx, s, true, x, wg, wu, wd, T, D, Dff, G, mask_bits, y, out_dtype, ws);
}

int wide_launch_oproj_decode_tc(wide_ctx* ctx, cudaStream_t s, const void* a_in, const void* wo, int T, int D,
                                int K, int G, const uint32_t* mask_bits, void* y, int out_dtype, void* ws) {
    if (T == 0) return WIDE_OK;
    return launch_decode(ctx, s, false, a_in, nullptr, nullptr, wo, T, D, K, G, mask_bits, y, out_dtype, ws);
}
