// Decode path (tokens <= 64) of wide_ffn / wide_oproj: memory-bound weight streaming in ONE
// persistent cooperative kernel (one CTA per SM).
//
// Reordering is bypassed (the paper does the same for T_q = 1 and dispatches GEMV-style kernels
// for tiny M); instead every CTA forms the union U of the groups selected by any token of the
// batch, and only the weight rows / columns of groups in U are read, each exactly once:
//
//   phase 1 (FFN)   stream W_gate / W_up rows of groups in U:  C^T[128 rows, NT tokens] +=
//                   W_tile * X_tile^T  (swap-AB: the weight tile is the 128-row UMMA operand, the
//                   padded batch is N).  Weight tiles arrive by TMA through an 8-stage ring
//                   (>= 128 KB in flight per SM), tcgen05 accumulates in TMEM, the epilogue adds
//                   the partial tile into an L2-resident fp32 accumulator with coalesced red.add.
//                   Items are ~128 KB of weights (K split), so every SM streams until the end.
//       (O-proj)    instead: a_masked = M ? attn_out : 0
//   grid barrier
//   phase 2 (FFN)   h = M ? silu(gate) * up : 0 -> bf16, accumulators re-zeroed on the way
//   grid barrier
//   phase 3         stream W_down (or W_o): 128-row tiles x chunks of groups in U, same pipeline,
//                   partial tiles added into the fp32 output accumulator
//   grid barrier
//   phase 4         accumulator -> output dtype, accumulator re-zeroed
//
// The fp32 accumulators belong to the context and are zero between calls; a call leaves them zero.
// Grid barriers are counters in the context with bounded spins.  One context must not run two
// decode calls concurrently.
#include <cuda.h>

#include "internal.h"
#include "ptx.cuh"

namespace {

using namespace wptx;

constexpr int kStagesD = 8;
constexpr int kRows = 128;                 // weight rows per tile (UMMA M)
constexpr int kBKD = 64;
constexpr int kWBytes = kRows * kBKD * 2;  // 16 KB
constexpr int kMaxNT = WIDE_DECODE_MAX_TOKENS;
constexpr int kActBytes = kMaxNT * kBKD * 2;  // 8 KB reserved per stage
constexpr int kStageBytesD = kWBytes + kActBytes;
constexpr int kAccColsD = 64;              // TMEM columns per accumulator buffer
constexpr int kThreadsD = 192;

enum { MODE_GATEUP = 0, MODE_DOWN = 1 };

struct DecodeArgs {
    int is_ffn;
    int B, NT;
    int D, inner, G, NG, words;
    int rows_valid;        // gate/up weight rows fetched per tile: min(G, 128)
    int blocks_per_group;  // gate/up: max(1, G / 128)
    int kchunk, ksplit;    // gate/up: k columns per item, items per row block
    int row_tiles;         // down: ceil(D / 128)
    int groups_per_item;   // down
    const uint32_t* mask_bits;
    const __nv_bfloat16* act_in;  // O-proj: attention output [B, inner]
    float* gate;           // [64, inner] fp32, zero on entry and on exit
    float* up;
    float* yacc;           // [64, D]
    __nv_bfloat16* h;      // [64, inner] bf16 scratch (caller workspace)
    void* y;
    int out_bf16;
    unsigned* bar;         // 3 grid-barrier counters
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
};

__device__ __forceinline__ void red_add_f32(float* p, float v) {
    asm volatile("red.global.add.f32 [%0], %1;" ::"l"(p), "f"(v) : "memory");
}
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

// All CTAs of the (co-resident) grid meet here.  Returns false if the wait expired.
__device__ bool grid_barrier(unsigned* counter, unsigned long long wait_ns, volatile int* abort_flag, int* status) {
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(counter, 1u);
        if (!*abort_flag) {
            const uint64_t start = globaltimer_ns();
            while (ld_acquire_u32(counter) < gridDim.x) {
                __nanosleep(32);
                if (globaltimer_ns() - start > wait_ns) {
                    *abort_flag = 1;
                    atomicExch(status, WIDE_ERR_TIMEOUT);
                    break;
                }
            }
        }
        __threadfence();
    }
    __syncthreads();
    return *abort_flag == 0;
}

// One streaming pass.  Every warp calls it; roles: warp 0 TMA producer, warp 1 UMMA issuer,
// warps 2..5 epilogue.  s_union / n_union: groups in U (shared memory).
__device__ void stream_phase(int mode, const DecodeArgs& a, const CUtensorMap* tmW0, const CUtensorMap* tmW1,
                             const CUtensorMap* tmAct, Pipe& P, const int* s_union, int n_union) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ksub = a.G / kBKD;
    int n_items;
    if (mode == MODE_GATEUP) {
        n_items = n_union * a.blocks_per_group * 2 * a.ksplit;
    } else {
        const int n_chunks = (n_union + a.groups_per_item - 1) / a.groups_per_item;
        n_items = a.row_tiles * n_chunks;
    }
    const int rows_valid = mode == MODE_GATEUP ? a.rows_valid : kRows;
    const uint32_t stage_tx = static_cast<uint32_t>(rows_valid * kBKD * 2 + a.NT * kBKD * 2);

    struct Item { int mat, row0, nsteps, col0, u0; };
    auto decode_item = [&](int item) {
        Item it;
        if (mode == MODE_GATEUP) {
            const int ks = item % a.ksplit;
            int r = item / a.ksplit;
            it.mat = r & 1;
            r >>= 1;
            const int blk = r % a.blocks_per_group, u = r / a.blocks_per_group;
            it.row0 = s_union[u] * a.G + blk * kRows;
            it.nsteps = a.kchunk / kBKD;
            it.col0 = ks * a.kchunk;
            it.u0 = 0;
        } else {
            const int rt = item % a.row_tiles, ch = item / a.row_tiles;
            it.mat = 0;
            it.row0 = rt * kRows;
            it.u0 = ch * a.groups_per_item;
            it.nsteps = min(a.groups_per_item, n_union - it.u0) * ksub;
            it.col0 = 0;
        }
        return it;
    };
    auto step_col = [&](const Item& it, int i) {
        if (mode == MODE_GATEUP) return it.col0 + i * kBKD;
        return s_union[it.u0 + i / ksub] * a.G + (i % ksub) * kBKD;
    };

    if (warp == 0) {
        if (lane == 0) {
            fence_proxy_async_all();  // activations written by other CTAs before the last grid barrier
            bool ok = *P.abort_flag == 0;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                const Item it = decode_item(item);
                const CUtensorMap* tw = it.mat ? tmW1 : tmW0;
                for (int i = 0; i < it.nsteps; ++i, ++P.n) {
                    const int s = P.n % kStagesD;
                    const uint32_t ph = (P.n / kStagesD) & 1;
                    if (!mbar_wait(P.empty + 8 * s, ph ^ 1u, a.wait_ns, P.abort_flag)) { ok = false; break; }
                    mbar_arrive_expect_tx(P.full + 8 * s, stage_tx);
                    const uint32_t dst = smem_u32(P.base + s * kStageBytesD);
                    const int col = step_col(it, i);
                    tma_load_2d(dst, tw, col, it.row0, P.full + 8 * s);
                    tma_load_2d(dst + kWBytes, tmAct, col, 0, P.full + 8 * s);
                }
            }
            if (!ok) {
                atomicExch(a.status, WIDE_ERR_TIMEOUT);
                for (int i = 0; i < 64; ++i) __nanosleep(1000);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(kRows, a.NT);
            bool ok = *P.abort_flag == 0;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++P.tc) {
                const Item it = decode_item(item);
                const int buf = P.tc & 1;
                const uint32_t tph = (P.tc >> 1) & 1;
                if (!mbar_wait(P.tempty + 8 * buf, tph ^ 1u, a.wait_ns, P.abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = P.tmem_base + buf * kAccColsD;
                for (int i = 0; i < it.nsteps; ++i, ++P.n) {
                    const int s = P.n % kStagesD;
                    const uint32_t ph = (P.n / kStagesD) & 1;
                    if (!mbar_wait(P.full + 8 * s, ph, a.wait_ns, P.abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t w_addr = smem_u32(P.base + s * kStageBytesD);
                    const uint64_t adesc = umma_desc_sw128(w_addr);
                    const uint64_t bdesc = umma_desc_sw128(w_addr + kWBytes);
#pragma unroll
                    for (int k4 = 0; k4 < kBKD / 16; ++k4)
                        umma_bf16(d_tmem, adesc + 2 * k4, bdesc + 2 * k4, idesc, (i > 0 || k4 > 0) ? 1u : 0u);
                    umma_commit(P.empty + 8 * s);
                }
                if (ok) umma_commit(P.tfull + 8 * buf);
            }
            if (!ok) atomicExch(a.status, WIDE_ERR_TIMEOUT);
        }
    } else {
        const int q = warp & 3;
        bool ok = *P.abort_flag == 0;
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++P.tc) {
            const Item it = decode_item(item);
            const int rloc = q * 32 + lane;
            const int row = it.row0 + rloc;
            const int rows_total = mode == MODE_GATEUP ? a.inner : a.D;
            const bool live = rloc < rows_valid && row < rows_total;
            float* out = mode == MODE_GATEUP ? (it.mat ? a.up : a.gate) : a.yacc;
            const long long ldo = mode == MODE_GATEUP ? a.inner : a.D;
            const int buf = P.tc & 1;
            const uint32_t tph = (P.tc >> 1) & 1;
            if (!mbar_wait(P.tfull + 8 * buf, tph, a.wait_ns, P.abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t taddr = P.tmem_base + (static_cast<uint32_t>(q * 32) << 16) + buf * kAccColsD;
            for (int c0 = 0; c0 < a.NT; c0 += 16) {
                uint32_t r[16];
                tmem_ld_32x16(taddr + c0, r);
                tmem_ld_wait();
                if (live) {
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (c0 + i < a.B) red_add_f32(out + (c0 + i) * ldo + row, __uint_as_float(r[i]));
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(P.tempty + 8 * buf);
        }
        if (!ok && lane == 0) atomicExch(a.status, WIDE_ERR_TIMEOUT);
    }
}

__global__ void __launch_bounds__(kThreadsD, 1)
decode_fused_kernel(const __grid_constant__ CUtensorMap tmG, const __grid_constant__ CUtensorMap tmU,
                    const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmWd,
                    const __grid_constant__ CUtensorMap tmH, const DecodeArgs a) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ int s_union[WIDE_MAX_GROUPS];
    __shared__ int s_nunion;
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + kStagesD * kStageBytesD);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStagesD + 4);
    Pipe P;
    P.base = base;
    P.full = smem_u32(bars);
    P.empty = smem_u32(bars + kStagesD);
    P.tfull = smem_u32(bars + 2 * kStagesD);
    P.tempty = smem_u32(bars + 2 * kStagesD + 2);
    P.abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    P.n = 0;
    P.tc = 0;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < kStagesD; ++s) {
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
        if (blockIdx.x == 0) a.bar[2] = 0u;  // last barrier of the previous call; nobody is near it yet
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

    // ---- phase 1
    if (a.is_ffn) {
        stream_phase(MODE_GATEUP, a, &tmG, &tmU, &tmX, P, s_union, n_union);
    } else {
        const int vec_per_row = a.inner / 8, vec_per_group = a.G / 8;
        const uint4* src = reinterpret_cast<const uint4*>(a.act_in);
        uint4* dst = reinterpret_cast<uint4*>(a.h);
        for (long long i = gtid; i < static_cast<long long>(a.B) * vec_per_row; i += gthreads) {
            const int t = static_cast<int>(i / vec_per_row);
            const int g = static_cast<int>(i % vec_per_row) / vec_per_group;
            dst[i] = wide_mask_bit(a.mask_bits, a.words, t, g) ? src[i] : make_uint4(0u, 0u, 0u, 0u);
        }
    }
    grid_barrier(a.bar + 0, a.wait_ns, P.abort_flag, a.status);

    // ---- phase 2: activation (FFN only); consumes and re-zeroes the gate/up accumulators
    if (a.is_ffn) {
        if (!*P.abort_flag) {
            const int per_group = a.B * a.G;  // elements of one group: b-major, c fastest
            const int total = n_union * per_group;
            for (long long i = gtid; i < total; i += gthreads) {
                const int u = static_cast<int>(i) / per_group;
                const int rem = static_cast<int>(i) - u * per_group;
                const int b = rem / a.G, c = rem - b * a.G;
                const int g = s_union[u];
                const size_t idx = static_cast<size_t>(b) * a.inner + static_cast<size_t>(g) * a.G + c;
                const float gv = __ldcg(a.gate + idx), uv = __ldcg(a.up + idx);
                a.gate[idx] = 0.f;
                a.up[idx] = 0.f;
                const float v = wide_mask_bit(a.mask_bits, a.words, b, g) ? gv / (1.f + __expf(-gv)) * uv : 0.f;
                a.h[idx] = __float2bfloat16_rn(v);
            }
        }
        grid_barrier(a.bar + 1, a.wait_ns, P.abort_flag, a.status);
    }

    // ---- phase 3: down / output projection
    stream_phase(MODE_DOWN, a, &tmWd, &tmWd, &tmH, P, s_union, n_union);
    grid_barrier(a.bar + 2, a.wait_ns, P.abort_flag, a.status);

    // ---- phase 4: write the output, leave the accumulator zero
    if (blockIdx.x == 0 && tid == 0) {
        a.bar[0] = 0u;
        a.bar[1] = 0u;
    }
    if (!*P.abort_flag) {
        const long long n = static_cast<long long>(a.B) * a.D;
        for (long long i = gtid; i < n; i += gthreads) {
            const float v = __ldcg(a.yacc + i);
            a.yacc[i] = 0.f;
            if (a.out_bf16) static_cast<__nv_bfloat16*>(a.y)[i] = __float2bfloat16_rn(v);
            else static_cast<float*>(a.y)[i] = v;
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

constexpr int kSmemD = kStagesD * kStageBytesD + (2 * kStagesD + 4) * 8 + 16 + 1024;

int pick_kchunk(int D) {
    for (int kc = 512; kc >= 64; kc >>= 1)
        if (D % kc == 0) return kc;
    return 64;
}

int launch_decode(wide_ctx* ctx, cudaStream_t s, bool is_ffn, const void* x_or_a, const void* wg, const void* wu,
                  const void* wd, int B, int D, int inner, int G, const uint32_t* mask_bits, void* y, int out_dtype,
                  void* ws) {
    if (static_cast<size_t>(kMaxNT) * (2 * static_cast<size_t>(inner) + D) > ctx->decode_acc_floats)
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
    a.kchunk = pick_kchunk(D);
    a.ksplit = D / a.kchunk;
    a.row_tiles = (D + kRows - 1) / kRows;
    a.groups_per_item = 512 / G > 0 ? 512 / G : 1;
    a.mask_bits = mask_bits;
    a.act_in = static_cast<const __nv_bfloat16*>(x_or_a);
    a.gate = ctx->decode_acc;
    a.up = ctx->decode_acc + static_cast<size_t>(kMaxNT) * inner;
    a.yacc = ctx->decode_acc + 2 * static_cast<size_t>(kMaxNT) * inner;
    a.h = static_cast<__nv_bfloat16*>(ws);
    a.y = y;
    a.out_bf16 = out_dtype == WIDE_BF16 ? 1 : 0;
    a.bar = reinterpret_cast<unsigned*>(ctx->d_status + 4);
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
    // cooperative: the grid barriers need every CTA resident (one per SM)
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
