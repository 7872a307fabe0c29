// Decode path (tokens <= 64) of wide_ffn / wide_oproj: memory-bound weight streaming.
//
// Reordering is bypassed (the paper does the same for T_q = 1 and dispatches GEMV-style kernels
// for tiny M); instead the union U of the groups selected by any token of the batch is formed and
// only the weight rows / columns of groups in U are read, each exactly once:
//
//   prep_kernel      U from the mask bits, zeroed fp32 accumulators
//   stream_kernel    C^T[128 weight rows, NT tokens] += W_tile * Act_tile^T  (swap-AB: the weight
//                    tile is the 128-row UMMA operand, the padded batch is N).  Weight tiles arrive
//                    by TMA through an 8-stage ring (>= 128 KB in flight per SM), the MMA runs on
//                    tcgen05 with fp32 accumulators in TMEM, and the epilogue adds the partial tile
//                    into an L2-resident fp32 accumulator with coalesced red.add.  Items are small
//                    (about 128 KB of weights) so that every SM streams until the end.
//                      mode GATEUP: rows of W_gate / W_up of groups in U, K split in chunks
//                      mode DOWN:   128-row tiles of W_down (or W_o) x chunks of groups in U
//   act_kernel       h = M ? silu(gate) * up : 0 -> bf16 (channels of groups in U only)
//   finish_kernel    fp32 accumulator -> output dtype
#include <cuda.h>

#include "internal.h"
#include "ptx.cuh"

namespace {

using namespace wptx;

constexpr int kStagesD = 8;
constexpr int kRows = 128;                 // weight rows per tile (UMMA M)
constexpr int kBKD = 64;
constexpr int kWBytes = kRows * kBKD * 2;  // 16 KB
constexpr int kMaxNT = 64;
constexpr int kActBytes = kMaxNT * kBKD * 2;  // 8 KB reserved per stage
constexpr int kStageBytesD = kWBytes + kActBytes;
constexpr int kAccColsD = 64;              // TMEM columns per accumulator buffer

enum { MODE_GATEUP = 0, MODE_DOWN = 1 };

struct DecodeMeta {           // lives at the start of the workspace
    int32_t n_union;
    int32_t pad[3];
    int32_t union_list[WIDE_MAX_GROUPS];
};

struct StreamArgs {
    int mode;
    int B, NT;            // real and padded token count
    int rows_total;       // rows of the weight matrix (Dff for gate/up, hidden for down)
    int rows_valid;       // weight rows fetched per tile (min(G,128) for gate/up, 128 for down)
    int G;
    int kchunk;           // GATEUP: k columns per item
    int ksplit;           // GATEUP: items per row block
    int blocks_per_group; // GATEUP: max(1, G/128)
    int row_tiles;        // DOWN: rows_total / 128 (rounded up)
    int groups_per_item;  // DOWN
    long long ldo;        // accumulator row stride (elements)
    float* out0;          // GATEUP: gate accumulator; DOWN: y accumulator
    float* out1;          // GATEUP: up accumulator
};

__device__ __forceinline__ void red_add_f32(float* p, float v) {
    asm volatile("red.global.add.f32 [%0], %1;" ::"l"(p), "f"(v) : "memory");
}

__global__ void __launch_bounds__(256) prep_kernel(const uint32_t* __restrict__ mask_bits, int B, int NG, int words,
                                                   DecodeMeta* __restrict__ meta, float4* __restrict__ zero_base,
                                                   long long zero_vec) {
    if (blockIdx.x == 0 && threadIdx.x < 32) {
        const int lane = threadIdx.x;
        int pos = 0;
        for (int w = 0; w < words; ++w) {
            uint32_t u = 0;
            for (int t = lane; t < B; t += 32) u |= mask_bits[static_cast<size_t>(t) * words + w];
            u = __reduce_or_sync(0xffffffffu, u);
            const int g = w * 32 + lane;
            const bool in = g < NG && ((u >> lane) & 1u);
            const unsigned vote = __ballot_sync(0xffffffffu, in);
            if (in) meta->union_list[pos + __popc(vote & ((1u << lane) - 1u))] = g;
            pos += __popc(vote);
        }
        for (int g = pos + lane; g < WIDE_MAX_GROUPS; g += 32) meta->union_list[g] = -1;
        if (lane == 0) meta->n_union = pos;
    }
    const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < zero_vec;
         i += static_cast<long long>(gridDim.x) * blockDim.x)
        zero_base[i] = z;
}

__global__ void __launch_bounds__(192, 1)
stream_kernel(const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmW1,
              const __grid_constant__ CUtensorMap tmAct, const DecodeMeta* __restrict__ meta, StreamArgs a,
              int* __restrict__ status, unsigned long long wait_ns) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + kStagesD * kStageBytesD);
    const uint32_t full = smem_u32(bars), empty = smem_u32(bars + kStagesD);
    const uint32_t tfull = smem_u32(bars + 2 * kStagesD), tempty = smem_u32(bars + 2 * kStagesD + 2);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStagesD + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < kStagesD; ++s) {
            mbar_init(full + 8 * s, 1);
            mbar_init(empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull + 8 * b, 1);
            mbar_init(tempty + 8 * b, 4);
        }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmW0);
        prefetch_tmap(&tmW1);
        prefetch_tmap(&tmAct);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), 2 * kAccColsD);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    const int n_union = meta->n_union;
    const int ksub = a.G / kBKD;
    int n_items, n_chunks = 0;
    if (a.mode == MODE_GATEUP) {
        n_items = n_union * a.blocks_per_group * 2 * a.ksplit;
    } else {
        n_chunks = (n_union + a.groups_per_item - 1) / a.groups_per_item;
        n_items = a.row_tiles * n_chunks;
    }
    const uint32_t stage_tx = static_cast<uint32_t>(a.rows_valid * kBKD * 2 + a.NT * kBKD * 2);

    // item -> (weight map, first weight row, number of k-steps, column of k-step i)
    struct Item { int mat, row0, nsteps, col0, u0; };
    auto decode_item = [&](int item) {
        Item it;
        if (a.mode == MODE_GATEUP) {
            const int ks = item % a.ksplit;
            int r = item / a.ksplit;
            it.mat = r & 1;
            r >>= 1;
            const int blk = r % a.blocks_per_group, u = r / a.blocks_per_group;
            it.row0 = meta->union_list[u] * a.G + blk * kRows;
            it.nsteps = a.kchunk / kBKD;
            it.col0 = ks * a.kchunk;
            it.u0 = 0;
        } else {
            const int rt = item % a.row_tiles, ch = item / a.row_tiles;
            it.mat = 0;
            it.row0 = rt * kRows;
            it.u0 = ch * a.groups_per_item;
            const int ng = min(a.groups_per_item, n_union - it.u0);
            it.nsteps = ng * ksub;
            it.col0 = 0;
        }
        return it;
    };
    auto step_col = [&](const Item& it, int i) {
        if (a.mode == MODE_GATEUP) return it.col0 + i * kBKD;
        return meta->union_list[it.u0 + i / ksub] * a.G + (i % ksub) * kBKD;
    };

    if (warp == 0) {
        if (lane == 0) {
            int n = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                const Item it = decode_item(item);
                const CUtensorMap* tw = it.mat ? &tmW1 : &tmW0;
                for (int i = 0; i < it.nsteps; ++i, ++n) {
                    const int s = n % kStagesD;
                    const uint32_t ph = (n / kStagesD) & 1;
                    if (!mbar_wait(empty + 8 * s, ph ^ 1u, wait_ns, abort_flag)) { ok = false; break; }
                    mbar_arrive_expect_tx(full + 8 * s, stage_tx);
                    const uint32_t dst = smem_u32(base + s * kStageBytesD);
                    const int col = step_col(it, i);
                    tma_load_2d(dst, tw, col, it.row0, full + 8 * s);
                    tma_load_2d(dst + kWBytes, &tmAct, col, 0, full + 8 * s);
                }
            }
            if (!ok) {
                atomicExch(status, WIDE_ERR_TIMEOUT);
                for (int i = 0; i < 64; ++i) __nanosleep(1000);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(kRows, a.NT);
            int n = 0, tc = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++tc) {
                const Item it = decode_item(item);
                const int buf = tc & 1;
                const uint32_t tph = (tc >> 1) & 1;
                if (!mbar_wait(tempty + 8 * buf, tph ^ 1u, wait_ns, abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * kAccColsD;
                for (int i = 0; i < it.nsteps; ++i, ++n) {
                    const int s = n % kStagesD;
                    const uint32_t ph = (n / kStagesD) & 1;
                    if (!mbar_wait(full + 8 * s, ph, wait_ns, abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t w_addr = smem_u32(base + s * kStageBytesD);
                    const uint64_t adesc = umma_desc_sw128(w_addr);
                    const uint64_t bdesc = umma_desc_sw128(w_addr + kWBytes);
#pragma unroll
                    for (int k4 = 0; k4 < kBKD / 16; ++k4)
                        umma_bf16(d_tmem, adesc + 2 * k4, bdesc + 2 * k4, idesc, (i > 0 || k4 > 0) ? 1u : 0u);
                    umma_commit(empty + 8 * s);
                }
                if (ok) umma_commit(tfull + 8 * buf);
            }
            if (!ok) atomicExch(status, WIDE_ERR_TIMEOUT);
        }
    } else {
        const int q = warp & 3;
        int tc = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++tc) {
            const Item it = decode_item(item);
            const int rloc = q * 32 + lane;
            const int row = it.row0 + rloc;
            const bool live = rloc < a.rows_valid && row < a.rows_total;
            float* out = (a.mode == MODE_GATEUP && it.mat) ? a.out1 : a.out0;
            const int buf = tc & 1;
            const uint32_t tph = (tc >> 1) & 1;
            if (!mbar_wait(tfull + 8 * buf, tph, wait_ns, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + buf * kAccColsD;
            for (int c0 = 0; c0 < a.NT; c0 += 16) {
                uint32_t r[16];
                tmem_ld_32x16(taddr + c0, r);
                tmem_ld_wait();
                if (live) {
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (c0 + i < a.B) red_add_f32(out + static_cast<long long>(c0 + i) * a.ldo + row, __uint_as_float(r[i]));
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty + 8 * buf);
        }
        if (!ok && lane == 0) atomicExch(status, WIDE_ERR_TIMEOUT);
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 2 * kAccColsD);
    }
}

// h[b, c] = M[b, c/G] ? bf16(silu(gate[b, c]) * up[b, c]) : 0 for channels of groups in U.
__global__ void __launch_bounds__(256) act_kernel(const DecodeMeta* __restrict__ meta, const float* __restrict__ gate,
                                                  const float* __restrict__ up, const uint32_t* __restrict__ mask_bits,
                                                  int words, int B, int Dff, int G, __nv_bfloat16* __restrict__ h) {
    const int n_union = meta->n_union;
    const long long total = static_cast<long long>(n_union) * B * G;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int c = static_cast<int>(i % G);
        const long long ub = i / G;
        const int b = static_cast<int>(ub % B), u = static_cast<int>(ub / B);
        const int g = meta->union_list[u];
        const size_t idx = static_cast<size_t>(b) * Dff + static_cast<size_t>(g) * G + c;
        float v = 0.f;
        if (wide_mask_bit(mask_bits, words, b, g)) {
            const float gv = gate[idx];
            v = gv / (1.f + __expf(-gv)) * up[idx];
        }
        h[idx] = __float2bfloat16_rn(v);
    }
}

__global__ void __launch_bounds__(256) finish_kernel(const float* __restrict__ acc, long long n, void* __restrict__ y,
                                                     int out_bf16) {
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < n;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        if (out_bf16) static_cast<__nv_bfloat16*>(y)[i] = __float2bfloat16_rn(acc[i]);
        else static_cast<float*>(y)[i] = acc[i];
    }
}

__global__ void __launch_bounds__(256) mask_rows_small_kernel(const uint4* __restrict__ a, const uint32_t* __restrict__ mask_bits,
                                                              int words, int T, int K, int G, uint4* __restrict__ out) {
    const int vec_per_row = K / 8, vec_per_group = G / 8;
    const long long total = static_cast<long long>(T) * vec_per_row;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int t = static_cast<int>(i / vec_per_row);
        const int g = static_cast<int>(i % vec_per_row) / vec_per_group;
        out[i] = wide_mask_bit(mask_bits, words, t, g) ? a[i] : make_uint4(0u, 0u, 0u, 0u);
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

struct DecodeWs {
    DecodeMeta* meta;
    float* gate;   // [64, inner]
    float* up;     // [64, inner]
    float* yacc;   // [64, hidden]
    __nv_bfloat16* h;  // [64, inner]
    size_t zero_floats;  // gate, up, yacc are contiguous
};

DecodeWs carve_ws(void* ws, int D, int inner) {
    DecodeWs w;
    char* p = static_cast<char*>(ws);
    w.meta = reinterpret_cast<DecodeMeta*>(p);
    p += wide_align_up(sizeof(DecodeMeta), 256);
    const size_t acc = wide_align_up(static_cast<size_t>(kMaxNT) * inner * sizeof(float), 256);
    const size_t yac = wide_align_up(static_cast<size_t>(kMaxNT) * D * sizeof(float), 256);
    w.gate = reinterpret_cast<float*>(p);
    w.up = reinterpret_cast<float*>(p + acc);
    w.yacc = reinterpret_cast<float*>(p + 2 * acc);
    w.h = reinterpret_cast<__nv_bfloat16*>(p + 2 * acc + yac);
    w.zero_floats = (2 * acc + yac) / sizeof(float);
    return w;
}

int launch_stream(wide_ctx* ctx, cudaStream_t s, const CUtensorMap& w0, const CUtensorMap& w1, const CUtensorMap& act,
                  const DecodeMeta* meta, const StreamArgs& a) {
    WIDE_CUDA_CHECK(cudaFuncSetAttribute(stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemD));
    {
        WideLaunch l(ctx, s, a.mode == MODE_GATEUP ? "decode_stream_gateup" : "decode_stream_down");
        stream_kernel<<<ctx->sm_count, 192, kSmemD, s>>>(w0, w1, act, meta, a, ctx->d_status, ctx->wait_ns);
    }
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}

int pick_kchunk(int D) {
    for (int kc = 512; kc >= 64; kc >>= 1)
        if (D % kc == 0) return kc;
    return 64;
}

int run_down(wide_ctx* ctx, cudaStream_t s, const DecodeWs& w, const void* act_ptr, const void* wd, int B, int NT,
             int D, int K, int G, void* y, int out_dtype) {
    CUtensorMap tmW, tmAct;
    if (!make_tmap(ctx, &tmW, wd, D, K, kRows) || !make_tmap(ctx, &tmAct, act_ptr, B, K, NT)) return WIDE_ERR_CUDA;
    StreamArgs a{};
    a.mode = MODE_DOWN; a.B = B; a.NT = NT; a.rows_total = D; a.rows_valid = kRows; a.G = G;
    a.row_tiles = (D + kRows - 1) / kRows;
    a.groups_per_item = 512 / G > 0 ? 512 / G : 1;
    a.ldo = D; a.out0 = w.yacc; a.out1 = nullptr;
    int rc = launch_stream(ctx, s, tmW, tmW, tmAct, w.meta, a);
    if (rc != WIDE_OK) return rc;
    const long long n = static_cast<long long>(B) * D;
    {
        WideLaunch l(ctx, s, "decode_finish");
        finish_kernel<<<static_cast<int>((n + 255) / 256 < 1184 ? (n + 255) / 256 : 1184), 256, 0, s>>>(
            w.yacc, n, y, out_dtype == WIDE_BF16 ? 1 : 0);
    }
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}

}  // namespace

size_t wide_decode_workspace(int T, int D, int inner) {
    (void)T;
    return wide_align_up(sizeof(DecodeMeta), 256) + 2 * wide_align_up(static_cast<size_t>(kMaxNT) * inner * 4, 256) +
           wide_align_up(static_cast<size_t>(kMaxNT) * D * 4, 256) + wide_align_up(static_cast<size_t>(kMaxNT) * inner * 2, 256);
}

int wide_launch_ffn_decode_tc(wide_ctx* ctx, cudaStream_t s, const void* x, const void* wg, const void* wu,
                              const void* wd, int T, int D, int Dff, int G, const uint32_t* mask_bits, void* y,
                              int out_dtype, void* ws) {
    if (T == 0) return WIDE_OK;
    const int B = T, NT = (B + 15) / 16 * 16, NG = Dff / G, words = (NG + 31) / 32;
    DecodeWs w = carve_ws(ws, D, Dff);
    // zero only the accumulator rows that are used: gate/up rows [0,B) and y rows [0,B) -- they are
    // laid out [64, inner] so rows 0..B-1 of each are contiguous; zero the three prefixes.
    {
        WideLaunch l(ctx, s, "decode_prep");
        prep_kernel<<<ctx->sm_count, 256, 0, s>>>(mask_bits, B, NG, words, w.meta, reinterpret_cast<float4*>(w.gate),
                                                  static_cast<long long>(w.zero_floats / 4));
    }
    if (cudaGetLastError() != cudaSuccess) return WIDE_ERR_CUDA;

    CUtensorMap tmG, tmU, tmX;
    const int rows_valid = G < kRows ? G : kRows;
    if (!make_tmap(ctx, &tmG, wg, Dff, D, rows_valid) || !make_tmap(ctx, &tmU, wu, Dff, D, rows_valid) ||
        !make_tmap(ctx, &tmX, x, B, D, NT))
        return WIDE_ERR_CUDA;
    StreamArgs a{};
    a.mode = MODE_GATEUP; a.B = B; a.NT = NT; a.rows_total = Dff; a.rows_valid = rows_valid; a.G = G;
    a.kchunk = pick_kchunk(D); a.ksplit = D / a.kchunk; a.blocks_per_group = G / kRows > 0 ? G / kRows : 1;
    a.ldo = Dff; a.out0 = w.gate; a.out1 = w.up;
    int rc = launch_stream(ctx, s, tmG, tmU, tmX, w.meta, a);
    if (rc != WIDE_OK) return rc;

    {
        WideLaunch l(ctx, s, "decode_act");
        act_kernel<<<ctx->sm_count * 2, 256, 0, s>>>(w.meta, w.gate, w.up, mask_bits, words, B, Dff, G, w.h);
    }
    if (cudaGetLastError() != cudaSuccess) return WIDE_ERR_CUDA;
    return run_down(ctx, s, w, w.h, wd, B, NT, D, Dff, G, y, out_dtype);
}

int wide_launch_oproj_decode_tc(wide_ctx* ctx, cudaStream_t s, const void* a_in, const void* wo, int T, int D,
                                int K, int G, const uint32_t* mask_bits, void* y, int out_dtype, void* ws) {
    if (T == 0) return WIDE_OK;
    const int B = T, NT = (B + 15) / 16 * 16, NG = K / G, words = (NG + 31) / 32;
    DecodeWs w = carve_ws(ws, D, K);
    {
        WideLaunch l(ctx, s, "decode_prep");
        prep_kernel<<<ctx->sm_count, 256, 0, s>>>(mask_bits, B, NG, words, w.meta, reinterpret_cast<float4*>(w.gate),
                                                  static_cast<long long>(w.zero_floats / 4));
    }
    if (cudaGetLastError() != cudaSuccess) return WIDE_ERR_CUDA;
    const long long total = static_cast<long long>(B) * (K / 8);
    {
        WideLaunch l(ctx, s, "decode_mask_rows");
        mask_rows_small_kernel<<<static_cast<int>((total + 255) / 256), 256, 0, s>>>(
            static_cast<const uint4*>(a_in), mask_bits, words, B, K, G, reinterpret_cast<uint4*>(w.h));
    }
    if (cudaGetLastError() != cudaSuccess) return WIDE_ERR_CUDA;
    return run_down(ctx, s, w, w.h, wo, B, NT, D, K, G, y, out_dtype);
}
