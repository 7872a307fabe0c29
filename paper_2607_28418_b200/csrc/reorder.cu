// wide_reorder: per-group stable partition of the routing mask (Eq. 6 / Algorithm 1) and the
// CTA-level predicate of Eq. 7-8, built with warp ballots and prefix sums -- no sort, no host
// read-back.  wide_unpermute: the scatter epilogue of Algorithm 2 as a standalone kernel.
#include "internal.h"

namespace {

constexpr int kPartThreads = 512;

__device__ void build_metadata(const int32_t* counts, int NG, int tile_m, int n_tiles, uint8_t* __restrict__ tile_map,
                               int32_t* __restrict__ work_list, int32_t* __restrict__ n_work,
                               int32_t* __restrict__ union_list, int32_t* __restrict__ n_union,
                               int32_t* __restrict__ offsets);

// Token clustering key, 8 bits.  Up to 32 groups: the decisions for groups 0..7 themselves, so that
// in sorted order a tile of tokens agrees on the leading decisions and the groups it agrees to skip
// drop out of the tile's K loop even when every token has a mask of its own.  More groups: the top
// byte of an FNV-1a style hash over the token's mask words (only equal masks can then share a tile
// on purpose).  Tokens with the same mask get the same key either way.
__device__ __forceinline__ unsigned mask_key(const uint32_t* __restrict__ row, int words, int NG) {
    if (NG <= 32) return row[0] & 0xFFu;
    uint32_t h = 0x811C9DC5u;
    for (int w = 0; w < words; ++w) h = (h ^ row[w]) * 0x01000193u;
    return h >> 24;
}

// Run by one whole CTA (kPartThreads threads): stable counting sort of the tokens by mask_key.
// order[p] = token at clustered position p, rank[t] = position of token t.  Tokens that share a
// mask end up next to each other, so token tiles taken in this order use few groups when the
// router's decisions cluster.
__device__ void cluster_tokens(const uint32_t* __restrict__ mask_bits, int T, int words, int NG, int32_t* __restrict__ order,
                               int32_t* __restrict__ rank) {
    constexpr int nwarps = kPartThreads / 32;
    __shared__ unsigned s_next[256];                // next free position of every bucket
    __shared__ unsigned short s_wcnt[nwarps][256];  // per-warp bucket counts of the current chunk
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid < 256) s_next[tid] = 0u;
    __syncthreads();
    for (int t = tid; t < T; t += kPartThreads) atomicAdd(&s_next[mask_key(mask_bits + static_cast<size_t>(t) * words, words, NG)], 1u);
    __syncthreads();
    if (warp == 0) {
        // exclusive prefix over the 256 buckets: 8 per lane
        unsigned v[8], sum = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) { v[i] = s_next[lane * 8 + i]; sum += v[i]; }
        unsigned incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned u = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += u;
        }
        unsigned run = incl - sum;
#pragma unroll
        for (int i = 0; i < 8; ++i) { s_next[lane * 8 + i] = run; run += v[i]; }
    }
    __syncthreads();
    for (int c0 = 0; c0 < T; c0 += kPartThreads) {
        const int t = c0 + tid;
        const unsigned key = t < T ? mask_key(mask_bits + static_cast<size_t>(t) * words, words, NG) : 0xFFFFFFFFu;
        for (int i = tid; i < nwarps * 256; i += kPartThreads) (&s_wcnt[0][0])[i] = 0;
        __syncthreads();
        const unsigned peers = __match_any_sync(0xffffffffu, key);
        const int in_warp = __popc(peers & ((1u << lane) - 1u));
        if (t < T && in_warp == 0) s_wcnt[warp][key] = static_cast<unsigned short>(__popc(peers));
        __syncthreads();
        if (t < T) {
            unsigned pos = s_next[key] + in_warp;
            for (int w = 0; w < warp; ++w) pos += s_wcnt[w][key];
            order[pos] = t;
            rank[t] = static_cast<int32_t>(pos);
        }
        __syncthreads();
        if (tid < 256) {
            unsigned add = 0;
#pragma unroll
            for (int w = 0; w < nwarps; ++w) add += s_wcnt[w][tid];
            s_next[tid] += add;
        }
        __syncthreads();
    }
}

// One CTA per group.  Every thread owns kPerThread consecutive tokens of a chunk, so a token's
// rank among the active rows is (active rows in earlier chunks) + (exclusive prefix over threads)
// + (bits below it in the thread's own nibble): one warp scan and one 16-entry block scan per
// chunk.  The group's total is needed before the inactive rows can be placed, so the counting
// sweep runs first (its loads stay in L1 for the placing sweep).
constexpr int kPerThread = 4;
constexpr int kChunk = kPartThreads * kPerThread;

__device__ __forceinline__ unsigned load_nibble(const uint32_t* __restrict__ mask_bits, int words, int w, int b,
                                                int t0, int T) {
    unsigned nib = 0;
#pragma unroll
    for (int i = 0; i < kPerThread; ++i) {
        const int t = t0 + i;
        if (t < T) nib |= ((mask_bits[static_cast<size_t>(t) * words + w] >> b) & 1u) << i;
    }
    return nib;
}

__global__ void __launch_bounds__(kPartThreads) partition_kernel(const uint32_t* __restrict__ mask_bits, int T,
                                                                 int NG, int words, int32_t* __restrict__ perm,
                                                                 int32_t* counts, int tile_m, int n_tiles,
                                                                 uint8_t* __restrict__ tile_map,
                                                                 int32_t* __restrict__ work_list,
                                                                 int32_t* __restrict__ n_work,
                                                                 int32_t* __restrict__ union_list,
                                                                 int32_t* __restrict__ n_union,
                                                                 int32_t* __restrict__ offsets, int* ticket,
                                                                 int32_t* __restrict__ token_order,
                                                                 int32_t* __restrict__ token_rank) {
    __shared__ int warp_cnt[kPartThreads / 32];
    __shared__ int s_total;
    __shared__ int s_last;
    if (static_cast<int>(blockIdx.x) == NG) {  // the extra CTA clusters the tokens
        cluster_tokens(mask_bits, T, words, NG, token_order, token_rank);
        return;
    }
    const int g = blockIdx.x;
    const int w = g >> 5, b = g & 31;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int nwarps = kPartThreads / 32;

    // sweep 1: total number of active rows
    int local = 0;
    for (int c0 = 0; c0 < T; c0 += kChunk) local += __popc(load_nibble(mask_bits, words, w, b, c0 + tid * kPerThread, T));
    local = __reduce_add_sync(0xffffffffu, local);
    if (lane == 0) warp_cnt[warp] = local;
    __syncthreads();
    if (tid == 0) {
        int tot = 0;
        for (int i = 0; i < nwarps; ++i) tot += warp_cnt[i];
        s_total = tot;
        counts[g] = tot;
    }
    __syncthreads();
    const int total = s_total;

    // sweep 2: place every row
    int32_t* out = perm + static_cast<size_t>(g) * T;
    int base = 0;  // active rows in earlier chunks
    for (int c0 = 0; c0 < T; c0 += kChunk) {
        const int t0 = c0 + tid * kPerThread;
        const unsigned nib = load_nibble(mask_bits, words, w, b, t0, T);
        const int mine = __popc(nib);
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        __syncthreads();  // warp_cnt of the previous round (or of sweep 1) has been consumed
        if (lane == 31) warp_cnt[warp] = incl;
        __syncthreads();
        int before = 0, chunk_total = 0;
#pragma unroll
        for (int i = 0; i < nwarps; ++i) {
            const int c = warp_cnt[i];
            before += (i < warp) ? c : 0;
            chunk_total += c;
        }
        int rank = base + before + incl - mine;  // active rows before token t0
#pragma unroll
        for (int i = 0; i < kPerThread; ++i) {
            const int t = t0 + i;
            if (t < T) {
                if ((nib >> i) & 1u) out[rank++] = t;
                else out[total + (t - rank)] = t;
            }
        }
        base += chunk_total;
    }

    // The CTA that finishes last has every group's count in view and builds the rest.
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const int done = atomicAdd(ticket, 1);
        s_last = (done == NG - 1) ? 1 : 0;
        if (s_last) *ticket = 0;  // ready for the next call on this context
    }
    __syncthreads();
    if (s_last) {
        __threadfence();
        build_metadata(counts, NG, tile_m, n_tiles, tile_map, work_list, n_work, union_list, n_union, offsets);
    }
}

// Run by one whole CTA: offsets, tile map, work list, union list.
__device__ void build_metadata(const int32_t* counts, int NG, int tile_m, int n_tiles, uint8_t* __restrict__ tile_map,
                               int32_t* __restrict__ work_list, int32_t* __restrict__ n_work,
                               int32_t* __restrict__ union_list, int32_t* __restrict__ n_union,
                               int32_t* __restrict__ offsets) {
    __shared__ int s_tiles[WIDE_MAX_GROUPS];      // active tiles of each group
    __shared__ int s_work_off[WIDE_MAX_GROUPS + 1];
    __shared__ int s_union_pos[WIDE_MAX_GROUPS + 1];
    const int tid = threadIdx.x;
    for (int g = tid; g < NG; g += blockDim.x) s_tiles[g] = (__ldcg(counts + g) + tile_m - 1) / tile_m;
    __syncthreads();
    if (tid < 32) {
        // exclusive prefix sums over the groups, 32 at a time
        int woff = 0, uoff = 0;
        for (int g0 = 0; g0 < NG; g0 += 32) {
            const int g = g0 + tid;
            const int tv = g < NG ? s_tiles[g] : 0;
            const int uv = (g < NG && __ldcg(counts + g) > 0) ? 1 : 0;
            int tp = tv, up = uv;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int a = __shfl_up_sync(0xffffffffu, tp, o), c = __shfl_up_sync(0xffffffffu, up, o);
                if (tid >= o) { tp += a; up += c; }
            }
            if (g < NG) {
                s_work_off[g] = woff + tp - tv;
                s_union_pos[g] = uoff + up - uv;
                offsets[g] = (woff + tp - tv) * tile_m;
            }
            woff += __shfl_sync(0xffffffffu, tp, 31);
            uoff += __shfl_sync(0xffffffffu, up, 31);
        }
        if (tid == 0) {
            s_work_off[NG] = woff;
            s_union_pos[NG] = uoff;
            offsets[NG] = woff * tile_m;
            *n_work = woff;
            *n_union = uoff;
        }
    }
    __syncthreads();
    const int total_work = s_work_off[NG], total_union = s_union_pos[NG];
    for (int i = tid; i < n_tiles * NG; i += blockDim.x) {
        const int m = i / NG, g = i - m * NG;
        tile_map[i] = (m < s_tiles[g]) ? 1 : 0;
        if (i >= total_work) {
            work_list[2 * i] = -1;
            work_list[2 * i + 1] = -1;
        }
    }
    for (int g = tid; g < NG; g += blockDim.x) {
        const int nt = s_tiles[g], wo = s_work_off[g];
        for (int m = 0; m < nt; ++m) {
            work_list[2 * (wo + m)] = m;
            work_list[2 * (wo + m) + 1] = g;
        }
        if (__ldcg(counts + g) > 0) union_list[s_union_pos[g]] = g;
        if (g >= total_union) union_list[g] = -1;
    }
}

// dst[perm[g][j], g*G:(g+1)*G] = j < counts[g] ? src[offsets[g] + j] : 0, in 16-byte pieces.
// perm is a full permutation per group, so every element of dst is written exactly once.
__global__ void __launch_bounds__(256) unpermute_kernel(const uint4* __restrict__ src, const int32_t* __restrict__ perm,
                                                        const int32_t* __restrict__ counts,
                                                        const int32_t* __restrict__ offsets, int T, int NG,
                                                        int vec_per_group, uint4* __restrict__ dst) {
    const long long total = static_cast<long long>(NG) * T * vec_per_group;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int v = static_cast<int>(i % vec_per_group);
        const long long gj = i / vec_per_group;
        const int j = static_cast<int>(gj % T);
        const int g = static_cast<int>(gj / T);
        const int tok = perm[static_cast<size_t>(g) * T + j];
        uint4 val = make_uint4(0u, 0u, 0u, 0u);
        if (j < counts[g]) val = src[(static_cast<size_t>(offsets[g]) + j) * vec_per_group + v];
        dst[(static_cast<size_t>(tok) * NG + g) * vec_per_group + v] = val;
    }
}

// out[t] = bits [g_begin, g_end) of row t, re-packed from bit 0 (unused high bits 0).
__global__ void __launch_bounds__(256) mask_slice_kernel(const uint32_t* __restrict__ mask_bits, int T, int words_in,
                                                         int g_begin, int g_end, int words_out, uint32_t* __restrict__ out) {
    const long long total = static_cast<long long>(T) * words_out;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int t = static_cast<int>(i / words_out), w = static_cast<int>(i % words_out);
        const int first = g_begin + 32 * w;                 // global index of this word's bit 0
        const uint32_t* row = mask_bits + static_cast<size_t>(t) * words_in;
        const int wi = first >> 5, sh = first & 31;
        uint32_t lo = row[wi] >> sh;
        if (sh != 0 && wi + 1 < words_in) lo |= row[wi + 1] << (32 - sh);
        const int keep = g_end - first;                     // bits of this word inside the range
        if (keep < 32) lo &= (1u << keep) - 1u;
        out[i] = lo;
    }
}

}  // namespace

int wide_launch_mask_slice(wide_ctx* ctx, cudaStream_t s, const uint32_t* mask_bits, int T, int NG, int g_begin, int g_end,
                           uint32_t* out) {
    const int words_out = (g_end - g_begin + 31) / 32;
    const long long total = static_cast<long long>(T) * words_out;
    if (total == 0) return WIDE_OK;
    long long blocks = (total + 255) / 256;
    if (blocks > ctx->sm_count * 8) blocks = ctx->sm_count * 8;
    WideLaunch l(ctx, s, "mask_slice");
    mask_slice_kernel<<<static_cast<int>(blocks), 256, 0, s>>>(mask_bits, T, (NG + 31) / 32, g_begin, g_end, words_out, out);
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}

int wide_launch_reorder(wide_ctx* ctx, cudaStream_t s, const uint32_t* mask_bits, int T, int NG,
                        int tile_m, int32_t* perm, int32_t* counts, uint8_t* tile_map,
                        int32_t* work_list, int32_t* n_work, int32_t* union_list, int32_t* n_union,
                        int32_t* offsets, int32_t* token_order, int32_t* token_rank) {
    const int words = (NG + 31) / 32;
    const int n_tiles = (T + tile_m - 1) / tile_m;
    const int extra = (token_order && token_rank) ? 1 : 0;
    WideLaunch l(ctx, s, "reorder_partition");
    partition_kernel<<<NG + extra, kPartThreads, 0, s>>>(mask_bits, T, NG, words, perm, counts, tile_m, n_tiles,
                                                         tile_map, work_list, n_work, union_list, n_union, offsets,
                                                         ctx->d_status + 1, token_order, token_rank);
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}

int wide_launch_unpermute(wide_ctx* ctx, cudaStream_t s, const void* src, const int32_t* perm, const int32_t* counts,
                          const int32_t* offsets, int T, int NG, int G, int elem_bytes, void* dst) {
    const int vec_per_group = G * elem_bytes / 16;
    const long long total = static_cast<long long>(NG) * T * vec_per_group;
    if (total == 0) return WIDE_OK;
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    WideLaunch l(ctx, s, "unpermute");
    unpermute_kernel<<<static_cast<int>(blocks), 256, 0, s>>>(static_cast<const uint4*>(src), perm, counts, offsets,
                                                              T, NG, vec_per_group, static_cast<uint4*>(dst));
    return cudaGetLastError() == cudaSuccess ? WIDE_OK : WIDE_ERR_CUDA;
}
