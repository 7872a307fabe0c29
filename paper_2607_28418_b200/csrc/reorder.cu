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

// One CTA per group: pass 1 counts the active rows, pass 2 places every row.
__global__ void __launch_bounds__(kPartThreads) partition_kernel(const uint32_t* __restrict__ mask_bits, int T,
                                                                 int NG, int words, int32_t* __restrict__ perm,
                                                                 int32_t* counts, int tile_m, int n_tiles,
                                                                 uint8_t* __restrict__ tile_map,
                                                                 int32_t* __restrict__ work_list,
                                                                 int32_t* __restrict__ n_work,
                                                                 int32_t* __restrict__ union_list,
                                                                 int32_t* __restrict__ n_union,
                                                                 int32_t* __restrict__ offsets, int* ticket) {
    __shared__ int warp_cnt[kPartThreads / 32];
    __shared__ int s_total;
    __shared__ int s_last;
    const int g = blockIdx.x;
    const int w = g >> 5, b = g & 31;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int nwarps = kPartThreads / 32;

    int local = 0;
    for (int t = tid; t < T; t += kPartThreads) local += (mask_bits[static_cast<size_t>(t) * words + w] >> b) & 1u;
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

    int32_t* out = perm + static_cast<size_t>(g) * T;
    int base = 0;  // active rows before this chunk
    for (int t0 = 0; t0 < T; t0 += kPartThreads) {
        const int t = t0 + tid;
        const unsigned bit = (t < T) ? ((mask_bits[static_cast<size_t>(t) * words + w] >> b) & 1u) : 0u;
        const unsigned vote = __ballot_sync(0xffffffffu, bit);
        __syncthreads();  // warp_cnt from the previous round has been consumed
        if (lane == 0) warp_cnt[warp] = __popc(vote);
        __syncthreads();
        int before = 0, chunk = 0;
        for (int i = 0; i < nwarps; ++i) {
            const int c = warp_cnt[i];
            before += (i < warp) ? c : 0;
            chunk += c;
        }
        const int rank = base + before + __popc(vote & ((1u << lane) - 1u));  // active rows before t
        if (t < T) {
            if (bit) out[rank] = t;
            else out[total + (t - rank)] = t;
        }
        base += chunk;
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
    if (tid == 0) {
        int woff = 0, uoff = 0, roff = 0;
        for (int g = 0; g < NG; ++g) {
            s_work_off[g] = woff;
            s_union_pos[g] = uoff;
            offsets[g] = roff;
            woff += s_tiles[g];
            uoff += __ldcg(counts + g) > 0 ? 1 : 0;
            roff += s_tiles[g] * tile_m;
        }
        s_work_off[NG] = woff;
        s_union_pos[NG] = uoff;
        offsets[NG] = roff;
        *n_work = woff;
        *n_union = uoff;
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

}  // namespace

int wide_launch_reorder(wide_ctx* ctx, cudaStream_t s, const uint32_t* mask_bits, int T, int NG,
                        int tile_m, int32_t* perm, int32_t* counts, uint8_t* tile_map,
                        int32_t* work_list, int32_t* n_work, int32_t* union_list, int32_t* n_union,
                        int32_t* offsets) {
    const int words = (NG + 31) / 32;
    const int n_tiles = (T + tile_m - 1) / tile_m;
    WideLaunch l(ctx, s, "reorder_partition");
    partition_kernel<<<NG, kPartThreads, 0, s>>>(mask_bits, T, NG, words, perm, counts, tile_m, n_tiles, tile_map,
                                                 work_list, n_work, union_list, n_union, offsets, ctx->d_status + 1);
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
