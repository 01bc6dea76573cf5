// Keep-index sampler (Sec. 3.2.1 index sets; Sec. 4 random and grid-wise masks).
//
// One thread block per sample.  Random mode finds the K-th smallest 64-bit score
// (philox word << 32 | position) with a four-pass, 8-bit radix select over the philox words -
// which are recomputed on every pass, never stored - and then emits the kept positions in
// ascending order with a block-wide prefix sum.  Grid mode evaluates the lattice predicate and
// uses the same ordered compaction; per-sample offsets come from closed-form counts.
#include "sbp_common.cuh"

namespace sbp {
namespace {

constexpr int kSampThreads = 512;
constexpr int kSampWarps = kSampThreads / 32;

struct SampShared {
    uint32_t hist[256];
    uint32_t warp_sums_a[kSampWarps];
    uint32_t warp_sums_b[kSampWarps];
    uint32_t sel_digit;
    uint32_t sel_below;
    uint64_t red64[kSampWarps];
};

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v, int lane) {
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t n = __shfl_up_sync(0xffffffffu, v, d);
        if (lane >= d) v += n;
    }
    return v;
}

// Exclusive prefix over the block of per-thread counts; returns (exclusive prefix, block total).
__device__ __forceinline__ uint2 block_excl_scan(uint32_t v, uint32_t* warp_sums) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t incl = warp_incl_scan(v, lane);
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    uint32_t ws = (lane < kSampWarps) ? warp_sums[lane] : 0u;
    const uint32_t ws_incl = warp_incl_scan(ws, lane);
    const uint32_t total = __shfl_sync(0xffffffffu, ws_incl, kSampWarps - 1);
    const uint32_t warp_base = __shfl_sync(0xffffffffu, ws_incl - ws, warp);
    __syncthreads();
    return make_uint2(warp_base + incl - v, total);
}

// words of the four positions 4q .. 4q+3 of sample gid
__device__ __forceinline__ PhiloxWords position_words(uint32_t q, uint32_t gid, uint32_t step,
                                                      uint32_t k0, uint32_t k1) {
    return philox4x32_10(q, gid, step, 0u, k0, k1);
}

__global__ void __launch_bounds__(kSampThreads)
sample_keep_random_kernel(uint32_t N, uint32_t K, uint32_t k0, uint32_t k1, uint32_t step,
                          uint32_t first_sample, int share_mask,
                          int32_t* __restrict__ keep_rows, int32_t* __restrict__ keep_offsets) {
    __shared__ SampShared sh;
    // the selection looks at every word five times: maps of up to 8192 positions keep their words here
    constexpr uint32_t kCacheGroups = 2048;
    __shared__ uint4 word_cache[kCacheGroups];
    pdl_launch_dependents();
    pdl_wait();                 // earlier kernels of the stream may still be reading the index buffers
    const uint32_t b = blockIdx.x;
    const uint32_t gid = share_mask ? 0u : first_sample + b;
    const uint32_t groups = (N + 3u) >> 2;
    const int64_t row_base = (int64_t)b * N;
    int32_t* out = keep_rows + (int64_t)b * K;
    if (threadIdx.x == 0) {
        keep_offsets[b + 1] = (int32_t)((b + 1) * (int64_t)K);
        if (b == 0) keep_offsets[0] = 0;
    }

    const bool cached = groups <= kCacheGroups && K < N;
    if (cached) {
        for (uint32_t q = threadIdx.x; q < groups; q += kSampThreads) {
            const PhiloxWords pw = position_words(q, gid, step, k0, k1);
            word_cache[q] = make_uint4(pw.w[0], pw.w[1], pw.w[2], pw.w[3]);
        }
        __syncthreads();
    }
    auto words_of = [&](uint32_t q) {
        if (!cached) return position_words(q, gid, step, k0, k1);
        const uint4 v = word_cache[q];
        PhiloxWords pw;
        pw.w[0] = v.x; pw.w[1] = v.y; pw.w[2] = v.z; pw.w[3] = v.w;
        return pw;
    };

    // ---- radix select: threshold word `prefix` and how many positions equal to it are kept ----
    uint32_t prefix = 0, known = 0, remaining = K;
    if (K < N) {
        for (int shift = 24; shift >= 0; shift -= 8) {
            for (int i = threadIdx.x; i < 256; i += kSampThreads) sh.hist[i] = 0;
            __syncthreads();
            for (uint32_t q = threadIdx.x; q < groups; q += kSampThreads) {
                const PhiloxWords pw = words_of(q);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t n = 4u * q + e;
                    if (n < N && (pw.w[e] & known) == prefix) atomicAdd(&sh.hist[(pw.w[e] >> shift) & 0xffu], 1u);
                }
            }
            __syncthreads();
            // exclusive scan over the 256 bins; the bin where the running count crosses `remaining` wins
            const uint32_t cnt = (threadIdx.x < 256) ? sh.hist[threadIdx.x] : 0u;
            const uint2 sc = block_excl_scan(cnt, sh.warp_sums_a);
            if (threadIdx.x < 256 && sc.x < remaining && remaining <= sc.x + cnt) {
                sh.sel_digit = threadIdx.x;
                sh.sel_below = sc.x;
            }
            __syncthreads();
            prefix |= sh.sel_digit << shift;
            known |= 0xffu << shift;
            remaining -= sh.sel_below;
            __syncthreads();
        }
    }
    const bool keep_all = (K >= N);
    const uint32_t threshold = prefix;       // kept: word < threshold, plus the first `remaining` equal to it

    // ---- ordered compaction, kSampThreads*4 positions per sweep ----
    uint32_t eq_seen = 0, written = 0;
    for (uint32_t q0 = 0; q0 < groups; q0 += kSampThreads) {
        const uint32_t q = q0 + threadIdx.x;
        uint32_t lt_mask = 0, eq_mask = 0;
        if (q < groups) {
            if (keep_all) {
#pragma unroll
                for (int e = 0; e < 4; ++e) if (4u * q + e < N) lt_mask |= 1u << e;
            } else {
                const PhiloxWords pw = words_of(q);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (4u * q + e < N) {
                        if (pw.w[e] < threshold) lt_mask |= 1u << e;
                        else if (pw.w[e] == threshold) eq_mask |= 1u << e;
                    }
                }
            }
        }
        uint32_t keep_mask = lt_mask;
        if (!keep_all) {
            const uint2 se = block_excl_scan(__popc(eq_mask), sh.warp_sums_a);
            uint32_t rank = eq_seen + se.x;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (eq_mask & (1u << e)) {
                    if (rank < remaining) keep_mask |= 1u << e;
                    ++rank;
                }
            }
            eq_seen += se.y;
        }
        const uint2 sk = block_excl_scan(__popc(keep_mask), sh.warp_sums_b);
        uint32_t pos = written + sk.x;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (keep_mask & (1u << e)) out[pos++] = (int32_t)(row_base + 4u * q + e);
        }
        written += sk.y;
    }
}

// ---- large maps: one sample spread over a cluster of C thread blocks ----
// Each block owns a contiguous slice of the positions.  The per-pass digit histograms stay in the
// blocks' shared memory and are summed through distributed shared memory, so every block derives
// the same threshold; slice counts exchanged the same way give each block its output offset.
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_load(const uint32_t* local_ptr, uint32_t rank) {
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(local_ptr);
    uint32_t ra, v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(a), "r"(rank));
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(ra) : "memory");
    return v;
}

template <int C>
__global__ void __launch_bounds__(kSampThreads)
sample_keep_random_cluster_kernel(uint32_t N, uint32_t K, uint32_t k0, uint32_t k1, uint32_t step,
                                  uint32_t first_sample, int share_mask, int cache_words,
                                  int32_t* __restrict__ keep_rows, int32_t* __restrict__ keep_offsets) {
    // The selection looks at every word six times (four digit passes, the tie count, the compaction).  When the
    // slice's words fit in shared memory they are generated once and kept there; otherwise each look recomputes them.
    extern __shared__ uint4 word_cache[];
    __shared__ SampShared sh;
    __shared__ uint32_t slice_counts[2];          // positions of this slice below / equal to the threshold
    // Two histograms used alternately: the one a pass clears was last read by the other blocks two passes
    // earlier, before the cluster barrier of the pass in between, so one barrier per pass is enough.
    __shared__ uint32_t hist2[2][256];
    pdl_launch_dependents();
    pdl_wait();
    const uint32_t rank = cluster_rank();
    const uint32_t b = blockIdx.x / C;
    const uint32_t gid = share_mask ? 0u : first_sample + b;
    const uint32_t groups = (N + 3u) >> 2;
    const uint32_t per = (groups + C - 1) / C;
    const uint32_t g_begin = rank * per;
    const uint32_t g_end = (g_begin + per < groups) ? g_begin + per : groups;
    const int64_t row_base = (int64_t)b * N;
    int32_t* out = keep_rows + (int64_t)b * K;
    if (rank == 0 && threadIdx.x == 0) {
        keep_offsets[b + 1] = (int32_t)((b + 1) * (int64_t)K);
        if (b == 0) keep_offsets[0] = 0;
    }

    if (cache_words) {
        for (uint32_t q = g_begin + threadIdx.x; q < g_end; q += kSampThreads) {
            const PhiloxWords pw = position_words(q, gid, step, k0, k1);
            word_cache[q - g_begin] = make_uint4(pw.w[0], pw.w[1], pw.w[2], pw.w[3]);
        }
        __syncthreads();
    }
    auto words_of = [&](uint32_t q) {
        if (!cache_words) return position_words(q, gid, step, k0, k1);
        const uint4 v = word_cache[q - g_begin];
        PhiloxWords pw;
        pw.w[0] = v.x; pw.w[1] = v.y; pw.w[2] = v.z; pw.w[3] = v.w;
        return pw;
    };

    uint32_t prefix = 0, known = 0, remaining = K;
    for (int shift = 24, pass = 0; shift >= 0; shift -= 8, ++pass) {
        uint32_t* hist = hist2[pass & 1];
        for (int i = threadIdx.x; i < 256; i += kSampThreads) hist[i] = 0;
        __syncthreads();
        for (uint32_t q = g_begin + threadIdx.x; q < g_end; q += kSampThreads) {
            const PhiloxWords pw = words_of(q);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const uint32_t n = 4u * q + e;
                if (n < N && (pw.w[e] & known) == prefix) atomicAdd(&hist[(pw.w[e] >> shift) & 0xffu], 1u);
            }
        }
        cluster_sync();                                   // every slice's histogram is complete
        uint32_t cnt = 0;
        if (threadIdx.x < 256)
            for (uint32_t r = 0; r < (uint32_t)C; ++r) cnt += cluster_load(&hist[threadIdx.x], r);
        const uint2 sc = block_excl_scan(cnt, sh.warp_sums_a);
        if (threadIdx.x < 256 && sc.x < remaining && remaining <= sc.x + cnt) {
            sh.sel_digit = threadIdx.x;
            sh.sel_below = sc.x;
        }
        __syncthreads();
        prefix |= sh.sel_digit << shift;
        known |= 0xffu << shift;
        remaining -= sh.sel_below;
        __syncthreads();                                  // sel_digit / sel_below are read before the next pass rewrites them
    }
    const uint32_t threshold = prefix;

    // slice counts -> rank of this slice's first tie and its first output slot
    uint32_t lt = 0, eq = 0;
    for (uint32_t q = g_begin + threadIdx.x; q < g_end; q += kSampThreads) {
        const PhiloxWords pw = words_of(q);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (4u * q + e < N) {
                lt += pw.w[e] < threshold;
                eq += pw.w[e] == threshold;
            }
        }
    }
    const uint32_t lt_total = block_excl_scan(lt, sh.warp_sums_a).y;
    const uint32_t eq_total = block_excl_scan(eq, sh.warp_sums_b).y;
    if (threadIdx.x == 0) { slice_counts[0] = lt_total; slice_counts[1] = eq_total; }
    cluster_sync();
    uint32_t eq_seen = 0, written = 0;
    for (uint32_t r = 0; r < rank; ++r) {
        const uint32_t lt_r = cluster_load(&slice_counts[0], r), eq_r = cluster_load(&slice_counts[1], r);
        const uint32_t room = remaining > eq_seen ? remaining - eq_seen : 0u;
        written += lt_r + (eq_r < room ? eq_r : room);
        eq_seen += eq_r;
    }

    // ordered compaction of this slice
    for (uint32_t q0 = g_begin; q0 < g_end; q0 += kSampThreads) {
        const uint32_t q = q0 + threadIdx.x;
        uint32_t lt_mask = 0, eq_mask = 0;
        if (q < g_end) {
            const PhiloxWords pw = words_of(q);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (4u * q + e < N) {
                    if (pw.w[e] < threshold) lt_mask |= 1u << e;
                    else if (pw.w[e] == threshold) eq_mask |= 1u << e;
                }
            }
        }
        uint32_t keep_mask = lt_mask;
        const uint2 se = block_excl_scan(__popc(eq_mask), sh.warp_sums_a);
        uint32_t tie_rank = eq_seen + se.x;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (eq_mask & (1u << e)) {
                if (tie_rank < remaining) keep_mask |= 1u << e;
                ++tie_rank;
            }
        }
        eq_seen += se.y;
        const uint2 sk = block_excl_scan(__popc(keep_mask), sh.warp_sums_b);
        uint32_t pos = written + sk.x;
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (keep_mask & (1u << e)) out[pos++] = (int32_t)(row_base + 4u * q + e);
        written += sk.y;
    }
    cluster_sync();                                       // the slice counts stay readable until every block is done
}

// ---- grid-wise masks: 2x2-periodic lattice with a per-sample phase ----
__device__ __forceinline__ uint32_t grid_phase(int family, uint32_t gid, uint32_t step, uint32_t k0, uint32_t k1) {
    if (family == 4) return 0u;
    const uint32_t word = philox4x32_10(0u, gid, step, 1u, k0, k1).w[0];
    return family == 2 ? (word & 1u) : (word & 3u);
}

__device__ __forceinline__ uint32_t grid_count(int family, uint32_t p, uint32_t H, uint32_t W) {
    const uint32_t quarter = ((H + 1u - (p >> 1)) >> 1) * ((W + 1u - (p & 1u)) >> 1);
    switch (family) {
        case 1: return quarter;
        case 2: return (H * W + 1u - p) >> 1;
        case 3: return H * W - quarter;
        default: return H * W;
    }
}

__device__ __forceinline__ bool grid_keeps(int family, uint32_t p, uint32_t h, uint32_t w) {
    const bool on_lattice = ((h & 1u) == (p >> 1)) && ((w & 1u) == (p & 1u));
    switch (family) {
        case 1: return on_lattice;
        case 2: return ((h + w) & 1u) == p;
        case 3: return !on_lattice;
        default: return true;
    }
}

__global__ void __launch_bounds__(kSampThreads)
sample_keep_grid_kernel(int family, uint32_t H, uint32_t W, uint32_t k0, uint32_t k1, uint32_t step,
                        uint32_t first_sample, int share_mask,
                        int32_t* __restrict__ keep_rows, int32_t* __restrict__ keep_offsets) {
    __shared__ SampShared sh;
    pdl_launch_dependents();
    pdl_wait();
    const uint32_t b = blockIdx.x;
    const uint32_t N = H * W;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    // offset of this sample = sum of the closed-form counts of the samples before it
    uint64_t before = 0;
    if (share_mask) {
        before = (uint64_t)b * grid_count(family, grid_phase(family, 0u, step, k0, k1), H, W);
    } else {
        uint64_t part = 0;
        for (uint32_t s = threadIdx.x; s < b; s += kSampThreads)
            part += grid_count(family, grid_phase(family, first_sample + s, step, k0, k1), H, W);
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) part += __shfl_xor_sync(0xffffffffu, part, d);
        if (lane == 0) sh.red64[warp] = part;
        __syncthreads();
        for (int i = 0; i < kSampWarps; ++i) before += sh.red64[i];
        __syncthreads();
    }
    const uint32_t gid = share_mask ? 0u : first_sample + b;
    const uint32_t p = grid_phase(family, gid, step, k0, k1);
    const uint32_t mine = grid_count(family, p, H, W);
    if (threadIdx.x == 0) {
        keep_offsets[b + 1] = (int32_t)(before + mine);
        if (b == 0) keep_offsets[0] = 0;
    }
    int32_t* out = keep_rows + before;
    const int64_t row_base = (int64_t)b * N;
    const uint32_t groups = (N + 3u) >> 2;
    uint32_t written = 0;
    for (uint32_t q0 = 0; q0 < groups; q0 += kSampThreads) {
        const uint32_t q = q0 + threadIdx.x;
        uint32_t keep_mask = 0;
        if (q < groups) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const uint32_t n = 4u * q + e;
                if (n < N && grid_keeps(family, p, n / W, n % W)) keep_mask |= 1u << e;
            }
        }
        const uint2 sk = block_excl_scan(__popc(keep_mask), sh.warp_sums_b);
        uint32_t pos = written + sk.x;
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (keep_mask & (1u << e)) out[pos++] = (int32_t)(row_base + 4u * q + e);
        written += sk.y;
    }
}


// ---------------------------------------------------------------------------------------------
// whole-frame masks for video (Sec. 3.1, 3.2.1: a subset of frames): T frames of P positions, the
// K_T frames with the smallest scores (word << 32) | f are kept, each with all of its positions.
// T is small (a clip has tens of frames), so one block ranks the frames by counting.
// ---------------------------------------------------------------------------------------------
constexpr uint32_t kMaxFrames = 2048;

// frames of family `family` (as the spatial grid families: every fourth, every second, all but every fourth, all)
// at phase p among T frames
__device__ __forceinline__ uint32_t frame_count(int family, uint32_t p, uint32_t T) {
    const uint32_t fourth = (T + 3u - p) >> 2;
    switch (family) {
        case 1: return fourth;
        case 2: return (T + 1u - p) >> 1;
        case 3: return T - fourth;
        default: return T;
    }
}
__device__ __forceinline__ bool frame_keeps(int family, uint32_t p, uint32_t f) {
    switch (family) {
        case 1: return (f & 3u) == p;
        case 2: return (f & 1u) == p;
        case 3: return (f & 3u) != p;
        default: return true;
    }
}

// family 0: the K_T frames with the smallest scores; families 1-4: frames on a lattice in time whose phase is
// drawn per sample like the spatial grid phase (counts, and so the offsets, then depend on the phases)
__global__ void __launch_bounds__(kSampThreads)
sample_keep_temporal_kernel(int family, uint32_t T, uint32_t P, uint32_t KT, uint32_t k0, uint32_t k1, uint32_t step,
                            uint32_t first_sample, int share_mask,
                            int32_t* __restrict__ keep_rows, int32_t* __restrict__ keep_offsets) {
    __shared__ unsigned long long score[kMaxFrames];
    __shared__ uint32_t kept[kMaxFrames];        // first a flag per frame, then the ascending list of kept frames
    __shared__ uint32_t list[kMaxFrames];
    pdl_launch_dependents();
    pdl_wait();
    const uint32_t b = blockIdx.x;
    const uint32_t gid = share_mask ? 0u : first_sample + b;
    uint64_t frames_before = (uint64_t)b * KT;                       // kept frames of the samples before this one
    if (family == 0) {
        for (uint32_t f = threadIdx.x; f < T; f += kSampThreads) {
            const uint32_t w = philox4x32_10(f >> 2, gid, step, 0u, k0, k1).w[f & 3u];
            score[f] = ((unsigned long long)w << 32) | f;
        }
        __syncthreads();
        for (uint32_t f = threadIdx.x; f < T; f += kSampThreads) {
            const unsigned long long mine = score[f];
            uint32_t rank = 0;
            for (uint32_t g = 0; g < T; ++g) rank += score[g] < mine;
            kept[f] = rank < KT ? 1u : 0u;
        }
    } else {
        const uint32_t p = grid_phase(family, gid, step, k0, k1);
        for (uint32_t f = threadIdx.x; f < T; f += kSampThreads) kept[f] = frame_keeps(family, p, f) ? 1u : 0u;
        KT = frame_count(family, p, T);
        // the offset of this sample is the sum of the closed-form counts of the samples before it
        if (share_mask) {
            frames_before = (uint64_t)b * KT;
        } else {
            __shared__ unsigned long long red[kSampThreads / 32];
            unsigned long long part = 0;
            for (uint32_t s2 = threadIdx.x; s2 < b; s2 += kSampThreads)
                part += frame_count(family, grid_phase(family, first_sample + s2, step, k0, k1), T);
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) part += __shfl_xor_sync(0xffffffffu, part, d);
            if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = part;
            __syncthreads();
            frames_before = 0;
            for (int i = 0; i < kSampThreads / 32; ++i) frames_before += red[i];
        }
    }
    __syncthreads();
    for (uint32_t f = threadIdx.x; f < T; f += kSampThreads) {
        if (kept[f]) {
            uint32_t pos = 0;
            for (uint32_t g = 0; g < f; ++g) pos += kept[g];
            list[pos] = f;
        }
    }
    __syncthreads();
    const uint64_t per_sample = (uint64_t)KT * P;
    int32_t* out = keep_rows + frames_before * P;
    for (uint64_t e = threadIdx.x; e < per_sample; e += kSampThreads) {
        const uint32_t k = (uint32_t)(e / P), q = (uint32_t)(e - (uint64_t)k * P);
        out[e] = (int32_t)(((uint64_t)b * T + list[k]) * P + q);
    }
    if (threadIdx.x == 0) {
        keep_offsets[b] = (int32_t)(frames_before * P);
        if (b + 1 == gridDim.x) keep_offsets[b + 1] = (int32_t)(frames_before * P + per_sample);
    }
}

}  // namespace

uint32_t sample_keep_max_frames() { return kMaxFrames; }

namespace {
constexpr size_t kClusterCacheMax = 160 * 1024;

template <int C>
cudaError_t launch_cluster_sampler(dim3 grid, dim3 block, size_t cache_bytes, cudaStream_t stream, int64_t N, int64_t K,
                                   uint32_t k0, uint32_t k1, uint32_t step, uint32_t first_sample, bool share_mask,
                                   int32_t* keep_rows, int32_t* keep_offsets) {
    const cudaError_t opt = opt_in_dynamic_smem<sample_keep_random_cluster_kernel<C>>((int)kClusterCacheMax);
    if (opt != cudaSuccess) return opt;
    return launch_pdl_cluster(sample_keep_random_cluster_kernel<C>, grid, block, cache_bytes, C, stream, (uint32_t)N,
                              (uint32_t)K, k0, k1, step, first_sample, share_mask ? 1 : 0, cache_bytes ? 1 : 0, keep_rows,
                              keep_offsets);
}
}  // namespace

cudaError_t launch_sample_keep(int mode, int grid_family, int64_t B, int64_t H, int64_t W, int64_t K,
                               uint64_t seed, uint32_t step, uint32_t first_sample, bool share_mask,
                               int32_t* keep_rows, int32_t* keep_offsets, cudaStream_t stream) {
    const uint32_t k0 = (uint32_t)(seed & 0xffffffffu), k1 = (uint32_t)(seed >> 32);
    const dim3 grid((unsigned)B), block(kSampThreads);
    if (mode == SBP_MASK_RANDOM) {
        const int64_t N = H * W;
        // large maps with few samples: spread each sample over a cluster so that more SMs take part
        int cluster = 1;
        if (K < N && N > 8192 && B * 8 <= 4 * kNumSMs) cluster = N > 32768 ? 8 : (N > 16384 ? 4 : 2);
        const dim3 cgrid((unsigned)(B * cluster));
        // shared-memory cache of the slice's words (16 bytes per group of four positions), when it fits
        const int64_t slice_groups = (((N + 3) / 4) + cluster - 1) / cluster;
        const size_t cache_bytes = (size_t)slice_groups * 16 <= kClusterCacheMax ? (size_t)slice_groups * 16 : 0;
        switch (cluster) {
            case 8: return launch_cluster_sampler<8>(cgrid, block, cache_bytes, stream, N, K, k0, k1, step, first_sample, share_mask, keep_rows, keep_offsets);
            case 4: return launch_cluster_sampler<4>(cgrid, block, cache_bytes, stream, N, K, k0, k1, step, first_sample, share_mask, keep_rows, keep_offsets);
            case 2: return launch_cluster_sampler<2>(cgrid, block, cache_bytes, stream, N, K, k0, k1, step, first_sample, share_mask, keep_rows, keep_offsets);
            default: break;
        }
        return launch_pdl(sample_keep_random_kernel, grid, block, 0, stream, (uint32_t)(H * W), (uint32_t)K, k0, k1,
                          step, first_sample, share_mask ? 1 : 0, keep_rows, keep_offsets);
    }
    if (mode == SBP_MASK_TEMPORAL || mode == SBP_MASK_TEMPORAL_GRID)      // H frames of W positions; K = kept frames x W
        return launch_pdl(sample_keep_temporal_kernel, grid, block, 0, stream, mode == SBP_MASK_TEMPORAL ? 0 : grid_family,
                          (uint32_t)H, (uint32_t)W, (uint32_t)(K / W),
                          k0, k1, step, first_sample, share_mask ? 1 : 0, keep_rows, keep_offsets);
    return launch_pdl(sample_keep_grid_kernel, grid, block, 0, stream, grid_family, (uint32_t)H, (uint32_t)W, k0, k1,
                      step, first_sample, share_mask ? 1 : 0, keep_rows, keep_offsets);
}

}  // namespace sbp
