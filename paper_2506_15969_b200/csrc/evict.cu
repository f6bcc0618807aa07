// Lagged eviction (Section 4 "MRI-Centric Eviction" of the paper):
//   score_fn       -- H1, H2 and Eq. (2), fp64
//   select_kernel  -- top-(B - R - S) of the unprotected slots by (score, recency): block-wide radix
//                     select on the fp64 score bits, then a prefix sum that turns keep flags into the
//                     list "slot src[j] moves to slot j" (Appendix A, Eq. (evic))
//   compact_kernel -- in-place, order-preserving gather of K, V, TS, MRI and positions (Algorithm 1,
//                     "update KV pairs")
#include "internal.h"

namespace lzk {

namespace {

// I_t[i] from the elapsed time d = t - TS[i] and MRI[i].
//   H1 = 2 sigma(-d / MRI)          (MRI = 0: 1 when d = 0, else 0 -- the ratio is +inf)
//   H2 = 2 sigma(-1 / (MRI - 1))    (0 for MRI = 0 by definition and for MRI = 1 as the limit)
//   Eq. (2): H1 + H2 when MRI != 0, H1 alone when MRI = 0.
// 2 sigma(-x) is evaluated as 2 / (1 + exp(x)).
__device__ __forceinline__ double score_fn(int d, int mri, int mode) {
    double h1, h2 = 0.0;
    if (mri == 0) {
        h1 = d == 0 ? 1.0 : 0.0;
    } else {
        h1 = 2.0 / (1.0 + exp((double)d / (double)mri));
        if (mri > 1) h2 = 2.0 / (1.0 + exp(1.0 / ((double)mri - 1.0)));
    }
    if (mode == 1) return h1;
    if (mode == 2) return h2;
    return h1 + h2;
}

constexpr int kSelThreads = 512;

// Exclusive prefix sum of one int per thread over the block; *total gets the block sum.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_sums, int* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += up;
    }
    __syncthreads();                       // warp_sums may still be read from a previous call
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        int s = lane < kSelThreads / 32 ? warp_sums[lane] : 0;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, s, o);
            if (lane >= o) s += up;
        }
        if (lane < kSelThreads / 32) warp_sums[lane] = s;      // inclusive sums of the warps
    }
    __syncthreads();
    *total = warp_sums[kSelThreads / 32 - 1];
    return inc - v + (warp > 0 ? warp_sums[warp - 1] : 0);
}

__global__ void __launch_bounds__(kSelThreads) select_kernel(Geometry geo, StateView st, EvictArgs a) {
    extern __shared__ __align__(16) unsigned long long keys[];
    __shared__ unsigned int hist[256];
    __shared__ unsigned long long sh_prefix;
    __shared__ int sh_krem, sh_first;
    __shared__ int warp_sums[kSelThreads / 32];

    const int u = blockIdx.x, tid = threadIdx.x;
    const int S = a.n_initial, R = a.n_recent;
    const int ncand = a.n - R - S;                 // unprotected slots [S, n - R)
    const int k = a.budget - R - S;                // how many of them stay
    const int32_t* ts = st.ts + (size_t)u * geo.capacity + S;
    const int32_t* mri = st.mri + (size_t)u * geo.capacity + S;
    int32_t* src = a.src + (size_t)u * a.budget;

    for (int i = tid; i < ncand; i += kSelThreads)
        keys[i] = (unsigned long long)__double_as_longlong(score_fn(a.t - ts[i], mri[i], a.score_mode));
    if (tid == 0) sh_first = ncand;
    __syncthreads();

    // Radix select, most significant byte first: the bit pattern of the k-th largest score.
    // Scores are >= 0, so their IEEE bit patterns order like unsigned integers.
    unsigned long long prefix = 0, mask = 0;
    int krem = k;
    for (int shift = 56; shift >= 0; shift -= 8) {
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
        for (int i = tid; i < ncand; i += kSelThreads) {
            const unsigned long long key = keys[i];
            if ((key & mask) == prefix) atomicAdd(&hist[(unsigned)(key >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (tid == 0) {
            int cum = 0, digit = 0;
            for (int b = 255; b >= 0; --b) {
                const int c = (int)hist[b];
                if (cum + c >= krem) {
                    digit = b;
                    break;
                }
                cum += c;
            }
            sh_prefix = prefix | ((unsigned long long)digit << shift);
            sh_krem = krem - cum;
        }
        __syncthreads();
        prefix = sh_prefix;
        krem = sh_krem;
        mask |= 0xFFull << shift;
    }
    const unsigned long long kth = prefix;         // keep every key > kth, and `krem` of the keys == kth

    // Ties are resolved towards the more recent token, i.e. the higher slot: keep the last `krem` ties.
    const int ipt = (ncand + kSelThreads - 1) / kSelThreads;
    const int b = min(ncand, tid * ipt), e = min(ncand, b + ipt);
    int ties = 0;
    for (int i = b; i < e; ++i) ties += keys[i] == kth;
    int total_ties;
    int tie_rank = block_exclusive_scan(ties, warp_sums, &total_ties);
    const int first_kept_tie = total_ties - krem;
    int kept = 0;
    {
        int r = tie_rank;
        for (int i = b; i < e; ++i) {
            const unsigned long long key = keys[i];
            bool keep = key > kth;
            if (key == kth) keep = r++ >= first_kept_tie;
            kept += keep;
        }
    }
    int total_kept;
    int dst = block_exclusive_scan(kept, warp_sums, &total_kept);
    {
        int r = tie_rank, first_evicted = ncand;
        for (int i = b; i < e; ++i) {
            const unsigned long long key = keys[i];
            bool keep = key > kth;
            if (key == kth) keep = r++ >= first_kept_tie;
            if (keep)
                src[S + dst++] = S + i;
            else if (first_evicted == ncand)
                first_evicted = i;
        }
        if (first_evicted < ncand) atomicMin(&sh_first, first_evicted);
    }
    for (int j = tid; j < S; j += kSelThreads) src[j] = j;
    for (int r = tid; r < R; r += kSelThreads) src[a.budget - R + r] = a.n - R + r;
    __syncthreads();
    if (tid == 0) {
        a.first_moved[u] = S + sh_first;
        if (total_kept != k) atomicOr(st.status, kStatusBadIndex);
    }
}

constexpr int kCompactThreads = 256;
constexpr int kRowsPerWarp = kPageTokens / (kCompactThreads / 32);     // 8

// One block per unit walks destination pages front to back.  Destination slot j
// receives slot src[j] >= j, and sources are strictly increasing in j, so once a
// tile's sources sit in registers (barrier) its destinations can be overwritten:
// they are sources only of this or of earlier tiles.
__global__ void __launch_bounds__(kCompactThreads) compact_kernel(Geometry geo, uint8_t* pool, StateView st,
                                                                 EvictArgs a) {
    const int u = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int32_t* src = a.src + (size_t)u * a.budget;
    const int32_t* pt = st.page_table + (size_t)u * geo.pages_per_unit;
    const int first = a.first_moved[u];
    const size_t sbase = (size_t)u * geo.capacity;
    const int half = lane < 16 ? 0 : kPageHalfBytes;      // lanes 0..15: K row, 16..31: V row
    const int cp = lane & 15;                             // physical chunk read from the source row

    for (int d0 = first / kPageTokens * kPageTokens; d0 < a.budget; d0 += kPageTokens) {
        uint4 val[kRowsPerWarp];
        int srow[kRowsPerWarp];
#pragma unroll
        for (int i = 0; i < kRowsPerWarp; ++i) {
            const int dj = d0 + warp + 8 * i;
            srow[i] = -1;
            if (dj >= first && dj < a.budget) {
                const int sj = src[dj];
                if (sj != dj) {
                    srow[i] = sj;
                    const uint8_t* row =
                        page_ptr(pool, pt[sj / kPageTokens]) + half + (sj % kPageTokens) * kRowBytes;
                    val[i] = *reinterpret_cast<const uint4*>(row + cp * 16);
                }
            }
        }
        int s_ts = 0, s_mri = 0, s_pos = 0, s_from = -1;
        if (tid < kPageTokens) {
            const int dj = d0 + tid;
            if (dj >= first && dj < a.budget) {
                const int sj = src[dj];
                if (sj != dj) {
                    s_from = sj;
                    s_ts = st.ts[sbase + sj];
                    s_mri = st.mri[sbase + sj];
                    s_pos = st.pos[sbase + sj];
                }
            }
        }
        __syncthreads();
        uint8_t* dpage = page_ptr(pool, pt[d0 / kPageTokens]) + half;
#pragma unroll
        for (int i = 0; i < kRowsPerWarp; ++i) {
            if (srow[i] >= 0) {
                const int dr = warp + 8 * i;
                const int c = cp ^ (srow[i] & 7);              // logical chunk held by this lane
                *reinterpret_cast<uint4*>(dpage + dr * kRowBytes + swz_chunk(c, dr) * 16) = val[i];
            }
        }
        if (s_from >= 0) {
            st.ts[sbase + d0 + tid] = s_ts;
            st.mri[sbase + d0 + tid] = s_mri;
            st.pos[sbase + d0 + tid] = s_pos;
        }
    }
}

__global__ void score_kernel(Geometry geo, StateView st, int unit_begin, int unit_count, int n, int t, int mode,
                             double* out) {
    const size_t total = (size_t)unit_count * geo.capacity;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int u = (int)(i / geo.capacity), s = (int)(i % geo.capacity);
        const size_t g = (size_t)(unit_begin + u) * geo.capacity + s;
        out[i] = s < n ? score_fn(t - st.ts[g], st.mri[g], mode) : 0.0;
    }
}

}  // namespace

size_t select_smem_bytes(int n_candidates) { return (size_t)n_candidates * sizeof(unsigned long long); }

cudaError_t select_prepare() {
    return cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
}

cudaError_t select_launch(const Geometry& geo, StateView st, const EvictArgs& a, cudaStream_t stream) {
    const int ncand = a.n - a.n_recent - a.n_initial;
    select_kernel<<<geo.units, kSelThreads, select_smem_bytes(ncand), stream>>>(geo, st, a);
    return cudaGetLastError();
}

cudaError_t compact_launch(const Geometry& geo, uint8_t* pool, StateView st, const EvictArgs& a,
                           cudaStream_t stream) {
    compact_kernel<<<geo.units, kCompactThreads, 0, stream>>>(geo, pool, st, a);
    return cudaGetLastError();
}

cudaError_t score_launch(const Geometry& geo, StateView st, int unit_begin, int unit_count, int n, int t,
                         int score_mode, double* out, cudaStream_t stream) {
    const size_t total = (size_t)unit_count * geo.capacity;
    const int blocks = (int)((total + 255) / 256 < 148 * 8 ? (total + 255) / 256 : 148 * 8);
    score_kernel<<<blocks, 256, 0, stream>>>(geo, st, unit_begin, unit_count, n, t, score_mode, out);
    return cudaGetLastError();
}

}  // namespace lzk
