// Lagged eviction (Section 4 "MRI-Centric Eviction" of the paper):
//   score_fn       -- H1, H2 and Eq. (2), fp64
//   select_fast_kernel -- top-(B - R - S) of the unprotected slots by (score, recency) when the k-th
//                     score is 0 (only zero / non-zero matters, no floating point), else lists the unit
//   select_kernel  -- the general route for listed units: fp64 scores, block-wide radix select on the
//                     score bits, then a prefix sum that turns keep flags into the list "slot src[j]
//                     moves to slot j" (Appendix A, Eq. (evic))
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
// Modes: 0 = Eq. (2); 1 = H1 only; 2 = H2 only (the paper's ablations); 3 = Eq. (2) with
// H2 = 2 sigma(-(MRI - 1)), a variant that decreases with MRI as the paper's prose asks.
__device__ __forceinline__ double h1_term(int d, int mri) {
    if (mri == 0) return d == 0 ? 1.0 : 0.0;
    return 2.0 / (1.0 + exp((double)d / (double)mri));
}

// The H2 term depends on MRI alone (mri >= 1 here; mode 1 never asks for it).
__device__ __forceinline__ double h2_term(int mri, int mode) {
    if (mode == 3) return 2.0 / (1.0 + exp((double)mri - 1.0));
    return mri > 1 ? 2.0 / (1.0 + exp(1.0 / ((double)mri - 1.0))) : 0.0;
}

__device__ __forceinline__ double combine_terms(double h1, double h2, int mode) {
    if (mode == 1) return h1;
    if (mode == 2) return h2;
    return h1 + h2;
}

__device__ __forceinline__ double score_fn(int d, int mri, int mode) {
    const double h1 = mode == 2 ? 0.0 : h1_term(d, mri);
    const double h2 = (mode == 1 || mri == 0) ? 0.0 : h2_term(mri, mode);
    return combine_terms(h1, h2, mode);
}

// The same value with the H2 term read from a table filled by h2_table_kernel with h2_term itself,
// so both routes give identical bits.
__device__ __forceinline__ double score_with_table(int d, int mri, int mode, const double* __restrict__ h2_table,
                                                   int h2_entries) {
    const double h1 = mode == 2 ? 0.0 : h1_term(d, mri);
    double h2 = 0.0;
    if (mode != 1 && mri != 0) h2 = mri < h2_entries ? h2_table[mri] : h2_term(mri, mode);
    return combine_terms(h1, h2, mode);
}

__global__ void h2_table_kernel(int mode, int entries, double* table) {
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m < entries) table[m] = m == 0 ? 0.0 : h2_term(m, mode);
}

constexpr int kSelThreads = 512;

// Block-wide sum of one int per thread.
__device__ __forceinline__ int block_sum(int v, int* warp_sums) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();                       // warp_sums may still be read from a previous call
    if (lane == 0) warp_sums[warp] = v;
    __syncthreads();
    int s = 0;
#pragma unroll
    for (int w = 0; w < kSelThreads / 32; ++w) s += warp_sums[w];
    return s;
}

struct SelectShared {
    unsigned int hist[256];
    unsigned long long prefix;
    unsigned long long surv[kSelThreads];          // the keys still in the race once they are few
    int krem, first, done, n_surv;
    int warp_sums[kSelThreads / 32];
};

// The selection of one unit with the k-th score found by radix passes (the general route).
__device__ void select_radix_unit(const int u, const Geometry& geo, const StateView& st, const EvictArgs& a,
                                  unsigned long long* keys, SelectShared& sh) {
    unsigned int* hist = sh.hist;
    unsigned long long& sh_prefix = sh.prefix;
    int &sh_krem = sh.krem, &sh_first = sh.first, &sh_done = sh.done;
    int* warp_sums = sh.warp_sums;

    const int tid = threadIdx.x, lane = tid & 31;
    const int S = a.n_initial, R = a.n_recent;
    const int ncand = a.n - R - S;                 // unprotected slots [S, n - R)
    const int k = a.budget - R - S;                // how many of them stay
    const int2* tsm = st.tsm + (size_t)u * geo.capacity + S;       // (TS, MRI) of the candidates
    int32_t* src = a.src + (size_t)u * a.budget;
    if (!in_bounds(S >= 0 && R >= 0 && ncand > 0 && k >= 0 && k <= ncand && a.n <= geo.capacity && a.budget <= a.n, st.status))
        return;

    // Each warp owns a contiguous segment of the candidates and walks it 32 at a time (also in the
    // ranking passes below, where ranks in slot order come from ballots over consecutive keys).
    constexpr int kWarps = kSelThreads / 32;
    const int warp = tid >> 5;
    const int seg = ((ncand + kWarps - 1) / kWarps + 31) / 32 * 32;
    const int seg_b = min(ncand, warp * seg), seg_e = min(ncand, seg_b + seg);
    const unsigned lt = (1u << lane) - 1u;

    // Scores are >= 0, so their IEEE bit patterns order like unsigned integers; a score of exactly 0
    // (never re-activated) has key 0.  Units come here because more of their scores are non-zero than
    // tokens are kept, so Eq. (2) is evaluated in fp64 for every candidate (tokens with MRI = 0 take the
    // short way through it); eight steps' loads are in flight before the first evaluation.
    int nonzero = 0;
    for (int i0 = seg_b; i0 < seg_e; i0 += 8 * 32) {
        int mm[8], tt[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int i = i0 + 32 * q + lane;
            const int2 w = i < seg_e ? __ldg(tsm + i) : make_int2(0, 0);
            tt[q] = w.x;
            mm[q] = w.y;
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int i = i0 + 32 * q + lane;
            if (i < seg_e) {
                const unsigned long long key = (unsigned long long)__double_as_longlong(
                    score_with_table(a.t - tt[q], mm[q], a.score_mode, a.h2_table, a.h2_entries));
                keys[i] = key;
                nonzero += key != 0ull;
            }
        }
    }
    if (tid == 0) sh_first = ncand;
    nonzero = block_sum(nonzero, warp_sums);       // (its barriers also publish keys[] and sh_first)

    // kth: bit pattern of the k-th largest score; krem: how many of the keys equal to it stay.
    unsigned long long kth = 0;
    int krem = k - nonzero;
    if (nonzero > k) {
        // More non-zero scores than tokens to keep: the k-th score is found by a radix select over the
        // non-zero keys, most significant byte first.  The histogram is built with
        // one shared-memory atomic per distinct digit and warp (scores cluster in a few exponents), and
        // the passes stop as soon as the k-th key's bin holds at most one key per thread.
        unsigned long long prefix = 0, mask = 0;
        krem = k;
        for (int shift = 56; shift >= 0; shift -= 8) {
            if (tid < 256) hist[tid] = 0;
            __syncthreads();
            for (int i0 = 0; i0 < ncand; i0 += kSelThreads) {
                const int i = i0 + tid;
                const unsigned long long key = i < ncand ? keys[i] : 0ull;
                const bool on = key != 0ull && (key & mask) == prefix;
                const unsigned digit = on ? (unsigned)(key >> shift) & 255u : 256u;
                const unsigned peers = __match_any_sync(0xffffffffu, digit);
                if (on && (int)(__ffs(peers) - 1) == lane) atomicAdd(&hist[digit], (unsigned)__popc(peers));
            }
            __syncthreads();
            if (tid < 32) {
                // The bin that holds the krem-th largest key, bins counted from the top: lane l sums bins
                // 8 l .. 8 l + 7, a suffix scan over the lanes finds the lane, eight steps find the bin.
                int c8[8], own = 0;
#pragma unroll
                for (int b = 0; b < 8; ++b) {
                    c8[b] = (int)hist[8 * lane + b];
                    own += c8[b];
                }
                int above = own;                   // inclusive suffix sum: this lane's bins and all higher ones
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int v = __shfl_down_sync(0xffffffffu, above, o);
                    if (lane + o < 32) above += v;
                }
                const bool here = above >= krem && above - own < krem;     // exactly one lane (krem >= 1 keys exist)
                if (here) {
                    int cum = above - own, digit = 8 * lane;
#pragma unroll
                    for (int b = 7; b >= 0; --b) {
                        if (cum + c8[b] >= krem) {
                            digit = 8 * lane + b;
                            break;
                        }
                        cum += c8[b];
                    }
                    sh_prefix = prefix | ((unsigned long long)digit << shift);
                    sh_krem = krem - cum;
                    sh_done = hist[digit] <= (unsigned)kSelThreads;
                }
            }
            __syncthreads();
            prefix = sh_prefix;
            krem = sh_krem;
            mask |= 0xFFull << shift;
            if (sh_done) break;                    // uniform: read from shared memory after the barrier
        }
        kth = prefix;
        if (mask != ~0ull) {
            // Stopped early: at most one key per thread shares the prefix.  They are gathered, and every
            // thread ranks its own among them: the k-th is the key with fewer than krem keys above it and
            // at least krem keys at or above it.
            if (tid == 0) sh.n_surv = 0;
            __syncthreads();
            for (int i = tid; i < ncand; i += kSelThreads) {
                const unsigned long long key = keys[i];
                if (key != 0ull && (key & mask) == prefix) sh.surv[atomicAdd(&sh.n_surv, 1)] = key;
            }
            __syncthreads();
            const int n_surv = sh.n_surv;
            if (tid < n_surv) {
                const unsigned long long mine = sh.surv[tid];
                int above = 0, equal = 0;
                for (int j = 0; j < n_surv; ++j) {
                    const unsigned long long other = sh.surv[j];
                    above += other > mine;
                    equal += other == mine;
                }
                if (above < krem && krem <= above + equal) {       // equal keys all write the same two values
                    sh_prefix = mine;
                    sh_krem = krem - above;
                }
            }
            __syncthreads();
            kth = sh_prefix;
            krem = sh_krem;
        }
    }
    // keep every key > kth, and `krem` of the keys == kth

    // Ties are resolved towards the more recent token, i.e. the higher slot: keep the last `krem` ties.
    // Ranks in slot order come from ballots over each warp's segment: lanes read consecutive keys (no
    // bank conflicts).
    int ties = 0;
    for (int i0 = seg_b; i0 < seg_e; i0 += 32) {
        const int i = i0 + lane;
        ties += __popc(__ballot_sync(0xffffffffu, i < seg_e && keys[i] == kth));
    }
    __syncthreads();
    if (lane == 0) warp_sums[warp] = ties;
    __syncthreads();
    int tie_rank = 0, total_ties = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        tie_rank += w < warp ? warp_sums[w] : 0;
        total_ties += warp_sums[w];
    }
    const int first_kept_tie = total_ties - krem;
    unsigned long long keep_bits = 0;              // bit j: this lane's candidate of step j stays (at most 50 steps)
    int kept = 0;
    {
        int step = 0;
        for (int i0 = seg_b; i0 < seg_e; i0 += 32, ++step) {
            const int i = i0 + lane;
            const unsigned long long key = i < seg_e ? keys[i] : 0ull;
            const bool tie = i < seg_e && key == kth;
            const unsigned tie_mask = __ballot_sync(0xffffffffu, tie);
            const bool keep = i < seg_e && (key > kth || (tie && tie_rank + __popc(tie_mask & lt) >= first_kept_tie));
            tie_rank += __popc(tie_mask);
            kept += __popc(__ballot_sync(0xffffffffu, keep));
            keep_bits |= (unsigned long long)keep << step;
        }
    }
    __syncthreads();
    if (lane == 0) warp_sums[warp] = kept;
    __syncthreads();
    int dst = 0, total_kept = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        dst += w < warp ? warp_sums[w] : 0;
        total_kept += warp_sums[w];
    }
    {
        int step = 0, first_evicted = ncand;
        for (int i0 = seg_b; i0 < seg_e; i0 += 32, ++step) {
            const int i = i0 + lane;
            const bool keep = (keep_bits >> step) & 1ull;
            const unsigned keep_mask = __ballot_sync(0xffffffffu, keep);
            if (keep && in_bounds(S + dst + __popc(keep_mask & lt) < a.budget - R, st.status))
                src[S + dst + __popc(keep_mask & lt)] = S + i;
            dst += __popc(keep_mask);
            const unsigned gone = __ballot_sync(0xffffffffu, i < seg_e && !keep);
            if (gone != 0u && first_evicted == ncand) first_evicted = i0 + __ffs(gone) - 1;
        }
        if (lane == 0 && first_evicted < ncand) atomicMin(&sh_first, first_evicted);
    }
    for (int j = tid; j < S; j += kSelThreads) src[j] = j;
    for (int r = tid; r < R; r += kSelThreads) src[a.budget - R + r] = a.n - R + r;
    __syncthreads();
    if (tid == 0) {
        a.first_moved[u] = S + sh_first;
        if (total_kept != k) atomicOr(st.status, kStatusBadIndex);
    }
}

// Blocks take the units that select_fast_kernel listed for the general route.
__global__ void __launch_bounds__(kSelThreads) select_kernel(Geometry geo, StateView st, EvictArgs a) {
    extern __shared__ __align__(16) unsigned long long keys[];
    __shared__ SelectShared sh;
    const int listed = *a.radix_count;
    for (int idx = blockIdx.x; idx < listed; idx += gridDim.x) {
        select_radix_unit(a.radix_list[idx], geo, st, a, keys, sh);
        __syncthreads();
    }
}

constexpr int kMaxSelSteps = 64;       // 32 candidates per step and warp: up to 32768 candidates per unit

// First stage of the selection, for every unit: classify every candidate's score as zero or not (no
// floating point, see select_radix_unit) into one bit per candidate.  If at most k scores are non-zero
// -- the usual case: the tokens an eviction removes are the ones never re-activated -- the k-th score is
// 0, every non-zero score stays, and of the zeros the most recent stay (the tie rule): the keep flags,
// their ranks and the source list all follow from the bit words, and the unit is done.  Otherwise the
// unit is put on the list for select_kernel.
__global__ void __launch_bounds__(kSelThreads) select_fast_kernel(Geometry geo, StateView st, EvictArgs a) {
    constexpr int kWarps = kSelThreads / 32;
    __shared__ uint32_t nzw[kWarps][kMaxSelSteps];      // bit = this candidate's score is not zero
    __shared__ uint32_t keepw[kWarps][kMaxSelSteps];    // bit = this candidate stays
    __shared__ int dbase[kWarps][kMaxSelSteps];         // kept candidates of the warp before this word
    __shared__ int warp_nz[kWarps], warp_kept[kWarps];
    __shared__ int sh_first;

    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int S = a.n_initial, R = a.n_recent;
    const int ncand = a.n - R - S, k = a.budget - R - S;
    const int2* tsm = st.tsm + (size_t)u * geo.capacity + S;       // (TS, MRI) of the candidates
    int32_t* src = a.src + (size_t)u * a.budget;
    if (!in_bounds(S >= 0 && R >= 0 && ncand > 0 && k >= 0 && k <= ncand && a.n <= geo.capacity && a.budget <= a.n, st.status))
        return;
    const int seg = ((ncand + kWarps - 1) / kWarps + 31) / 32 * 32;
    const int seg_b = min(ncand, warp * seg), seg_e = min(ncand, seg_b + seg);
    const int nsteps = (seg_e - seg_b + 31) / 32;
    const unsigned lt = (1u << lane) - 1u;

    // (eight steps at a time: all eight loads of a lane are in flight before the first ballot, which
    // is what keeps this pass bound by bandwidth and not by one memory latency per step)
    int nz_warp = 0;
    for (int s0 = 0; s0 < nsteps; s0 += 8) {
        int mm[8], tt[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int i = seg_b + (s0 + q) * 32 + lane;
            const bool in = s0 + q < nsteps && i < seg_e;
            const int2 w = in ? __ldg(tsm + i) : make_int2(a.t - 1, 0);    // outside: MRI = 0, elapsed 1 -> a zero score
            tt[q] = w.x;
            mm[q] = w.y;
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int m = mm[q], d = a.t - tt[q];
            bool nz;
            if (a.score_mode == 2)
                nz = m > 1;
            else if (m == 0)
                nz = d == 0;
            else if ((long long)d > 700ll * m)
                nz = score_with_table(d, m, a.score_mode, a.h2_table, a.h2_entries) != 0.0;
            else
                nz = true;
            const unsigned word = __ballot_sync(0xffffffffu, nz);
            if (lane == 0 && s0 + q < nsteps) nzw[warp][s0 + q] = word;
            nz_warp += __popc(word);
        }
    }
    if (lane == 0) warp_nz[warp] = nz_warp;
    if (tid == 0) sh_first = ncand;
    __syncthreads();
    int nonzero = 0, zeros_before = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        nonzero += warp_nz[w];
        const int wb = min(ncand, w * seg), we = min(ncand, wb + seg);
        zeros_before += w < warp ? (we - wb) - warp_nz[w] : 0;
    }
    if (nonzero > k) {                             // the k-th score is not zero: the general route
        if (tid == 0) {
            a.radix_list[atomicAdd(a.radix_count, 1)] = u;
            atomicAdd(st.status + kCounterRadixUnits, 1);
        }
        return;
    }
    if (tid == 0) atomicAdd(st.status + kCounterZeroCutUnits, 1);

    // Of the zeros, the first `drop_total` in slot order go (ties are resolved towards the more recent
    // token); lane l of a warp handles the warp's words l and l + 32.
    const int drop_total = (ncand - nonzero) - (k - nonzero);
    int tie_carry = zeros_before, kept_carry = 0, first_gone = ncand;
    for (int c = 0; c * 32 < nsteps; ++c) {
        const int step = c * 32 + lane;
        const bool valid = step < nsteps;
        const int left = valid ? min(32, seg_e - (seg_b + step * 32)) : 0;
        const unsigned in_mask = left >= 32 ? 0xffffffffu : ((1u << left) - 1u);
        const unsigned nz = valid ? nzw[warp][step] : 0u;
        const unsigned z = ~nz & in_mask;
        const int cz = __popc(z), ck_nz = __popc(nz);
        int incl = cz;                             // zeros of this warp up to and including this word
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        const int rank0 = tie_carry + incl - cz;   // rank among all zeros of this word's first zero
        const int drop = min(max(drop_total - rank0, 0), cz);
        unsigned zk = z;
        if (drop >= cz)
            zk = 0u;
        else
            for (int q = 0; q < drop; ++q) zk &= zk - 1u;      // clears the lowest set bit
        const unsigned kw = nz | zk;
        const int ck = ck_nz + __popc(zk);
        int inclk = ck;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, inclk, o);
            if (lane >= o) inclk += up;
        }
        if (valid) {
            keepw[warp][step] = kw;
            dbase[warp][step] = kept_carry + inclk - ck;
            const unsigned gone = in_mask & ~kw;
            if (gone != 0u) first_gone = min(first_gone, seg_b + step * 32 + __ffs(gone) - 1);
        }
        tie_carry += __shfl_sync(0xffffffffu, incl, 31);
        kept_carry += __shfl_sync(0xffffffffu, inclk, 31);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) first_gone = min(first_gone, __shfl_xor_sync(0xffffffffu, first_gone, o));
    if (lane == 0) {
        warp_kept[warp] = kept_carry;
        if (first_gone < ncand) atomicMin(&sh_first, first_gone);
    }
    __syncthreads();
    int warp_dst = 0, total_kept = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        warp_dst += w < warp ? warp_kept[w] : 0;
        total_kept += warp_kept[w];
    }
    // source list: kept candidate number j of the unit moves to slot S + j
    for (int step = 0; step < nsteps; ++step) {
        const unsigned kw = keepw[warp][step];
        const int j = warp_dst + dbase[warp][step] + __popc(kw & lt);
        if (((kw >> lane) & 1u) && in_bounds(j < k, st.status)) src[S + j] = S + seg_b + step * 32 + lane;
    }
    for (int j = tid; j < S; j += kSelThreads) src[j] = j;
    for (int r = tid; r < R; r += kSelThreads) src[a.budget - R + r] = a.n - R + r;
    if (tid == 0) {
        a.first_moved[u] = S + sh_first;
        if (total_kept != k) atomicOr(st.status, kStatusBadIndex);
    }
}

constexpr int kCompactThreads = 256;
constexpr int kRowsPerWarp = kPageTokens / (kCompactThreads / 32);     // 8
constexpr int kMaxPagesInSmem = 1024;                                  // page-table entries cached per block

// One block per unit walks destination pages front to back.  Destination slot j
// receives slot src[j] >= j, and sources are strictly increasing in j, so once a
// tile's sources sit in registers (barrier) its destinations can be overwritten:
// they are sources only of this or of earlier tiles.  The source indices of the
// next tile are fetched while the rows of the current one are in flight, and the
// unit's page table sits in shared memory, so a tile costs one global round trip.
__global__ void __launch_bounds__(kCompactThreads, 3) compact_kernel(Geometry geo, uint8_t* pool, StateView st,
                                                                 EvictArgs a) {
    __shared__ int32_t pt_s[kMaxPagesInSmem];
    const int u = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int32_t* src = a.src + (size_t)u * a.budget;
    const int32_t* pt_g = st.page_table + (size_t)u * geo.pages_per_unit;
    const int first = in_bounds(a.first_moved[u] >= 0, st.status) ? a.first_moved[u] : a.budget;
    const size_t sbase = (size_t)u * geo.capacity;
    const int half = lane < 16 ? 0 : kPageHalfBytes;      // lanes 0..15: K row, 16..31: V row
    const int cp = lane & 15;                             // physical chunk read from the source row
    const bool pt_cached = geo.pages_per_unit <= kMaxPagesInSmem;
    if (pt_cached)
        for (int i = tid; i < geo.pages_per_unit; i += kCompactThreads) pt_s[i] = pt_g[i];
    __syncthreads();
    const int32_t* pt = pt_cached ? pt_s : pt_g;

    // source slot of destination slot dj, or -1 when the row stays where it is
    auto source_of = [&](int dj) -> int {
        if (dj < first || dj >= a.budget) return -1;
        const int sj = src[dj];
        if (!in_bounds(sj >= dj && sj < a.n, st.status)) return -1;
        return sj != dj ? sj : -1;
    };
    // physical page of logical page `lp` of this unit (checked in the debug build)
    auto page_of = [&](int lp) -> int32_t {
        if (!in_bounds(lp >= 0 && lp < geo.pages_per_unit, st.status)) return 0;
        const int32_t pp = pt[lp];
        return in_bounds(pp >= 0 && pp < geo.units * geo.pages_per_unit, st.status) ? pp : 0;
    };

    int d0 = first / kPageTokens * kPageTokens;
    int srow[kRowsPerWarp], s_from = -1;
#pragma unroll
    for (int i = 0; i < kRowsPerWarp; ++i) srow[i] = source_of(d0 + warp + 8 * i);
    if (tid < kPageTokens) s_from = source_of(d0 + tid);

    for (; d0 < a.budget; d0 += kPageTokens) {
        uint4 val[kRowsPerWarp];
#pragma unroll
        for (int i = 0; i < kRowsPerWarp; ++i)
            if (srow[i] >= 0) {
                const uint8_t* row =
                    page_ptr(pool, page_of(srow[i] / kPageTokens)) + half + (srow[i] % kPageTokens) * kRowBytes;
                val[i] = *reinterpret_cast<const uint4*>(row + cp * 16);
            }
        int2 s_tsm = make_int2(0, 0);
        int s_pos = 0;
        if (s_from >= 0) {
            s_tsm = st.tsm[sbase + s_from];
            s_pos = st.pos[sbase + s_from];
        }
        // next tile's source indices: in flight together with this tile's rows
        int srow_next[kRowsPerWarp], s_from_next = -1;
#pragma unroll
        for (int i = 0; i < kRowsPerWarp; ++i) srow_next[i] = source_of(d0 + kPageTokens + warp + 8 * i);
        if (tid < kPageTokens) s_from_next = source_of(d0 + kPageTokens + tid);

        __syncthreads();       // every source row of this tile is in registers
        uint8_t* dpage = page_ptr(pool, page_of(d0 / kPageTokens)) + half;
#pragma unroll
        for (int i = 0; i < kRowsPerWarp; ++i) {
            if (srow[i] >= 0) {
                const int dr = warp + 8 * i;
                const int c = cp ^ (srow[i] & 7);              // logical chunk held by this lane
                *reinterpret_cast<uint4*>(dpage + dr * kRowBytes + swz_chunk(c, dr) * 16) = val[i];
            }
            srow[i] = srow_next[i];
        }
        if (s_from >= 0) {
            st.tsm[sbase + d0 + tid] = s_tsm;
            st.pos[sbase + d0 + tid] = s_pos;
        }
        s_from = s_from_next;
    }
}

__global__ void score_kernel(Geometry geo, StateView st, int unit_begin, int unit_count, int n, int t, int mode,
                             double* out) {
    const size_t total = (size_t)unit_count * geo.capacity;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int u = (int)(i / geo.capacity), s = (int)(i % geo.capacity);
        const size_t g = (size_t)(unit_begin + u) * geo.capacity + s;
        const int2 w = st.tsm[g];
        out[i] = s < n ? score_fn(t - w.x, w.y, mode) : 0.0;
    }
}

// Histogram of MRI over the cached tokens of a range of units (Section 4, "Discussion about the
// choice of W and alpha": W is read off the distribution of MRI).  hist[b] counts tokens with MRI = b
// for b < bins - 1; the last bin takes every larger value.  Blocks stride over units, count the
// first kHistSmemBins values in shared memory and flush what is non-zero with one atomic per bin.
constexpr int kHistSmemBins = 8192;

__global__ void __launch_bounds__(256) mri_histogram_kernel(Geometry geo, StateView st, int unit_begin,
                                                           int unit_count, int n, int bins,
                                                           unsigned long long* hist) {
    __shared__ unsigned int local[kHistSmemBins];
    const int nlocal = min(bins, kHistSmemBins);
    for (int b = threadIdx.x; b < nlocal; b += blockDim.x) local[b] = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31;
    for (int u = unit_begin + blockIdx.x; u < unit_begin + unit_count; u += gridDim.x) {
        const int2* tsm = st.tsm + (size_t)u * geo.capacity;
        for (int i0 = 0; i0 < n; i0 += blockDim.x) {
            const int i = i0 + threadIdx.x;
            const bool on = i < n;
            const int v = on ? tsm[i].y : -1;
            const int b = v < 0 ? 0 : min(v, bins - 1);
            // most tokens share one value (0): one atomic per distinct value and warp
            const unsigned peers = __match_any_sync(0xffffffffu, on ? b : -1);
            if (on && (int)(__ffs(peers) - 1) == lane) {
                if (b < nlocal)
                    atomicAdd(&local[b], (unsigned)__popc(peers));
                else
                    atomicAdd(&hist[b], (unsigned long long)__popc(peers));
            }
        }
    }
    __syncthreads();
    for (int b = threadIdx.x; b < nlocal; b += blockDim.x)
        if (local[b] != 0u) atomicAdd(&hist[b], (unsigned long long)local[b]);
}

}  // namespace

size_t select_smem_bytes(int n_candidates) { return (size_t)n_candidates * sizeof(unsigned long long); }

cudaError_t select_prepare() {
    return cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
}

cudaError_t select_launch(const Geometry& geo, StateView st, const EvictArgs& a, int num_sms, cudaStream_t stream) {
    const int ncand = a.n - a.n_recent - a.n_initial;
    if (ncand > 32 * kMaxSelSteps * (kSelThreads / 32)) return cudaErrorInvalidValue;
    cudaError_t e = cudaMemsetAsync(a.radix_count, 0, sizeof(int32_t), stream);
    if (e != cudaSuccess) return e;
    select_fast_kernel<<<geo.units, kSelThreads, 0, stream>>>(geo, st, a);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    // the general route for the units the first stage listed: a grid that fills the GPU once
    const size_t smem = select_smem_bytes(ncand);
    int per_sm = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, select_kernel, kSelThreads, smem) != cudaSuccess || per_sm < 1) {
        cudaGetLastError();
        per_sm = 1;
    }
    const int blocks = geo.units < num_sms * per_sm ? geo.units : num_sms * per_sm;
    select_kernel<<<blocks, kSelThreads, smem, stream>>>(geo, st, a);
    return cudaGetLastError();
}

cudaError_t h2_table_launch(int score_mode, int entries, double* table, cudaStream_t stream) {
    h2_table_kernel<<<(entries + 255) / 256, 256, 0, stream>>>(score_mode, entries, table);
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

cudaError_t mri_histogram_launch(const Geometry& geo, StateView st, int unit_begin, int unit_count, int n, int bins,
                                 unsigned long long* hist, cudaStream_t stream) {
    cudaError_t e = cudaMemsetAsync(hist, 0, (size_t)bins * sizeof(unsigned long long), stream);
    if (e != cudaSuccess) return e;
    const int blocks = unit_count < 148 * 4 ? unit_count : 148 * 4;
    mri_histogram_kernel<<<blocks, 256, 0, stream>>>(geo, st, unit_begin, unit_count, n, bins, hist);
    return cudaGetLastError();
}

}  // namespace lzk
