// GQA flash-decode over the paged, swizzled KV pool with per-token probability
// emission and the fused recurrence-statistics update.
//
// Computes, for every cache unit (Appendix A, Eq. (attn) of the paper):
//   s_g[i] = q_g . k_i / sqrt(D),  p_g = softmax_i(s_g),  out_g = sum_i p_g[i] v_i
// and, fused (Section 4 "Recurrence Interval Tracking", Eq. (1), Algorithm 1):
//   pbar[i] = mean_g p_g[i];  if pbar[i] >= alpha: MRI[i] = max(MRI[i], t - TS[i]); TS[i] = t.
//
// Structure: persistent blocks, one block per SM.  A block -- or, when a unit's
// logits do not fit one SM, a cluster of `splits` blocks that split the unit's
// pages -- walks units round-robin.  Inside a block one producer warp streams
// 32 KiB pages into a shared-memory ring with linear bulk copies (TMA engine,
// mbarrier completion).  Consumer warps come in groups of four; a group takes a
// whole page, 16 tokens per warp, and with two groups consecutive pages are
// worked on concurrently.
//
// Per 16 tokens a warp runs S^T = K Q^T (tokens are the M rows, query heads the
// N columns) and O^T += V^T P^T (head dimensions are the M rows) on mma.sync
// m16n8k16, so both operands that come from the cache fill the whole A tile and
// the eight query-head columns fill the N = 8 tile.  P goes from the accumulator
// layout of the first product to the B layout of the second with movmatrix
// transposes, as two bf16 terms (hi + lo).  Softmax is online against a per-warp,
// per-head reference value that is raised (and O, l rescaled) only when a logit
// exceeds it by more than 2^8, found with one warp vote per tile; any reference
// gives the same sums.
//
// The scaled logits of the block's chunk stay on chip: in tensor memory (TMEM,
// used as 512 private 32-bit words per consumer thread through tcgen05.ld / st),
// and in shared memory for the pages beyond the 128 that fit there.  After the
// chunk the warps merge (reference, l, O) through per-warp shared-memory slots
// and the cluster's blocks through distributed shared memory, which gives the
// exact log-sum-exp.  The probabilities of a unit are produced while the block's
// NEXT unit streams: the warp that is about to overwrite the logits of a
// 16-token tile first turns the old ones into pbar, writes it and updates
// TS / MRI.  K and V are read from HBM exactly once and nothing but the outputs
// is written.
#include "internal.h"

namespace lzk {

namespace {

constexpr int kXchgRow = kHeadDim + 4;    // row stride = 4 (mod 32) floats: conflict-free fragment stores

struct Xchg {
    float o[kMaxGroup][kXchgRow];         // partial output, relative to m
    float m[kMaxGroup];                   // reference value of the partial sums (log2 domain)
    float l[kMaxGroup];                   // sum of exp2(x - m)
};

struct DecodeParams {
    uint8_t* pool;
    const int32_t* page_table;
    const __nv_bfloat16* q;
    __nv_bfloat16* out;
    float* pbar;
    int2* tsm;                                      // (TS, MRI) per token
    int32_t* status;
    int unit_begin, unit_end, group, pages_per_unit, capacity, total_pages;     // this launch walks units [begin, end)
    int n, t;
    float alpha, scale_log2, inv_group;
    int splits, stages, pages_per_cta, logit_stride, tmem_pages, tmem_cols;
    int off_logits, off_xchg, off_wml, off_slots, off_misc, off_bars;
    unsigned long long wait_limit_ns;               // a wait that lasts this long is a failure, not a delay
    int stop_after_pages;                           // diagnostics: the producer issues no copy beyond this many (-1: off)
    int rounds_before;                              // rounds of the round-robin walk that earlier launches of this step took
    // Step S1 inside this launch (small problems: one launch less per step): the new token's K / V rows
    // [units][128] bf16, written into slot n - 1 by the block that streams the slot's page.
    const uint4* k_new;                             // nullptr: the append ran as a launch of its own
    const uint4* v_new;
    int32_t* pos;
    int append_position;
};

constexpr float kRaiseMargin = 8.f;                // log2 units a logit may exceed the softmax reference by

// Bounded wait on an mbarrier phase.  On time-out the block-wide abort flag and
// the device status word are set; once the flag is up no wait blocks any more,
// so that every thread still reaches the cluster barriers and the kernel ends.
__device__ __forceinline__ bool wait_phase(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                           unsigned long long limit_ns, bool honour_abort = true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (honour_abort && *abort_flag) return false;
    uint32_t spins = 0;
    uint64_t t_start = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0xFF) == 0) {
            if (honour_abort && *abort_flag) return false;
            const uint64_t now = global_timer_ns();
            if (t_start == 0) {
                t_start = now;
            } else if (now - t_start > limit_ns) {
                *abort_flag = 1;
                atomicOr(status, kStatusWaitTimeout);
                return false;
            }
        }
    }
    return true;
}

__device__ __forceinline__ float ld_rank_f32(const float* local_ptr, uint32_t rank, bool clustered) {
    if (!clustered) return *local_ptr;
    return ld_dsmem_f32(map_to_rank(smem_u32(local_ptr), rank));
}

// NG groups of four consumer warps plus one producer warp.
template <int NG>
__global__ void __launch_bounds__((4 * NG + 1) * 32, 1) decode_kernel(const DecodeParams p) {
    constexpr int NW = 4 * NG;
    constexpr int kConsumers = NW * 32;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* ring = smem;
    float* spill = reinterpret_cast<float*>(smem + p.off_logits);       // logits of the pages beyond tensor memory
    Xchg* xchg = reinterpret_cast<Xchg*>(smem + p.off_xchg);          // [2], alternating per unit
    float* wml = reinterpret_cast<float*>(smem + p.off_wml);            // [NW][16]: m[8], l[8] per warp
    float* slots = reinterpret_cast<float*>(smem + p.off_slots);        // [NW][8][kXchgRow]: O^T of every warp
    float* lse_s = reinterpret_cast<float*>(smem + p.off_misc);         // [8]
    float* sc_s = lse_s + kMaxGroup;                                    // [splits <= 8][8]
    float* scw = sc_s + 8 * kMaxGroup;                                  // [NW <= 8][8]: scale of every warp's partial sums
    volatile int* abort_flag = reinterpret_cast<volatile int*>(scw + 8 * kMaxGroup);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(scw + 8 * kMaxGroup) + 1;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + p.off_bars);
    uint64_t* empty = full + p.stages;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = p.splits, NS = p.stages, G = p.group, LS = p.logit_stride;
    const bool clustered = S > 1;
    const uint32_t rank = clustered ? cluster_ctarank() : 0u;
    const int cluster_id = blockIdx.x / S, n_clusters = gridDim.x / S;

    if (threadIdx.x == 0) {
        for (int i = 0; i < NS; ++i) {
            mbar_init(&full[i], 1);
            mbar_init(&empty[i], 4);           // the four warps of the group that owns the page release it
        }
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 0) {                           // tensor memory for the logits: allocated and freed by warp 0
        tmem_alloc(tmem_slot, (uint32_t)p.tmem_cols);
        tmem_relinquish_alloc_permit();
    }
    tmem_fence_before_sync();
    __syncthreads();
    tmem_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    if (clustered) {   // every block of the cluster is resident before any remote access
        cluster_arrive();
        cluster_wait();
    }

    const int np = (p.n + kPageTokens - 1) / kPageTokens;       // pages in use per unit
    const int pg0 = min(np, (int)rank * p.pages_per_cta);
    const int pg1 = min(np, pg0 + p.pages_per_cta);
    const int npg = pg1 - pg0;
    const int n_units = p.unit_end - p.unit_begin;
    const int my_units = cluster_id < n_units ? (n_units - cluster_id + n_clusters - 1) / n_clusters : 0;

    if (warp == NW) {
        // ------------------------------------------------------------ producer
        uint32_t pc = 0, stage = 0, parity = 1;     // parity of the "empty" phase that frees the stage
        int it = 0;
        bool stopped = false;
        for (int u = p.unit_begin + cluster_id; u < p.unit_end && !stopped; u += n_clusters, ++it) {
            const int32_t* pt = p.page_table + (size_t)u * p.pages_per_unit + pg0;
            for (int base = 0; base < npg && !stopped; base += 32) {
                const int cnt = min(32, npg - base);
                const int32_t entry = lane < cnt ? pt[base + lane] : 0;
                for (int j = 0; j < cnt; ++j, ++pc) {
                    // Diagnostics (one block per unit only): stop feeding the ring, so that the consumers'
                    // bounded waits run out.  Every copy issued so far was armed, so the drain below is exact.
                    if (!clustered && p.stop_after_pages >= 0 && pc >= (uint32_t)p.stop_after_pages) {
                        stopped = true;
                        break;
                    }
                    int32_t pp = __shfl_sync(0xffffffffu, entry, j);
                    if (pc >= (uint32_t)NS) wait_phase(&empty[stage], parity, abort_flag, p.status, p.wait_limit_ns);
                    if (pp < 0 || pp >= p.total_pages) {
                        if (lane == 0) atomicOr(p.status, kStatusBadIndex);
                        pp = 0;
                    }
                    if (p.k_new != nullptr && pg0 + base + j == (p.n - 1) / kPageTokens &&
                        in_bounds(p.n >= 1 && p.n <= p.capacity, p.status)) {
                        // The new token (Section 4: TS = t, MRI = 0) goes into slot n - 1 of this page before the
                        // page is streamed: lanes 0..15 move the K row's chunks, lanes 16..31 the V row's.  The
                        // bulk copy below reads global memory through the async proxy, so the rows are fenced
                        // across the proxies first; the state words become visible to the consumer warps with
                        // the page (the barrier's release / acquire).
                        const int r = (p.n - 1) % kPageTokens, c = lane & 15;
                        const uint4 v = (lane < 16 ? p.k_new : p.v_new)[(size_t)u * kChunksPerRow + c];
                        uint8_t* row = p.pool + (size_t)pp * kPageBytes + (lane < 16 ? 0 : kPageHalfBytes) + r * kRowBytes;
                        *reinterpret_cast<uint4*>(row + swz_chunk(c, r) * 16) = v;
                        if (lane == 0) {
                            const size_t sl = (size_t)u * p.capacity + (p.n - 1);
                            p.tsm[sl] = make_int2(p.t, 0);
                            p.pos[sl] = p.append_position;
                        }
                        asm volatile("fence.proxy.async.global;" ::: "memory");
                        __syncwarp();
                    }
                    if (lane == 0) {
                        mbar_arrive_expect_tx(&full[stage], kPageBytes);
                        bulk_load(ring + (size_t)stage * kPageBytes, p.pool + (size_t)pp * kPageBytes, kPageBytes,
                                  &full[stage]);
                    }
                    __syncwarp();
                    if (++stage == (uint32_t)NS) {
                        stage = 0;
                        parity ^= 1;
                    }
                }
            }
            if (clustered) {   // this warp's share of the per-unit cluster barrier, split so it can run ahead
                if (it > 0) cluster_wait();
                cluster_arrive();
            }
        }
        if (clustered && it > 0) cluster_wait();
        if (*abort_flag || stopped) {   // consumers stopped waiting: let the copies in flight land before the block exits
            const uint32_t last = pc < (uint32_t)NS ? pc : (uint32_t)NS;
            for (uint32_t k = pc - last; k < pc; ++k)
                wait_phase(&full[k % NS], (k / NS) & 1, abort_flag, p.status, p.wait_limit_ns, false);
        }
    } else {
        // ------------------------------------------------------------ consumers
        // Fragment coordinates of this lane: row g (and g + 8), column pair 2 qd, 2 qd + 1.
        // In S^T rows are tokens and columns query heads; in O^T rows are head dimensions.
        const int g = lane >> 2, qd = lane & 3;
        const int h0 = 2 * qd, h1 = h0 + 1;
        const bool h0_on = h0 < G, h1_on = h1 < G;
        const int ctid = threadIdx.x;                 // consumer thread id: warps 0..NW-1
        const int grp = warp >> 2, wq = warp & 3;
        const uint32_t ring_base = smem_u32(ring);
        const uint32_t lrow = lane & 7;
        // ldmatrix row addresses.  K tile (16 tokens x 16 dims) as the A operand: matrices are
        // (tokens 0-7, chunk c), (tokens 8-15, c), (tokens 0-7, c + 1), (tokens 8-15, c + 1).
        // V tile through .trans (16 dims x 16 tokens): (tokens 0-7, c), (tokens 0-7, c + 1),
        // (tokens 8-15, c), (tokens 8-15, c + 1).  Chunk c of row r sits at c ^ (r & 7): for
        // k-step ks the lane's byte offset is lane_term ^ (ks << 5); ks bit 2 only adds 128.
        const uint32_t tok_off = 16 * wq;             // this warp's 16 tokens inside a page
        const uint32_t k_row = (tok_off + (lane & 7) + 8 * ((lane >> 3) & 1)) * kRowBytes;
        const uint32_t v_row = kPageHalfBytes + (tok_off + (lane & 7) + 8 * (lane >> 4)) * kRowBytes;
        const uint32_t k_term = ((lane >> 4) ^ lrow) << 4, v_term = (((lane >> 3) & 1) ^ lrow) << 4;
        uint32_t k_off[4], v_off[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            k_off[i] = k_row + (k_term ^ (i << 5));
            v_off[i] = v_row + (v_term ^ (i << 5));
        }
        // Logits of page j of the chunk: tensor-memory columns 4 j .. 4 j + 3 of this thread's lane
        // (x00, x01, x10, x11), or the shared-memory spill area for the pages beyond tensor memory.
        const uint32_t tmem_lane = tmem_base + ((uint32_t)(32 * wq) << 16);
        const int tmem_pages = p.tmem_pages;
        const uint32_t pc_total = (uint32_t)my_units * (uint32_t)npg;
        const int tok0 = pg0 * kPageTokens;           // first token of this block's chunk
        uint32_t pc_base = 0;                         // pages of this block before the current unit
        // Which group takes which page of a unit depends on how many pages the block has seen before it;
        // the order in which the partial sums are added follows from that.  When the walk over the units
        // is split over several launches, a launch starts where the one before it left off, so that every
        // unit gets the same bits whichever launch it falls into.
        uint32_t pc_mod = (uint32_t)(((long long)p.rounds_before * npg) % NG);   // pages before the current unit, mod NG
        uint32_t st_base = 0;                         // ring stage of page pc_base
        uint32_t pc_seen = 0, st_seen = 0, par_seen = 0;   // next page whose "full" phase this warp observes
        float lse0 = 0.f, lse1 = 0.f;                 // log-sum-exp of the previous unit, heads h0 and h1
        int u_prev = -1;
        int it = 0;

        // Every warp observes every page's "full" barrier exactly once and in page order: a parity
        // wait is only valid for a waiter that saw the previous phase of that barrier.
        auto observe_through = [&](uint32_t last) {
            while (pc_seen <= last && pc_seen < pc_total) {
                wait_phase(&full[st_seen], par_seen, abort_flag, p.status, p.wait_limit_ns);
                ++pc_seen;
                if (++st_seen == (uint32_t)NS) {
                    st_seen = 0;
                    par_seen ^= 1;
                }
            }
        };

        auto load_logits = [&](int j, float& x00, float& x01, float& x10, float& x11) {
            if (j < tmem_pages) {
                tmem_ld4(tmem_lane + 4 * j, x00, x01, x10, x11);
                tmem_wait_ld();
            } else {
                const int i = (j - tmem_pages) * kPageTokens + (int)tok_off + g;
                if (!in_bounds(i >= 0 && i + 8 < LS, p.status)) {
                    x00 = x01 = x10 = x11 = 0.f;
                    return;
                }
                x00 = h0_on ? spill[h0 * LS + i] : 0.f;
                x10 = h0_on ? spill[h0 * LS + i + 8] : 0.f;
                x01 = h1_on ? spill[h1 * LS + i] : 0.f;
                x11 = h1_on ? spill[h1 * LS + i + 8] : 0.f;
            }
        };
        auto store_logits = [&](int j, float x00, float x01, float x10, float x11) {
            if (j < tmem_pages) {
                tmem_st4(tmem_lane + 4 * j, x00, x01, x10, x11);
            } else {
                const int i = (j - tmem_pages) * kPageTokens + (int)tok_off + g;
                if (!in_bounds(i >= 0 && i + 8 < LS, p.status)) return;
                if (h0_on) {
                    spill[h0 * LS + i] = x00;
                    spill[h0 * LS + i + 8] = x10;
                }
                if (h1_on) {
                    spill[h1 * LS + i] = x01;
                    spill[h1 * LS + i + 8] = x11;
                }
            }
        };

        // pbar, TS and MRI of tokens (base + g) and (base + g + 8) of the previous unit from its logits
        // (base: token index inside the block's chunk).
        // Eq. (1) for an activated token needs its old TS.  The load is issued when the activation is
        // found and its result is used one emit_previous call later (a page's worth of work), so the
        // update never stalls the warp that holds a ring stage; at most one token per half is pending.
        long long pend_idx0 = -1, pend_idx1 = -1;
        int2 pend_old0 = make_int2(0, 0), pend_old1 = make_int2(0, 0);
        auto retire_pending = [&]() {
            if (pend_idx0 >= 0) {
                // MRI = max(MRI, t - TS), TS = t: the token belongs to this lane alone, one 8-byte store
                p.tsm[pend_idx0] = make_int2(p.t, max(pend_old0.y, p.t - pend_old0.x));
                pend_idx0 = -1;
            }
            if (pend_idx1 >= 0) {
                p.tsm[pend_idx1] = make_int2(p.t, max(pend_old1.y, p.t - pend_old1.x));
                pend_idx1 = -1;
            }
        };
        auto emit_previous = [&](int base, float x00, float x01, float x10, float x11) {
            float a0 = h0_on ? fast_exp2(x00 - lse0) : 0.f;
            float a1 = h0_on ? fast_exp2(x10 - lse0) : 0.f;
            if (h1_on) {
                a0 += fast_exp2(x01 - lse1);
                a1 += fast_exp2(x11 - lse1);
            }
            a0 += __shfl_xor_sync(0xffffffffu, a0, 1);
            a1 += __shfl_xor_sync(0xffffffffu, a1, 1);
            a0 += __shfl_xor_sync(0xffffffffu, a0, 2);
            a1 += __shfl_xor_sync(0xffffffffu, a1, 2);
            if (qd == 0) {
                retire_pending();
                const size_t row = (size_t)u_prev * p.capacity + tok0;
                const int i0 = base + g, i1 = base + g + 8;
                if (!in_bounds(u_prev >= p.unit_begin && u_prev < p.unit_end && p.n <= p.capacity, p.status)) return;
                if (tok0 + i0 < p.n) {
                    const float pb = a0 * p.inv_group;
                    p.pbar[row + i0] = pb;
                    if (pb >= p.alpha) {
                        pend_idx0 = (long long)(row + i0);
                        pend_old0 = p.tsm[row + i0];
                    }
                }
                if (tok0 + i1 < p.n) {
                    const float pb = a1 * p.inv_group;
                    p.pbar[row + i1] = pb;
                    if (pb >= p.alpha) {
                        pend_idx1 = (long long)(row + i1);
                        pend_old1 = p.tsm[row + i1];
                    }
                }
            }
        };

        // Q^T as the B operand: b0 = Q[head g][16 ks + 2 qd, +1], b1 = the same 8 dims further.  The
        // fragments of the next unit are fetched while the current one streams.
        uint32_t qb[8][2];
        auto load_q = [&](int u, uint32_t (&dst)[8][2]) {
            const __nv_bfloat16* qrow = p.q + ((size_t)u * G + g) * kHeadDim;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                dst[ks][0] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 2 * qd) : 0u;
                dst[ks][1] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 8 + 2 * qd) : 0u;
            }
        };
        if (my_units > 0) load_q(p.unit_begin + cluster_id, qb);

        // Pages belong to the groups in turn (page pc of the block's walk to group pc mod NG, across unit
        // boundaries), and a warp looks at the barriers up to its own next page before it releases the
        // page it holds; the producer refills a stage only after the pages before it were released, so it
        // cannot lap a barrier that some warp has not looked at -- provided every warp has looked at the
        // first NG pages before the first release.  With fewer pages per unit than groups a group's first
        // page lies behind the first unit's merge, so that is made sure of here, once.
        if (NG > 1) {
            observe_through((uint32_t)(NG - 1));
            named_barrier_sync(1, kConsumers);
        }

        for (int u = p.unit_begin + cluster_id; u < p.unit_end; u += n_clusters, ++it) {
            uint32_t qn[8][2] = {};
            if (u + n_clusters < p.unit_end) load_q(u + n_clusters, qn);
            float mref0 = -INFINITY, mref1 = -INFINITY, l0 = 0.f, l1 = 0.f;
            float o[8][4];      // O^T: [m-tile][(dim g, h0), (dim g, h1), (dim g + 8, h0), (dim g + 8, h1)]
#pragma unroll
            for (int i = 0; i < 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;

            // this group's pages of the unit: j = j0, j0 + NG, ...
            const int j0 = NG == 1 ? 0 : (int)((grp + NG - pc_mod) % NG);
            uint32_t stage = st_base + j0;
            if (stage >= (uint32_t)NS) stage -= NS;
            for (int j = j0; j < npg; j += NG) {
                const uint32_t pc = pc_base + j;
                observe_through(pc);
                const uint32_t page = ring_base + stage * kPageBytes;
                const int base = j * kPageTokens + (int)tok_off;

                // S^T = K Q^T for this warp's 16 tokens, two accumulator chains over the 8 k-steps
                float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int ks = 0; ks < 8; ks += 2) {
                    uint32_t a0, a1, a2, a3;
                    ldmatrix_x4(a0, a1, a2, a3, page + k_off[ks & 3] + 128 * (ks >> 2));
                    mma_bf16_16816(sa, a0, a1, a2, a3, qb[ks][0], qb[ks][1]);
                    ldmatrix_x4(a0, a1, a2, a3, page + k_off[(ks + 1) & 3] + 128 * (ks >> 2));
                    mma_bf16_16816(sb, a0, a1, a2, a3, qb[ks + 1][0], qb[ks + 1][1]);
                }

                if (it > 0) {      // the previous unit's logits of these slots, before they are overwritten
                    float y00, y01, y10, y11;
                    load_logits(j, y00, y01, y10, y11);
                    emit_previous(base, y00, y01, y10, y11);
                }

                // scale to the log2 domain, mask the slots past n, keep the logits for the next pass
                float x00 = (sa[0] + sb[0]) * p.scale_log2;      // token g,     head h0
                float x01 = (sa[1] + sb[1]) * p.scale_log2;      // token g,     head h1
                float x10 = (sa[2] + sb[2]) * p.scale_log2;      // token g + 8, head h0
                float x11 = (sa[3] + sb[3]) * p.scale_log2;      // token g + 8, head h1
                if (tok0 + base + 16 > p.n) {                    // only the unit's last page can be ragged
                    if (tok0 + base + g >= p.n) x00 = x01 = -INFINITY;
                    if (tok0 + base + g + 8 >= p.n) x10 = x11 = -INFINITY;
                }
                store_logits(j, x00, x01, x10, x11);

                // raise the reference only when some logit is more than 2^8 above it (always on the first tile)
                float mx0 = fmaxf(x00, x10), mx1 = fmaxf(x01, x11);
                if (__any_sync(0xffffffffu, mx0 > mref0 + kRaiseMargin || mx1 > mref1 + kRaiseMargin)) {
#pragma unroll
                    for (int s = 4; s < 32; s <<= 1) {
                        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, s));
                        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, s));
                    }
                    const float n0 = fmaxf(mref0, mx0), n1 = fmaxf(mref1, mx1);
                    const float c0 = n0 == mref0 ? 1.f : fast_exp2(mref0 - n0);
                    const float c1 = n1 == mref1 ? 1.f : fast_exp2(mref1 - n1);
                    mref0 = n0;
                    mref1 = n1;
                    l0 *= c0;
                    l1 *= c1;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        o[i][0] *= c0;
                        o[i][1] *= c1;
                        o[i][2] *= c0;
                        o[i][3] *= c1;
                    }
                }
                // a reference of -inf means that every slot seen so far lies past n: all weights are zero
                const float r0 = mref0 == -INFINITY ? 0.f : mref0, r1 = mref1 == -INFINITY ? 0.f : mref1;
                const float p00 = fast_exp2(x00 - r0), p01 = fast_exp2(x01 - r1);
                const float p10 = fast_exp2(x10 - r0), p11 = fast_exp2(x11 - r1);
                l0 += p00 + p10;
                l1 += p01 + p11;

                // O^T += V^T P^T.  P enters the tensor core as two bf16 terms, p = hi + lo, so that the
                // weights carry 16 mantissa bits: with a single bf16 term a dominant token's weight would
                // be off by up to 2^-9 whenever the reference is not exactly its logit.  l stays fp32.
                const uint32_t hi0 = pack_bf16(p00, p01), hi1 = pack_bf16(p10, p11);
                const uint32_t lo0 = pack_bf16(p00 - bf16_lo_as_float(hi0), p01 - bf16_hi_as_float(hi0));
                const uint32_t lo1 = pack_bf16(p10 - bf16_lo_as_float(hi1), p11 - bf16_hi_as_float(hi1));
                const uint32_t bh0 = movmatrix_trans(hi0), bh1 = movmatrix_trans(hi1);   // tokens 0-7 / 8-15:
                const uint32_t bl0 = movmatrix_trans(lo0), bl1 = movmatrix_trans(lo1);   // (k = 2 qd, +1; head g)
#pragma unroll
                for (int mt = 0; mt < 8; ++mt) {
                    uint32_t a0, a1, a2, a3;
                    ldmatrix_x4_trans(a0, a1, a2, a3, page + v_off[mt & 3] + 128 * (mt >> 2));
                    mma_bf16_16816(o[mt], a0, a1, a2, a3, bh0, bh1);
                    mma_bf16_16816(o[mt], a0, a1, a2, a3, bl0, bl1);
                }
                // Before the page goes back, look at the barriers of the other groups' pages up to this
                // group's next one: the producer cannot reuse their stages while this one is held.
                if (NG > 1) observe_through(pc + NG - 1);
                if (j < tmem_pages) tmem_wait_st();
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[stage]);
                stage += NG;
                if (stage >= (uint32_t)NS) stage -= NS;
            }
            // ring position of the next unit's first page
            pc_base += npg;
            pc_mod = (pc_mod + npg) % NG;
            st_base = (st_base + (uint32_t)npg) % NS;

            // ---- merge the warps of this block ---------------------------------
            // Every warp leaves its (reference, l) pair and its unscaled O^T in a slot of its own; after
            // one barrier 8 x NW threads turn the references into per-warp scales and the block's
            // (reference, l), and after a second one all threads add the slots up in warp order (the
            // sum is the same in every run).
#pragma unroll
            for (int s = 4; s < 32; s <<= 1) {
                l0 += __shfl_xor_sync(0xffffffffu, l0, s);
                l1 += __shfl_xor_sync(0xffffffffu, l1, s);
            }
            if (g == 0) {
                wml[warp * 16 + h0] = mref0;
                wml[warp * 16 + h1] = mref1;
                wml[warp * 16 + 8 + h0] = l0;
                wml[warp * 16 + 8 + h1] = l1;
            }
            {
                float* slot = slots + warp * (kMaxGroup * kXchgRow);
#pragma unroll
                for (int mt = 0; mt < 8; ++mt) {
                    float* d0 = slot + h0 * kXchgRow + 16 * mt + g;
                    float* d1 = slot + h1 * kXchgRow + 16 * mt + g;
                    d0[0] = o[mt][0];
                    d1[0] = o[mt][1];
                    d0[8] = o[mt][2];
                    d1[8] = o[mt][3];
                }
            }
            named_barrier_sync(1, kConsumers);
            if (!clustered) {
                // One block owns the unit: every warp finishes 8 / NW heads on its own -- the block's
                // reference, the per-warp scales, l, the log-sum-exp and the normalised output -- so one
                // more barrier (for the log-sum-exp) ends the unit.
                constexpr int kHeadsPerWarp = kMaxGroup / NW;
#pragma unroll
                for (int hh = 0; hh < kHeadsPerWarp; ++hh) {
                    const int h = warp * kHeadsPerWarp + hh;
                    float mc = -INFINITY;
#pragma unroll
                    for (int k = 0; k < NW; ++k) mc = fmaxf(mc, wml[k * 16 + h]);
                    float sc[NW], lc = 0.f;
#pragma unroll
                    for (int k = 0; k < NW; ++k) {
                        const float mk = wml[k * 16 + h];
                        sc[k] = mk == -INFINITY ? 0.f : fast_exp2(mk - mc);
                        lc += wml[k * 16 + 8 + h] * sc[k];
                    }
                    const float inv = 1.f / lc;
                    if (lane == 0) lse_s[h] = mc + log2f(lc);
                    if (h < G) {
#pragma unroll
                        for (int k4 = 0; k4 < kHeadDim / 32; ++k4) {
                            const int d = lane + 32 * k4;
                            float acc = 0.f;
#pragma unroll
                            for (int k = 0; k < NW; ++k) acc += slots[k * (kMaxGroup * kXchgRow) + h * kXchgRow + d] * sc[k];
                            p.out[((size_t)u * G + h) * kHeadDim + d] = __float2bfloat16_rn(acc * inv);
                        }
                    }
                }
                named_barrier_sync(1, kConsumers);
                lse0 = lse_s[h0];
                lse1 = lse_s[h1];
                u_prev = u;
            } else {
                Xchg* xb = xchg + (it & 1);
                if (ctid < kMaxGroup * NW) {
                    const int w = ctid >> 3, h = ctid & 7;
                    float mc = -INFINITY;
#pragma unroll
                    for (int k = 0; k < NW; ++k) mc = fmaxf(mc, wml[k * 16 + h]);
                    const float mw = wml[w * 16 + h];
                    scw[w * kMaxGroup + h] = mw == -INFINITY ? 0.f : fast_exp2(mw - mc);
                    if (w == 0) {
                        float lc = 0.f;
#pragma unroll
                        for (int k = 0; k < NW; ++k) {
                            const float mk = wml[k * 16 + h];
                            lc += mk == -INFINITY ? 0.f : wml[k * 16 + 8 + h] * fast_exp2(mk - mc);
                        }
                        xb->m[h] = mc;
                        xb->l[h] = lc;
                    }
                }
                named_barrier_sync(1, kConsumers);
                for (int e = ctid; e < kMaxGroup * kHeadDim; e += kConsumers) {
                    const int h = e >> 7, d = e & (kHeadDim - 1);
                    float acc = 0.f;
#pragma unroll
                    for (int k = 0; k < NW; ++k) acc += slots[k * (kMaxGroup * kXchgRow) + h * kXchgRow + d] * scw[k * kMaxGroup + h];
                    xb->o[h][d] = acc;
                }
                if (clustered) {
                    cluster_arrive();
                    cluster_wait();
                } else {
                    named_barrier_sync(1, kConsumers);
                }

                // ---- merge the blocks of the cluster: exact log-sum-exp per head -----
                if (ctid < kMaxGroup) {
                    float M = -INFINITY, L = 0.f;
                    for (int r = 0; r < S; ++r) M = fmaxf(M, ld_rank_f32(&xb->m[ctid], r, clustered));
                    for (int r = 0; r < S; ++r) {
                        const float mr = ld_rank_f32(&xb->m[ctid], r, clustered);
                        L += mr == -INFINITY ? 0.f : ld_rank_f32(&xb->l[ctid], r, clustered) * exp2f(mr - M);
                    }
                    lse_s[ctid] = M + log2f(L);
                    for (int r = 0; r < S; ++r) {
                        const float mr = ld_rank_f32(&xb->m[ctid], r, clustered);
                        sc_s[r * kMaxGroup + ctid] = mr == -INFINITY ? 0.f : exp2f(mr - M) / L;
                    }
                }
                named_barrier_sync(1, kConsumers);
                lse0 = lse_s[h0];
                lse1 = lse_s[h1];
                u_prev = u;

                // out[g][d]: each block of the cluster finishes a slice of the head dimension
                {
                    const int d_lo = kHeadDim * (int)rank / S, d_hi = kHeadDim * ((int)rank + 1) / S;
                    const int dper = d_hi - d_lo;
                    for (int e = ctid; e < G * dper; e += kConsumers) {
                        const int gg = e / dper, d = d_lo + e % dper;
                        float acc = 0.f;
                        for (int r = 0; r < S; ++r)
                            acc += ld_rank_f32(&xb->o[gg][d], r, clustered) * sc_s[r * kMaxGroup + gg];
                        p.out[((size_t)u * G + gg) * kHeadDim + d] = __float2bfloat16_rn(acc);
                    }
                }
            }
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                qb[ks][0] = qn[ks][0];
                qb[ks][1] = qn[ks][1];
            }
            // No barrier here: lse_s and sc_s are rewritten only after the barriers of the next unit's
            // merge, the exchange buffer alternates, and every logit slot is read and rewritten by
            // the same lane (or, across units, on either side of those barriers).
        }

        // probabilities and statistics of the block's last unit
        if (it > 0) {
            for (int j = grp; j < npg; j += NG) {
                float y00, y01, y10, y11;
                load_logits(j, y00, y01, y10, y11);
                emit_previous(j * kPageTokens + (int)tok_off, y00, y01, y10, y11);
            }
        }
        retire_pending();
    }

    // No block may exit while a peer can still read its shared memory; tensor memory goes back last.
    tmem_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tmem_fence_after_sync();
        tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
    if (clustered) {
        cluster_arrive();
        cluster_wait();
    }
}

constexpr int kMaxGroups = 2;
constexpr int kTmemPages = 128;            // 512 columns / 4 per page
constexpr size_t kMinSmemBytes = 120 * 1024;

template <int NG>
cudaError_t launch_impl(const DecodeParams& p, const DecodePlan& plan, int clusters, cudaStream_t stream,
                        int* max_clusters) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((max_clusters ? 1 : clusters) * plan.splits, 1, 1);
    cfg.blockDim = dim3((4 * NG + 1) * 32, 1, 1);
    cfg.dynamicSmemBytes = plan.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = plan.splits;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (max_clusters) return cudaOccupancyMaxActiveClusters(max_clusters, decode_kernel<NG>, &cfg);
    return cudaLaunchKernelEx(&cfg, decode_kernel<NG>, p);
}

}  // namespace

// Shared-memory layout for a given cluster size and ring depth; returns the total bytes.
static size_t layout(const DecodeConfig& c, int np, int s, int ns, DecodePlan* plan) {
    const int ppc = (np + s - 1) / s;
    // Logits live in tensor memory, four columns per page and lane (128 pages at most); the pages
    // beyond that spill to shared memory, one row per head with a stride = 4 (mod 32) floats, so
    // that the rows of a lane's two heads and of the four lanes of a fragment row fall into
    // different banks.
    const int tp = ppc < kTmemPages ? ppc : kTmemPages;
    int cols = 32;
    while (cols < 4 * tp) cols *= 2;
    const int ls = (ppc - tp) * kPageTokens + 4;
    size_t off = (size_t)ns * kPageBytes;
    plan->off_logits = (int)off;
    if (ppc > tp) off += ((size_t)c.group * ls * sizeof(float) + 127) / 128 * 128;
    plan->off_xchg = (int)off;
    off += 2 * sizeof(Xchg);
    plan->off_wml = (int)off;
    off += 4 * kMaxGroups * 16 * sizeof(float);
    plan->groups = c.force_groups > 0 ? c.force_groups : 2;
    plan->off_slots = (int)off;
    off += (size_t)4 * plan->groups * kMaxGroup * kXchgRow * sizeof(float);
    plan->off_misc = (int)off;
    off += 256 * sizeof(float);
    plan->off_bars = (int)off;
    off += 2 * (size_t)ns * sizeof(uint64_t);
    plan->splits = s;
    plan->stages = ns;
    plan->pages_per_cta = ppc;
    plan->logit_stride = ls;
    plan->tmem_pages = tp;
    plan->tmem_cols = cols;
    // More than half of an SM's shared memory: one block per SM, so the tensor-memory allocation
    // of one block never waits for another block's.
    if (off < kMinSmemBytes) off = kMinSmemBytes;
    plan->smem_bytes = (int)off;
    return off;
}

int decode_plan(const DecodeConfig& c, int n, int max_smem, int splits, DecodePlan* plan) {
    const int np = (n + kPageTokens - 1) / kPageTokens;
    constexpr int kMaxStages = 6;
    const int min_stages = 2;      // a stage per group being worked on      // a stage per group being worked on
    if (c.force_stages > 0)
        return c.force_stages >= min_stages && layout(c, np, splits, c.force_stages, plan) <= (size_t)max_smem ? 0 : -1;
    for (int ns = kMaxStages; ns >= min_stages; --ns)
        if (layout(c, np, splits, ns, plan) <= (size_t)max_smem) return 0;
    return -1;
}

cudaError_t decode_prepare() {
    cudaError_t e = cudaFuncSetAttribute(decode_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(decode_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
}

cudaError_t decode_max_clusters(const DecodePlan& plan, int* clusters) {
    DecodeParams none = {};
    return plan.groups == 2 ? launch_impl<2>(none, plan, 1, nullptr, clusters)
                            : launch_impl<1>(none, plan, 1, nullptr, clusters);
}

cudaError_t decode_launch(const DecodeConfig& c, const DecodePlan& plan, int clusters, const DecodeArgs& a,
                          cudaStream_t stream) {
    DecodeParams p;
    p.pool = const_cast<uint8_t*>(a.pool);
    p.k_new = reinterpret_cast<const uint4*>(a.k_new);
    p.v_new = reinterpret_cast<const uint4*>(a.v_new);
    p.pos = a.state.pos;
    p.append_position = a.append_position;
    p.page_table = a.state.page_table;
    p.q = reinterpret_cast<const __nv_bfloat16*>(a.q);
    p.out = reinterpret_cast<__nv_bfloat16*>(a.out);
    p.pbar = a.state.pbar;
    p.tsm = a.state.tsm;
    p.status = a.state.status;
    p.unit_begin = a.unit_begin;
    p.unit_end = a.unit_begin + a.unit_count;
    p.group = c.group;
    p.pages_per_unit = c.pages_per_unit;
    p.capacity = c.capacity;
    p.total_pages = c.units * c.pages_per_unit;
    p.n = a.n;
    p.t = a.t;
    p.alpha = c.alpha;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)kHeadDim);
    p.inv_group = 1.0f / (float)c.group;
    p.splits = plan.splits;
    p.stages = plan.stages;
    p.pages_per_cta = plan.pages_per_cta;
    p.logit_stride = plan.logit_stride;
    p.tmem_pages = plan.tmem_pages;
    p.tmem_cols = plan.tmem_cols;
    p.off_logits = plan.off_logits;
    p.off_xchg = plan.off_xchg;
    p.off_wml = plan.off_wml;
    p.off_slots = plan.off_slots;
    p.off_misc = plan.off_misc;
    p.off_bars = plan.off_bars;
    p.wait_limit_ns = c.wait_limit_ns;
    p.stop_after_pages = c.stop_after_pages;
    p.rounds_before = a.rounds_before;
    return plan.groups == 2 ? launch_impl<2>(p, plan, clusters, stream, nullptr)
                            : launch_impl<1>(p, plan, clusters, stream, nullptr);
}

}  // namespace lzk
