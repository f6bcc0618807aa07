// GQA flash-decode over the paged, swizzled KV pool with per-token probability
// emission and the fused recurrence-statistics update.
//
// Computes, for every cache unit (Appendix A, Eq. (attn) of the paper):
//   s_g[i] = q_g . k_i / sqrt(D),  p_g = softmax_i(s_g),  out_g = sum_i p_g[i] v_i
// and, fused (Section 4 "Recurrence Interval Tracking", Eq. (1), Algorithm 1):
//   pbar[i] = mean_g p_g[i];  if pbar[i] >= alpha: MRI[i] = max(MRI[i], t - TS[i]); TS[i] = t.
//
// Structure: persistent blocks, one block per SM, grouped in clusters of
// `splits` blocks.  A cluster walks units round-robin; its blocks split the
// unit's pages.  Inside a block one producer warp streams 32 KiB pages into a
// shared-memory ring with linear bulk copies (TMA engine, mbarrier completion);
// the four consumer warps share every page, 16 tokens each: S = Q K^T and
// O += P V run on mma.sync m16n8k16 with the query heads as the M rows, softmax
// is online per warp, and the scaled logits of the block's chunk stay in shared
// memory.
// After the chunk the warps and then the cluster's blocks merge (m, l, O)
// through (distributed) shared memory, which gives the exact log-sum-exp; each
// block then turns its own logits into probabilities, writes pbar and updates
// TS / MRI.  K and V are read from HBM exactly once and nothing but the outputs
// is written.
#include "internal.h"

namespace lzk {

namespace {

constexpr int kXchgRow = kHeadDim + 8;    // padded row of the O exchange buffer (floats)

struct Xchg {
    float o[kMaxGroup][kXchgRow];         // partial output, relative to m
    float m[kMaxGroup];                   // running maximum (log2 domain)
    float l[kMaxGroup];                   // sum of exp2(x - m)
};

struct DecodeParams {
    const uint8_t* pool;
    const int32_t* page_table;
    const __nv_bfloat16* q;
    __nv_bfloat16* out;
    float* pbar;
    int32_t* ts;
    int32_t* mri;
    int32_t* status;
    int units, group, pages_per_unit, capacity, total_pages;
    int n, t;
    float alpha, scale_log2, inv_group;
    int splits, stages, pages_per_cta, logit_stride;
    int off_logits, off_xchg, off_wml, off_misc, off_bars;
};

constexpr uint64_t kWaitLimitNs = 2000000000ull;   // a wait that lasts 2 s is a failure, not a delay

// Bounded wait on an mbarrier phase.  On time-out the block-wide abort flag and
// the device status word are set; once the flag is up no wait blocks any more,
// so that every thread still reaches the cluster barriers and the kernel ends.
__device__ __forceinline__ bool wait_phase(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                           bool honour_abort = true) {
    if (honour_abort && *abort_flag) return false;
    uint32_t spins = 0;
    uint64_t t_start = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0xFF) == 0) {
            if (honour_abort && *abort_flag) return false;
            const uint64_t now = global_timer_ns();
            if (t_start == 0) {
                t_start = now;
            } else if (now - t_start > kWaitLimitNs) {
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

template <int NW>
__global__ void __launch_bounds__((NW + 1) * 32, 1) decode_kernel(const DecodeParams p) {
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* ring = smem;
    float* logits = reinterpret_cast<float*>(smem + p.off_logits);
    Xchg* xchg = reinterpret_cast<Xchg*>(smem + p.off_xchg);          // [2], alternating per unit
    float* wml = reinterpret_cast<float*>(smem + p.off_wml);            // [NW][16]: m[8], l[8] per warp
    float* lse_s = reinterpret_cast<float*>(smem + p.off_misc);         // [8]
    float* sc_s = lse_s + kMaxGroup;                                    // [splits <= 8][8]
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sc_s + 8 * kMaxGroup);
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
            mbar_init(&empty[i], NW);          // every consumer warp releases the stage
        }
        *abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();
    if (clustered) {   // every block of the cluster is resident before any remote access
        cluster_arrive();
        cluster_wait();
    }

    const int np = (p.n + kPageTokens - 1) / kPageTokens;       // pages in use per unit
    const int pg0 = min(np, (int)rank * p.pages_per_cta);
    const int pg1 = min(np, pg0 + p.pages_per_cta);
    const int npg = pg1 - pg0;

    if (warp == NW) {
        // ------------------------------------------------------------ producer
        uint32_t pc = 0;
        int it = 0;
        for (int u = cluster_id; u < p.units; u += n_clusters, ++it) {
            const int32_t* pt = p.page_table + (size_t)u * p.pages_per_unit + pg0;
            for (int base = 0; base < npg; base += 32) {
                const int cnt = min(32, npg - base);
                const int32_t entry = lane < cnt ? pt[base + lane] : 0;
                for (int j = 0; j < cnt; ++j, ++pc) {
                    int32_t pp = __shfl_sync(0xffffffffu, entry, j);
                    const uint32_t stage = pc % NS, use = pc / NS;
                    if (use > 0) wait_phase(&empty[stage], (use - 1) & 1, abort_flag, p.status);
                    if (lane == 0) {
                        if (pp < 0 || pp >= p.total_pages) {
                            atomicOr(p.status, kStatusBadIndex);
                            pp = 0;
                        }
                        mbar_arrive_expect_tx(&full[stage], kPageBytes);
                        bulk_load(ring + (size_t)stage * kPageBytes, p.pool + (size_t)pp * kPageBytes, kPageBytes,
                                  &full[stage]);
                    }
                    __syncwarp();
                }
            }
            if (clustered) {   // this warp's share of the per-unit cluster barrier, split so it can run ahead
                if (it > 0) cluster_wait();
                cluster_arrive();
            }
        }
        if (clustered && it > 0) cluster_wait();
        if (*abort_flag) {   // consumers stopped waiting: let the copies in flight land before the block exits
            const uint32_t last = pc < (uint32_t)NS ? pc : (uint32_t)NS;
            for (uint32_t k = pc - last; k < pc; ++k)
                wait_phase(&full[k % NS], (k / NS) & 1, abort_flag, p.status, false);
        }
    } else {
        // ------------------------------------------------------------ consumers
        const int g = lane >> 2, qd = lane & 3;
        const int ctid = threadIdx.x;                 // consumer thread id: warps 0..NW-1
        constexpr int kConsumers = NW * 32;
        const uint32_t ring_base = smem_u32(ring);
        const uint32_t lrow = lane & 7, lmat = lane >> 3;
        const uint32_t tok_off = 16 * warp;           // this warp's 16 tokens inside every page
        uint32_t pc = 0;
        int it = 0;
        for (int u = cluster_id; u < p.units; u += n_clusters, ++it) {
            uint32_t qa[8][2];
            {
                const __nv_bfloat16* qrow = p.q + ((size_t)u * G + g) * kHeadDim;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    qa[ks][0] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 2 * qd) : 0u;
                    qa[ks][1] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 8 + 2 * qd) : 0u;
                }
            }
            float m_run = -INFINITY, l_run = 0.f;
            float o[16][4];
#pragma unroll
            for (int i = 0; i < 16; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;

            for (int j = 0; j < npg; ++j, ++pc) {
                // All consumer warps work on the same page, 16 tokens each, so a stage is held only
                // for a quarter of a page's arithmetic and goes back to the producer early.  (It also
                // means every warp sees every phase of every "full" barrier, in order, which a parity
                // wait needs.)
                const uint32_t stage = pc % NS;
                wait_phase(&full[stage], (pc / NS) & 1, abort_flag, p.status);
                const uint32_t kb = ring_base + stage * kPageBytes + tok_off * kRowBytes;
                const uint32_t vb = kb + kPageHalfBytes;

                // S[g][token] = Q K^T for this warp's 16 tokens (2 tiles of 8 tokens)
                float sacc[2][4];
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.f;
#pragma unroll
                for (int kp = 0; kp < 4; ++kp) {
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt) {
                        uint32_t b0, b1, b2, b3;
                        ldmatrix_x4(b0, b1, b2, b3,
                                    kb + (8 * nt + lrow) * kRowBytes + (((4 * kp + lmat) ^ lrow) << 4));
                        mma_bf16_16816(sacc[nt], qa[2 * kp][0], 0u, qa[2 * kp][1], 0u, b0, b1);
                        mma_bf16_16816(sacc[nt], qa[2 * kp + 1][0], 0u, qa[2 * kp + 1][1], 0u, b2, b3);
                    }
                }

                // scale to the log2 domain, mask the slots past n, keep the logits for the epilogue
                const int tok_base = (pg0 + j) * kPageTokens + tok_off;
                float tmax = -INFINITY;
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    const int t0 = tok_base + 8 * nt + 2 * qd;
                    const float x0 = t0 < p.n ? sacc[nt][0] * p.scale_log2 : -INFINITY;
                    const float x1 = t0 + 1 < p.n ? sacc[nt][1] * p.scale_log2 : -INFINITY;
                    sacc[nt][0] = x0;
                    sacc[nt][1] = x1;
                    tmax = fmaxf(tmax, fmaxf(x0, x1));
                    if (g < G)
                        *reinterpret_cast<float2*>(&logits[g * LS + j * kPageTokens + tok_off + 8 * nt + 2 * qd]) =
                            make_float2(x0, x1);
                }
                tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
                tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
                const float m_new = fmaxf(m_run, tmax);
                if (m_new != -INFINITY) {            // this warp's 16 slots may all lie past n in the last page
                    if (m_new != m_run) {
                        const float corr = fast_exp2(m_run - m_new);
                        m_run = m_new;
                        l_run *= corr;
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            o[i][0] *= corr;
                            o[i][1] *= corr;
                        }
                    }
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt) {
                        const float p0 = fast_exp2(sacc[nt][0] - m_new), p1 = fast_exp2(sacc[nt][1] - m_new);
                        l_run += p0 + p1;
                        sacc[nt][0] = p0;
                        sacc[nt][1] = p1;
                    }
                } else {
                    sacc[0][0] = sacc[0][1] = sacc[1][0] = sacc[1][1] = 0.f;
                }

                // O[g][d] += P V  (P rounded to bf16 for the tensor core; l stays fp32)
                {
                    const uint32_t a0 = pack_bf16(sacc[0][0], sacc[0][1]);
                    const uint32_t a2 = pack_bf16(sacc[1][0], sacc[1][1]);
#pragma unroll
                    for (int ntp = 0; ntp < 8; ++ntp) {
                        uint32_t b0, b1, b2, b3;
                        ldmatrix_x4_trans(b0, b1, b2, b3,
                                          vb + (8 * (lmat & 1) + lrow) * kRowBytes +
                                              (((2 * ntp + (lmat >> 1)) ^ lrow) << 4));
                        mma_bf16_16816(o[2 * ntp], a0, 0u, a2, 0u, b0, b1);
                        mma_bf16_16816(o[2 * ntp + 1], a0, 0u, a2, 0u, b2, b3);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[stage]);
            }

            // ---- merge the warps of this block ---------------------------------
            l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
            l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
            if (qd == 0) {
                wml[warp * 16 + g] = m_run;
                wml[warp * 16 + 8 + g] = l_run;
            }
            named_barrier_sync(1, kConsumers);
            float m_cta = -INFINITY, l_cta = 0.f;
#pragma unroll
            for (int w = 0; w < NW; ++w) m_cta = fmaxf(m_cta, wml[w * 16 + g]);
#pragma unroll
            for (int w = 0; w < NW; ++w) {
                const float mw = wml[w * 16 + g];
                l_cta += mw == -INFINITY ? 0.f : wml[w * 16 + 8 + g] * fast_exp2(mw - m_cta);
            }
            const float f = m_run == -INFINITY ? 0.f : fast_exp2(m_run - m_cta);
            Xchg* xb = xchg + (it & 1);
            for (int w = 0; w < NW; ++w) {     // fixed order: the sum is the same in every run
                if (warp == w) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        float2* dst = reinterpret_cast<float2*>(&xb->o[g][8 * i + 2 * qd]);
                        float2 v = make_float2(o[i][0] * f, o[i][1] * f);
                        if (w > 0) {
                            const float2 old = *dst;
                            v.x += old.x;
                            v.y += old.y;
                        }
                        *dst = v;
                    }
                }
                named_barrier_sync(1, kConsumers);
            }
            if (warp == 0 && qd == 0) {
                xb->m[g] = m_cta;
                xb->l[g] = l_cta;
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

            // probabilities of this block's tokens, and the statistics update
            {
                const int tok0 = pg0 * kPageTokens;
                const int cn = min(p.n, pg1 * kPageTokens) - tok0;
                const size_t row = (size_t)u * p.capacity + tok0;
                for (int i = ctid; i < cn; i += kConsumers) {
                    float acc = 0.f;
                    for (int gg = 0; gg < G; ++gg) acc += fast_exp2(logits[gg * LS + i] - lse_s[gg]);
                    const float pb = acc * p.inv_group;
                    p.pbar[row + i] = pb;
                    if (pb >= p.alpha) {
                        const int32_t ts_old = p.ts[row + i];
                        const int32_t gap = p.t - ts_old;
                        const int32_t mri_old = p.mri[row + i];
                        if (gap > mri_old) p.mri[row + i] = gap;
                        p.ts[row + i] = p.t;
                    }
                }
            }
            named_barrier_sync(1, kConsumers);   // logits, lse and scales are free for the next unit
        }
    }

    // No block may exit while a peer can still read its shared memory.
    __syncthreads();
    if (clustered) {
        cluster_arrive();
        cluster_wait();
    }
}

constexpr int kConsumerWarps = 4;
static_assert(kConsumerWarps * 16 == kPageTokens, "each consumer warp takes 16 tokens of a page");

}  // namespace

// Shared-memory layout for a given cluster size and ring depth; returns the total bytes.
static size_t layout(const DecodeConfig& c, int np, int s, int ns, DecodePlan* plan) {
    const int ppc = (np + s - 1) / s;
    const int ls = ppc * kPageTokens + 8;      // +8 floats: rows of different heads start in different banks
    size_t off = (size_t)ns * kPageBytes;
    plan->off_logits = (int)off;
    off += ((size_t)c.group * ls * sizeof(float) + 127) / 128 * 128;
    plan->off_xchg = (int)off;
    off += 2 * sizeof(Xchg);
    plan->off_wml = (int)off;
    off += kConsumerWarps * 16 * sizeof(float);
    plan->off_misc = (int)off;
    off += 128 * sizeof(float);
    plan->off_bars = (int)off;
    off += 2 * (size_t)ns * sizeof(uint64_t);
    plan->splits = s;
    plan->stages = ns;
    plan->pages_per_cta = ppc;
    plan->logit_stride = ls;
    plan->smem_bytes = (int)off;
    return off;
}

int decode_plan(const DecodeConfig& c, int n, int max_smem, int splits, DecodePlan* plan) {
    const int np = (n + kPageTokens - 1) / kPageTokens;
    constexpr int kMaxStages = 6;
    if (c.force_stages > 0) return layout(c, np, splits, c.force_stages, plan) <= (size_t)max_smem ? 0 : -1;
    for (int ns = kMaxStages; ns >= 2; --ns)
        if (layout(c, np, splits, ns, plan) <= (size_t)max_smem) return 0;
    return -1;
}

cudaError_t decode_prepare() {
    return cudaFuncSetAttribute(decode_kernel<kConsumerWarps>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                227 * 1024);
}

cudaError_t decode_max_clusters(const DecodePlan& plan, int* clusters) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(plan.splits, 1, 1);
    cfg.blockDim = dim3((kConsumerWarps + 1) * 32, 1, 1);
    cfg.dynamicSmemBytes = plan.smem_bytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = plan.splits;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaOccupancyMaxActiveClusters(clusters, decode_kernel<kConsumerWarps>, &cfg);
}

cudaError_t decode_launch(const DecodeConfig& c, const DecodePlan& plan, int clusters, const DecodeArgs& a,
                          cudaStream_t stream) {
    DecodeParams p;
    p.pool = a.pool;
    p.page_table = a.state.page_table;
    p.q = reinterpret_cast<const __nv_bfloat16*>(a.q);
    p.out = reinterpret_cast<__nv_bfloat16*>(a.out);
    p.pbar = a.state.pbar;
    p.ts = a.state.ts;
    p.mri = a.state.mri;
    p.status = a.state.status;
    p.units = c.units;
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
    p.off_logits = plan.off_logits;
    p.off_xchg = plan.off_xchg;
    p.off_wml = plan.off_wml;
    p.off_misc = plan.off_misc;
    p.off_bars = plan.off_bars;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(clusters * plan.splits, 1, 1);
    cfg.blockDim = dim3((kConsumerWarps + 1) * 32, 1, 1);
    cfg.dynamicSmemBytes = plan.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = plan.splits;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, decode_kernel<kConsumerWarps>, p);
}

}  // namespace lzk
